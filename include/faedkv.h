/*
 * faedkv.h -- C ABI of the FAEDKV / IWDFT hot path on one NVIDIA B200 (sm_100a).
 *
 * The library keeps an LLM KV cache compressed as the retained bins of its
 * discrete Fourier transform along the token axis (FAEDKV, Sec. 4).  It owns
 * three things and nothing else: the per-layer bin plan, small device tables
 * derived from it, and a scratch area that is sized while layers are planned
 * (faedkv_plan() allocates it on the first plan and re-allocates the parts
 * that depend on the bin count whenever a plan brings a larger M than any
 * before it; no other call allocates).  Every tensor, every coefficient plane
 * and every token counter belongs to the caller.
 *
 * Conventions
 *   P        DFT grid size (the paper's N / N_DFT), fixed at create time.
 *   bins[]   ascending retained ONE-SIDED bin indices in [0, P/2]; M = count.
 *            K/V are real, so bin k stands for the conjugate pair (k, P-k);
 *            w_k = 1 for k = 0 and k = P/2 (P even), else 2.
 *   coef     float32, layout [batch][n_kv_heads][2][M][head_dim]; plane 0 is
 *            the real part, plane 1 the imaginary part; head_dim contiguous.
 *            Coefficients are always float32, whatever kv_dtype is.
 *   t_len    int32 [batch], tokens folded into each sequence so far.  One
 *            counter array per layer (append advances it).
 *   K, V     [batch][n_kv_heads][T][head_dim] contiguous, element type kv_dtype.
 *   q, out   [batch][n_q_heads][head_dim], element type kv_dtype; query head g
 *            reads kv head g / (n_q_heads / n_kv_heads).
 *   stream   a cudaStream_t passed as void* (NULL = the default stream).
 *
 * Pointers are DEVICE pointers unless a comment says "host".  Tensor and
 * coefficient pointers must be 16-byte aligned, t_len 4-byte aligned.  Calls
 * validate their arguments on the
 * host and enqueue work on `stream`; apart from faedkv_create(), faedkv_plan()
 * and faedkv_device_status() they do not synchronise and do not allocate.
 * Return value: 0 on success, a negative faedkv_status otherwise;
 * faedkv_last_error() gives the text of the last failure on that context.
 * There is no CPU fallback: what the kernels do not support is an error.
 * A context must not be used from two host threads at once.
 */
#ifndef FAEDKV_H
#define FAEDKV_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct faedkv_ctx faedkv_ctx; /* opaque */

typedef enum { FAEDKV_F32 = 0, FAEDKV_BF16 = 1 } faedkv_dtype;

typedef enum {
    FAEDKV_OK = 0,
    FAEDKV_ERR_INVALID_ARG = -1, /* NULL pointer, negative size, bad enum            */
    FAEDKV_ERR_NOT_PLANNED = -2, /* layer has no plan yet                            */
    FAEDKV_ERR_SHAPE = -3,       /* batch / length outside what the context was made for */
    FAEDKV_ERR_UNSUPPORTED = -4, /* configuration the kernels do not implement       */
    FAEDKV_ERR_ALIGN = -5,       /* device pointer not 16-byte aligned               */
    FAEDKV_ERR_CUDA = -6,        /* a CUDA call failed; see faedkv_last_error()      */
    FAEDKV_ERR_TIMEOUT = -7      /* a bounded device-side wait gave up (see faedkv_device_status) */
} faedkv_status;

/* How the prefill transform is evaluated (faedkv_config.prefill_mode). */
typedef enum {
    FAEDKV_PREFILL_AUTO = 0,  /* bf16 K/V: tensor-core contraction; float32 K/V: FFT-shaped when P is a
                                 power of two in [64, 2^19] (and decode_mode allows FFT), else float32 SIMT */
    FAEDKV_PREFILL_SIMT = 1,  /* float32 FMA contraction, twiddles exact to float32     */
    FAEDKV_PREFILL_UMMA = 2,  /* tcgen05 tensor-core contraction, bf16 operands, float32 accumulate */
    FAEDKV_PREFILL_FFT = 3    /* float32 two-pass FFT of every channel, then a gather of the retained
                                 bins (power-of-two P; needs decode_mode AUTO, FFT or FFT_TWO_PASS): O(T log T) per
                                 channel instead of O(T * M), float32-exact                          */
} faedkv_prefill_mode;

/* How reconstruction and the two transforms inside decode attention are evaluated
 * (faedkv_config.decode_mode). */
typedef enum {
    FAEDKV_DECODE_AUTO = 0,  /* P a power of two in [64, 2^19]: FFT-shaped transforms; otherwise
                                bf16 tensors: tensor-core path; float32 tensors: float32 SIMT path */
    FAEDKV_DECODE_SIMT = 1,  /* float32 FMA contractions, twiddles exact to float32            */
    FAEDKV_DECODE_UMMA = 2,  /* tcgen05 contractions with f16 operands, float32 accumulate (bf16 tensors only) */
    FAEDKV_DECODE_FFT = 3,   /* float32 shared-memory FFTs (power-of-two P only; one kernel per column for
                                P <= 16384, two passes through an L2-resident array above): O(P log P) per
                                query head instead of O(P * M)                                 */
    FAEDKV_DECODE_FFT_TWO_PASS = 4  /* FAEDKV_DECODE_FFT restricted to the two-pass kernels at every P */
} faedkv_decode_mode;

typedef struct {
    int n_layers;      /* >= 1                                                     */
    int n_kv_heads;    /* >= 1                                                     */
    int n_q_heads;     /* multiple of n_kv_heads; 1 to 8 query heads per kv head (any value:
                          e.g. 7 for a 28 / 4 grouped-query model)                  */
    int head_dim;      /* must be 128                                              */
    int n_dft;         /* P >= 2; need not be a power of two                       */
    int max_batch;     /* >= 1; sizes the scratch area                             */
    int kv_dtype;      /* faedkv_dtype of K, V, q, out                             */
    int prefill_mode;  /* faedkv_prefill_mode                                      */
    int twiddle_terms; /* tensor-core prefill only: 1 = twiddles rounded to one bf16
                          (rel. error ~1e-3), 2 = bf16 hi+lo pair (~1e-5, twice the
                          MMA work); 0 = default (1)                                */
    int decode_mode;   /* faedkv_decode_mode                                       */
    int n_sink;        /* S >= 0: first tokens kept in the time domain (Sec. 4.2; the paper
                          uses 10).  Only the *_windowed calls look at n_sink / n_recent */
    int n_recent;      /* R >= 0: most recent tokens kept in the time domain (the paper
                          uses 50); n_sink + n_recent <= 1024                        */
    int n_defer;       /* D: 0 or 1 = the paper's step, one token folded per step (Eq. 12);
                          2 .. 128 = block-deferred fold, see the window section       */
    int recon_engine;  /* FFT-shaped reconstruction: 0 = default (one persistent kernel that runs both
                          passes for P <= 2^15, the two-kernel engine above that), 1 = always the
                          two-kernel engine (one launch per pass and group of units), 2 = the
                          persistent kernel wherever it exists (P <= 2^17)                    */
} faedkv_config;

/* Create a context on the CURRENT CUDA device.  Allocates only a few counters; the scratch area
 * (a few floats per (batch, query head, position of the grid) and per retained bin) is allocated
 * by faedkv_plan().  max_batch * n_kv_heads and max_batch * n_q_heads / 16 must not exceed 65535 (they
 * index a grid dimension).  host: cfg, out. */
int faedkv_create(const faedkv_config *cfg, faedkv_ctx **out);

/* Free the context, its plans and its scratch.  NULL is allowed. */
void faedkv_destroy(faedkv_ctx *ctx);

/* Text of the last error on this context ("" if none).  The pointer stays
 * valid until the next failing call or faedkv_destroy(). */
const char *faedkv_last_error(const faedkv_ctx *ctx);

/* Plan a layer: the pruning rule of Eq. 6 as a keep-list.  bin_mask (host,
 * length P/2 + 1): nonzero = retain one-sided bin k and, implicitly, its
 * mirror P-k.  Builds the ascending bin list and its device copy; replaces an
 * earlier plan of the same layer (the caller must not have work of that layer
 * in flight).  *n_bins_out (host, may be NULL) receives M.  M = 0 is an error.
 * Allocates, and synchronises the device: the first plan of a context sizes the
 * scratch area, and a plan whose M exceeds every earlier M of the context frees
 * and re-allocates the M-dependent parts of it -- buffers that calls of OTHER
 * layers in flight may still be using.  So plan all layers before the first
 * transform call, or make sure the context has no work in flight when planning. */
int faedkv_plan(faedkv_ctx *ctx, int layer, const uint8_t *bin_mask, int *n_bins_out);

/* Number of retained bins of a planned layer, or a negative status. */
int faedkv_n_bins(const faedkv_ctx *ctx, int layer);

/* Copy the layer's bin list to bins_out (host, room for M int32). */
int faedkv_get_bins(const faedkv_ctx *ctx, int layer, int32_t *bins_out);

/* Bytes of ONE coefficient tensor (K or V) of a planned layer at this batch:
 * batch * n_kv_heads * 2 * M * head_dim * 4.  0 if the layer is not planned. */
size_t faedkv_coef_bytes(const faedkv_ctx *ctx, int layer, int batch);

/* Synthetic mask generators used by the tests and the benchmark in place of
 * the paper's ablation-study selection (Sec. 3.2), which needs a model and a
 * corpus.  mask_out: host, length P/2 + 1.
 *   lowpass: bins 0 .. M-1.
 *   mixed:   chunks of 16 bins; the lowest floor((M/2)/16)*16 bins, plus
 *            (M - that)/16 further chunks picked by a Fisher-Yates shuffle of
 *            the remaining chunks below P/2, driven by the 64-bit LCG
 *            s <- s*6364136223846793005 + 1442695040888963407 (draw = s >> 33),
 *            s0 = seed*2654435761 + layer.  M must be a multiple of 16. */
int faedkv_mask_lowpass(int n_dft, int n_keep, uint8_t *mask_out);
int faedkv_mask_mixed(int n_dft, int n_keep, int layer, uint64_t seed, uint8_t *mask_out);

/* Prefill transform (Sec. 4.2.1; Eq. 4 restricted to the retained bins by Eq. 6):
 *   coef[k, c] = sum_{n < T} x[n, c] * exp(-j*2*pi*bins[k]*n / P)
 * for every (batch, kv head) of K and of V.  SETS coefK, coefV and
 * t_len[b] = T for b < batch.  T >= 1 may be smaller than, equal to or larger
 * than P (positions wrap modulo P). */
int faedkv_compress_prefill(faedkv_ctx *ctx, int layer, const void *K, const void *V,
                            int batch, int T, float *coefK, float *coefV,
                            int32_t *t_len, void *stream);

/* IWDFT update (Sec. 4.1 Eq. 9 in its unnormalised, start-referenced form;
 * Sec. 4.2.2 Eq. 12): fold one new token per sequence into the coefficients
 * with unit weight,
 *   coef[k, c] += x_new[c] * exp(-j*2*pi*bins[k]*t / P),  t = t_len[b],
 * then t_len[b] += 1.  k_new, v_new: [batch][n_kv_heads][head_dim].  Only the
 * retained bins exist, which equals updating every bin and pruning again. */
int faedkv_append(faedkv_ctx *ctx, int layer, const void *k_new, const void *v_new,
                  int batch, float *coefK, float *coefV, int32_t *t_len, void *stream);

/* Reconstruction (Sec. 4.2.2 Eq. 11; Eq. 5 with every pruned bin zero):
 *   x~[n, c] = (1/P) * sum_k w_k * (Re coef[k,c]*cos(2*pi*bins[k]*n/P)
 *                                   - Im coef[k,c]*sin(2*pi*bins[k]*n/P))
 * written to K_out, V_out [batch][n_kv_heads][L][head_dim] (kv_dtype) for
 * n < min(t_len[b], P); rows from there up to L are written as zero.
 * 1 <= L <= P.  Either of (coefK, K_out) or (coefV, V_out) may be a NULL pair. */
int faedkv_reconstruct(faedkv_ctx *ctx, int layer, const float *coefK, const float *coefV,
                       const int32_t *t_len, int batch, int L, void *K_out, void *V_out,
                       void *stream);

/* Decode attention (Eq. 3 on the reconstruction of Eq. 11):
 *   out[g] = softmax_n( scale * q[g] . K~[n] ) * V~,  n < min(t_len[b], P)
 * evaluated in the frequency domain, without writing K~ or V~ to memory.
 * scale = 0 means 1/sqrt(head_dim).  A sequence with t_len[b] = 0 has no token
 * to attend to: its rows of out are written as zero (the empty sum of Eq. 3).
 * Uses the context's scratch area: two calls on the same context must not
 * overlap on the GPU. */
int faedkv_decode_attn(faedkv_ctx *ctx, int layer, const void *q, const float *coefK,
                       const float *coefV, const int32_t *t_len, int batch, float scale,
                       void *out, void *stream);

/* IWDFT update and decode attention of one step in one call: exactly
 * faedkv_append() followed by faedkv_decode_attn() (the new token is visible
 * to the attention), but the update rides on the two passes that attention
 * makes over the coefficient planes anyway, so the planes are read once and
 * written once per step instead of read twice more.  coefK, coefV and t_len
 * are updated in place; results equal those of the two separate calls. */
int faedkv_append_decode_attn(faedkv_ctx *ctx, int layer, const void *k_new, const void *v_new,
                              const void *q, int batch, float *coefK, float *coefV, int32_t *t_len,
                              float scale, void *out, void *stream);

/* ---- sink and recent window (Sec. 4.2; Eq. 10, 12, 13) -------------------------------------------
 * The paper's own workflow keeps the first S = n_sink tokens and the last R = n_recent tokens of a
 * sequence in the time domain; only the tokens between them live in the frequency domain.  A
 * window tensor (one for K, one for V; caller-owned, kv_dtype) has the layout
 *   [batch][n_kv_heads][S + R][head_dim]:  rows [0, S) the sink tokens, rows [S, S + R) a ring in
 *   which token n >= S occupies slot (n - S) mod R while it is among the last R tokens.
 * t_len counts ALL tokens of a sequence; the transformed segment holds t_len - S - R of them, at
 * positions 0, 1, ... (token n sits at position n - S), wrapping modulo P like everywhere else.
 *
 * Block-deferred fold (n_defer = D >= 2).  Eq. 12 costs a read and a write of every coefficient per
 * step.  Because the update is linear, tokens may instead wait in the time domain and be folded D at
 * a time: the ring then has R + D slots (rows [S, S + R + D); token n in slot (n - S) mod (R + D)),
 * the transformed segment holds  folded(t) = D * floor((t - S - R) / D)  tokens (0 while t < S + R),
 * and a step whose token brings t - S - R to a multiple of D folds the D oldest waiting tokens,
 * oldest first, with exactly the arithmetic of D single-token updates.  Whenever t - S - R is a
 * multiple of D the state equals that of the per-step form; in between, up to D - 1 more tokens are
 * attended exactly instead of through their retained bins.  Every other step only READS the planes. */

/* Bytes of ONE window tensor (K or V) at this batch. */
size_t faedkv_window_bytes(const faedkv_ctx *ctx, int batch);

/* Prefill (Eq. 10): tokens [0, S) are copied to the sink rows, tokens [T - R, T) to their ring
 * slots, and the tokens between them are transformed into coefK, coefV as in
 * faedkv_compress_prefill (planes are zero when there is none).  SETS t_len[b] = T.
 * With n_defer = D >= 2 the transformed tokens are [S, S + folded(T)) and the ring takes the rest.
 * T >= S + R is required (FAEDKV_ERR_SHAPE otherwise).  With S = R = 0 this is
 * faedkv_compress_prefill and winK, winV may be NULL. */
int faedkv_prefill_windowed(faedkv_ctx *ctx, int layer, const void *K, const void *V, int batch,
                            int T, float *coefK, float *coefV, void *winK, void *winV,
                            int32_t *t_len, void *stream);

/* One decode step of the paper's workflow for every sequence, t = t_len[b]:
 *   update (Eq. 12)  the token leaving the recent window, t - R, is folded into the coefficients
 *                    at position t - R - S with unit weight (with R = 0: the new token itself);
 *   attend (Eq. 13, Eq. 3)  out = softmax(scale * q . [K_sink | K~ | K_recent]) [V_sink | V~ | V_recent]
 *                    over the S sink tokens, the reconstruction of min(t + 1 - S - R, P) positions
 *                    and the R most recent tokens including the new one -- one softmax, evaluated
 *                    without writing K~, V~ or the scores to memory;
 *   commit           the new token takes the ring slot of the one that left; t_len[b] += 1.
 * With n_defer = D >= 2: the D oldest waiting tokens are folded if t + 1 - S - R is a multiple of D
 * (per sequence; ragged batches fold at different steps), attention runs over the sink, the
 * reconstruction of min(folded(t + 1), P) positions and all waiting tokens including the new one,
 * then the new token takes its ring slot and t_len[b] += 1.
 * Needs the FFT-shaped decode path (P a power of two in [64, 2^19]); FAEDKV_ERR_UNSUPPORTED
 * otherwise.  The segment Eq. 10 transforms, N - S - R tokens, is rarely a power of two: create the
 * context with n_dft = the next power of two at or above the longest segment that must not alias
 * (e.g. 16324 tokens of a 16384-token prompt on P = 16384); positions the segment has not reached yet
 * are masked out of the softmax, so a grid longer than the segment changes no result.
 * winK, winV, coefK, coefV and t_len are updated in place. */
int faedkv_step_windowed(faedkv_ctx *ctx, int layer, const void *k_new, const void *v_new,
                         const void *q, int batch, float *coefK, float *coefV, void *winK,
                         void *winV, int32_t *t_len, float scale, void *out, void *stream);

/* Eq. 13 written out: K_out, V_out [batch][n_kv_heads][L][head_dim] (kv_dtype) receive, per sequence, the
 * cache the windowed attention attends over, in order: the S sink tokens, the reconstruction (Eq. 11) of
 * the min(folded, P) positions of the transformed segment, the tokens still in the time domain (the last
 * R; R .. R + D - 1 with the block-deferred fold), and zeros up to row L.  Rows past L are not written; a
 * sequence longer than L is cut.  For callers that run their own attention on the reconstructed cache;
 * faedkv_step_windowed itself never materialises these rows.  Call it between steps.  Needs the
 * FFT-shaped path like the other windowed calls. */
int faedkv_reconstruct_windowed(faedkv_ctx *ctx, int layer, const float *coefK, const float *coefV,
                                const void *winK, const void *winV, const int32_t *t_len, int batch,
                                int L, void *K_out, void *V_out, void *stream);

/* ---- frequency ablation and bin selection (Sec. 3.2) -----------------------------------------------
 * The paper chooses each layer's retained bins once per model: the P two-sided bins are cut into C
 * contiguous chunks (C = 22 in the paper), each chunk is zeroed in turn in the DFT of the layer's K and
 * V caches (Eq. 6), the perplexity change Delta is measured, and the r*C chunks with the largest Delta
 * are kept.  The perplexity runs need a model and a corpus and are the caller's; these calls are the
 * rest of the procedure. */

/* Two-sided bins [*lo, *hi) of chunk `chunk` of n_chunks: chunks of floor(P / n_chunks) bins, the
 * last one running to P.  host: lo, hi. */
int faedkv_chunk_range(int n_dft, int n_chunks, int chunk, int *lo, int *hi);

/* One-sided view of zeroing the two-sided bins [lo, hi) of a real signal.  mask_out, gain_out: host,
 * length P/2 + 1.  mask_out[k] = 1 when bin k or its mirror P - k is zeroed; gain_out[k] = the share
 * of that conjugate pair's real component that disappears from Re(IDFT): 1 when both are zeroed (or k
 * is its own mirror), 1/2 when only one of them is, 0 elsewhere. */
int faedkv_ablation_bins(int n_dft, int lo, int hi, uint8_t *mask_out, float *gain_out);

/* Greedy selection: keeps the n_keep = max(1, floor(ratio * n_chunks + 1/2)) chunks with the largest
 * delta (host, n_chunks doubles; ties go to the lower chunk index) and writes the one-sided keep-mask
 * for faedkv_plan (a bin is kept when it or its mirror lies in a kept chunk).  *n_keep_out may be NULL. */
int faedkv_mask_from_scores(int n_dft, int n_chunks, const double *delta, double ratio,
                            uint8_t *mask_out, int *n_keep_out);

/* The ablated caches (Eq. 6, then Eq. 5, real part):  X_out = X - sum_i gain[i] * (component of
 * retained bin i of X), for X = K and X = V, [batch][n_kv_heads][T][head_dim], T <= P (rows beyond T
 * count as zero; the paper's N is the sequence length, i.e. create the context with n_dft = T).
 * The layer must be planned with the mask from faedkv_ablation_bins; gain: DEVICE float[M], the
 * gains of the retained bins in ascending bin order.  wsK, wsV (faedkv_coef_bytes each) and ws_len
 * (int32[batch]) are workspaces the call overwrites.  Runs compress_prefill, a scaling of the planes,
 * reconstruct and a subtraction on `stream`. */
int faedkv_ablate(faedkv_ctx *ctx, int layer, const void *K, const void *V, int batch, int T,
                  const float *gain, float *wsK, float *wsV, int32_t *ws_len, void *K_out, void *V_out,
                  void *stream);

/* ---- the state in the forms the paper's equations print (Sec. 4.1) ---------------------------------
 * Every call of this library keeps the unnormalised, start-referenced sum
 *   SUM       C_t[k] = sum_{n<t} x[n] exp(-j*2*pi*k*n/P).
 * Eq. 9 with its exact factors (t-1)/t and 1/t keeps the running mean, and Eq. 8 / Eq. 9 as recursions
 * that multiply the whole state by W_k = exp(-j*2*pi*k/P) each step keep a newest-token-referenced state:
 *   MEAN      S_t[k] = C_t[k] / t
 *   ROTATING  R_t[k] = W_k^t * conj(C_t[k])          (R <- W_k (R + x) from R_0 = 0)
 * For real K/V the three hold the same information; this call converts a coefficient tensor between
 * them, for exchanging state with an implementation that follows the printed recursions.  t = t_len[b];
 * coef_in and coef_out have the coefficient layout and may be the same buffer. */
typedef enum { FAEDKV_STATE_SUM = 0, FAEDKV_STATE_MEAN = 1, FAEDKV_STATE_ROTATING = 2 } faedkv_state_form;
int faedkv_convert_state(faedkv_ctx *ctx, int layer, const float *coef_in, const int32_t *t_len,
                         int batch, int from_form, int to_form, float *coef_out, void *stream);

/* Device-side status word of the context (host read; synchronises `stream`):
 * 0, or a nonzero code left by a kernel whose bounded wait on an mbarrier gave
 * up.  Such a kernel returns early instead of hanging; its output is invalid. */
int faedkv_device_status(faedkv_ctx *ctx, void *stream);

/* Clear the device-side status word (enqueued on `stream`), so that a context whose kernel gave up a wait can be
 * used, and watched, again. */
int faedkv_reset_device_status(faedkv_ctx *ctx, void *stream);

/* Test and diagnostics hooks of the tensor-core prefill (host state of the context; they apply to the calls
 * that follow).  wait_limit_ns: time limit of each bounded mbarrier wait of that kernel (0 = the default,
 * about one second).  withhold_step: 0 = off; s >= 1 = at pipeline step s (64 tokens per step) one producer
 * warp of every CTA skips its "tile full" signal, so that every wait of the CTA runs out after wait_limit_ns:
 * the kernel then records a code in the status word, waits for its own bulk copies, frees its tensor memory
 * and returns -- the give-up path, exercised without any fault.  The output of such a call is invalid. */
int faedkv_test_hooks(faedkv_ctx *ctx, unsigned long long wait_limit_ns, int withhold_step);

/* Checked build.  The same sources compiled with -DFAEDKV_DEBUG (python -m paper_2507_20030_b200.build --debug
 * -> lib/libfaedkv_debug.so) test every index that the kernels compute from data (bins, plan slots, ring
 * slots, rows, tile offsets) against its bound before using it; a failed test records where it happened and
 * skips the access, and the kernel returns normally.  faedkv_debug_build() is 1 in that build, else 0.
 * faedkv_debug_word() synchronises `stream`, returns (file tag << 16 | source line) of the first failed test
 * since the last call, or 0, and clears the word; it is always 0 in the normal build.  (The word is per
 * process and device, not per context.) */
int faedkv_debug_build(void);
long long faedkv_debug_word(faedkv_ctx *ctx, void *stream);

/* Decode attention for callers that cannot allocate -- the paper has no
 * counterpart; this is a packaging of faedkv_decode_attn() for hosts that
 * must not call cudaMalloc where they need it: code that runs while a CUDA
 * graph is being captured, a serving loop whose device memory was handed out
 * once by an external pool, a plugin that only gets the tensors it is called
 * with.  It takes no context (creating and planning one allocates): the bin
 * list `bins` (DEVICE, int32[n_bins], ascending one-sided bins as produced by
 * faedkv_get_bins) comes with the other inputs, and all intermediates live in
 * a fixed device array of FAEDKV_STATIC_SCRATCH_BYTES that is part of the
 * library image -- every GPU that loads the library holds that much until
 * the process exits.  It calls no allocation routine of any kind.
 *
 * Same arguments, layouts and result as faedkv_decode_attn() (float32
 * kernels); kv_dtype is the faedkv_dtype of q and out.  Sizes whose
 * intermediates, about 4*batch*HQP*(n_dft + 4*n_bins + n_dft/32) bytes with
 * HQP = n_q_heads rounded up to 32, exceed the array, and sizes with
 * batch * n_kv_heads or batch * HQP / 32 above 65535 (a grid dimension), are
 * refused with FAEDKV_ERR_SHAPE before anything is launched.  On any failure a
 * text is written to err_msg (host, err_len bytes; may be NULL).
 *
 * All calls share the one array, which keeps the previous call's contents.
 * Nothing in it needs to start at zero, so nothing is cleared; but calls that
 * overlap on the GPU (two streams, two host threads) race on it: serialise
 * them.  The first call on each device resolves the array's device address;
 * make that first call outside any stream capture. */
#define FAEDKV_STATIC_SCRATCH_BYTES (8u << 20)
int faedkv_decode_attn_static(int n_dft, int n_kv_heads, int n_q_heads, int kv_dtype,
                              const int32_t *bins, int n_bins, const void *q, const float *coefK,
                              const float *coefV, const int32_t *t_len, int batch, float scale,
                              void *out, void *stream, char *err_msg, size_t err_len);

/* Number of kernels this context has enqueued since it was created (host
 * counter; the benchmark reports its difference over the timed region). */
unsigned long long faedkv_launch_count(const faedkv_ctx *ctx);

#ifdef __cplusplus
}
#endif
#endif /* FAEDKV_H */
