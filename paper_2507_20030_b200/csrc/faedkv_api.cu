// Host side of the FAEDKV C ABI: context, per-layer plans, argument checks and
// kernel launches.  See include/faedkv.h for the contract of every call.
#include <algorithm>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <new>
#include <string>
#include <vector>

#include <nvtx3/nvToolsExt.h>

#include "../../include/faedkv.h"
#include "common.cuh"
#include "k_append.cuh"
#include "k_attn.cuh"
#include "k_dft_simt.cuh"
#include "k_prefill_umma.cuh"
#include "k_idft_umma.cuh"
#include "k_attn_umma.cuh"
#include "k_attn_fft.cuh"
#include "k_attn_fft2.cuh"
#include "k_attn_col.cuh"
#include "k_recon_fft.cuh"
#include "k_recon2.cuh"
#include "k_prefill_fft.cuh"
#include "k_ablate.cuh"
#include "k_state.cuh"

using namespace faedkv;

namespace {

// An NVTX range around a C-ABI call: names the call on a profiler's timeline; a no-op when no tool is attached.
struct CallRange {
    explicit CallRange(const char *name) { nvtxRangePushA(name); }
    ~CallRange() { nvtxRangePop(); }
    CallRange(const CallRange &) = delete;
    CallRange &operator=(const CallRange &) = delete;
};

struct LayerPlan {
    int M = 0;
    std::vector<int32_t> bins;
    int32_t *d_bins = nullptr;
    float *d_tab = nullptr;   // [M][16] per-bin phasors e^{jwk i}, i = 1..8 (tensor-core inverse transform)
    int32_t *d_slot = nullptr;  // [P/2 + 1] bin -> index in bins[] or -1 (FFT-shaped transforms)
};

constexpr int kSplitsCap = 8;   // most position splits of the probability spectrum

// Scratch of the tensor-core decode / reconstruct path (bf16 tensors only).
struct TcScratch {
    __half *Qf16 = nullptr, *P16 = nullptr, *C16K = nullptr, *C16V = nullptr;
    float *S = nullptr, *tile_max = nullptr, *cmax = nullptr, *psum = nullptr, *colsum = nullptr, *PfS = nullptr;
    int gtot_max = 0, max_M = 0;
};

// Scratch of the FFT-shaped decode attention (power-of-two P).
struct FftScratch {
    float2 *Qs = nullptr, *Y = nullptr, *Zf = nullptr;
    float2 *Yr = nullptr;                 // two-pass array of the FFT-shaped reconstruction / prefill, [N][recon_units * 128]
    float2 *Zr = nullptr;                 // second array of the FFT-shaped prefill (full spectrum before the gather)
    int recon_units = 0;                  // units (sequence, kv head) per launch group of the reconstruction
    float *mloc = nullptr, *sloc = nullptr, *colsum = nullptr;   // [N1 + 1][Gp] (last row: the window), [2][Gp]
    float *o_win = nullptr;               // [Gp][128] unnormalised attention output over the sink + recent window
    float2 *Wg = nullptr;                 // [Gp][max_M] probability-spectrum weights (one-kernel column transform)
    float2 *colE = nullptr, *colB = nullptr, *colP = nullptr;   // its twiddle tables (see k_col_tables)
    cudaStream_t side = nullptr;          // second stream: the window kernel runs beside the FFT kernels
    cudaEvent_t ev_fork = nullptr, ev_join = nullptr;
    cudaStream_t side2 = nullptr;         // third stream: the second run of sequences of a call cut in two
    cudaEvent_t ev_cut = nullptr, ev_merge = nullptr;
    float2 *a2_tabI = nullptr;            // inter-pass twiddles of the two-column attention transforms (P <= 2^17)
    unsigned int a2_attr[3] = {0, 0, 0};  // their instances already opted in to large shared memory
    // second reconstruction engine (one persistent kernel; P <= 2^17)
    float2 *r2_tabP = nullptr, *r2_tabI = nullptr;
    unsigned int *r2_sync = nullptr;      // ticket, exit counter, per-column-block pass counters; zero between calls
    size_t yr_bytes = 0;                  // size of Yr
    unsigned int r2_attr = 0;             // instances already opted in to large shared memory
    int r2_ctas_per_sm[2][32] = {};       // occupancy of each instance (0 = not asked yet)
    unsigned int *tickets = nullptr;      // [max_batch * H + max_batch], zero between calls
    int max_M = 0;
    unsigned int attr_mask[11] = {0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0};  // per kernel: transform lengths already opted in to large shared memory
};

}  // namespace

struct faedkv_ctx {
    faedkv_config cfg;
    int device = 0;
    int n_sm = 1;  // multiprocessors of the device (grid sizing)
    int gq = 1;    // query heads per kv head
    int hqp = 32;  // n_q_heads rounded up to a multiple of 32
    int max_M = 0;
    int out_slices_cap = 0;
    std::vector<LayerPlan> plans;
    // scratch (device)
    float *Qf = nullptr, *Pf = nullptr, *S = nullptr, *tile_max = nullptr, *colmax = nullptr,
          *partial = nullptr;
    unsigned int *tick = nullptr;      // [n_layers] tickets of k_append
    unsigned int *dev_status = nullptr;  // one word, set by a kernel whose bounded wait gave up
    UmmaPrefillState umma;             // tensor maps etc. of the tensor-core prefill
    TcScratch tc;
    bool use_tc = false;               // bf16 tensors and decode_mode != SIMT
    bool use_fft = false;              // power-of-two P: FFT-shaped transforms in decode attention and reconstruction
    bool use_col = false;              // ... and P <= 16384: decode attention's transforms as one kernel per column
    bool prefill_fft = false;          // FFT-shaped prefill transform
    FftScratch fs;
    unsigned long long launches = 0;   // kernels enqueued by this context so far
    std::string err;
};

namespace {

int fail(faedkv_ctx *ctx, int code, const char *fmt, ...) {
    if (ctx != nullptr) {
        char buf[512];
        va_list ap;
        va_start(ap, fmt);
        vsnprintf(buf, sizeof(buf), fmt, ap);
        va_end(ap);
        ctx->err = buf;
    }
    return code;
}

#define CUDA_TRY(ctx, expr)                                                                   \
    do {                                                                                      \
        cudaError_t e_ = (expr);                                                              \
        if (e_ != cudaSuccess)                                                                \
            return fail(ctx, FAEDKV_ERR_CUDA, "%s failed: %s", #expr, cudaGetErrorString(e_)); \
    } while (0)

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
bool aligned4(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 3u) == 0; }

int check_layer(faedkv_ctx *ctx, int layer, const LayerPlan **plan) {
    if (ctx == nullptr) return FAEDKV_ERR_INVALID_ARG;
    if (layer < 0 || layer >= ctx->cfg.n_layers)
        return fail(ctx, FAEDKV_ERR_INVALID_ARG, "layer %d outside [0, %d)", layer, ctx->cfg.n_layers);
    const LayerPlan &p = ctx->plans[layer];
    if (p.M == 0) return fail(ctx, FAEDKV_ERR_NOT_PLANNED, "layer %d has no plan", layer);
    *plan = &p;
    return FAEDKV_OK;
}

int check_batch(faedkv_ctx *ctx, int batch) {
    if (batch < 1 || batch > ctx->cfg.max_batch)
        return fail(ctx, FAEDKV_ERR_SHAPE, "batch %d outside [1, max_batch=%d]", batch, ctx->cfg.max_batch);
    return FAEDKV_OK;
}

int check_ptrs(faedkv_ctx *ctx, std::initializer_list<const void *> ptrs) {
    for (const void *p : ptrs)
        if (!aligned16(p)) return fail(ctx, FAEDKV_ERR_ALIGN, "device pointer %p is not 16-byte aligned", p);
    return FAEDKV_OK;
}

int check_tlen(faedkv_ctx *ctx, const void *t_len) {
    if (!aligned4(t_len)) return fail(ctx, FAEDKV_ERR_ALIGN, "t_len %p is not 4-byte aligned", t_len);
    return FAEDKV_OK;
}

int launch_check(faedkv_ctx *ctx, const char *what) {
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return fail(ctx, FAEDKV_ERR_CUDA, "launch of %s failed: %s", what, cudaGetErrorString(e));
    ctx->launches += 1;
    return FAEDKV_OK;
}

int out_slices(const faedkv_ctx *ctx, int batch, int M) {
    // enough CTAs to fill the GPU twice over, at least 64 bins per slice
    const int units = batch * ctx->cfg.n_kv_heads;
    int s = (2 * ctx->n_sm + units - 1) / units;
    int cap = (M + 63) / 64;
    if (s > cap) s = cap;
    if (s < 1) s = 1;
    return s;
}

void free_scratch(faedkv_ctx *ctx) {
    cudaFree(ctx->Qf); cudaFree(ctx->Pf); cudaFree(ctx->S);
    cudaFree(ctx->tile_max); cudaFree(ctx->colmax); cudaFree(ctx->partial);
    ctx->Qf = ctx->Pf = ctx->S = ctx->tile_max = ctx->colmax = ctx->partial = nullptr;
    TcScratch &t = ctx->tc;
    cudaFree(t.Qf16); cudaFree(t.P16); cudaFree(t.C16K); cudaFree(t.C16V); cudaFree(t.S); cudaFree(t.tile_max);
    cudaFree(t.cmax); cudaFree(t.psum); cudaFree(t.colsum); cudaFree(t.PfS);
    t = TcScratch();
    FftScratch &f = ctx->fs;
    cudaFree(f.Qs); cudaFree(f.Y); cudaFree(f.Zf); cudaFree(f.mloc); cudaFree(f.sloc); cudaFree(f.colsum); cudaFree(f.o_win); cudaFree(f.Wg); cudaFree(f.colE); cudaFree(f.colB); cudaFree(f.colP); cudaFree(f.tickets); cudaFree(f.Yr); cudaFree(f.Zr); cudaFree(f.r2_tabP); cudaFree(f.r2_tabI); cudaFree(f.r2_sync); cudaFree(f.a2_tabI);
    if (f.side != nullptr) cudaStreamDestroy(f.side);
    if (f.ev_fork != nullptr) cudaEventDestroy(f.ev_fork);
    if (f.ev_join != nullptr) cudaEventDestroy(f.ev_join);
    if (f.side2 != nullptr) cudaStreamDestroy(f.side2);
    if (f.ev_cut != nullptr) cudaEventDestroy(f.ev_cut);
    if (f.ev_merge != nullptr) cudaEventDestroy(f.ev_merge);
    f = FftScratch();
}

// (Re)size the parts of the scratch area that depend on the largest M planned so far.
int ensure_scratch(faedkv_ctx *ctx, int M) {
    const faedkv_config &c = ctx->cfg;
    const size_t B = (size_t)c.max_batch, P = (size_t)c.n_dft, HQP = (size_t)ctx->hqp;
    const bool attn_simt = !ctx->use_fft && !ctx->use_tc, attn_tc = !ctx->use_fft && ctx->use_tc;
    if (attn_simt && ctx->S == nullptr) {
        const size_t n_tiles = (P + kTilePos - 1) / kTilePos;
        CUDA_TRY(ctx, cudaMalloc(&ctx->S, B * P * HQP * sizeof(float)));
        CUDA_TRY(ctx, cudaMalloc(&ctx->tile_max, B * n_tiles * HQP * sizeof(float)));
        CUDA_TRY(ctx, cudaMalloc(&ctx->colmax, B * HQP * sizeof(float)));
    }
    if (M > ctx->max_M) {
        cudaFree(ctx->Qf); cudaFree(ctx->Pf); cudaFree(ctx->partial);
        ctx->Qf = ctx->Pf = ctx->partial = nullptr;
        if (attn_simt) {
            CUDA_TRY(ctx, cudaMalloc(&ctx->Qf, B * 2 * (size_t)M * HQP * sizeof(float)));
            CUDA_TRY(ctx, cudaMalloc(&ctx->Pf, B * 2 * (size_t)M * HQP * sizeof(float)));
        }
        // the slice count never exceeds twice the SM count (units >= 1), nor ceil(M/64)
        int cap = (M + 63) / 64;
        if (cap > 2 * ctx->n_sm) cap = 2 * ctx->n_sm;
        ctx->out_slices_cap = cap;
        CUDA_TRY(ctx, cudaMalloc(&ctx->partial, B * c.n_kv_heads * (size_t)cap * ctx->gq * kHeadDim * sizeof(float)));
        ctx->max_M = M;
    }
    if (ctx->use_fft) {
        FftScratch &f = ctx->fs;
        const fft::Geometry g = fft::make_geometry(c.n_dft, c.max_batch * c.n_q_heads);
        if (f.Y == nullptr) {
            CUDA_TRY(ctx, cudaMalloc(&f.Y, (size_t)g.N * g.Gp * sizeof(float2)));
            CUDA_TRY(ctx, cudaMalloc(&f.Zf, (size_t)g.N * g.Gp * sizeof(float2)));
            CUDA_TRY(ctx, cudaMalloc(&f.mloc, (size_t)(g.N1 + 1) * g.Gp * sizeof(float)));
            CUDA_TRY(ctx, cudaMalloc(&f.sloc, (size_t)(g.N1 + 1) * g.Gp * sizeof(float)));
            CUDA_TRY(ctx, cudaMalloc(&f.colsum, (size_t)2 * g.Gp * sizeof(float)));
            if (c.n_sink + c.n_recent > 0 || c.n_defer > 1) {
                CUDA_TRY(ctx, cudaMalloc(&f.o_win, (size_t)g.Gp * kHeadDim * sizeof(float)));
                CUDA_TRY(ctx, cudaStreamCreateWithFlags(&f.side, cudaStreamNonBlocking));
                CUDA_TRY(ctx, cudaEventCreateWithFlags(&f.ev_fork, cudaEventDisableTiming));
                CUDA_TRY(ctx, cudaEventCreateWithFlags(&f.ev_join, cudaEventDisableTiming));
            }
            const size_t n_tickets = (size_t)c.max_batch * c.n_kv_heads + c.max_batch;
            CUDA_TRY(ctx, cudaMalloc(&f.tickets, n_tickets * sizeof(unsigned int)));
            CUDA_TRY(ctx, cudaMemset(f.tickets, 0, n_tickets * sizeof(unsigned int)));
            // reconstruction / FFT-shaped prefill: units per launch group, bounded by a 128 MB two-pass array.
            // (These kernels are instruction-bound, not bandwidth-bound: measured, larger launches win over
            // keeping the array L2-resident, up to about this size.)
            const size_t unit_bytes = (size_t)g.N * kHeadDim * sizeof(float2);
            size_t ru = (128u << 20) / unit_bytes;
            if (ru < 1) ru = 1;
            if (ru > (size_t)c.max_batch * c.n_kv_heads) ru = (size_t)c.max_batch * c.n_kv_heads;
            f.recon_units = (int)ru;
            f.yr_bytes = ru * unit_bytes;
            CUDA_TRY(ctx, cudaMalloc(&f.Yr, ru * unit_bytes));
            if (rfft2::supported(c.n_dft)) {
                const size_t n_sync = 2 + 2 * (size_t)2 * c.max_batch * c.n_kv_heads * (kHeadDim / rfft2::kCW);
                CUDA_TRY(ctx, cudaMalloc(&f.r2_tabP, ((size_t)g.N + 1) * sizeof(float2)));
                CUDA_TRY(ctx, cudaMalloc(&f.r2_tabI, (size_t)g.N * sizeof(float2)));
                CUDA_TRY(ctx, cudaMalloc(&f.r2_sync, n_sync * sizeof(unsigned int)));
                CUDA_TRY(ctx, cudaMemset(f.r2_sync, 0, n_sync * sizeof(unsigned int)));
                rfft2::k_recon2_tables<<<64, 256>>>(f.r2_tabP, f.r2_tabI, (uint32_t)c.n_dft, g.N2);
                CUDA_TRY(ctx, cudaMalloc(&f.a2_tabI, (size_t)g.N * sizeof(float2)));
                afft2::k_afft2_tables<<<64, 256>>>(f.a2_tabI, (uint32_t)g.N, g.N2);
                CUDA_TRY(ctx, cudaDeviceSynchronize());
            }
            if (ctx->prefill_fft) CUDA_TRY(ctx, cudaMalloc(&f.Zr, ru * unit_bytes));
        }
        if (M > f.max_M) {
            cudaFree(f.Qs); cudaFree(f.Wg);
            f.Qs = f.Wg = nullptr;
            CUDA_TRY(ctx, cudaMalloc(&f.Qs, (size_t)M * g.Gp * sizeof(float2)));
            if (ctx->use_col) CUDA_TRY(ctx, cudaMalloc(&f.Wg, (size_t)M * g.Gp * sizeof(float2)));
            f.max_M = M;
        }
        if (ctx->use_col && f.colE == nullptr) {
            CUDA_TRY(ctx, cudaMalloc(&f.colE, sizeof(float2) << colfft::kLgE));
            CUDA_TRY(ctx, cudaMalloc(&f.colB, sizeof(float2) << colfft::kLgE));
            CUDA_TRY(ctx, cudaMalloc(&f.colP, sizeof(float2) * ((size_t)g.N + 1)));
            CUDA_TRY(ctx, cudaStreamCreateWithFlags(&f.side2, cudaStreamNonBlocking));
            CUDA_TRY(ctx, cudaEventCreateWithFlags(&f.ev_cut, cudaEventDisableTiming));
            CUDA_TRY(ctx, cudaEventCreateWithFlags(&f.ev_merge, cudaEventDisableTiming));
            colfft::k_col_tables<<<32, 256>>>(f.colE, f.colB, f.colP, (uint32_t)c.n_dft);
            CUDA_TRY(ctx, cudaDeviceSynchronize());
        }
    }
    if (ctx->use_tc) {
        TcScratch &t = ctx->tc;
        if (attn_tc && t.S == nullptr) {
            t.gtot_max = (c.max_batch * c.n_q_heads + 63) / 64 * 64;
            const size_t G = (size_t)t.gtot_max;
            CUDA_TRY(ctx, cudaMalloc(&t.S, P * G * sizeof(float)));
            CUDA_TRY(ctx, cudaMalloc(&t.tile_max, ((P + 31) / 32) * G * sizeof(float)));
            CUDA_TRY(ctx, cudaMalloc(&t.cmax, G * sizeof(float)));
            CUDA_TRY(ctx, cudaMalloc(&t.colsum, G * sizeof(float)));
            CUDA_TRY(ctx, cudaMalloc(&t.psum, ((P + kSoftmaxRows - 1) / kSoftmaxRows) * G * sizeof(float)));
            CUDA_TRY(ctx, cudaMalloc(&t.P16, P * G * sizeof(__half)));
        }
        if (M > t.max_M) {
            cudaFree(t.Qf16); cudaFree(t.PfS); cudaFree(t.C16K); cudaFree(t.C16V);
            t.Qf16 = nullptr; t.PfS = nullptr; t.C16K = t.C16V = nullptr;
            if (attn_tc) {
                const size_t G = (size_t)t.gtot_max;
                CUDA_TRY(ctx, cudaMalloc(&t.Qf16, 2 * (size_t)M * G * sizeof(__half)));
                CUDA_TRY(ctx, cudaMemset(t.Qf16, 0, 2 * (size_t)M * G * sizeof(__half)));   // padded columns stay finite
                CUDA_TRY(ctx, cudaMalloc(&t.PfS, (size_t)kSplitsCap * 2 * M * G * sizeof(float)));
            }
            if (!ctx->use_fft) {   // f16 copies of the planes: operands of the tensor-core reconstruction
                const size_t cbytes = B * c.n_kv_heads * 2 * (size_t)M * kHeadDim * sizeof(__half);
                CUDA_TRY(ctx, cudaMalloc(&t.C16K, cbytes));
                CUDA_TRY(ctx, cudaMalloc(&t.C16V, cbytes));
            }
            t.max_M = M;
        }
    }
    return FAEDKV_OK;
}

// 3-D tiled tensor map with 128-byte swizzle and zero fill outside the tensor.
int make_map3(faedkv_ctx *ctx, CUtensorMap *map, const void *base, CUtensorMapDataType dt, size_t elem, uint64_t d0,
              uint64_t d1, uint64_t d2, uint64_t stride1_elems, uint64_t stride2_elems, uint32_t b0, uint32_t b1) {
    char msg[200];
    if (int r = umma_resolve_encode(ctx->umma, msg, sizeof(msg))) return fail(ctx, r, "%s", msg);
    cuuint64_t dims[3] = {d0, d1, d2};
    cuuint64_t strides[2] = {stride1_elems * elem, stride2_elems * elem};
    cuuint32_t box[3] = {b0, b1, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = ctx->umma.encode(map, dt, 3, const_cast<void *>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                  CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(ctx, FAEDKV_ERR_CUDA, "cuTensorMapEncodeTiled failed with code %d", (int)r);
    return FAEDKV_OK;
}

template <typename K>
int opt_in_smem(faedkv_ctx *ctx, K kernel, uint32_t bytes) {
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
    if (e != cudaSuccess) return fail(ctx, FAEDKV_ERR_CUDA, "cannot opt in to %u bytes of shared memory: %s", bytes, cudaGetErrorString(e));
    return FAEDKV_OK;
}

template <int NCOLS, int NT, int MODE>
int launch_idft(faedkv_ctx *ctx, const CUtensorMap &m0, const CUtensorMap &m1, const idft::Args &a, dim3 grid, cudaStream_t st) {
    using C = idft::Cfg<NCOLS, NT>;
    if (int r = opt_in_smem(ctx, k_idft_umma<NCOLS, NT, MODE>, C::kSmemBytes)) return r;
    k_idft_umma<NCOLS, NT, MODE><<<grid, idft::kThreads, C::kSmemBytes, st>>>(m0, m1, a);
    return launch_check(ctx, "k_idft_umma");
}

template <int NCOLS>
int launch_pspec(faedkv_ctx *ctx, const CUtensorMap &mp, const LayerPlan &p, int P, int rows_per_split, int Gtot, dim3 grid,
                 cudaStream_t st) {
    using C = pspec::Cfg<NCOLS>;
    if (int r = opt_in_smem(ctx, k_pspec_umma<NCOLS>, C::kSmemBytes)) return r;
    k_pspec_umma<NCOLS><<<grid, pspec::kThreads, C::kSmemBytes, st>>>(mp, p.d_bins, p.M, (uint32_t)P, rows_per_split, Gtot,
                                                                       ctx->tc.PfS, ctx->dev_status);
    return launch_check(ctx, "k_pspec_umma");
}

// Reconstruction on tensor cores (bf16 outputs): convert the planes to scaled f16, then one inverse-transform launch.
int launch_reconstruct_tc(faedkv_ctx *ctx, const LayerPlan &p, const float *coefK, const float *coefV, const int32_t *t_len,
                          int batch, int L, void *K_out, void *V_out, cudaStream_t st) {
    const faedkv_config &c = ctx->cfg;
    TcScratch &t = ctx->tc;
    const int units = batch * c.n_kv_heads, M = p.M, P = c.n_dft;
    const size_t n_vec = (size_t)units * 2 * M * kHeadDim / 8;
    const float *src[2] = {coefK, coefV};
    __half *dst[2] = {t.C16K, t.C16V};
    CUtensorMap maps[2];
    int nt = 0;
    void *outs[2] = {nullptr, nullptr};
    for (int i = 0; i < 2; ++i) {
        if (src[i] == nullptr) continue;
        k_coef_to_half<<<(unsigned)((n_vec + 255) / 256), 256, 0, st>>>(src[i], dst[nt], p.d_bins, M, (uint32_t)P, n_vec);
        if (int r = launch_check(ctx, "k_coef_to_half")) return r;
        if (int r = make_map3(ctx, &maps[nt], dst[nt], CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, kHeadDim, (uint64_t)M,
                              (uint64_t)units * 2, kHeadDim, (uint64_t)M * kHeadDim, 64, idft::kBinsPerStage))
            return r;
        outs[nt] = (i == 0) ? K_out : V_out;
        ++nt;
    }
    idft::Args a{};
    a.bins = p.d_bins; a.tab = p.d_tab; a.t_len = t_len; a.M = M; a.P = (uint32_t)P; a.Lrows = L;
    a.outK = outs[0]; a.outV = outs[1]; a.H = c.n_kv_heads; a.status = ctx->dev_status;
    if (nt == 2) {
        dim3 grid((L + 255) / 256, units);
        return launch_idft<256, 2, 0>(ctx, maps[0], maps[1], a, grid, st);
    }
    dim3 grid((L + 255) / 256, units);
    return launch_idft<128, 2, 0>(ctx, maps[0], maps[0], a, grid, st);
}

template <typename TQ, int GQ>
int launch_attn_tc(faedkv_ctx *ctx, const LayerPlan &p, const void *q, const float *coefK, const float *coefV,
                   const int32_t *t_len, int batch, float scale, void *out, cudaStream_t st) {
    const faedkv_config &c = ctx->cfg;
    TcScratch &t = ctx->tc;
    const int H = c.n_kv_heads, HQ = c.n_q_heads, M = p.M, P = c.n_dft;
    const int n_cols = batch * HQ;
    const int Gtot = (n_cols + 63) / 64 * 64;
    const int ncols = (Gtot % 256 == 0) ? 256 : (Gtot % 128 == 0) ? 128 : 64;
    const int col_blocks = Gtot / ncols;
    constexpr int KB = attn_bins_per_warp(GQ);
    // (1) scaled query spectrum in f16
    {
        dim3 grid((M + kAttnWarps * KB - 1) / (kAttnWarps * KB), batch * H);
        k_attn_qf16<TQ, GQ><<<grid, kAttnWarps * 32, 0, st>>>(static_cast<const TQ *>(q), coefK, p.d_bins, t.Qf16, M, H, HQ,
                                                              Gtot, (uint32_t)P, scale / (float)P);
        if (int r = launch_check(ctx, "k_attn_qf16")) return r;
    }
    // (2) scores
    {
        CUtensorMap mq;
        if (int r = make_map3(ctx, &mq, t.Qf16, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, (uint64_t)Gtot, (uint64_t)M, 2,
                              (uint64_t)Gtot, (uint64_t)M * Gtot, 64, idft::kBinsPerStage))
            return r;
        idft::Args a{};
        a.bins = p.d_bins; a.tab = p.d_tab; a.t_len = t_len; a.M = M; a.P = (uint32_t)P; a.Lrows = P;
        a.S = t.S; a.tile_max = t.tile_max; a.Gtot = Gtot; a.HQ = HQ; a.n_seq_cols = n_cols; a.status = ctx->dev_status;
        const int tiles2 = (P + 255) / 256;
        const bool two = tiles2 * col_blocks >= ctx->n_sm;
        dim3 grid(two ? tiles2 : (P + 127) / 128, col_blocks);
        int r;
        if (ncols == 256) r = two ? launch_idft<256, 2, 1>(ctx, mq, mq, a, grid, st) : launch_idft<256, 1, 1>(ctx, mq, mq, a, grid, st);
        else if (ncols == 128) r = two ? launch_idft<128, 2, 1>(ctx, mq, mq, a, grid, st) : launch_idft<128, 1, 1>(ctx, mq, mq, a, grid, st);
        else r = two ? launch_idft<64, 2, 1>(ctx, mq, mq, a, grid, st) : launch_idft<64, 1, 1>(ctx, mq, mq, a, grid, st);
        if (r) return r;
    }
    // (3) softmax numerators in f16 + normalisers
    const int n_groups = (P + 31) / 32, n_sblocks = (P + kSoftmaxRows - 1) / kSoftmaxRows;
    {
        k_colmax_par<<<Gtot / 32, 256, 0, st>>>(t.tile_max, n_groups, Gtot, t.cmax);
        if (int r = launch_check(ctx, "k_colmax_par")) return r;
        dim3 grid(n_sblocks, Gtot / 64);
        k_softmax_half<<<grid, 256, 0, st>>>(t.S, t.cmax, t_len, t.P16, t.psum, P, Gtot, HQ, n_cols);
        if (int r = launch_check(ctx, "k_softmax_half")) return r;
        k_colsum<<<Gtot / 32, 32, 0, st>>>(t.psum, n_sblocks, Gtot, t.colsum);
        if (int r = launch_check(ctx, "k_colsum")) return r;
    }
    // (4) probability spectrum, positions split over CTAs
    const int bin_tiles = (M + 127) / 128;
    int splits = (2 * ctx->n_sm + bin_tiles * col_blocks - 1) / (bin_tiles * col_blocks);
    if (splits > kSplitsCap) splits = kSplitsCap;
    if (splits > (P + 511) / 512) splits = (P + 511) / 512;
    if (splits < 1) splits = 1;
    const int rows_per_split = ((P + splits - 1) / splits + 63) / 64 * 64;
    {
        CUtensorMap mp;
        if (int r = make_map3(ctx, &mp, t.P16, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, (uint64_t)Gtot, (uint64_t)P, 1, (uint64_t)Gtot,
                              (uint64_t)P * Gtot, 64, pspec::kTileTok))
            return r;
        dim3 grid(bin_tiles, col_blocks, splits);
        int r;
        if (ncols == 256) r = launch_pspec<256>(ctx, mp, p, P, rows_per_split, Gtot, grid, st);
        else if (ncols == 128) r = launch_pspec<128>(ctx, mp, p, P, rows_per_split, Gtot, grid, st);
        else r = launch_pspec<64>(ctx, mp, p, P, rows_per_split, Gtot, grid, st);
        if (r) return r;
    }
    // (5) value stream
    {
        const int slices = out_slices(ctx, batch, M);
        const int per = (M + slices - 1) / slices;
        dim3 grid(slices, batch * H);
        k_attn_out2<GQ><<<grid, kAttnWarps * 32, 0, st>>>(coefV, t.PfS, p.d_bins, ctx->partial, M, H, HQ, Gtot, splits, (uint32_t)P, per);
        if (int r = launch_check(ctx, "k_attn_out2")) return r;
        k_attn_out_reduce2<TQ><<<batch * H * GQ, kHeadDim, 0, st>>>(ctx->partial, t.colsum, static_cast<TQ *>(out), slices, GQ,
                                                                   1.0f / (float)P);
        if (int r = launch_check(ctx, "k_attn_out_reduce2")) return r;
    }
    return FAEDKV_OK;
}

// Launch one of the three FFT kernels for a transform length of 2^lg rows.
#define FAEDKV_FFT_SWITCH(lg, lo, CALL)                                                     \
    switch (lg) {                                                                           \
        case 2: if (lo <= 2) { CALL(2); } break;                                            \
        case 3: CALL(3); break;                                                             \
        case 4: CALL(4); break;                                                             \
        case 5: CALL(5); break;                                                             \
        case 6: CALL(6); break;                                                             \
        case 7: CALL(7); break;                                                             \
        case 8: CALL(8); break;                                                             \
        case 9: CALL(9); break;                                                             \
        default: break;                                                                     \
    }

// The instance with compile-time tile indexing when the launch uses the tile shape it was built for,
// else the instance that takes the shape at run time.
#define FFT_PICK(KERNEL, LG, lg_t) ((lg_t) == fft::fast_lg_transforms(LG) ? KERNEL<LG, fft::fast_lg_transforms(LG)> : KERNEL<LG, -1>)
#define FFT_PICK_T(KERNEL, LG, lg_t, T) \
    ((lg_t) == fft::fast_lg_transforms(LG) ? KERNEL<LG, fft::fast_lg_transforms(LG), T> : KERNEL<LG, -1, T>)

// Launch with programmatic stream serialisation: the kernel may begin (up to its pdl_wait()) before the
// previous kernel of the stream has finished.
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

template <typename K>
int fft_opt_in(faedkv_ctx *ctx, K kernel, size_t bytes, unsigned int &done_mask, int lg) {
    if (bytes <= 48 * 1024 || (done_mask >> lg) & 1u) return FAEDKV_OK;
    if (int r = opt_in_smem(ctx, kernel, (uint32_t)bytes)) return r;
    done_mask |= 1u << lg;
    return FAEDKV_OK;
}

// FFT-shaped reconstruction of one tensor: pairs of (pass A, pass B) launches over runs of units.
template <typename TOut>
int launch_reconstruct_fft_tensor(faedkv_ctx *ctx, const LayerPlan &p, const float *coef, const int32_t *t_len, int units,
                                  int L, void *out, cudaStream_t st, ReconRows rows = ReconRows{0, -1, 0, 1}) {
    if (rows.unit_rows < 0) rows.unit_rows = L;
    const faedkv_config &c = ctx->cfg;
    FftScratch &f = ctx->fs;
    constexpr int kOutKind = sizeof(TOut) == 2 ? 4 : 5;
    for (int u0 = 0; u0 < units; u0 += f.recon_units) {
        const int uc = units - u0 < f.recon_units ? units - u0 : f.recon_units;
        const fft::Geometry g = fft::make_geometry(c.n_dft, uc * kHeadDim);
        const int col_blocks = g.Gp / fft::kCW;
        const int lgKT = fft::ilog2(fft::transforms_per_cta(g.N1, g.N2, col_blocks, ctx->n_sm));
        const int lgMT = fft::ilog2(fft::transforms_per_cta(g.N2, g.N1, col_blocks, ctx->n_sm));
        int rc = FAEDKV_ERR_UNSUPPORTED;
        {
            const dim3 grid(g.N2 >> lgKT, col_blocks);
            const size_t smem = afft_smem_a(g.lgN1, lgKT, true);
#define CALL(LG)                                                                                         \
            rc = fft_opt_in(ctx, FFT_PICK(k_rfft_inv_a, LG, lgKT), smem, f.attr_mask[3], LG + ((lgKT) == fft::fast_lg_transforms(LG) ? 16 : 0));                            \
            if (rc == 0) FFT_PICK(k_rfft_inv_a, LG, lgKT)<<<grid, fft::kThreads, smem, st>>>(g, p.d_slot, coef, p.M, u0, f.Yr, lgKT)
            FAEDKV_FFT_SWITCH(g.lgN1, 3, CALL)
#undef CALL
            if (rc) return rc == FAEDKV_ERR_UNSUPPORTED ? fail(ctx, rc, "no FFT kernel for 2^%d rows", g.lgN1) : rc;
            if (int r = launch_check(ctx, "k_rfft_inv_a")) return r;
        }
        rc = FAEDKV_ERR_UNSUPPORTED;
        {
            const dim3 grid(g.N1 >> lgMT, col_blocks);
            const size_t smem = rfft_smem_b(g.lgN2, lgMT);
#define CALL(LG)                                                                                         \
            rc = fft_opt_in(ctx, FFT_PICK_T(k_rfft_inv_b, LG, lgMT, TOut), smem, f.attr_mask[kOutKind], LG + ((lgMT) == fft::fast_lg_transforms(LG) ? 16 : 0));               \
            if (rc == 0) FFT_PICK_T(k_rfft_inv_b, LG, lgMT, TOut)<<<grid, fft::kThreads, smem, st>>>(g, f.Yr, t_len, c.n_kv_heads, u0, L, static_cast<TOut *>(out), lgMT, rows)
            FAEDKV_FFT_SWITCH(g.lgN2, 2, CALL)
#undef CALL
            if (rc) return rc == FAEDKV_ERR_UNSUPPORTED ? fail(ctx, rc, "no FFT kernel for 2^%d rows", g.lgN2) : rc;
            if (int r = launch_check(ctx, "k_rfft_inv_b")) return r;
        }
    }
    return FAEDKV_OK;
}

// Which reconstruction engine a call takes: the persistent one where it exists and is the faster of the two (measured:
// 1.3 - 1.4x faster up to 128 x 128 points per channel, slower at 256-point passes, whose radix-16 x 16 butterflies
// leave it three CTAs per SM), unless the configuration asks for the two-kernel engine.
bool use_recon2(const faedkv_ctx *ctx) {
    if (ctx->fs.r2_sync == nullptr || ctx->cfg.recon_engine == 1) return false;
    if (ctx->cfg.recon_engine == 2) return true;
    return ctx->cfg.n_dft <= (1 << 15);
}

// Second engine: both tensors, both passes, one persistent launch (k_recon2.cuh).
template <int LG1, int LG2, typename TOut>
int launch_recon2_t(faedkv_ctx *ctx, rfft2::Args &a, int inst, cudaStream_t st) {
    FftScratch &f = ctx->fs;
    constexpr size_t smem = rfft2::smem_bytes<LG1, LG2>();
    constexpr int kind = sizeof(TOut) == 2 ? 0 : 1;
    auto kernel = rfft2::k_recon2<LG1, LG2, TOut>;
    const unsigned int bit = 1u << (inst + 16 * kind);
    if (smem > 48 * 1024 && !(f.r2_attr & bit)) {
        if (int r = opt_in_smem(ctx, kernel, (uint32_t)smem)) return r;
        f.r2_attr |= bit;
    }
    int &occ = f.r2_ctas_per_sm[kind][inst];
    if (occ == 0) {
        CUDA_TRY(ctx, cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, kernel, rfft2::kThreads, smem));
        if (occ < 1) return fail(ctx, FAEDKV_ERR_CUDA, "the reconstruction kernel does not fit an SM");
    }
    constexpr int nA = (1 << LG2) >> rfft2::lg_per_tile(LG1, LG2), nB = (1 << LG1) >> rfft2::lg_per_tile(LG2, LG1);
    const int n_cb = a.n_tensors * a.units * (kHeadDim / rfft2::kCW);
    const long long n_items = (long long)n_cb * (nA + nB);
    long long grid = (long long)occ * ctx->n_sm;
    if (grid > n_items) grid = n_items;
    // pass B of a block is claimed `lag` blocks after its pass A: about the blocks the running CTAs span, plus one;
    // the ring of the array between the passes holds twice that (and must hold more than the lag)
    const size_t cb_bytes = ((size_t)1 << (LG1 + LG2)) * rfft2::kCP * sizeof(rfft2::C2);
    long long ring_max = (long long)(f.yr_bytes / cb_bytes);
    int lag = (int)((grid + nA - 1) / nA) + 1;
    if (ring_max < 2) return fail(ctx, FAEDKV_ERR_UNSUPPORTED, "two-pass array too small for the reconstruction ring");
    if (lag > ring_max - 1) lag = (int)ring_max - 1;
    if (lag > n_cb) lag = n_cb;
    long long ring = 2LL * lag + 2;
    if (ring > ring_max) ring = ring_max;
    a.lag = lag;
    a.ring = (int)ring;
    kernel<<<(unsigned)grid, rfft2::kThreads, smem, st>>>(a);
    return launch_check(ctx, "k_recon2");
}

template <typename TOut>
int launch_recon2(faedkv_ctx *ctx, const LayerPlan &p, const float *coefK, const float *coefV, const int32_t *t_len, int units,
                  int L, void *K_out, void *V_out, cudaStream_t st, ReconRows rows = ReconRows{0, -1, 0, 1}) {
    if (rows.unit_rows < 0) rows.unit_rows = L;
    const faedkv_config &c = ctx->cfg;
    FftScratch &f = ctx->fs;
    rfft2::Args a{};
    a.n_tensors = 0;
    if (coefK != nullptr) { a.coef[a.n_tensors] = coefK; a.out[a.n_tensors] = K_out; ++a.n_tensors; }
    if (coefV != nullptr) { a.coef[a.n_tensors] = coefV; a.out[a.n_tensors] = V_out; ++a.n_tensors; }
    a.units = units; a.M = p.M; a.H = c.n_kv_heads; a.Lrows = L;
    a.slot = p.d_slot; a.t_len = t_len; a.tabP = f.r2_tabP; a.tabI = f.r2_tabI;
    a.Y = reinterpret_cast<rfft2::C2 *>(f.Yr);
    a.sync = f.r2_sync; a.status = ctx->dev_status; a.rows = rows;
    const fft::Geometry g = fft::make_geometry(c.n_dft, kHeadDim);
#define R2CASE(L1, L2, INST) if (g.lgN1 == L1 && g.lgN2 == L2) return launch_recon2_t<L1, L2, TOut>(ctx, a, INST, st)
    R2CASE(3, 2, 0); R2CASE(3, 3, 1); R2CASE(4, 3, 2); R2CASE(4, 4, 3); R2CASE(5, 4, 4); R2CASE(5, 5, 5);
    R2CASE(6, 5, 6); R2CASE(6, 6, 7); R2CASE(7, 6, 8); R2CASE(7, 7, 9); R2CASE(8, 7, 10); R2CASE(8, 8, 11);
#undef R2CASE
    return fail(ctx, FAEDKV_ERR_UNSUPPORTED, "no reconstruction kernel for 2^%d x 2^%d points", g.lgN1, g.lgN2);
}

template <typename TOut>
int launch_reconstruct_fft(faedkv_ctx *ctx, const LayerPlan &p, const float *coefK, const float *coefV, const int32_t *t_len,
                           int batch, int L, void *K_out, void *V_out, cudaStream_t st) {
    const int units = batch * ctx->cfg.n_kv_heads;
    if (use_recon2(ctx))
        return launch_recon2<TOut>(ctx, p, coefK, coefV, t_len, units, L, K_out, V_out, st);
    if (coefK != nullptr)
        if (int r = launch_reconstruct_fft_tensor<TOut>(ctx, p, coefK, t_len, units, L, K_out, st)) return r;
    if (coefV != nullptr)
        if (int r = launch_reconstruct_fft_tensor<TOut>(ctx, p, coefV, t_len, units, L, V_out, st)) return r;
    return FAEDKV_OK;
}

// FFT-shaped prefill of one tensor: (pass A', pass B', gather) over runs of units.
template <typename TIn>
int launch_prefill_fft_tensor(faedkv_ctx *ctx, const LayerPlan &p, const void *x, int units, int T, int T_stride, float *coef,
                              cudaStream_t st) {
    const faedkv_config &c = ctx->cfg;
    FftScratch &f = ctx->fs;
    constexpr int kInKind = sizeof(TIn) == 2 ? 6 : 7;
    const int per = f.recon_units > 1 ? f.recon_units / 2 : 1;      // two arrays live at once: half the units each
    for (int u0 = 0; u0 < units; u0 += per) {
        const int uc = units - u0 < per ? units - u0 : per;
        const fft::Geometry g = fft::make_geometry(c.n_dft, uc * kHeadDim);
        const int col_blocks = g.Gp / fft::kCW;
        const int lgKT = fft::ilog2(fft::transforms_per_cta(g.N1, g.N2, col_blocks, ctx->n_sm));
        const int lgMT = fft::ilog2(fft::transforms_per_cta(g.N2, g.N1, col_blocks, ctx->n_sm));
        int rc = FAEDKV_ERR_UNSUPPORTED;
        {
            const dim3 grid(g.N1 >> lgMT, col_blocks);
            const size_t smem = pfft_smem_a(g.lgN2, lgMT);
#define CALL(LG)                                                                                         \
            rc = fft_opt_in(ctx, FFT_PICK_T(k_pfft_fwd_a, LG, lgMT, TIn), smem, f.attr_mask[kInKind], LG + ((lgMT) == fft::fast_lg_transforms(LG) ? 16 : 0));                 \
            if (rc == 0) FFT_PICK_T(k_pfft_fwd_a, LG, lgMT, TIn)<<<grid, fft::kThreads, smem, st>>>(g, static_cast<const TIn *>(x), T, T_stride, u0, f.Yr, lgMT)
            FAEDKV_FFT_SWITCH(g.lgN2, 2, CALL)
#undef CALL
            if (rc) return rc == FAEDKV_ERR_UNSUPPORTED ? fail(ctx, rc, "no FFT kernel for 2^%d rows", g.lgN2) : rc;
            if (int r = launch_check(ctx, "k_pfft_fwd_a")) return r;
        }
        rc = FAEDKV_ERR_UNSUPPORTED;
        {
            const dim3 grid(g.N2 >> lgKT, col_blocks);
            const size_t smem = pfft_smem_b(g.lgN1, lgKT);
#define CALL(LG)                                                                                         \
            rc = fft_opt_in(ctx, FFT_PICK(k_pfft_fwd_b, LG, lgKT), smem, f.attr_mask[8], LG + ((lgKT) == fft::fast_lg_transforms(LG) ? 16 : 0));                            \
            if (rc == 0) FFT_PICK(k_pfft_fwd_b, LG, lgKT)<<<grid, fft::kThreads, smem, st>>>(g, f.Yr, f.Zr, lgKT)
            FAEDKV_FFT_SWITCH(g.lgN1, 3, CALL)
#undef CALL
            if (rc) return rc == FAEDKV_ERR_UNSUPPORTED ? fail(ctx, rc, "no FFT kernel for 2^%d rows", g.lgN1) : rc;
            if (int r = launch_check(ctx, "k_pfft_fwd_b")) return r;
        }
        {
            const dim3 grid((p.M + 7) / 8, uc);
            k_pfft_gather<<<grid, 256, 0, st>>>(g, f.Zr, p.d_bins, p.M, u0, coef);
            if (int r = launch_check(ctx, "k_pfft_gather")) return r;
        }
    }
    return FAEDKV_OK;
}

// Steps (2)-(4) through the two-column kernels (k_attn_fft2.cuh).  `join`: event to wait for before the last kernel
// (the window statistics), or nullptr.
template <int LG1, int LG2>
int launch_afft2_t(faedkv_ctx *ctx, int inst, const fft::Geometry &g, const LayerPlan &p, const int32_t *t_len, int HQ, int t_add,
                   int t_quant, int n_extra, cudaEvent_t join, cudaStream_t st) {
    FftScratch &f = ctx->fs;
    constexpr int lgKT = afft2::lg_per_tile(LG1, LG2), lgMT = afft2::lg_per_tile(LG2, LG1);
    const afft2::Tables tb{f.r2_tabP, f.a2_tabI};
    rfft2::C2 *Y2 = reinterpret_cast<rfft2::C2 *>(f.Y);
    const int n_cb = g.Gp / afft2::kCW;
    const unsigned int bit = 1u << inst;
    constexpr size_t sa = afft2::smem_a<LG1, LG2>(), sm = afft2::smem_mid<LG1, LG2>(), sf = afft2::smem_fwd_b<LG1, LG2>();
    if (sa > 48 * 1024 && !(f.a2_attr[0] & bit)) { if (int r = opt_in_smem(ctx, afft2::k_afft2_inv_a<LG1, LG2>, (uint32_t)sa)) return r; f.a2_attr[0] |= bit; }
    if (sm > 48 * 1024 && !(f.a2_attr[1] & bit)) { if (int r = opt_in_smem(ctx, afft2::k_afft2_mid<LG1, LG2>, (uint32_t)sm)) return r; f.a2_attr[1] |= bit; }
    if (sf > 48 * 1024 && !(f.a2_attr[2] & bit)) { if (int r = opt_in_smem(ctx, afft2::k_afft2_fwd_b<LG1, LG2>, (uint32_t)sf)) return r; f.a2_attr[2] |= bit; }
    launch_pdl(afft2::k_afft2_inv_a<LG1, LG2>, dim3((1 << LG2) >> lgKT, n_cb), dim3(afft2::kThreads), sa, st, g.Gp, p.d_slot, f.Qs, tb, Y2);
    if (int r = launch_check(ctx, "k_afft2_inv_a")) return r;
    launch_pdl(afft2::k_afft2_mid<LG1, LG2>, dim3((1 << LG1) >> lgMT, n_cb), dim3(afft2::kThreads), sm, st, g.Gp, g.G, Y2, tb, t_len, HQ,
               t_add, t_quant, f.mloc, f.sloc);
    if (int r = launch_check(ctx, "k_afft2_mid")) return r;
    if (join != nullptr) CUDA_TRY(ctx, cudaStreamWaitEvent(st, join, 0));
    launch_pdl(afft2::k_afft2_fwd_b<LG1, LG2>, dim3((1 << LG2) >> lgKT, n_cb), dim3(afft2::kThreads), sf, st, g.Gp, Y2, tb, f.mloc, f.sloc,
               f.Zf, f.colsum, n_extra);
    return launch_check(ctx, "k_afft2_fwd_b");
}

// Whether the two-pass transforms of decode attention take the two-column kernels, and how many softmax tiles they make.
bool use_afft2(const faedkv_ctx *ctx, const fft::Geometry &g) { return ctx->fs.a2_tabI != nullptr && g.lgN1 <= afft2::kMaxLg; }

int launch_afft2(faedkv_ctx *ctx, const fft::Geometry &g, const LayerPlan &p, const int32_t *t_len, int HQ, int t_add, int t_quant,
                 int n_extra, cudaEvent_t join, cudaStream_t st) {
#define A2CASE(L1, L2, INST) if (g.lgN1 == L1 && g.lgN2 == L2) return launch_afft2_t<L1, L2>(ctx, INST, g, p, t_len, HQ, t_add, t_quant, n_extra, join, st)
    A2CASE(3, 2, 0); A2CASE(3, 3, 1); A2CASE(4, 3, 2); A2CASE(4, 4, 3); A2CASE(5, 4, 4); A2CASE(5, 5, 5);
    A2CASE(6, 5, 6); A2CASE(6, 6, 7); A2CASE(7, 6, 8); A2CASE(7, 7, 9); A2CASE(8, 7, 10); A2CASE(8, 8, 11);
#undef A2CASE
    return fail(ctx, FAEDKV_ERR_UNSUPPORTED, "no two-column transform for 2^%d x 2^%d points", g.lgN1, g.lgN2);
}

// FFT-shaped decode attention; with APPEND the IWDFT update of K and V rides on the two coefficient
// streams and the token counters advance at the end.
// A windowed step (winK != nullptr) folds the token leaving the recent ring instead of the new one, lets the
// sink + recent tokens join the softmax as one more tile, and ends by committing the new token to the ring.
template <typename TQ, int GQ, bool APPEND>
int launch_attn_fft(faedkv_ctx *ctx, const LayerPlan &p, const void *q, const void *k_new, const void *v_new,
                    float *coefK, float *coefV, int32_t *t_len, int batch, float scale, void *out, cudaStream_t st,
                    void *winK = nullptr, void *winV = nullptr) {
    const faedkv_config &c = ctx->cfg;
    FftScratch &f = ctx->fs;
    const bool windowed = winK != nullptr;
    const int S = windowed ? c.n_sink : 0, R = windowed ? c.n_recent : 0;
    // block-deferred fold (D > 1, APPEND == false): the caller has folded already; this call attends over the
    // whole blocks in the planes plus every waiting token, then commits the new token and advances t_len
    const int D = windowed ? c.n_defer : 1, Rc = win_ring(R, D);
    const bool counts_new = APPEND || D > 1;
    const int n_extra = (windowed && (S + R > 0 || D > 1)) ? 1 : 0;
    // the folded token: the call's new token, or with a ring the token that leaves it
    const FoldSrc fold{(windowed && R > 0) ? S + R : 1, S, R};
    const void *foldK = (windowed && R > 0) ? winK : k_new, *foldV = (windowed && R > 0) ? winV : v_new;
    const int H = c.n_kv_heads, HQ = c.n_q_heads, M = p.M, P = c.n_dft;
    const fft::Geometry g = fft::make_geometry(P, batch * HQ);
    const int col_blocks = g.Gp / fft::kCW;
    const bool two_col = !ctx->use_col && use_afft2(ctx, g);
    const int lgKT = fft::ilog2(fft::transforms_per_cta(g.N1, g.N2, col_blocks, ctx->n_sm));
    const int lgMT = two_col ? afft2::lg_per_tile(g.lgN2, g.lgN1) : fft::ilog2(fft::transforms_per_cta(g.N2, g.N1, col_blocks, ctx->n_sm));
    constexpr int KB = attn_bins_per_warp(GQ);
    // step (5) for the sequences [b0, b1) on stream s
    auto launch_out = [&](int b0, int b1, cudaStream_t s) -> int {
        const int nb = b1 - b0;
        const int slices = out_slices(ctx, nb, M);
        // one stride for every launch of the call, whatever its own slice count: runs never share a partial slot
        const int slice_stride = ctx->out_slices_cap;
        const int per = (M + slices - 1) / slices;
        dim3 grid(slices, nb * H);
        launch_pdl(k_attn_out_fft<TQ, GQ, APPEND>, grid, dim3(kAttnWarps * 32), 0, s,
                   coefV, static_cast<const TQ *>(foldV), t_len, f.Zf, f.colsum, p.d_bins, ctx->partial, f.tickets,
                   static_cast<TQ *>(out), M, H, HQ, g, per, 1.0f / (float)P, fold, n_extra ? f.o_win : nullptr, counts_new ? 1 : 0,
                   windowed ? WindowArgs{winK, winV, k_new, v_new, S, R, D, Rc, 0.f, nullptr, nullptr, nullptr} : WindowArgs{},
                   ctx->use_col ? f.Wg : nullptr, b0 * H, batch * H, slice_stride);
        return launch_check(ctx, "k_attn_out_fft");
    };
    if (n_extra) {
        // the window's scores, statistics (one more "tile" row) and unnormalised output depend on nothing this call
        // computes: they run on the context's second stream from the top of the call, beside the pass over
        // C_K, and are joined before the kernel that reads the statistics
        const int n_tiles = g.N1 >> lgMT;
        const WindowArgs wa{winK, winV, k_new, v_new, S, R, D, Rc, scale, f.mloc + (size_t)n_tiles * g.Gp,
                            f.sloc + (size_t)n_tiles * g.Gp, f.o_win};
        CUDA_TRY(ctx, cudaEventRecord(f.ev_fork, st));
        CUDA_TRY(ctx, cudaStreamWaitEvent(f.side, f.ev_fork, 0));
        k_attn_window<TQ, GQ><<<dim3(batch * H, GQ), kWinWarps * 32, 0, f.side>>>(static_cast<const TQ *>(q), wa, t_len, H);
        if (int r = launch_check(ctx, "k_attn_window")) return r;
        CUDA_TRY(ctx, cudaEventRecord(f.ev_join, f.side));
    }
    {
        dim3 grid((M + kAttnWarps * KB - 1) / (kAttnWarps * KB), batch * H);
        k_attn_qs<TQ, GQ, APPEND><<<grid, kAttnWarps * 32, 0, st>>>(
            static_cast<const TQ *>(q), coefK, static_cast<const TQ *>(foldK), t_len, p.d_bins, f.Qs, M, H, HQ, g.Gp,
            (uint32_t)P, scale / (float)P, fold, ctx->use_col ? 1 : 0);
        if (int r = launch_check(ctx, "k_attn_qs")) return r;
    }
    int rc = FAEDKV_ERR_UNSUPPORTED;
    if (ctx->use_col) {
        // steps (2)-(4) in one kernel: a CTA per column holds the whole packed signal in shared memory
        if (n_extra) CUDA_TRY(ctx, cudaStreamWaitEvent(st, f.ev_join, 0));
        const int n_tiles = g.N1 >> lgMT;
        const float *m_w = n_extra ? f.mloc + (size_t)n_tiles * g.Gp : nullptr, *s_w = n_extra ? f.sloc + (size_t)n_tiles * g.Gp : nullptr;
        // With more columns than the GPU holds at once (two CTAs per SM at 8192 points) the last wave of the column kernel leaves
        // SMs idle and the whole kernel leaves DRAM idle: the batch is then cut into two runs of sequences, each
        // with its own column kernel and pass over C_V, the second on another stream, so that the first run's
        // pass over C_V streams while the second run's columns are still being transformed.
        const int lgn = g.lgN1 + g.lgN2;
        const int ctas_per_sm = lgn >= 13 ? 2 : (lgn == 12 ? 3 : (lgn == 11 ? 7 : 16));   // registers / shared memory
        const int b_cut = (batch >= 2 && batch * HQ > ctas_per_sm * ctx->n_sm) ? batch / 2 : batch;
        auto launch_col = [&](int b0, int b1, cudaStream_t s) -> int {
            int rcc = FAEDKV_ERR_UNSUPPORTED;
#define CALL(LG)                                                                                         \
            rcc = fft_opt_in(ctx, colfft::k_afft_col<LG>, colfft::smem_bytes<LG>(), f.attr_mask[10], LG);  \
            if (rcc == 0) launch_pdl(colfft::k_afft_col<LG>, dim3((b1 - b0) * HQ), dim3(colfft::threads<LG>()), colfft::smem_bytes<LG>(), s, \
                                     (uint32_t)P, M, p.d_bins, f.Qs, f.colE, f.colB, f.colP, t_len, HQ,   \
                                     (counts_new ? 1 : 0) - S - R, D, m_w, s_w, f.Wg, f.colsum, g.Gp, b0 * HQ)
            switch (g.lgN1 + g.lgN2) {
                case 5: CALL(5); break;
                case 6: CALL(6); break;
                case 7: CALL(7); break;
                case 8: CALL(8); break;
                case 9: CALL(9); break;
                case 10: CALL(10); break;
                case 11: CALL(11); break;
                case 12: CALL(12); break;
                case 13: CALL(13); break;
                default: break;
            }
#undef CALL
            if (rcc) return rcc == FAEDKV_ERR_UNSUPPORTED ? fail(ctx, rcc, "no column kernel for 2^%d points", g.lgN1 + g.lgN2) : rcc;
            return launch_check(ctx, "k_afft_col");
        };
        if (b_cut < batch) {
            CUDA_TRY(ctx, cudaEventRecord(f.ev_cut, st));
            CUDA_TRY(ctx, cudaStreamWaitEvent(f.side2, f.ev_cut, 0));
        }
        if (int r = launch_col(0, b_cut, st)) return r;
        if (b_cut < batch) {
            if (int r = launch_col(b_cut, batch, f.side2)) return r;
        }
        if (int r = launch_out(0, b_cut, st)) return r;
        if (b_cut < batch) {
            if (int r = launch_out(b_cut, batch, f.side2)) return r;
            CUDA_TRY(ctx, cudaEventRecord(f.ev_merge, f.side2));
            CUDA_TRY(ctx, cudaStreamWaitEvent(st, f.ev_merge, 0));
        }
        rc = FAEDKV_OK;
    } else if (two_col) {
        if (int r = launch_afft2(ctx, g, p, t_len, HQ, (counts_new ? 1 : 0) - S - R, D, n_extra, n_extra ? f.ev_join : nullptr, st)) return r;
    } else {
    rc = FAEDKV_ERR_UNSUPPORTED;
    {
        const dim3 grid(g.N2 >> lgKT, col_blocks);
        const size_t smem = afft_smem_a(g.lgN1, lgKT, true);
#define CALL(LG)                                                                                         \
        rc = fft_opt_in(ctx, FFT_PICK(k_afft_inv_a, LG, lgKT), smem, f.attr_mask[0], LG + ((lgKT) == fft::fast_lg_transforms(LG) ? 16 : 0));                                \
        if (rc == 0) launch_pdl(FFT_PICK(k_afft_inv_a, LG, lgKT), grid, dim3(fft::kThreads), smem, st, g, p.d_slot, f.Qs, f.Y, lgKT)
        FAEDKV_FFT_SWITCH(g.lgN1, 3, CALL)
#undef CALL
        if (rc) return rc == FAEDKV_ERR_UNSUPPORTED ? fail(ctx, rc, "no FFT kernel for 2^%d rows", g.lgN1) : rc;
        if (int r = launch_check(ctx, "k_afft_inv_a")) return r;
    }
    rc = FAEDKV_ERR_UNSUPPORTED;
    {
        const dim3 grid(g.N1 >> lgMT, col_blocks);
        const size_t smem = afft_smem_mid(g.lgN2, lgMT);
#define CALL(LG)                                                                                         \
        rc = fft_opt_in(ctx, FFT_PICK(k_afft_mid, LG, lgMT), smem, f.attr_mask[1], LG + ((lgMT) == fft::fast_lg_transforms(LG) ? 16 : 0));                                  \
        if (rc == 0) launch_pdl(FFT_PICK(k_afft_mid, LG, lgMT), grid, dim3(fft::kThreads), smem, st, g, f.Y, t_len, HQ, (counts_new ? 1 : 0) - S - R, D, f.mloc, f.sloc, lgMT)
        FAEDKV_FFT_SWITCH(g.lgN2, 2, CALL)
#undef CALL
        if (rc) return rc == FAEDKV_ERR_UNSUPPORTED ? fail(ctx, rc, "no FFT kernel for 2^%d rows", g.lgN2) : rc;
        if (int r = launch_check(ctx, "k_afft_mid")) return r;
    }
    if (n_extra) CUDA_TRY(ctx, cudaStreamWaitEvent(st, f.ev_join, 0));
    rc = FAEDKV_ERR_UNSUPPORTED;
    {
        const dim3 grid(g.N2 >> lgKT, col_blocks);
        const size_t smem = afft_smem_fwd_b(g.lgN1, lgKT, lgMT);
#define CALL(LG)                                                                                         \
        rc = fft_opt_in(ctx, FFT_PICK(k_afft_fwd_b, LG, lgKT), smem, f.attr_mask[2], LG + ((lgKT) == fft::fast_lg_transforms(LG) ? 16 : 0));                                \
        if (rc == 0) launch_pdl(FFT_PICK(k_afft_fwd_b, LG, lgKT), grid, dim3(fft::kThreads), smem, st, g, f.Y, f.mloc, f.sloc, lgMT, f.Zf, f.colsum, lgKT, n_extra)
        FAEDKV_FFT_SWITCH(g.lgN1, 3, CALL)
#undef CALL
        if (rc) return rc == FAEDKV_ERR_UNSUPPORTED ? fail(ctx, rc, "no FFT kernel for 2^%d rows", g.lgN1) : rc;
        if (int r = launch_check(ctx, "k_afft_fwd_b")) return r;
    }
    }
    if (!ctx->use_col) {
        if (int r = launch_out(0, batch, st)) return r;
    }
    return FAEDKV_OK;
}

template <typename TQ, bool APPEND>
int dispatch_attn_fft(faedkv_ctx *ctx, const LayerPlan &p, const void *q, const void *k_new, const void *v_new,
                      float *coefK, float *coefV, int32_t *t_len, int batch, float scale, void *out, cudaStream_t st,
                      void *winK = nullptr, void *winV = nullptr) {
    switch (ctx->gq) {
        case 1: return launch_attn_fft<TQ, 1, APPEND>(ctx, p, q, k_new, v_new, coefK, coefV, t_len, batch, scale, out, st, winK, winV);
        case 2: return launch_attn_fft<TQ, 2, APPEND>(ctx, p, q, k_new, v_new, coefK, coefV, t_len, batch, scale, out, st, winK, winV);
        case 3: return launch_attn_fft<TQ, 3, APPEND>(ctx, p, q, k_new, v_new, coefK, coefV, t_len, batch, scale, out, st, winK, winV);
        case 4: return launch_attn_fft<TQ, 4, APPEND>(ctx, p, q, k_new, v_new, coefK, coefV, t_len, batch, scale, out, st, winK, winV);
        case 5: return launch_attn_fft<TQ, 5, APPEND>(ctx, p, q, k_new, v_new, coefK, coefV, t_len, batch, scale, out, st, winK, winV);
        case 6: return launch_attn_fft<TQ, 6, APPEND>(ctx, p, q, k_new, v_new, coefK, coefV, t_len, batch, scale, out, st, winK, winV);
        case 7: return launch_attn_fft<TQ, 7, APPEND>(ctx, p, q, k_new, v_new, coefK, coefV, t_len, batch, scale, out, st, winK, winV);
        case 8: return launch_attn_fft<TQ, 8, APPEND>(ctx, p, q, k_new, v_new, coefK, coefV, t_len, batch, scale, out, st, winK, winV);
    }
    return fail(ctx, FAEDKV_ERR_UNSUPPORTED, "query heads per kv head must be between 1 and 8");
}

__global__ void k_set_tlen(int32_t *t_len, int batch, int T) {
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < batch) t_len[i] = T;
}

template <typename TIn>
int launch_prefill_simt(faedkv_ctx *ctx, const LayerPlan &p, const void *K, const void *V, int batch,
                        int T, int T_stride, float *coefK, float *coefV, cudaStream_t st) {
    const faedkv_config &c = ctx->cfg;
    DftUnitArgs a{};
    a.x[0] = K; a.x[1] = V;
    a.y[0] = coefK; a.y[1] = coefV;
    a.x_unit = (long long)T_stride * kHeadDim;
    a.y_unit = 2LL * p.M * kHeadDim;
    a.y_plane = (long long)p.M * kHeadDim;
    a.x_row = kHeadDim; a.y_row = kHeadDim; a.col_blocks = 1;
    dim3 grid((p.M + kTileBins - 1) / kTileBins, batch * c.n_kv_heads, 2);
    k_dft_forward_simt<TIn, kHeadDim, false><<<grid, kSimtThreads, 0, st>>>(
        a, p.d_bins, p.M, (uint32_t)c.n_dft, T, nullptr, 1, 0u, -1.0f, 0, nullptr);
    return launch_check(ctx, "k_dft_forward_simt");
}

template <typename TOut>
int launch_reconstruct(faedkv_ctx *ctx, const LayerPlan &p, const float *coefK, const float *coefV,
                       const int32_t *t_len, int batch, int L, void *K_out, void *V_out, cudaStream_t st) {
    const faedkv_config &c = ctx->cfg;
    DftUnitArgs a{};
    int nt = 0;
    if (coefK != nullptr) { a.x[nt] = K_out; a.y[nt] = const_cast<float *>(coefK); ++nt; }
    if (coefV != nullptr) { a.x[nt] = V_out; a.y[nt] = const_cast<float *>(coefV); ++nt; }
    a.x_unit = (long long)L * kHeadDim;
    a.y_unit = 2LL * p.M * kHeadDim;
    a.y_plane = (long long)p.M * kHeadDim;
    a.x_row = kHeadDim; a.y_row = kHeadDim; a.col_blocks = 1;
    dim3 grid((L + kTilePos - 1) / kTilePos, batch * c.n_kv_heads, nt);
    k_dft_inverse_simt<TOut, kHeadDim><<<grid, kSimtThreads, 0, st>>>(
        a, p.d_bins, p.M, (uint32_t)c.n_dft, L, t_len, c.n_kv_heads, 1.0f / (float)c.n_dft, nullptr);
    return launch_check(ctx, "k_dft_inverse_simt");
}

template <typename TQ, int GQ>
int launch_attn(faedkv_ctx *ctx, const LayerPlan &p, const void *q, const float *coefK,
                const float *coefV, const int32_t *t_len, int batch, float scale, void *out,
                cudaStream_t st) {
    const faedkv_config &c = ctx->cfg;
    const int H = c.n_kv_heads, HQ = c.n_q_heads, HQP = ctx->hqp, M = p.M, P = c.n_dft;
    const int col_blocks = HQP / 32;
    constexpr int KB = attn_bins_per_warp(GQ);
    // (1) query spectrum
    {
        dim3 grid((M + kAttnWarps * KB - 1) / (kAttnWarps * KB), batch * H);
        k_attn_qf<TQ, GQ><<<grid, kAttnWarps * 32, 0, st>>>(static_cast<const TQ *>(q), coefK, ctx->Qf, M, H, HQ, HQP);
        if (int r = launch_check(ctx, "k_attn_qf")) return r;
    }
    // (2) scores over positions, with per-tile column maxima
    const int n_tiles = (P + kTilePos - 1) / kTilePos;
    {
        DftUnitArgs a{};
        a.x[0] = ctx->S; a.y[0] = ctx->Qf;
        a.x_unit = (long long)P * HQP;
        a.y_unit = 2LL * M * HQP;
        a.y_plane = (long long)M * HQP;
        a.x_row = HQP; a.y_row = HQP; a.col_blocks = col_blocks;
        dim3 grid(n_tiles, batch * col_blocks, 1);
        k_dft_inverse_simt<float, 32><<<grid, kSimtThreads, 0, st>>>(
            a, p.d_bins, M, (uint32_t)P, P, t_len, 1, scale / (float)P, ctx->tile_max);
        if (int r = launch_check(ctx, "k_dft_inverse_simt(scores)")) return r;
        k_colmax<<<batch * col_blocks, 32, 0, st>>>(ctx->tile_max, n_tiles, 32, ctx->colmax);
        if (int r = launch_check(ctx, "k_colmax")) return r;
    }
    // (3)+(4) softmax fused into the forward transform of the probabilities
    {
        DftUnitArgs a{};
        a.x[0] = ctx->S; a.y[0] = ctx->Pf;
        a.x_unit = (long long)P * HQP;
        a.y_unit = 2LL * M * HQP;
        a.y_plane = (long long)M * HQP;
        a.x_row = HQP; a.y_row = HQP; a.col_blocks = col_blocks;
        dim3 grid((M + kTileBins - 1) / kTileBins, batch * col_blocks, 1);
        k_dft_forward_simt<float, 32, true><<<grid, kSimtThreads, 0, st>>>(
            a, p.d_bins, M, (uint32_t)P, 0, t_len, 1, 0u, 1.0f, 0, ctx->colmax);
        if (int r = launch_check(ctx, "k_dft_forward_simt(probabilities)")) return r;
    }
    // (5) value stream
    {
        const int slices = out_slices(ctx, batch, M);
        const int per = (M + slices - 1) / slices;
        dim3 grid(slices, batch * H);
        k_attn_out<GQ><<<grid, kAttnWarps * 32, 0, st>>>(coefV, ctx->Pf, p.d_bins, ctx->partial, M, H, HQP, (uint32_t)P, per);
        if (int r = launch_check(ctx, "k_attn_out")) return r;
        k_attn_out_reduce<TQ><<<batch * H * GQ, kHeadDim, 0, st>>>(ctx->partial, static_cast<TQ *>(out), slices, GQ, 1.0f / (float)P);
        if (int r = launch_check(ctx, "k_attn_out_reduce")) return r;
    }
    return FAEDKV_OK;
}

// The prefill transform of rows [0, T) of every unit of K and V (units T_stride rows apart) into the planes,
// by whichever evaluation the context was configured for.
int prefill_core(faedkv_ctx *ctx, const LayerPlan &p, const void *K, const void *V, int batch, int T, int T_stride,
                 float *coefK, float *coefV, cudaStream_t st) {
    const faedkv_config &c = ctx->cfg;
    int mode = c.prefill_mode;
    if (mode == FAEDKV_PREFILL_AUTO)
        mode = (c.kv_dtype == FAEDKV_BF16 && umma_prefill_available()) ? FAEDKV_PREFILL_UMMA : FAEDKV_PREFILL_SIMT;
    if (ctx->prefill_fft) {
        const int units = batch * c.n_kv_heads;
        if (c.kv_dtype == FAEDKV_BF16) {
            if (int r = launch_prefill_fft_tensor<__nv_bfloat16>(ctx, p, K, units, T, T_stride, coefK, st)) return r;
            return launch_prefill_fft_tensor<__nv_bfloat16>(ctx, p, V, units, T, T_stride, coefV, st);
        }
        if (int r = launch_prefill_fft_tensor<float>(ctx, p, K, units, T, T_stride, coefK, st)) return r;
        return launch_prefill_fft_tensor<float>(ctx, p, V, units, T, T_stride, coefV, st);
    }
    if (mode == FAEDKV_PREFILL_UMMA) {
        char msg[256] = {0};
        int r = umma_prefill_launch(ctx->umma, K, V, batch, c.n_kv_heads, T, T_stride, p.d_bins, p.M, c.n_dft,
                                    c.twiddle_terms == 2 ? 2 : 1, coefK, coefV, ctx->dev_status, st, msg, sizeof(msg));
        if (r != 0) return fail(ctx, r, "%s", msg);
        ctx->launches += 1;
        return FAEDKV_OK;
    }
    if (c.kv_dtype == FAEDKV_BF16) return launch_prefill_simt<__nv_bfloat16>(ctx, p, K, V, batch, T, T_stride, coefK, coefV, st);
    return launch_prefill_simt<float>(ctx, p, K, V, batch, T, T_stride, coefK, coefV, st);
}

template <typename TQ>
int dispatch_attn(faedkv_ctx *ctx, const LayerPlan &p, const void *q, const float *coefK,
                  const float *coefV, const int32_t *t_len, int batch, float scale, void *out,
                  cudaStream_t st) {
    if (ctx->use_fft)
        return dispatch_attn_fft<TQ, false>(ctx, p, q, nullptr, nullptr, const_cast<float *>(coefK), const_cast<float *>(coefV),
                                            const_cast<int32_t *>(t_len), batch, scale, out, st);
    if (ctx->use_tc) {
        switch (ctx->gq) {
            case 1: return launch_attn_tc<TQ, 1>(ctx, p, q, coefK, coefV, t_len, batch, scale, out, st);
            case 2: return launch_attn_tc<TQ, 2>(ctx, p, q, coefK, coefV, t_len, batch, scale, out, st);
            case 3: return launch_attn_tc<TQ, 3>(ctx, p, q, coefK, coefV, t_len, batch, scale, out, st);
            case 4: return launch_attn_tc<TQ, 4>(ctx, p, q, coefK, coefV, t_len, batch, scale, out, st);
            case 5: return launch_attn_tc<TQ, 5>(ctx, p, q, coefK, coefV, t_len, batch, scale, out, st);
            case 6: return launch_attn_tc<TQ, 6>(ctx, p, q, coefK, coefV, t_len, batch, scale, out, st);
            case 7: return launch_attn_tc<TQ, 7>(ctx, p, q, coefK, coefV, t_len, batch, scale, out, st);
            case 8: return launch_attn_tc<TQ, 8>(ctx, p, q, coefK, coefV, t_len, batch, scale, out, st);
        }
    }
    switch (ctx->gq) {
        case 1: return launch_attn<TQ, 1>(ctx, p, q, coefK, coefV, t_len, batch, scale, out, st);
        case 2: return launch_attn<TQ, 2>(ctx, p, q, coefK, coefV, t_len, batch, scale, out, st);
        case 3: return launch_attn<TQ, 3>(ctx, p, q, coefK, coefV, t_len, batch, scale, out, st);
        case 4: return launch_attn<TQ, 4>(ctx, p, q, coefK, coefV, t_len, batch, scale, out, st);
        case 5: return launch_attn<TQ, 5>(ctx, p, q, coefK, coefV, t_len, batch, scale, out, st);
        case 6: return launch_attn<TQ, 6>(ctx, p, q, coefK, coefV, t_len, batch, scale, out, st);
        case 7: return launch_attn<TQ, 7>(ctx, p, q, coefK, coefV, t_len, batch, scale, out, st);
        case 8: return launch_attn<TQ, 8>(ctx, p, q, coefK, coefV, t_len, batch, scale, out, st);
    }
    return fail(ctx, FAEDKV_ERR_UNSUPPORTED, "query heads per kv head must be between 1 and 8");
}

}  // namespace

// ------------------------------------------------------------------------------------------------
extern "C" {

int faedkv_create(const faedkv_config *cfg, faedkv_ctx **out) {
    if (cfg == nullptr || out == nullptr) return FAEDKV_ERR_INVALID_ARG;
    *out = nullptr;
    if (cfg->n_layers < 1 || cfg->n_kv_heads < 1 || cfg->n_q_heads < 1 || cfg->max_batch < 1 ||
        cfg->n_dft < 2 || cfg->n_dft > (1 << 24))
        return FAEDKV_ERR_INVALID_ARG;
    if (cfg->kv_dtype != FAEDKV_F32 && cfg->kv_dtype != FAEDKV_BF16) return FAEDKV_ERR_INVALID_ARG;
    if (cfg->prefill_mode < FAEDKV_PREFILL_AUTO || cfg->prefill_mode > FAEDKV_PREFILL_FFT) return FAEDKV_ERR_INVALID_ARG;
    if (cfg->twiddle_terms < 0 || cfg->twiddle_terms > 2) return FAEDKV_ERR_INVALID_ARG;
    if (cfg->decode_mode < FAEDKV_DECODE_AUTO || cfg->decode_mode > FAEDKV_DECODE_FFT_TWO_PASS) return FAEDKV_ERR_INVALID_ARG;
    if (cfg->decode_mode == FAEDKV_DECODE_UMMA && cfg->kv_dtype != FAEDKV_BF16) return FAEDKV_ERR_UNSUPPORTED;
    if ((cfg->decode_mode == FAEDKV_DECODE_FFT || cfg->decode_mode == FAEDKV_DECODE_FFT_TWO_PASS) && !fft::supported(cfg->n_dft))
        return FAEDKV_ERR_UNSUPPORTED;
    if (cfg->n_sink < 0 || cfg->n_recent < 0 || cfg->n_sink + cfg->n_recent > 1024) return FAEDKV_ERR_INVALID_ARG;
    if (cfg->n_defer < 0 || cfg->n_defer > 128) return FAEDKV_ERR_INVALID_ARG;
    if (cfg->recon_engine < 0 || cfg->recon_engine > 2) return FAEDKV_ERR_INVALID_ARG;
    if (cfg->head_dim != kHeadDim) return FAEDKV_ERR_UNSUPPORTED;
    if (cfg->n_q_heads % cfg->n_kv_heads != 0) return FAEDKV_ERR_UNSUPPORTED;
    const int gq = cfg->n_q_heads / cfg->n_kv_heads;
    if (gq < 1 || gq > 8) return FAEDKV_ERR_UNSUPPORTED;
    // units and column blocks index gridDim.y
    if ((long long)cfg->max_batch * cfg->n_kv_heads > 65535 || (long long)cfg->max_batch * cfg->n_q_heads / 16 > 65535)
        return FAEDKV_ERR_UNSUPPORTED;
    if (cfg->prefill_mode == FAEDKV_PREFILL_UMMA && cfg->kv_dtype != FAEDKV_BF16) return FAEDKV_ERR_UNSUPPORTED;

    faedkv_ctx *ctx = new (std::nothrow) faedkv_ctx();
    if (ctx == nullptr) return FAEDKV_ERR_INVALID_ARG;
    ctx->cfg = *cfg;
    ctx->gq = gq;
    ctx->hqp = (cfg->n_q_heads + 31) / 32 * 32;
    ctx->use_tc = cfg->kv_dtype == FAEDKV_BF16 && cfg->decode_mode != FAEDKV_DECODE_SIMT;
    const bool fft_ok = fft::supported(cfg->n_dft) && fft::fits_32bit_index(cfg->n_dft, cfg->max_batch * cfg->n_q_heads);
    const bool fft_mode = cfg->decode_mode == FAEDKV_DECODE_FFT || cfg->decode_mode == FAEDKV_DECODE_FFT_TWO_PASS;
    if (fft_mode && !fft_ok) { delete ctx; return FAEDKV_ERR_UNSUPPORTED; }
    ctx->use_fft = fft_ok && (cfg->decode_mode == FAEDKV_DECODE_AUTO || fft_mode);
    ctx->use_col = ctx->use_fft && cfg->decode_mode != FAEDKV_DECODE_FFT_TWO_PASS && cfg->n_dft <= (2 << colfft::kMaxLg);
    // the FFT-shaped prefill shares the decode path's scratch, so it needs that path too
    if (cfg->prefill_mode == FAEDKV_PREFILL_FFT && !ctx->use_fft) { delete ctx; return FAEDKV_ERR_UNSUPPORTED; }
    ctx->prefill_fft = ctx->use_fft && (cfg->prefill_mode == FAEDKV_PREFILL_FFT ||
                                        (cfg->prefill_mode == FAEDKV_PREFILL_AUTO && cfg->kv_dtype == FAEDKV_F32));
    ctx->plans.resize(cfg->n_layers);
    if (cudaGetDevice(&ctx->device) != cudaSuccess ||
        cudaDeviceGetAttribute(&ctx->n_sm, cudaDevAttrMultiProcessorCount, ctx->device) != cudaSuccess || ctx->n_sm < 1 ||
        cudaMalloc(&ctx->tick, sizeof(unsigned int) * (cfg->n_layers + 1)) != cudaSuccess ||
        cudaMemset(ctx->tick, 0, sizeof(unsigned int) * (cfg->n_layers + 1)) != cudaSuccess) {
        cudaGetLastError();
        delete ctx;
        return FAEDKV_ERR_CUDA;
    }
    ctx->dev_status = ctx->tick + cfg->n_layers;
    *out = ctx;
    return FAEDKV_OK;
}

void faedkv_destroy(faedkv_ctx *ctx) {
    if (ctx == nullptr) return;
    for (LayerPlan &p : ctx->plans) { cudaFree(p.d_bins); cudaFree(p.d_tab); cudaFree(p.d_slot); }
    free_scratch(ctx);
    cudaFree(ctx->tick);
    delete ctx;
}

const char *faedkv_last_error(const faedkv_ctx *ctx) { return ctx ? ctx->err.c_str() : "null context"; }

int faedkv_plan(faedkv_ctx *ctx, int layer, const uint8_t *bin_mask, int *n_bins_out) {
    const CallRange nvtx_range("faedkv_plan");
    if (ctx == nullptr) return FAEDKV_ERR_INVALID_ARG;
    if (bin_mask == nullptr) return fail(ctx, FAEDKV_ERR_INVALID_ARG, "bin_mask is NULL");
    if (layer < 0 || layer >= ctx->cfg.n_layers)
        return fail(ctx, FAEDKV_ERR_INVALID_ARG, "layer %d outside [0, %d)", layer, ctx->cfg.n_layers);
    const int n1 = ctx->cfg.n_dft / 2 + 1;
    std::vector<int32_t> bins;
    bins.reserve(n1);
    for (int k = 0; k < n1; ++k)
        if (bin_mask[k] != 0) bins.push_back(k);
    if (bins.empty()) return fail(ctx, FAEDKV_ERR_INVALID_ARG, "mask of layer %d retains no bin", layer);
    if (int r = ensure_scratch(ctx, (int)bins.size())) return r;
    LayerPlan &p = ctx->plans[layer];
    int32_t *d = nullptr;
    CUDA_TRY(ctx, cudaMalloc(&d, bins.size() * sizeof(int32_t)));
    cudaError_t e = cudaMemcpy(d, bins.data(), bins.size() * sizeof(int32_t), cudaMemcpyHostToDevice);
    if (e != cudaSuccess) {
        cudaFree(d);
        return fail(ctx, FAEDKV_ERR_CUDA, "upload of the bin list failed: %s", cudaGetErrorString(e));
    }
    float *tab = nullptr;
    if (ctx->use_tc) {
        e = cudaMalloc(&tab, bins.size() * 16 * sizeof(float));
        if (e != cudaSuccess) {
            cudaFree(d);
            return fail(ctx, FAEDKV_ERR_CUDA, "allocation of the phasor table failed: %s", cudaGetErrorString(e));
        }
        const int n = (int)bins.size() * 8;
        k_bin_tables<<<(n + 255) / 256, 256>>>(d, (int)bins.size(), (uint32_t)ctx->cfg.n_dft, tab);
        e = cudaDeviceSynchronize();
        if (e != cudaSuccess) {
            cudaFree(d); cudaFree(tab);
            return fail(ctx, FAEDKV_ERR_CUDA, "building the phasor table failed: %s", cudaGetErrorString(e));
        }
    }
    int32_t *slot = nullptr;
    if (ctx->use_fft) {
        std::vector<int32_t> hs(n1, -1);
        for (size_t i = 0; i < bins.size(); ++i) hs[bins[i]] = (int32_t)i;
        e = cudaMalloc(&slot, (size_t)n1 * sizeof(int32_t));
        if (e == cudaSuccess) e = cudaMemcpy(slot, hs.data(), (size_t)n1 * sizeof(int32_t), cudaMemcpyHostToDevice);
        if (e != cudaSuccess) {
            cudaFree(d); cudaFree(tab); cudaFree(slot);
            return fail(ctx, FAEDKV_ERR_CUDA, "upload of the bin slot map failed: %s", cudaGetErrorString(e));
        }
    }
    cudaFree(p.d_bins);
    cudaFree(p.d_tab);
    cudaFree(p.d_slot);
    p.d_bins = d;
    p.d_tab = tab;
    p.d_slot = slot;
    p.M = (int)bins.size();
    p.bins.swap(bins);
    if (n_bins_out != nullptr) *n_bins_out = p.M;
    return FAEDKV_OK;
}

int faedkv_n_bins(const faedkv_ctx *ctx, int layer) {
    if (ctx == nullptr || layer < 0 || layer >= ctx->cfg.n_layers) return FAEDKV_ERR_INVALID_ARG;
    if (ctx->plans[layer].M == 0) return FAEDKV_ERR_NOT_PLANNED;
    return ctx->plans[layer].M;
}

int faedkv_get_bins(const faedkv_ctx *ctx, int layer, int32_t *bins_out) {
    if (ctx == nullptr || bins_out == nullptr || layer < 0 || layer >= ctx->cfg.n_layers) return FAEDKV_ERR_INVALID_ARG;
    const LayerPlan &p = ctx->plans[layer];
    if (p.M == 0) return FAEDKV_ERR_NOT_PLANNED;
    std::memcpy(bins_out, p.bins.data(), sizeof(int32_t) * p.M);
    return FAEDKV_OK;
}

size_t faedkv_coef_bytes(const faedkv_ctx *ctx, int layer, int batch) {
    if (ctx == nullptr || layer < 0 || layer >= ctx->cfg.n_layers || batch < 1) return 0;
    const LayerPlan &p = ctx->plans[layer];
    return (size_t)batch * ctx->cfg.n_kv_heads * 2 * (size_t)p.M * kHeadDim * sizeof(float);
}

int faedkv_mask_lowpass(int n_dft, int n_keep, uint8_t *mask_out) {
    if (mask_out == nullptr || n_dft < 2) return FAEDKV_ERR_INVALID_ARG;
    const int n1 = n_dft / 2 + 1;
    if (n_keep < 0 || n_keep > n1) return FAEDKV_ERR_INVALID_ARG;
    std::memset(mask_out, 0, n1);
    std::memset(mask_out, 1, n_keep);
    return FAEDKV_OK;
}

int faedkv_mask_mixed(int n_dft, int n_keep, int layer, uint64_t seed, uint8_t *mask_out) {
    constexpr int kChunk = 16;
    if (mask_out == nullptr || n_dft < 2 || n_keep <= 0 || n_keep % kChunk != 0) return FAEDKV_ERR_INVALID_ARG;
    const int n1 = n_dft / 2 + 1;
    const int low_chunks = (n_keep / 2) / kChunk;        // always-kept low chunks
    const int extra_chunks = n_keep / kChunk - low_chunks;  // drawn chunks
    const int pool_end = (n_dft / 2) / kChunk;           // chunks wholly below P/2
    std::vector<int> pool;
    for (int c = low_chunks; c < pool_end; ++c) pool.push_back(c);
    if ((int)pool.size() < extra_chunks) return FAEDKV_ERR_INVALID_ARG;
    std::memset(mask_out, 0, n1);
    std::memset(mask_out, 1, (size_t)low_chunks * kChunk);
    uint64_t state = seed * 2654435761ULL + (uint64_t)layer;
    for (int i = 0; i < extra_chunks; ++i) {
        state = state * 6364136223846793005ULL + 1442695040888963407ULL;
        const uint64_t remaining = (uint64_t)(pool.size() - i);
        std::swap(pool[i], pool[i + (size_t)((state >> 33) % remaining)]);
        std::memset(mask_out + (size_t)pool[i] * kChunk, 1, kChunk);
    }
    return FAEDKV_OK;
}

int faedkv_compress_prefill(faedkv_ctx *ctx, int layer, const void *K, const void *V, int batch,
                            int T, float *coefK, float *coefV, int32_t *t_len, void *stream) {
    const CallRange nvtx_range("faedkv_compress_prefill");
    const LayerPlan *p = nullptr;
    if (int r = check_layer(ctx, layer, &p)) return r;
    if (int r = check_batch(ctx, batch)) return r;
    if (K == nullptr || V == nullptr || coefK == nullptr || coefV == nullptr || t_len == nullptr)
        return fail(ctx, FAEDKV_ERR_INVALID_ARG, "NULL tensor passed to faedkv_compress_prefill");
    if (T < 1) return fail(ctx, FAEDKV_ERR_SHAPE, "T = %d must be >= 1", T);
    if (int r = check_ptrs(ctx, {K, V, coefK, coefV})) return r;
    if (int r = check_tlen(ctx, t_len)) return r;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (int r = prefill_core(ctx, *p, K, V, batch, T, T, coefK, coefV, st)) return r;
    k_set_tlen<<<(batch + 127) / 128, 128, 0, st>>>(t_len, batch, T);
    return launch_check(ctx, "k_set_tlen");
}

int faedkv_append(faedkv_ctx *ctx, int layer, const void *k_new, const void *v_new, int batch,
                  float *coefK, float *coefV, int32_t *t_len, void *stream) {
    const CallRange nvtx_range("faedkv_append");
    const LayerPlan *p = nullptr;
    if (int r = check_layer(ctx, layer, &p)) return r;
    if (int r = check_batch(ctx, batch)) return r;
    if (k_new == nullptr || v_new == nullptr || coefK == nullptr || coefV == nullptr || t_len == nullptr)
        return fail(ctx, FAEDKV_ERR_INVALID_ARG, "NULL tensor passed to faedkv_append");
    if (int r = check_ptrs(ctx, {k_new, v_new, coefK, coefV})) return r;
    if (int r = check_tlen(ctx, t_len)) return r;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const faedkv_config &c = ctx->cfg;
    dim3 grid((p->M + kAppendWarps - 1) / kAppendWarps, batch);
    if (c.kv_dtype == FAEDKV_BF16)
        k_append<__nv_bfloat16><<<grid, kAppendWarps * 32, 0, st>>>(
            static_cast<const __nv_bfloat16 *>(k_new), static_cast<const __nv_bfloat16 *>(v_new), coefK, coefV,
            t_len, p->d_bins, p->M, c.n_kv_heads, (uint32_t)c.n_dft, ctx->tick + layer);
    else
        k_append<float><<<grid, kAppendWarps * 32, 0, st>>>(
            static_cast<const float *>(k_new), static_cast<const float *>(v_new), coefK, coefV, t_len,
            p->d_bins, p->M, c.n_kv_heads, (uint32_t)c.n_dft, ctx->tick + layer);
    return launch_check(ctx, "k_append");
}

int faedkv_reconstruct(faedkv_ctx *ctx, int layer, const float *coefK, const float *coefV,
                       const int32_t *t_len, int batch, int L, void *K_out, void *V_out, void *stream) {
    const CallRange nvtx_range("faedkv_reconstruct");
    const LayerPlan *p = nullptr;
    if (int r = check_layer(ctx, layer, &p)) return r;
    if (int r = check_batch(ctx, batch)) return r;
    if (t_len == nullptr) return fail(ctx, FAEDKV_ERR_INVALID_ARG, "t_len is NULL");
    if ((coefK == nullptr) != (K_out == nullptr) || (coefV == nullptr) != (V_out == nullptr) ||
        (coefK == nullptr && coefV == nullptr))
        return fail(ctx, FAEDKV_ERR_INVALID_ARG, "coefficient / output pointers must come in non-NULL pairs");
    if (L < 1 || L > ctx->cfg.n_dft) return fail(ctx, FAEDKV_ERR_SHAPE, "L = %d outside [1, P=%d]", L, ctx->cfg.n_dft);
    if (int r = check_ptrs(ctx, {coefK, coefV, K_out, V_out})) return r;
    if (int r = check_tlen(ctx, t_len)) return r;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (ctx->use_fft) {
        if (ctx->cfg.kv_dtype == FAEDKV_BF16)
            return launch_reconstruct_fft<__nv_bfloat16>(ctx, *p, coefK, coefV, t_len, batch, L, K_out, V_out, st);
        return launch_reconstruct_fft<float>(ctx, *p, coefK, coefV, t_len, batch, L, K_out, V_out, st);
    }
    if (ctx->use_tc) return launch_reconstruct_tc(ctx, *p, coefK, coefV, t_len, batch, L, K_out, V_out, st);
    if (ctx->cfg.kv_dtype == FAEDKV_BF16)
        return launch_reconstruct<__nv_bfloat16>(ctx, *p, coefK, coefV, t_len, batch, L, K_out, V_out, st);
    return launch_reconstruct<float>(ctx, *p, coefK, coefV, t_len, batch, L, K_out, V_out, st);
}

int faedkv_decode_attn(faedkv_ctx *ctx, int layer, const void *q, const float *coefK, const float *coefV,
                       const int32_t *t_len, int batch, float scale, void *out, void *stream) {
    const CallRange nvtx_range("faedkv_decode_attn");
    const LayerPlan *p = nullptr;
    if (int r = check_layer(ctx, layer, &p)) return r;
    if (int r = check_batch(ctx, batch)) return r;
    if (q == nullptr || coefK == nullptr || coefV == nullptr || t_len == nullptr || out == nullptr)
        return fail(ctx, FAEDKV_ERR_INVALID_ARG, "NULL tensor passed to faedkv_decode_attn");
    if (!(scale >= 0.0f)) return fail(ctx, FAEDKV_ERR_INVALID_ARG, "scale must be >= 0");
    if (int r = check_ptrs(ctx, {q, coefK, coefV, out})) return r;
    if (int r = check_tlen(ctx, t_len)) return r;
    if (scale == 0.0f) scale = 1.0f / sqrtf((float)ctx->cfg.head_dim);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (ctx->cfg.kv_dtype == FAEDKV_BF16)
        return dispatch_attn<__nv_bfloat16>(ctx, *p, q, coefK, coefV, t_len, batch, scale, out, st);
    return dispatch_attn<float>(ctx, *p, q, coefK, coefV, t_len, batch, scale, out, st);
}

int faedkv_append_decode_attn(faedkv_ctx *ctx, int layer, const void *k_new, const void *v_new, const void *q,
                              int batch, float *coefK, float *coefV, int32_t *t_len, float scale, void *out,
                              void *stream) {
    const CallRange nvtx_range("faedkv_append_decode_attn");
    const LayerPlan *p = nullptr;
    if (int r = check_layer(ctx, layer, &p)) return r;
    if (int r = check_batch(ctx, batch)) return r;
    if (k_new == nullptr || v_new == nullptr || q == nullptr || coefK == nullptr || coefV == nullptr ||
        t_len == nullptr || out == nullptr)
        return fail(ctx, FAEDKV_ERR_INVALID_ARG, "NULL tensor passed to faedkv_append_decode_attn");
    if (!(scale >= 0.0f)) return fail(ctx, FAEDKV_ERR_INVALID_ARG, "scale must be >= 0");
    if (int r = check_ptrs(ctx, {k_new, v_new, q, coefK, coefV, out})) return r;
    if (int r = check_tlen(ctx, t_len)) return r;
    if (!ctx->use_fft) {
        if (int r = faedkv_append(ctx, layer, k_new, v_new, batch, coefK, coefV, t_len, stream)) return r;
        return faedkv_decode_attn(ctx, layer, q, coefK, coefV, t_len, batch, scale, out, stream);
    }
    if (scale == 0.0f) scale = 1.0f / sqrtf((float)ctx->cfg.head_dim);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (ctx->cfg.kv_dtype == FAEDKV_BF16)
        return dispatch_attn_fft<__nv_bfloat16, true>(ctx, *p, q, k_new, v_new, coefK, coefV, t_len, batch, scale, out, st);
    return dispatch_attn_fft<float, true>(ctx, *p, q, k_new, v_new, coefK, coefV, t_len, batch, scale, out, st);
}

size_t faedkv_window_bytes(const faedkv_ctx *ctx, int batch) {
    if (ctx == nullptr || batch < 1) return 0;
    const size_t elem = ctx->cfg.kv_dtype == FAEDKV_BF16 ? 2 : 4;
    return (size_t)batch * ctx->cfg.n_kv_heads * (ctx->cfg.n_sink + win_ring(ctx->cfg.n_recent, ctx->cfg.n_defer)) * kHeadDim * elem;
}

int faedkv_prefill_windowed(faedkv_ctx *ctx, int layer, const void *K, const void *V, int batch, int T, float *coefK,
                            float *coefV, void *winK, void *winV, int32_t *t_len, void *stream) {
    const CallRange nvtx_range("faedkv_prefill_windowed");
    const LayerPlan *p = nullptr;
    if (int r = check_layer(ctx, layer, &p)) return r;
    if (int r = check_batch(ctx, batch)) return r;
    const faedkv_config &c = ctx->cfg;
    const int S = c.n_sink, R = c.n_recent, D = c.n_defer, Rc = win_ring(R, D);
    if (K == nullptr || V == nullptr || coefK == nullptr || coefV == nullptr || t_len == nullptr ||
        (S + Rc > 0 && (winK == nullptr || winV == nullptr)))
        return fail(ctx, FAEDKV_ERR_INVALID_ARG, "NULL tensor passed to faedkv_prefill_windowed");
    if (T < S + R || T < 1)
        return fail(ctx, FAEDKV_ERR_SHAPE, "T = %d must cover the sink and recent windows (%d + %d)", T, S, R);
    if (int r = check_ptrs(ctx, {K, V, coefK, coefV, winK, winV})) return r;
    if (int r = check_tlen(ctx, t_len)) return r;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t elem = c.kv_dtype == FAEDKV_BF16 ? 2 : 4;
    const int mid = win_folded(T, S, R, D);
    if (mid > 0) {
        // rows [S, S + mid) of every unit, at positions 0 .. mid - 1 of the transformed segment (Eq. 10)
        const char *Km = static_cast<const char *>(K) + (size_t)S * kHeadDim * elem;
        const char *Vm = static_cast<const char *>(V) + (size_t)S * kHeadDim * elem;
        if (int r = prefill_core(ctx, *p, Km, Vm, batch, mid, T, coefK, coefV, st)) return r;
    } else {
        const size_t bytes = faedkv_coef_bytes(ctx, layer, batch);
        CUDA_TRY(ctx, cudaMemsetAsync(coefK, 0, bytes, st));
        CUDA_TRY(ctx, cudaMemsetAsync(coefV, 0, bytes, st));
    }
    if (T - mid > 0) {
        dim3 grid(T - mid, batch * c.n_kv_heads);      // sink rows + the tokens that stay in the time domain
        if (c.kv_dtype == FAEDKV_BF16)
            k_window_fill<__nv_bfloat16><<<grid, kHeadDim, 0, st>>>(static_cast<const __nv_bfloat16 *>(K), static_cast<const __nv_bfloat16 *>(V),
                                                                   static_cast<__nv_bfloat16 *>(winK), static_cast<__nv_bfloat16 *>(winV), T, S, Rc, mid);
        else
            k_window_fill<float><<<grid, kHeadDim, 0, st>>>(static_cast<const float *>(K), static_cast<const float *>(V),
                                                           static_cast<float *>(winK), static_cast<float *>(winV), T, S, Rc, mid);
        if (int r = launch_check(ctx, "k_window_fill")) return r;
    }
    k_set_tlen<<<(batch + 127) / 128, 128, 0, st>>>(t_len, batch, T);
    return launch_check(ctx, "k_set_tlen");
}

int faedkv_step_windowed(faedkv_ctx *ctx, int layer, const void *k_new, const void *v_new, const void *q, int batch,
                         float *coefK, float *coefV, void *winK, void *winV, int32_t *t_len, float scale, void *out,
                         void *stream) {
    const CallRange nvtx_range("faedkv_step_windowed");
    const LayerPlan *p = nullptr;
    if (int r = check_layer(ctx, layer, &p)) return r;
    if (int r = check_batch(ctx, batch)) return r;
    if (k_new == nullptr || v_new == nullptr || q == nullptr || coefK == nullptr || coefV == nullptr ||
        winK == nullptr || winV == nullptr || t_len == nullptr || out == nullptr)
        return fail(ctx, FAEDKV_ERR_INVALID_ARG, "NULL tensor passed to faedkv_step_windowed");
    if (!(scale >= 0.0f)) return fail(ctx, FAEDKV_ERR_INVALID_ARG, "scale must be >= 0");
    if (int r = check_ptrs(ctx, {k_new, v_new, q, coefK, coefV, winK, winV, out})) return r;
    if (int r = check_tlen(ctx, t_len)) return r;
    if (!ctx->use_fft)
        return fail(ctx, FAEDKV_ERR_UNSUPPORTED, "the windowed step needs the FFT-shaped decode path (P a power of two in [64, 2^19])");
    if (scale == 0.0f) scale = 1.0f / sqrtf((float)ctx->cfg.head_dim);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const faedkv_config &c = ctx->cfg;
    if (c.n_defer > 1) {
        // block-deferred fold: fold the sequences that reach a block boundary (the others' CTAs return at
        // once), then attend without touching the planes again
        const int D = c.n_defer;
        const WindowArgs wa{winK, winV, k_new, v_new, c.n_sink, c.n_recent, D, win_ring(c.n_recent, D), 0.f, nullptr, nullptr, nullptr};
        // work items (sequence, 32 bins, share of the 2H planes); the planes are split until the items fill the SMs
        const int n_groups = (p->M + kFoldGroup - 1) / kFoldGroup;
        int splits = 1;
        while (splits < 2 * c.n_kv_heads && batch * n_groups * splits < 4 * ctx->n_sm) splits *= 2;
        const int n_items = batch * n_groups * splits;
        const dim3 grid(n_items < 4 * ctx->n_sm ? n_items : 4 * ctx->n_sm);
        const size_t smem = block_fold_smem(D);
        if (c.kv_dtype == FAEDKV_BF16) {
            if (int r = fft_opt_in(ctx, k_block_fold<__nv_bfloat16>, smem, ctx->fs.attr_mask[9], 0)) return r;
            k_block_fold<__nv_bfloat16><<<grid, kFoldWarps * 32, smem, st>>>(coefK, coefV, t_len, p->d_bins, wa, p->M, c.n_kv_heads, batch, (uint32_t)c.n_dft, splits);
        } else {
            if (int r = fft_opt_in(ctx, k_block_fold<float>, smem, ctx->fs.attr_mask[9], 1)) return r;
            k_block_fold<float><<<grid, kFoldWarps * 32, smem, st>>>(coefK, coefV, t_len, p->d_bins, wa, p->M, c.n_kv_heads, batch, (uint32_t)c.n_dft, splits);
        }
        if (int r = launch_check(ctx, "k_block_fold")) return r;
        if (c.kv_dtype == FAEDKV_BF16)
            return dispatch_attn_fft<__nv_bfloat16, false>(ctx, *p, q, k_new, v_new, coefK, coefV, t_len, batch, scale, out, st, winK, winV);
        return dispatch_attn_fft<float, false>(ctx, *p, q, k_new, v_new, coefK, coefV, t_len, batch, scale, out, st, winK, winV);
    }
    if (c.kv_dtype == FAEDKV_BF16)
        return dispatch_attn_fft<__nv_bfloat16, true>(ctx, *p, q, k_new, v_new, coefK, coefV, t_len, batch, scale, out, st, winK, winV);
    return dispatch_attn_fft<float, true>(ctx, *p, q, k_new, v_new, coefK, coefV, t_len, batch, scale, out, st, winK, winV);
}

int faedkv_reconstruct_windowed(faedkv_ctx *ctx, int layer, const float *coefK, const float *coefV, const void *winK,
                                const void *winV, const int32_t *t_len, int batch, int L, void *K_out, void *V_out,
                                void *stream) {
    const CallRange nvtx_range("faedkv_reconstruct_windowed");
    const LayerPlan *p = nullptr;
    if (int r = check_layer(ctx, layer, &p)) return r;
    if (int r = check_batch(ctx, batch)) return r;
    const faedkv_config &c = ctx->cfg;
    const int S = c.n_sink, R = c.n_recent, D = c.n_defer, Rc = win_ring(R, D);
    if (coefK == nullptr || coefV == nullptr || t_len == nullptr || K_out == nullptr || V_out == nullptr ||
        (S + Rc > 0 && (winK == nullptr || winV == nullptr)))
        return fail(ctx, FAEDKV_ERR_INVALID_ARG, "NULL tensor passed to faedkv_reconstruct_windowed");
    if (L < 1) return fail(ctx, FAEDKV_ERR_SHAPE, "L = %d must be at least 1", L);
    if (int r = check_ptrs(ctx, {coefK, coefV, winK, winV, K_out, V_out})) return r;
    if (int r = check_tlen(ctx, t_len)) return r;
    if (!ctx->use_fft)
        return fail(ctx, FAEDKV_ERR_UNSUPPORTED, "the windowed calls need the FFT-shaped path (P a power of two in [64, 2^19])");
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int units = batch * c.n_kv_heads;
    // the reconstructed segment at rows [S, S + min(L - S, P)), zeros past its live positions ...
    const int Lmid = L - S < c.n_dft ? L - S : c.n_dft;
    if (Lmid > 0 && use_recon2(ctx)) {
        const ReconRows rows{S, L, -(S + R), D > 1 ? D : 1};
        int r = c.kv_dtype == FAEDKV_BF16
                    ? launch_recon2<__nv_bfloat16>(ctx, *p, coefK, coefV, t_len, units, Lmid, K_out, V_out, st, rows)
                    : launch_recon2<float>(ctx, *p, coefK, coefV, t_len, units, Lmid, K_out, V_out, st, rows);
        if (r) return r;
    } else if (Lmid > 0) {
        const ReconRows rows{S, L, -(S + R), D > 1 ? D : 1};
        for (int kv = 0; kv < 2; ++kv) {
            const float *coef = kv == 0 ? coefK : coefV;
            void *out = kv == 0 ? K_out : V_out;
            int r = c.kv_dtype == FAEDKV_BF16
                        ? launch_reconstruct_fft_tensor<__nv_bfloat16>(ctx, *p, coef, t_len, units, Lmid, out, st, rows)
                        : launch_reconstruct_fft_tensor<float>(ctx, *p, coef, t_len, units, Lmid, out, st, rows);
            if (r) return r;
        }
    }
    // ... then the sink rows, the waiting tokens right behind the live positions, and zeros to the end
    for (int kv = 0; kv < 2; ++kv) {
        const void *win = kv == 0 ? winK : winV;
        void *out = kv == 0 ? K_out : V_out;
        const dim3 grid(L, units);
        if (c.kv_dtype == FAEDKV_BF16)
            k_window_place<__nv_bfloat16><<<grid, kHeadDim, 0, st>>>(static_cast<const __nv_bfloat16 *>(win), static_cast<__nv_bfloat16 *>(out),
                                                                    t_len, c.n_kv_heads, L, S, R, D, Rc, c.n_dft);
        else
            k_window_place<float><<<grid, kHeadDim, 0, st>>>(static_cast<const float *>(win), static_cast<float *>(out), t_len,
                                                            c.n_kv_heads, L, S, R, D, Rc, c.n_dft);
        if (int r = launch_check(ctx, "k_window_place")) return r;
    }
    return FAEDKV_OK;
}

int faedkv_chunk_range(int n_dft, int n_chunks, int chunk, int *lo, int *hi) {
    if (n_dft < 2 || n_chunks < 1 || n_chunks > n_dft || chunk < 0 || chunk >= n_chunks || lo == nullptr || hi == nullptr)
        return FAEDKV_ERR_INVALID_ARG;
    const int w = n_dft / n_chunks;
    *lo = chunk * w;
    *hi = chunk == n_chunks - 1 ? n_dft : (chunk + 1) * w;
    return FAEDKV_OK;
}

int faedkv_ablation_bins(int n_dft, int lo, int hi, uint8_t *mask_out, float *gain_out) {
    if (n_dft < 2 || lo < 0 || hi > n_dft || lo >= hi || mask_out == nullptr || gain_out == nullptr)
        return FAEDKV_ERR_INVALID_ARG;
    for (int k = 0; k <= n_dft / 2; ++k) {
        const int mirror = (n_dft - k) % n_dft;
        const bool a = lo <= k && k < hi, b = lo <= mirror && mirror < hi;
        mask_out[k] = (a || b) ? 1 : 0;
        gain_out[k] = (a && b) ? 1.0f : ((a || b) ? 0.5f : 0.0f);
    }
    return FAEDKV_OK;
}

int faedkv_mask_from_scores(int n_dft, int n_chunks, const double *delta, double ratio, uint8_t *mask_out,
                            int *n_keep_out) {
    if (n_dft < 2 || n_chunks < 1 || n_chunks > n_dft || delta == nullptr || mask_out == nullptr || !(ratio >= 0.0))
        return FAEDKV_ERR_INVALID_ARG;
    int n_keep = (int)std::floor(ratio * n_chunks + 0.5);
    if (n_keep < 1) n_keep = 1;
    if (n_keep > n_chunks) n_keep = n_chunks;
    std::vector<int> order(n_chunks);
    for (int c = 0; c < n_chunks; ++c) order[c] = c;
    std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return delta[a] > delta[b]; });   // ties keep index order
    std::vector<uint8_t> two(n_dft, 0);
    for (int i = 0; i < n_keep; ++i) {
        int lo, hi;
        faedkv_chunk_range(n_dft, n_chunks, order[i], &lo, &hi);
        std::fill(two.begin() + lo, two.begin() + hi, (uint8_t)1);
    }
    for (int k = 0; k <= n_dft / 2; ++k) mask_out[k] = (two[k] | two[(n_dft - k) % n_dft]) ? 1 : 0;
    if (n_keep_out != nullptr) *n_keep_out = n_keep;
    return FAEDKV_OK;
}

int faedkv_ablate(faedkv_ctx *ctx, int layer, const void *K, const void *V, int batch, int T, const float *gain,
                  float *wsK, float *wsV, int32_t *ws_len, void *K_out, void *V_out, void *stream) {
    const CallRange nvtx_range("faedkv_ablate");
    const LayerPlan *p = nullptr;
    if (int r = check_layer(ctx, layer, &p)) return r;
    if (int r = check_batch(ctx, batch)) return r;
    if (K == nullptr || V == nullptr || gain == nullptr || wsK == nullptr || wsV == nullptr || ws_len == nullptr ||
        K_out == nullptr || V_out == nullptr)
        return fail(ctx, FAEDKV_ERR_INVALID_ARG, "NULL tensor passed to faedkv_ablate");
    if (T < 1 || T > ctx->cfg.n_dft) return fail(ctx, FAEDKV_ERR_SHAPE, "T = %d outside [1, P=%d]", T, ctx->cfg.n_dft);
    if (int r = check_ptrs(ctx, {K, V, gain, wsK, wsV, K_out, V_out})) return r;
    if (int r = check_tlen(ctx, ws_len)) return r;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const faedkv_config &c = ctx->cfg;
    // spectrum of the touched bins, weighted by the share of each that the zeroing removes ...
    if (int r = faedkv_compress_prefill(ctx, layer, K, V, batch, T, wsK, wsV, ws_len, stream)) return r;
    const size_t n_vec = (size_t)batch * c.n_kv_heads * 2 * p->M * (kHeadDim / 4);
    for (float *ws : {wsK, wsV}) {
        k_scale_planes<<<(unsigned)((n_vec + 255) / 256), 256, 0, st>>>(ws, gain, p->M, n_vec);
        if (int r = launch_check(ctx, "k_scale_planes")) return r;
    }
    // ... back to the time domain, and out of the input
    if (int r = faedkv_reconstruct(ctx, layer, wsK, wsV, ws_len, batch, T, K_out, V_out, stream)) return r;
    const size_t n = (size_t)batch * c.n_kv_heads * T * kHeadDim;
    const void *xs[2] = {K, V};
    void *ys[2] = {K_out, V_out};
    for (int i = 0; i < 2; ++i) {
        if (c.kv_dtype == FAEDKV_BF16)
            k_subtract_from<__nv_bfloat16><<<(unsigned)((n + 255) / 256), 256, 0, st>>>(static_cast<const __nv_bfloat16 *>(xs[i]),
                                                                                     static_cast<__nv_bfloat16 *>(ys[i]), n);
        else
            k_subtract_from<float><<<(unsigned)((n + 255) / 256), 256, 0, st>>>(static_cast<const float *>(xs[i]),
                                                                             static_cast<float *>(ys[i]), n);
        if (int r = launch_check(ctx, "k_subtract_from")) return r;
    }
    return FAEDKV_OK;
}

int faedkv_convert_state(faedkv_ctx *ctx, int layer, const float *coef_in, const int32_t *t_len, int batch, int from_form,
                         int to_form, float *coef_out, void *stream) {
    const CallRange nvtx_range("faedkv_convert_state");
    const LayerPlan *p = nullptr;
    if (int r = check_layer(ctx, layer, &p)) return r;
    if (int r = check_batch(ctx, batch)) return r;
    if (coef_in == nullptr || coef_out == nullptr || t_len == nullptr)
        return fail(ctx, FAEDKV_ERR_INVALID_ARG, "NULL tensor passed to faedkv_convert_state");
    if (from_form < FAEDKV_STATE_SUM || from_form > FAEDKV_STATE_ROTATING || to_form < FAEDKV_STATE_SUM ||
        to_form > FAEDKV_STATE_ROTATING)
        return fail(ctx, FAEDKV_ERR_INVALID_ARG, "unknown state form");
    if (int r = check_ptrs(ctx, {coef_in, coef_out})) return r;
    if (int r = check_tlen(ctx, t_len)) return r;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    dim3 grid((p->M + 7) / 8, batch * ctx->cfg.n_kv_heads);
    k_convert_state<<<grid, 256, 0, st>>>(coef_in, coef_out, p->d_bins, t_len, p->M, ctx->cfg.n_kv_heads,
                                          (uint32_t)ctx->cfg.n_dft, from_form, to_form);
    return launch_check(ctx, "k_convert_state");
}

unsigned long long faedkv_launch_count(const faedkv_ctx *ctx) { return ctx ? ctx->launches : 0ULL; }

int faedkv_reset_device_status(faedkv_ctx *ctx, void *stream) {
    if (ctx == nullptr) return FAEDKV_ERR_INVALID_ARG;
    CUDA_TRY(ctx, cudaMemsetAsync(ctx->dev_status, 0, sizeof(unsigned int), static_cast<cudaStream_t>(stream)));
    return FAEDKV_OK;
}

int faedkv_debug_build(void) {
#ifdef FAEDKV_DEBUG
    return 1;
#else
    return 0;
#endif
}

long long faedkv_debug_word(faedkv_ctx *ctx, void *stream) {
    if (ctx == nullptr) return FAEDKV_ERR_INVALID_ARG;
#ifdef FAEDKV_DEBUG
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    unsigned int w = 0, zero = 0;
    CUDA_TRY(ctx, cudaStreamSynchronize(st));
    CUDA_TRY(ctx, cudaMemcpyFromSymbol(&w, g_faedkv_debug_word, sizeof(w)));
    CUDA_TRY(ctx, cudaMemcpyToSymbol(g_faedkv_debug_word, &zero, sizeof(zero)));
    if (w != 0) fail(ctx, FAEDKV_ERR_INVALID_ARG, "bounds check failed: file tag %u, line %u", w >> 16, w & 0xffffu);
    return (long long)w;
#else
    (void)stream;
    return 0;
#endif
}

int faedkv_test_hooks(faedkv_ctx *ctx, unsigned long long wait_limit_ns, int withhold_step) {
    if (ctx == nullptr || withhold_step < 0) return FAEDKV_ERR_INVALID_ARG;
    ctx->umma.wait_limit_ns = wait_limit_ns == 0 ? umma::kWaitLimitNs : wait_limit_ns;
    ctx->umma.withhold_step = withhold_step;
    return FAEDKV_OK;
}

int faedkv_device_status(faedkv_ctx *ctx, void *stream) {
    if (ctx == nullptr) return FAEDKV_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    unsigned int w = 0;
    CUDA_TRY(ctx, cudaMemcpyAsync(&w, ctx->dev_status, sizeof(w), cudaMemcpyDeviceToHost, st));
    CUDA_TRY(ctx, cudaStreamSynchronize(st));
    if (w != 0) {
        fail(ctx, FAEDKV_ERR_TIMEOUT, "device status word = 0x%x (a bounded wait gave up)", w);
        return (int)w;
    }
    return 0;
}

}  // extern "C"
