// Sink and recent window (Sec. 4.2: the first S tokens and the most recent R tokens stay in the time
// domain; Eq. 13 attends over [sink | reconstructed middle | recent]).
//
// Window tensors winK, winV: [units][S + R][128] in the storage type; rows [0, S) are the sink tokens,
// rows [S, S + R) a ring: token n (n >= S) lives in slot (n - S) mod R while it is among the last R.
// When token t arrives, the token leaving the window, t - R, sits in the slot the new one will take; it
// is folded into the coefficients at middle position t - R - S (Eq. 12) before being overwritten.
#pragma once
#include "common.cuh"

namespace faedkv {

// Where the token folded by a fused update comes from, and at which position of the transformed segment.
struct FoldSrc {
    int unit_rows;   // rows between consecutive units of the source (1: a [units][128] token tensor)
    int S, R;        // sink and ring sizes (0, 0: no window)
};
__device__ __forceinline__ void fold_locate(const FoldSrc &f, int t, int unit, uint32_t P, size_t &row, uint32_t &pos) {
    if (f.R > 0) {
        int mid = t - f.S - f.R;                       // tokens already in the transformed segment
        if (!FAEDKV_IN_BOUNDS(kTagWindow, mid >= 0 && f.S + f.R <= f.unit_rows)) mid = 0;
        row = (size_t)unit * f.unit_rows + f.S + mid % f.R;
        pos = (uint32_t)mid % P;
    } else {
        row = (size_t)unit * f.unit_rows;
        pos = (uint32_t)(t - f.S) % P;
    }
}

// Block-deferred fold (defer = D > 1): unfolded tokens wait in a ring of Rc = R + D slots and the D oldest are
// folded in one go whenever R + D are waiting, i.e. when (tokens - S - R) reaches a multiple of D.  The number
// of tokens in the transformed segment is therefore a function of the token count alone.
__host__ __device__ __forceinline__ int win_folded(int total, int S, int R, int D) {
    const int m = total - S - R;
    return m <= 0 ? 0 : (D > 1 ? m / D * D : m);
}
__host__ __device__ __forceinline__ int win_ring(int R, int D) { return D > 1 ? R + D : R; }

// Prefill: copy the sink rows and place the unfolded tokens [S + folded, T) in their ring slots.
// grid = (S + T - S - folded, units); block = 128.  K, V: [units][T][128]; win: [units][S + Rc][128].
template <typename T>
__global__ void k_window_fill(const T *__restrict__ K, const T *__restrict__ V, T *__restrict__ winK, T *__restrict__ winV,
                              int Ttot, int S, int Rc, int folded) {
    const int w = blockIdx.x, unit = blockIdx.y, c = threadIdx.x;
    int src, dst;
    if (w < S) {
        src = w; dst = w;
    } else {
        src = S + folded + (w - S);
        dst = S + (src - S) % Rc;
    }
    const size_t so = ((size_t)unit * Ttot + src) * kHeadDim + c, d_o = ((size_t)unit * (S + Rc) + dst) * kHeadDim + c;
    winK[d_o] = K[so];
    winV[d_o] = V[so];
}

// Eq. 13 materialised: the rows of [sink | reconstructed segment | waiting tokens] that are NOT the reconstructed
// segment (which the inverse transform writes at rows [S, S + live)).  Row n of a unit: n < S the sink token n;
// S + live <= n < S + live + u the waiting tokens in order; zero from there to L.  t_len is at rest (no step
// in flight): every token sits in its ring slot.
// grid = (L, units); block = 128.
template <typename T>
__global__ void k_window_place(const T *__restrict__ win, T *__restrict__ out, const int32_t *__restrict__ t_len,
                               int H, int L, int S, int R, int D, int Rc, int P) {
    const int n = blockIdx.x, unit = blockIdx.y, c = threadIdx.x;
    const int t = t_len[unit / H];
    const int folded = win_folded(t, S, R, D);
    const int live = folded < P ? folded : P;
    const int u = t - S - folded;                    // waiting tokens
    T *dst = out + ((size_t)unit * L + n) * kHeadDim + c;
    const T *src = nullptr;
    if (n < S) {
        if (n < t) src = win + ((size_t)unit * (S + Rc) + n) * kHeadDim + c;
    } else if (n < S + live) {
        return;                                      // written by the inverse transform
    } else if (n - S - live < u) {
        src = win + ((size_t)unit * (S + Rc) + S + (folded + n - S - live) % Rc) * kHeadDim + c;   // u > 0 implies Rc > 0
    }
    if (src != nullptr) *dst = *src;
    else store1(dst, 0.f);
}

// Attention over the time-domain tokens of one (sequence, kv head) for its GQ query heads, in the same
// unnormalised form as a tile of the transformed segment: per column the maximum score m, the sum of
// exp(s - m), and o_w[col][c] = sum_w exp(s_w - m) v_w[c].  Rows: the S sink tokens, then the unfolded tokens
// [S + folded(t + 1), t] in token order, where t = t_len is the step's new token; its ring slot is written only
// at the end of the step, so k_new / v_new stand in for that row.  No rows at all: m = -inf, sum = 0, o = 0.
//
// Nothing here depends on the rest of the step, so the host starts it on a second stream at the top of the
// call, beside the pass over C_K, and joins it before the kernel that reads the statistics.  Beside a
// bandwidth-saturating pass every dependent round of loads costs microseconds and every register held is one
// the pass cannot use: a CTA is 128 threads of at most 64 registers and takes one query head; each of its 4
// warps reads the K and V rows of kWinRows tokens at once (rows w = warp mod 4; kept in the storage type
// until used) and runs an online softmax over them in registers (a lane holds 4 of the 128 channels); the
// paper's window (60 rows; 110 with a deferred block of 50) takes 2 to 4 rounds.
// grid = (units, GQ); block = 128.
struct WindowArgs {
    const void *winK, *winV, *k_new, *v_new;   // storage type of the context
    int S, R, D, Rc;                           // sink, recent, defer block, ring capacity (win_ring(R, D))
    float scale;
    float *m_w, *s_w, *o_w;                    // statistics row of the window, [Gp] each; output [Gp][128]
};

template <typename T> struct WinRaw;
template <> struct WinRaw<float> {
    using type = float4;
    static __device__ __forceinline__ type load(const float *p) { return *reinterpret_cast<const float4 *>(p); }
    static __device__ __forceinline__ float4 cvt(type r) { return r; }
};
template <> struct WinRaw<__nv_bfloat16> {
    using type = uint2;
    static __device__ __forceinline__ type load(const __nv_bfloat16 *p) { return *reinterpret_cast<const uint2 *>(p); }
    static __device__ __forceinline__ float4 cvt(type r) {
        return make_float4(bf16_bits_to_float(r.x & 0xffffu), __uint_as_float(r.x & 0xffff0000u),
                           bf16_bits_to_float(r.y & 0xffffu), __uint_as_float(r.y & 0xffff0000u));
    }
};

constexpr int kWinWarps = 4;                   // row shares of a query head

template <typename TQ, int GQ>
__global__ void __launch_bounds__(kWinWarps * 32, 8)
k_attn_window(const TQ *__restrict__ q, WindowArgs wa, const int32_t *__restrict__ t_len, int H) {
    using Raw = WinRaw<TQ>;
    constexpr int RS = kWinWarps;
    constexpr int kWinRows = sizeof(TQ) == 2 ? 8 : 4;          // rows a warp has in flight
    __shared__ float4 o_s[RS][32];
    __shared__ float m_s[RS], s_s[RS];
    const TQ *winK = static_cast<const TQ *>(wa.winK), *winV = static_cast<const TQ *>(wa.winV);
    const TQ *k_new = static_cast<const TQ *>(wa.k_new), *v_new = static_cast<const TQ *>(wa.v_new);
    const int S = wa.S, Rc = wa.Rc, Wcap = S + Rc;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int rs = warp;                                       // share of the rows
    const int bh = blockIdx.x, b = bh / H, col = bh * GQ + (int)blockIdx.y;     // one query head per CTA
    const float4 qv = load4(q + (size_t)col * kHeadDim + lane * 4);
    const int t = t_len[b];
    const int first = win_folded(t + 1, S, wa.R, wa.D);       // offset (from S) of the oldest unfolded token
    const int W = S + (t + 1 - S - first);
    const int slot0 = Rc > 0 ? first % Rc : 0;                // ring slot of the oldest unfolded token
    const TQ *kbase = winK + (size_t)bh * Wcap * kHeadDim + lane * 4, *vbase = winV + (size_t)bh * Wcap * kHeadDim + lane * 4;
    const TQ *kn = k_new + (size_t)bh * kHeadDim + lane * 4, *vn = v_new + (size_t)bh * kHeadDim + lane * 4;
    float m_run = -INFINITY, sum = 0.f;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int w0 = rs; w0 < W; w0 += RS * kWinRows) {
        typename Raw::type kr[kWinRows], vr[kWinRows];
#pragma unroll
        for (int u = 0; u < kWinRows; ++u) {
            const int w = min(w0 + RS * u, W - 1);   // rows past W repeat the last one; their scores are dropped
            // row of the window tensor, or the step's new token
            const int n = first + w - S;             // offset from S of an unfolded token (w >= S)
            const bool is_new = w >= S && n == t - S;
            int slot = slot0 + w - S;                // n mod Rc: at most Rc tokens wait, so one wrap at most
            if (slot >= Rc) slot -= Rc;
            const size_t off = (size_t)(w < S ? w : S + slot) * kHeadDim;
            kr[u] = Raw::load(is_new ? kn : kbase + off);
            vr[u] = Raw::load(is_new ? vn : vbase + off);
        }
        float d[kWinRows];
#pragma unroll
        for (int u = 0; u < kWinRows; ++u) {
            const float4 k4 = Raw::cvt(kr[u]);
            d[u] = k4.x * qv.x + k4.y * qv.y + k4.z * qv.z + k4.w * qv.w;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1)
#pragma unroll
            for (int u = 0; u < kWinRows; ++u) d[u] += __shfl_xor_sync(0xffffffffu, d[u], o);   // independent chains
        float m_new = m_run;
#pragma unroll
        for (int u = 0; u < kWinRows; ++u) {
            d[u] = w0 + RS * u < W ? d[u] * wa.scale : -INFINITY;
            m_new = fmaxf(m_new, d[u]);
        }
        const float f = m_run == -INFINITY ? 0.f : __expf(m_run - m_new);      // m_new is finite: row w0 exists
        sum *= f;
        acc.x *= f; acc.y *= f; acc.z *= f; acc.w *= f;
#pragma unroll
        for (int u = 0; u < kWinRows; ++u) {
            const float p = __expf(d[u] - m_new);                              // 0 for the rows past W
            const float4 v4 = Raw::cvt(vr[u]);
            sum += p;
            acc.x = fmaf(p, v4.x, acc.x); acc.y = fmaf(p, v4.y, acc.y);
            acc.z = fmaf(p, v4.z, acc.z); acc.w = fmaf(p, v4.w, acc.w);
        }
        m_run = m_new;
    }
    // the row shares meet in shared memory
    o_s[rs][lane] = acc;
    if (lane == 0) {
        m_s[rs] = m_run;
        s_s[rs] = sum;
    }
    __syncthreads();
    {
        const int c = threadIdx.x;                             // 128 threads, 128 channels
        float m = m_s[0];
#pragma unroll
        for (int r = 1; r < RS; ++r) m = fmaxf(m, m_s[r]);
        float o = 0.f, sm = 0.f;
#pragma unroll
        for (int r = 0; r < RS; ++r) {
            const float f = m_s[r] == -INFINITY ? 0.f : __expf(m_s[r] - m);
            sm = fmaf(s_s[r], f, sm);
            o = fmaf(reinterpret_cast<const float *>(&o_s[r][0])[c], f, o);
        }
        wa.o_w[(size_t)col * kHeadDim + c] = o;
        if (c == 0) {
            wa.m_w[col] = m;
            wa.s_w[col] = sm;
        }
    }
}

// Block fold (Eq. 12 for D tokens at once): for every sequence whose token count reaches a block boundary with
// this step's token, the D oldest unfolded tokens are folded into C_K and C_V at the next D positions of the
// transformed segment, oldest first, with the very FMAs of D single-token updates (bit-identical planes:
// x * (-s) is -(x * s) exactly).  t_len is not changed.
//
// Work items are (sequence, group of 64 bins, share of the 2H {kv head, K or V} planes), dealt round-robin to a
// grid of a few CTAs per SM; items of sequences that do not fold this step cost one look at t_len, so the
// launch is nearly free on the steps without a fold.  Per item the 64 x D twiddles are computed once (they
// depend on bin and position only) and kept in shared memory as (c, -s), token-major; per plane the D token rows
// are staged as float, then each warp owns 8 bins (a lane holds 4 of the 128 channels): per token one 16-byte
// read of the token row and four 16-byte broadcast reads of twiddles, all at fixed offsets from one running
// pointer each, feed 64 FMAs -- the kernel is bound by FMA issue, not by HBM.
// grid = (n_ctas); block = 256; dynamic smem = block_fold_smem(D).
constexpr int kFoldBins = 8;                       // bins per warp
constexpr int kFoldWarps = 8;
constexpr int kFoldGroup = kFoldBins * kFoldWarps; // bins per work item
inline size_t block_fold_smem(int D) {
    return (size_t)D * kHeadDim * sizeof(float) + (size_t)kFoldGroup * D * sizeof(float2);
}

template <typename T>
__global__ void __launch_bounds__(kFoldWarps * 32, 3)
k_block_fold(float *__restrict__ coefK, float *__restrict__ coefV, const int32_t *__restrict__ t_len,
             const int32_t *__restrict__ bins, WindowArgs wa, int M, int H, int batch, uint32_t P, int splits) {
    extern __shared__ __align__(16) unsigned char fold_smem[];
    const int S = wa.S, R = wa.R, D = wa.D, Rc = wa.Rc;
    float *xs = reinterpret_cast<float *>(fold_smem);                                                    // [D][128]
    float2 *tws = reinterpret_cast<float2 *>(fold_smem + (size_t)D * kHeadDim * sizeof(float));          // [D][64]
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_groups = (M + kFoldGroup - 1) / kFoldGroup, combos = 2 * H, per_split = (combos + splits - 1) / splits;
    const int n_items = batch * n_groups * splits;
    const size_t plane = (size_t)M * kHeadDim;
    for (int item = blockIdx.x; item < n_items; item += gridDim.x) {
        const int sp = item % splits, grp = (item / splits) % n_groups, b = item / (splits * n_groups);
        const int t = t_len[b];
        const int cnt = t + 1 - S - R;               // unfolded tokens beyond the recent window, with the new one
        if (cnt <= 0 || cnt % D != 0) continue;      // the whole CTA agrees: t depends on the sequence only
        const int first = cnt - D;                   // tokens already folded = position of the oldest waiting one
        const int k0 = grp * kFoldGroup;
        __syncthreads();                             // the previous item's tables are no longer read
        for (int e = threadIdx.x; e < kFoldGroup * D; e += blockDim.x) {
            const int i = e / kFoldGroup, j = e % kFoldGroup;
            float cs, sn;                            // columns past the last bin repeat it; nothing stores their results
            twiddle(phase_mod((uint32_t)bins[min(k0 + j, M - 1)], (uint32_t)(first + i) % P, P), P, cs, sn);
            tws[e] = make_float2(cs, -sn);
        }
        const int kb = k0 + warp * kFoldBins, nb = max(0, min(kFoldBins, M - kb));
        for (int cb = sp * per_split; cb < min(combos, (sp + 1) * per_split); ++cb) {
            const int unit = b * H + (cb >> 1), kv = cb & 1;
            const T *win = static_cast<const T *>(kv == 0 ? wa.winK : wa.winV);
            const T *x_new = static_cast<const T *>(kv == 0 ? wa.k_new : wa.v_new);
            __syncthreads();                         // the previous plane's token rows are no longer read
            for (int i = warp; i < D; i += kFoldWarps) {
                const int n = first + i;             // token S + n
                const T *row = (S + n == t) ? x_new + (size_t)unit * kHeadDim
                                            : win + ((size_t)unit * (S + Rc) + S + n % Rc) * kHeadDim;
                *reinterpret_cast<float4 *>(xs + i * kHeadDim + lane * 4) = load4(row + lane * 4);
            }
            __syncthreads();
            if (nb == 0) continue;
            float *base = (kv == 0 ? coefK : coefV) + (size_t)unit * 2 * plane;
            float4 re[kFoldBins], im[kFoldBins];
#pragma unroll
            for (int j = 0; j < kFoldBins; ++j) {
                re[j] = im[j] = make_float4(0.f, 0.f, 0.f, 0.f);
                if (j < nb) {
                    const float *rp = base + (size_t)(kb + j) * kHeadDim + lane * 4;
                    re[j] = ld_stream(rp);
                    im[j] = ld_stream(rp + plane);
                }
            }
            const float4 *tp = reinterpret_cast<const float4 *>(tws + warp * kFoldBins);   // two bins' (c, -s) per read
            const float4 *xp = reinterpret_cast<const float4 *>(xs) + lane;
#pragma unroll 2
            for (int i = 0; i < D; ++i, tp += kFoldGroup / 2, xp += kHeadDim / 4) {
                const float4 x = *xp;
#pragma unroll
                for (int j = 0; j < kFoldBins; j += 2) {
                    const float4 w = tp[j / 2];
                    re[j].x = fmaf(x.x, w.x, re[j].x); im[j].x = fmaf(x.x, w.y, im[j].x);
                    re[j].y = fmaf(x.y, w.x, re[j].y); im[j].y = fmaf(x.y, w.y, im[j].y);
                    re[j].z = fmaf(x.z, w.x, re[j].z); im[j].z = fmaf(x.z, w.y, im[j].z);
                    re[j].w = fmaf(x.w, w.x, re[j].w); im[j].w = fmaf(x.w, w.y, im[j].w);
                    re[j + 1].x = fmaf(x.x, w.z, re[j + 1].x); im[j + 1].x = fmaf(x.x, w.w, im[j + 1].x);
                    re[j + 1].y = fmaf(x.y, w.z, re[j + 1].y); im[j + 1].y = fmaf(x.y, w.w, im[j + 1].y);
                    re[j + 1].z = fmaf(x.z, w.z, re[j + 1].z); im[j + 1].z = fmaf(x.z, w.w, im[j + 1].z);
                    re[j + 1].w = fmaf(x.w, w.z, re[j + 1].w); im[j + 1].w = fmaf(x.w, w.w, im[j + 1].w);
                }
            }
#pragma unroll
            for (int j = 0; j < kFoldBins; ++j) {
                if (j < nb) {
                    float *wp = base + (size_t)(kb + j) * kHeadDim + lane * 4;
                    st_stream(wp, re[j]);
                    st_stream(wp + plane, im[j]);
                }
            }
        }
    }
}

}  // namespace faedkv
