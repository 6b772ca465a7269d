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
        const int mid = t - f.S - f.R;                 // tokens already in the transformed segment
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

// Attention over the time-domain tokens of one (sequence, kv head) for its GQ query heads, in the same
// unnormalised form as a tile of the transformed segment: per column the maximum score m, the sum of
// exp(s - m), and o_w[col][c] = sum_w exp(s_w - m) v_w[c].  Rows: the S sink tokens, then the unfolded tokens
// [S + folded(t + 1), t] in token order, where t = t_len is the step's new token; its ring slot is written only
// at the end of the step, so k_new / v_new stand in for that row.  No rows at all: m = -inf, sum = 0, o = 0.
// The host runs it on a second stream beside the first two FFT kernels, which leave the memory system idle:
// beside a bandwidth-saturating pass its dependent loads would each cost many microseconds.
// grid = (units, GQ): one CTA per query head; block = 256; dynamic smem = (S + Rc) floats.
struct WindowArgs {
    const void *winK, *winV, *k_new, *v_new;   // storage type of the context
    int S, R, D, Rc;                           // sink, recent, defer block, ring capacity (win_ring(R, D))
    float scale;
    float *m_w, *s_w, *o_w;                    // statistics row of the window, [Gp] each; output [Gp][128]
};

template <typename TQ, int GQ>
__global__ void __launch_bounds__(256)
k_attn_window(const TQ *__restrict__ q, WindowArgs wa, const int32_t *__restrict__ t_len, int H) {
    extern __shared__ float sc[];                     // [W] scores, then exp(s - m)
    __shared__ float part[kHeadDim];
    const TQ *winK = static_cast<const TQ *>(wa.winK), *winV = static_cast<const TQ *>(wa.winV);
    const TQ *k_new = static_cast<const TQ *>(wa.k_new), *v_new = static_cast<const TQ *>(wa.v_new);
    const int S = wa.S, Rc = wa.Rc, Wcap = S + Rc;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int bh = blockIdx.x, b = bh / H, col = bh * GQ + (int)blockIdx.y;     // one query head per CTA
    const int t = t_len[b];
    const int first = win_folded(t + 1, S, wa.R, wa.D);       // offset (from S) of the oldest unfolded token
    const int W = S + (t + 1 - S - first);
    // row w -> its row in the window tensor, or -1 for the step's new token
    auto locate = [&](int w) { return w < S ? w : (first + w - S == t - S ? -1 : S + (first + w - S) % Rc); };
    const float4 qv = load4(q + (size_t)col * kHeadDim + lane * 4);
    // scores: a warp takes rows w = warp + 8u, all loads of a batch of 8 issued before any is used
    for (int w0 = warp; w0 < W; w0 += 64) {
        float4 kv[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int w = w0 + 8 * u;
            kv[u] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (w < W) {
                const int row = locate(w);
                const TQ *krow = row < 0 ? k_new + (size_t)bh * kHeadDim : winK + ((size_t)bh * Wcap + row) * kHeadDim;
                kv[u] = load4(krow + lane * 4);
            }
        }
        float d[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) d[u] = kv[u].x * qv.x + kv[u].y * qv.y + kv[u].z * qv.z + kv[u].w * qv.w;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1)
#pragma unroll
            for (int u = 0; u < 8; ++u) d[u] += __shfl_xor_sync(0xffffffffu, d[u], o);     // 8 independent chains
        if (lane < 8 && w0 + 8 * lane < W) {
            float v = d[0];
#pragma unroll
            for (int u = 1; u < 8; ++u) v = lane == u ? d[u] : v;
            sc[w0 + 8 * lane] = v * wa.scale;
        }
    }
    __syncthreads();
    if (warp == 0) {
        float m = -INFINITY;
        for (int w = lane; w < W; w += 32) m = fmaxf(m, sc[w]);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
        float sum = 0.f;
        for (int w = lane; w < W; w += 32) {
            const float p = __expf(sc[w] - m);
            sc[w] = p;
            sum += p;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
        if (lane == 0) {
            wa.m_w[col] = m;
            wa.s_w[col] = sum;
        }
    }
    __syncthreads();
    // output: thread (channel c, half) sums the rows of its parity, 8 loads in flight; halves meet in shared memory
    const int c = threadIdx.x & (kHeadDim - 1), half = threadIdx.x >> 7;
    float acc = 0.f;
    for (int w0 = half; w0 < W; w0 += 16) {
        float vv[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int w = w0 + 2 * u;
            vv[u] = 0.f;
            if (w < W) {
                const int row = locate(w);
                const TQ *vrow = row < 0 ? v_new + (size_t)bh * kHeadDim : winV + ((size_t)bh * Wcap + row) * kHeadDim;
                vv[u] = load1(vrow + c);
            }
        }
#pragma unroll
        for (int u = 0; u < 8; ++u)
            if (w0 + 2 * u < W) acc = fmaf(sc[w0 + 2 * u], vv[u], acc);
    }
    if (half == 1) part[c] = acc;
    __syncthreads();
    if (half == 0) wa.o_w[(size_t)col * kHeadDim + c] = acc + part[c];
}

// Block fold (Eq. 12 for D tokens at once): for every sequence whose token count reaches a block boundary with
// this step's token, the D oldest unfolded tokens are folded into C_K and C_V at the next D positions of the
// transformed segment, oldest first, with the very FMAs of D single-token updates (bit-identical planes).
// The other sequences' CTAs return at once.  t_len is not changed here.
// A warp owns kFoldBins bins at a time (a lane holds 4 of the 128 channels); the D tokens of the unit sit in
// shared memory as float, the D twiddles of each bin are computed by the lanes and broadcast through shared
// memory, so one token row read feeds kFoldBins * 8 FMAs.
// grid = (ceil(M / (8 * kFoldBins)), units, 2 {K, V}); block = 256;
// dynamic smem = D * 128 floats + 8 warps * kFoldBins * D float2.
constexpr int kFoldBins = 4;
constexpr int kFoldWarps = 8;
inline size_t block_fold_smem(int D) {
    return (size_t)D * kHeadDim * sizeof(float) + (size_t)kFoldWarps * kFoldBins * D * sizeof(float2);
}

template <typename T>
__global__ void __launch_bounds__(kFoldWarps * 32)
k_block_fold(float *__restrict__ coefK, float *__restrict__ coefV, const int32_t *__restrict__ t_len,
             const int32_t *__restrict__ bins, WindowArgs wa, int M, int H, uint32_t P) {
    extern __shared__ __align__(16) unsigned char fold_smem[];
    const int S = wa.S, R = wa.R, D = wa.D, Rc = wa.Rc;
    const int unit = blockIdx.y, b = unit / H, kv = blockIdx.z;
    const int t = t_len[b];
    const int cnt = t + 1 - S - R;                   // unfolded tokens beyond the recent window, with the new one
    if (cnt <= 0 || cnt % D != 0) return;
    const int first = cnt - D;                       // tokens already folded = position of the oldest unfolded one
    float *xs = reinterpret_cast<float *>(fold_smem);                                        // [D][128]
    float2 *tws = reinterpret_cast<float2 *>(fold_smem + (size_t)D * kHeadDim * sizeof(float));
    const T *win = static_cast<const T *>(kv == 0 ? wa.winK : wa.winV);
    const T *x_new = static_cast<const T *>(kv == 0 ? wa.k_new : wa.v_new);
    for (int e = threadIdx.x; e < D * kHeadDim; e += blockDim.x) {
        const int i = e / kHeadDim, c = e % kHeadDim;
        const int n = first + i;                     // token S + n
        const T *row = (S + n == t) ? x_new + (size_t)unit * kHeadDim
                                    : win + ((size_t)unit * (S + Rc) + S + n % Rc) * kHeadDim;
        xs[e] = load1(row + c);
    }
    __syncthreads();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    float2 *twl = tws + (size_t)warp * kFoldBins * D;
    const size_t plane = (size_t)M * kHeadDim;
    float *base = (kv == 0 ? coefK : coefV) + (size_t)unit * 2 * plane;
    const int k0 = (blockIdx.x * kFoldWarps + warp) * kFoldBins;
    if (k0 >= M) return;
    const int nb = min(kFoldBins, M - k0);
    for (int e = lane; e < nb * D; e += 32) {
        const int j = e / D, i = e % D;
        float cs, sn;
        twiddle(phase_mod((uint32_t)bins[k0 + j], (uint32_t)(first + i) % P, P), P, cs, sn);
        twl[j * D + i] = make_float2(cs, sn);
    }
    float4 re[kFoldBins], im[kFoldBins];
#pragma unroll
    for (int j = 0; j < kFoldBins; ++j) {
        re[j] = im[j] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (j < nb) {
            const float *rp = base + (size_t)(k0 + j) * kHeadDim + lane * 4;
            re[j] = ld_stream(rp);
            im[j] = ld_stream(rp + plane);
        }
    }
    __syncwarp();
    for (int i = 0; i < D; ++i) {
        const float4 x = *reinterpret_cast<const float4 *>(xs + i * kHeadDim + lane * 4);
#pragma unroll
        for (int j = 0; j < kFoldBins; ++j) {
            const float2 cs = twl[j * D + i];        // rows past nb hold stale values; their results are dropped
            re[j].x = fmaf(x.x, cs.x, re[j].x); im[j].x = fmaf(-x.x, cs.y, im[j].x);
            re[j].y = fmaf(x.y, cs.x, re[j].y); im[j].y = fmaf(-x.y, cs.y, im[j].y);
            re[j].z = fmaf(x.z, cs.x, re[j].z); im[j].z = fmaf(-x.z, cs.y, im[j].z);
            re[j].w = fmaf(x.w, cs.x, re[j].w); im[j].w = fmaf(-x.w, cs.y, im[j].w);
        }
    }
#pragma unroll
    for (int j = 0; j < kFoldBins; ++j) {
        if (j < nb) {
            float *wp = base + (size_t)(k0 + j) * kHeadDim + lane * 4;
            st_stream(wp, re[j]);
            st_stream(wp + plane, im[j]);
        }
    }
}

}  // namespace faedkv
