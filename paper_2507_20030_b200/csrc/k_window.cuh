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

// Prefill: copy the sink rows and place the last R tokens in their ring slots.
// grid = (S + R, units); block = 128.  K, V: [units][T][128].
template <typename T>
__global__ void k_window_fill(const T *__restrict__ K, const T *__restrict__ V, T *__restrict__ winK, T *__restrict__ winV,
                              int Ttot, int S, int R) {
    const int w = blockIdx.x, unit = blockIdx.y, c = threadIdx.x;
    int src, dst;
    if (w < S) {
        src = w; dst = w;
    } else {
        src = Ttot - R + (w - S);
        dst = S + (src - S) % R;
    }
    const size_t so = ((size_t)unit * Ttot + src) * kHeadDim + c, d_o = ((size_t)unit * (S + R) + dst) * kHeadDim + c;
    winK[d_o] = K[so];
    winV[d_o] = V[so];
}

// Attention over the window tokens of one (sequence, kv head) for its GQ query heads, in the same
// unnormalised form as a tile of the transformed segment: per column the maximum score m, the sum of
// exp(s - m), and o_w[col][c] = sum_w exp(s_w - m) v_w[c].  The slot of the step's new token still holds
// the token that leaves the window, so k_new / v_new stand in for that row.
// The host runs it on a second stream beside the first two FFT kernels, which leave the memory system idle:
// beside a bandwidth-saturating pass its dependent loads would each cost many microseconds.
// grid = (units, GQ): one CTA per query head; block = 256; dynamic smem = (S + R) floats.
struct WindowArgs {
    const void *winK, *winV, *k_new, *v_new;   // storage type of the context
    int S, R;
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
    const int S = wa.S, R = wa.R, W = S + R;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int bh = blockIdx.x, b = bh / H, col = bh * GQ + (int)blockIdx.y;     // one query head per CTA
    const int t = t_len[b];
    const int slot_new = R > 0 ? S + (t - S) % R : -1;
    const float4 qv = load4(q + (size_t)col * kHeadDim + lane * 4);
    // scores: a warp takes rows w = warp + 8u, all loads of a batch of 8 issued before any is used
    for (int w0 = warp; w0 < W; w0 += 64) {
        float4 kv[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int w = w0 + 8 * u;
            kv[u] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (w < W) {
                const TQ *krow = (w == slot_new) ? k_new + (size_t)bh * kHeadDim : winK + ((size_t)bh * W + w) * kHeadDim;
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
                const TQ *vrow = (w == slot_new) ? v_new + (size_t)bh * kHeadDim : winV + ((size_t)bh * W + w) * kHeadDim;
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

}  // namespace faedkv
