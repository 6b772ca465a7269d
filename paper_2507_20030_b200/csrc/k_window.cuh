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
// grid = units; block = 256; dynamic smem = GQ * (S + R) floats.
template <typename TQ, int GQ>
__global__ void __launch_bounds__(256)
k_attn_window(const TQ *__restrict__ q, const TQ *__restrict__ winK, const TQ *__restrict__ winV,
              const TQ *__restrict__ k_new, const TQ *__restrict__ v_new, const int32_t *__restrict__ t_len, int H,
              int S, int R, float scale, float *__restrict__ m_w, float *__restrict__ s_w, float *__restrict__ o_w) {
    extern __shared__ float sc[];                     // [GQ][W]

    const int W = S + R;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int bh = blockIdx.x, b = bh / H;
    const int t = t_len[b];
    const int slot_new = R > 0 ? S + (t - S) % R : -1;
    const int col0 = bh * GQ;
    float4 qv[GQ];
#pragma unroll
    for (int g = 0; g < GQ; ++g) qv[g] = load4(q + (size_t)(col0 + g) * kHeadDim + lane * 4);
    for (int w = warp; w < W; w += 8) {
        const TQ *krow = (w == slot_new) ? k_new + (size_t)bh * kHeadDim : winK + ((size_t)bh * W + w) * kHeadDim;
        const float4 kv = load4(krow + lane * 4);
#pragma unroll
        for (int g = 0; g < GQ; ++g) {
            float d = kv.x * qv[g].x + kv.y * qv[g].y + kv.z * qv[g].z + kv.w * qv[g].w;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) d += __shfl_xor_sync(0xffffffffu, d, o);
            if (lane == 0) sc[g * W + w] = d * scale;
        }
    }
    __syncthreads();
    if (warp < GQ) {
        float m = -INFINITY;
        for (int w = lane; w < W; w += 32) m = fmaxf(m, sc[warp * W + w]);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
        float sum = 0.f;
        for (int w = lane; w < W; w += 32) {
            const float p = __expf(sc[warp * W + w] - m);
            sc[warp * W + w] = p;
            sum += p;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
        if (lane == 0) {
            m_w[col0 + warp] = m;
            s_w[col0 + warp] = sum;
        }
    }
    __syncthreads();
    const int c = threadIdx.x & (kHeadDim - 1);
    for (int g = threadIdx.x >> 7; g < GQ; g += 2) {
        float acc = 0.f;
        for (int w = 0; w < W; ++w) {
            const TQ *vrow = (w == slot_new) ? v_new + (size_t)bh * kHeadDim : winV + ((size_t)bh * W + w) * kHeadDim;
            acc = fmaf(sc[g * W + w], load1(vrow + c), acc);
        }
        o_w[(size_t)(col0 + g) * kHeadDim + c] = acc;
    }
}

// End of a windowed step: the new token takes its ring slot (R > 0) and the token counters advance.
// grid = batch; block = 128.
template <typename T>
__global__ void k_window_commit(const T *__restrict__ k_new, const T *__restrict__ v_new, T *__restrict__ winK,
                                T *__restrict__ winV, int32_t *__restrict__ t_len, int H, int S, int R) {
    const int b = blockIdx.x, c = threadIdx.x;
    const int t = t_len[b];
    if (R > 0) {
        const int slot = S + (t - S) % R;
        for (int h = 0; h < H; ++h) {
            const size_t unit = (size_t)b * H + h;
            winK[(unit * (S + R) + slot) * kHeadDim + c] = k_new[unit * kHeadDim + c];
            winV[(unit * (S + R) + slot) * kHeadDim + c] = v_new[unit * kHeadDim + c];
        }
    }
    __syncthreads();
    if (c == 0) t_len[b] = t + 1;
}

}  // namespace faedkv
