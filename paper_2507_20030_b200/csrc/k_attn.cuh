// The two coefficient streams of frequency-domain decode attention (Eq. 3 on
// the reconstruction of Eq. 11, rewritten by linearity of the inverse DFT):
//
//   (1) Qf[g,k]   = sum_c q[g,c] * C_K[k,c]                  (k_attn_qf: reads C_K once)
//   (2) s[g,n]    = scale/P * sum_k w_k Re(Qf[g,k] e^{+jwkn})   (inverse transform, M -> L)
//   (3) p         = softmax_n(s)
//   (4) Pf[g,k]   = sum_n p[g,n] e^{+jwkn}                     (forward transform, L -> M)
//   (5) out[g,c]  = 1/P * sum_k w_k Re(C_V[k,c] * Pf[g,k])     (k_attn_out: reads C_V once)
//
// so that  out = softmax(scale * q K~^T) V~  without K~ or V~ ever being written.
// The query heads that share a kv head (GQ of them) share one pass over the
// planes of that head.
//
// Scratch layouts (float32): Qf, Pf [batch][2][M][HQP], HQP = n_q_heads rounded
// up to 32, query head contiguous; partial outputs [batch*H][slices][GQ][128].
#pragma once
#include "common.cuh"

namespace faedkv {

constexpr int kAttnWarps = 8;

// Sum 32 per-lane values across the warp in 31 shuffles; afterwards lane l
// holds the total of value l in v[0].
__device__ __forceinline__ float warp_transpose_reduce32(float (&v)[32], int lane) {
#pragma unroll
    for (int s = 16; s >= 1; s >>= 1) {
        const bool up = (lane & s) != 0;
#pragma unroll
        for (int i = 0; i < s; ++i) {
            float send = up ? v[i] : v[i + s];
            float keep = up ? v[i + s] : v[i];
            v[i] = keep + __shfl_xor_sync(0xffffffffu, send, s);
        }
    }
    return v[0];
}

// Bins a warp of the C_K pass takes: KB bins x 2 planes x GQ query heads are the (at most 32) dot products
// that one transpose-reduce finishes; any GQ from 1 to 8 (with GQ = 3, 5, 6, 7 a few of the 32 slots stay empty).
__host__ __device__ constexpr int attn_bins_per_warp(int GQ) { return 16 / GQ; }

// (1) grid = (ceil(M / (8 * KB)), batch * H); block = 256; KB = attn_bins_per_warp(GQ).
template <typename TQ, int GQ>
__global__ void __launch_bounds__(kAttnWarps * 32)
k_attn_qf(const TQ *__restrict__ q, const float *__restrict__ coefK, float *__restrict__ Qf,
          int M, int H, int HQ, int HQP) {
    constexpr int KB = attn_bins_per_warp(GQ);  // KB * 2 planes * GQ heads <= 32 values
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int bh = blockIdx.y, b = bh / H, h = bh % H;
    const int k0 = (blockIdx.x * kAttnWarps + warp) * KB;
    if (k0 >= M) return;
    float4 qv[GQ];
#pragma unroll
    for (int g = 0; g < GQ; ++g)
        qv[g] = load4(q + ((size_t)b * HQ + h * GQ + g) * kHeadDim + lane * 4);
    const size_t plane = (size_t)M * kHeadDim;
    const float *base = coefK + (size_t)bh * 2 * plane;
    float4 row[KB][2];
#pragma unroll
    for (int kk = 0; kk < KB; ++kk)
#pragma unroll
        for (int pl = 0; pl < 2; ++pl) {
            row[kk][pl] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (k0 + kk < M)
                row[kk][pl] = ld_stream(base + pl * plane + (size_t)(k0 + kk) * kHeadDim + lane * 4);
        }
    float v[32];
#pragma unroll
    for (int i = KB * 2 * GQ; i < 32; ++i) v[i] = 0.f;
#pragma unroll
    for (int kk = 0; kk < KB; ++kk)
#pragma unroll
        for (int pl = 0; pl < 2; ++pl)
#pragma unroll
            for (int g = 0; g < GQ; ++g) {
                const float4 r = row[kk][pl];
                v[(kk * 2 + pl) * GQ + g] = r.x * qv[g].x + r.y * qv[g].y + r.z * qv[g].z + r.w * qv[g].w;
            }
    const float tot = warp_transpose_reduce32(v, lane);
    const int kk = lane / (2 * GQ), pl = (lane / GQ) & 1, g = lane % GQ;
    if (kk < KB && k0 + kk < M)
        Qf[(((size_t)b * 2 + pl) * M + (k0 + kk)) * HQP + h * GQ + g] = tot;
}

// (5) grid = (slices, batch * H); block = 256.  Each CTA reduces its slice of
// bins for the GQ heads of one kv head and writes a [GQ][128] partial.
template <int GQ>
__global__ void __launch_bounds__(kAttnWarps * 32)
k_attn_out(const float *__restrict__ coefV, const float *__restrict__ Pf,
           const int32_t *__restrict__ bins, float *__restrict__ partial, int M, int H, int HQP,
           uint32_t P, int bins_per_slice) {
    __shared__ __align__(16) float red[kAttnWarps][GQ][kHeadDim];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int bh = blockIdx.y, b = bh / H, h = bh % H;
    const int kbeg = blockIdx.x * bins_per_slice;
    const int kend = min(M, kbeg + bins_per_slice);
    const size_t plane = (size_t)M * kHeadDim;
    const float *base = coefV + (size_t)bh * 2 * plane;
    const float *pre = Pf + ((size_t)b * 2) * M * HQP + h * GQ;
    const float *pim = pre + (size_t)M * HQP;
    float4 acc[GQ];
#pragma unroll
    for (int g = 0; g < GQ; ++g) acc[g] = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int k = kbeg + warp; k < kend; k += kAttnWarps) {
        const float4 re = ld_stream(base + (size_t)k * kHeadDim + lane * 4);
        const float4 im = ld_stream(base + plane + (size_t)k * kHeadDim + lane * 4);
        const float w = hermitian_weight((uint32_t)bins[k], P);
#pragma unroll
        for (int g = 0; g < GQ; ++g) {
            const float a = w * pre[(size_t)k * HQP + g];
            const float c = -w * pim[(size_t)k * HQP + g];
            acc[g].x = fmaf(re.x, a, fmaf(im.x, c, acc[g].x));
            acc[g].y = fmaf(re.y, a, fmaf(im.y, c, acc[g].y));
            acc[g].z = fmaf(re.z, a, fmaf(im.z, c, acc[g].z));
            acc[g].w = fmaf(re.w, a, fmaf(im.w, c, acc[g].w));
        }
    }
#pragma unroll
    for (int g = 0; g < GQ; ++g) *reinterpret_cast<float4 *>(&red[warp][g][lane * 4]) = acc[g];
    __syncthreads();
    for (int e = threadIdx.x; e < GQ * kHeadDim; e += blockDim.x) {
        const int g = e / kHeadDim, c = e % kHeadDim;
        float s = 0.f;
#pragma unroll
        for (int w = 0; w < kAttnWarps; ++w) s += red[w][g][c];
        partial[(((size_t)bh * gridDim.x + blockIdx.x) * GQ + g) * kHeadDim + c] = s;
    }
}

// Sum the slice partials, apply 1/P, convert to the output type.
// grid = batch * H * GQ; block = 128.
template <typename TOut>
__global__ void k_attn_out_reduce(const float *__restrict__ partial, TOut *__restrict__ out,
                                  int slices, int GQ, float inv_P) {
    const int bh = blockIdx.x / GQ, g = blockIdx.x % GQ, c = threadIdx.x;
    float s = 0.f;
    for (int sl = 0; sl < slices; ++sl)
        s += partial[(((size_t)bh * slices + sl) * GQ + g) * kHeadDim + c];
    // out is [batch][HQ][128] with HQ = H * GQ, so (bh, g) is already the flat head index
    store1(out + ((size_t)bh * GQ + g) * kHeadDim + c, s * inv_P);
}

}  // namespace faedkv
