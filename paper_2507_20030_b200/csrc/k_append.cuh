// IWDFT update (Sec. 4.1 Eq. 9 in unnormalised start-referenced form; Eq. 12):
//   coef[b,h,re,k,c] += x[b,h,c] * cos(2*pi*bins[k]*t/P)
//   coef[b,h,im,k,c] -= x[b,h,c] * sin(2*pi*bins[k]*t/P),   t = t_len[b]
// for K and V in one launch, then t_len[b] += 1.
//
// A pure stream over the coefficient planes: every float is read once and
// written once, 1 FMA each.  One warp owns one bin: a lane holds 4 of the 128
// channels, so each warp access is one 512-byte row; the twiddle of the bin is
// computed once per warp and reused for all kv heads of K and V (it depends on
// (sequence, bin) only).  Loads of four heads are issued before their FMAs to
// keep >= 8 x 16 B per thread in flight.
#pragma once
#include "common.cuh"

namespace faedkv {

constexpr int kAppendWarps = 8;  // bins per CTA

template <typename TIn>
__global__ void __launch_bounds__(kAppendWarps * 32)
k_append(const TIn *__restrict__ k_new, const TIn *__restrict__ v_new, float *__restrict__ coefK,
         float *__restrict__ coefV, int32_t *__restrict__ t_len, const int32_t *__restrict__ bins,
         int M, int H, uint32_t P, unsigned int *__restrict__ tick) {
    const int b = blockIdx.y;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int k = blockIdx.x * kAppendWarps + warp;
    if (k < M && FAEDKV_IN_BOUNDS(kTagAppend, (uint32_t)bins[k] <= P / 2 && t_len[b] >= 0)) {
        const uint32_t t = (uint32_t)t_len[b];
        float c, s;
        twiddle(phase_mod((uint32_t)bins[k], t % P, P), P, c, s);
        const size_t plane = (size_t)M * kHeadDim;
        const size_t row = (size_t)k * kHeadDim + lane * 4;
#pragma unroll
        for (int kv = 0; kv < 2; ++kv) {
            float *coef = kv == 0 ? coefK : coefV;
            const TIn *xn = kv == 0 ? k_new : v_new;
            if (coef == nullptr) continue;
            int h = 0;
            for (; h + 4 <= H; h += 4) {
                float4 re[4], im[4], x[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    float *base = coef + ((size_t)(b * H + h + i) * 2) * plane + row;
                    re[i] = ld_stream(base);
                    im[i] = ld_stream(base + plane);
                    x[i] = load4(xn + (size_t)(b * H + h + i) * kHeadDim + lane * 4);
                }
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    float *base = coef + ((size_t)(b * H + h + i) * 2) * plane + row;
                    re[i].x = fmaf(x[i].x, c, re[i].x); im[i].x = fmaf(-x[i].x, s, im[i].x);
                    re[i].y = fmaf(x[i].y, c, re[i].y); im[i].y = fmaf(-x[i].y, s, im[i].y);
                    re[i].z = fmaf(x[i].z, c, re[i].z); im[i].z = fmaf(-x[i].z, s, im[i].z);
                    re[i].w = fmaf(x[i].w, c, re[i].w); im[i].w = fmaf(-x[i].w, s, im[i].w);
                    st_stream(base, re[i]);
                    st_stream(base + plane, im[i]);
                }
            }
            for (; h < H; ++h) {
                float *base = coef + ((size_t)(b * H + h) * 2) * plane + row;
                float4 re = ld_stream(base), im = ld_stream(base + plane);
                float4 x = load4(xn + (size_t)(b * H + h) * kHeadDim + lane * 4);
                re.x = fmaf(x.x, c, re.x); im.x = fmaf(-x.x, s, im.x);
                re.y = fmaf(x.y, c, re.y); im.y = fmaf(-x.y, s, im.y);
                re.z = fmaf(x.z, c, re.z); im.z = fmaf(-x.z, s, im.z);
                re.w = fmaf(x.w, c, re.w); im.w = fmaf(-x.w, s, im.w);
                st_stream(base, re);
                st_stream(base + plane, im);
            }
        }
    }
    // The last CTA to finish advances the token counters: every other CTA has
    // read t_len before it took its ticket.
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        const unsigned int total = gridDim.x * gridDim.y;
        if (atomicAdd(tick, 1u) == total - 1u) {
            for (int i = 0; i < (int)gridDim.y; ++i) t_len[i] += 1;
            *tick = 0u;
            __threadfence();
        }
    }
}

}  // namespace faedkv
