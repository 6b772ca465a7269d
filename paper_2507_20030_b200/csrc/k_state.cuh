// Conversions between the library's state and the two forms the paper's equations print (Sec. 4.1):
//   SUM       C_t[k] = sum_{n<t} x[n] e^{-j w k n}                (what every call here keeps)
//   MEAN      S_t[k] = C_t[k] / t                                  (Eq. 9 with its exact factors (t-1)/t, 1/t)
//   ROTATING  R_t[k] = e^{-j w k t} * conj(C_t[k])                 (Eq. 8 / Eq. 9 without normalisation:
//                                                                   R <- W_k (R + x), newest-token-referenced)
// For real x the three hold the same information.  ROTATING <-> SUM is its own inverse.
#pragma once
#include "common.cuh"

namespace faedkv {

enum { kStateSum = 0, kStateMean = 1, kStateRotating = 2 };

// One warp per (unit, bin); grid = (ceil(M / 8), units); block = 256.  in, out: [units][2][M][128]
// (may alias).  Converts `from` -> SUM -> `to` in registers.
__global__ void __launch_bounds__(256)
k_convert_state(const float *in, float *out, const int32_t *__restrict__ bins, const int32_t *__restrict__ t_len,
                int M, int H, uint32_t P, int from, int to) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int i = blockIdx.x * 8 + warp, unit = blockIdx.y;
    if (i >= M) return;
    const int t = t_len[unit / H];
    const size_t plane = (size_t)M * kHeadDim, off = ((size_t)unit * 2 * M + i) * kHeadDim + lane * 4;
    float4 re = *reinterpret_cast<const float4 *>(in + off), im = *reinterpret_cast<const float4 *>(in + off + plane);
    float c = 1.f, s = 0.f;
    if (from == kStateRotating || to == kStateRotating) twiddle(phase_mod((uint32_t)bins[i], (uint32_t)t % P, P), P, c, s);
    auto rotate = [&](float4 &a, float4 &b) {        // (a + jb) -> conj((c + js)(a + jb)) = (ca - sb) - j(cb + sa)
        const float4 na = make_float4(c * a.x - s * b.x, c * a.y - s * b.y, c * a.z - s * b.z, c * a.w - s * b.w);
        b = make_float4(-(c * b.x + s * a.x), -(c * b.y + s * a.y), -(c * b.z + s * a.z), -(c * b.w + s * a.w));
        a = na;
    };
    auto scale = [&](float4 &a, float f) { a.x *= f; a.y *= f; a.z *= f; a.w *= f; };
    if (from == kStateMean) { scale(re, (float)t); scale(im, (float)t); }
    if (from == kStateRotating) rotate(re, im);
    if (to == kStateMean) { const float f = t > 0 ? 1.0f / (float)t : 0.f; scale(re, f); scale(im, f); }
    if (to == kStateRotating) rotate(re, im);
    *reinterpret_cast<float4 *>(out + off) = re;
    *reinterpret_cast<float4 *>(out + off + plane) = im;
}

}  // namespace faedkv
