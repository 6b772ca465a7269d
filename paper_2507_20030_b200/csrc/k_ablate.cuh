// Small kernels of the frequency-ablation transform (Sec. 3.2, Eq. 6): scale the coefficient planes by
// a per-bin gain, and subtract the reconstructed component from the input.
#pragma once
#include "common.cuh"

namespace faedkv {

// coef[unit][plane][i][c] *= gain[i].  One thread per 4 channels; n_vec = units * 2 * M * 32.
__global__ void k_scale_planes(float *__restrict__ coef, const float *__restrict__ gain, int M, size_t n_vec) {
    const size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= n_vec) return;
    const float g = gain[(int)((e >> 5) % (size_t)M)];
    float4 v = *reinterpret_cast<float4 *>(coef + e * 4);
    v.x *= g; v.y *= g; v.z *= g; v.w *= g;
    *reinterpret_cast<float4 *>(coef + e * 4) = v;
}

// y = x - y, elementwise over n values of the storage type (y holds the reconstructed component).
template <typename T>
__global__ void k_subtract_from(const T *__restrict__ x, T *__restrict__ y, size_t n) {
    const size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (e < n) store1(y + e, load1(x + e) - load1(y + e));
}

}  // namespace faedkv
