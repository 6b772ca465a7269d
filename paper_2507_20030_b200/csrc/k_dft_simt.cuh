// Float32 SIMT evaluation of the two pruned transforms, with twiddles that are
// exact to float32 (integer-reduced phase, then sincospif):
//
//   forward  (Eq. 4 on the retained bins):
//       Yre[k,c] = sum_n x[n,c] cos(w k n),  Yim[k,c] = sgn * sum_n x[n,c] sin(w k n)
//       (sgn = -1: the DFT of the prefill; sgn = +1: its conjugate, used for the
//        probability spectrum of decode attention)
//   inverse  (Eq. 5 with pruned bins zero and Hermitian mirrors implied):
//       x~[n,c] = scale * sum_k w_k (Yre[k,c] cos(w k n) - Yim[k,c] sin(w k n))
//
// "Columns" c are the channels of one unit (NCOL = 128: a kv head's head_dim)
// or the query heads of one sequence (NCOL = n_q_heads) in decode attention.
// These kernels are the exact-float32 path (float32 K/V, reconstruction, the
// two transforms inside decode attention) and the reference point for the
// tensor-core kernels.
#pragma once
#include "common.cuh"

namespace faedkv {

constexpr int kSimtThreads = 256;
constexpr int kTileBins = 32;  // bins per tile
constexpr int kTilePos = 32;   // positions per tile

struct DftUnitArgs {
    const void *x[2];   // forward: inputs of tensor 0/1; inverse: outputs
    float *y[2];        // coefficient planes of tensor 0/1 (re plane, im plane = re + y_plane)
    long long x_unit;   // element stride between units of x
    long long y_unit;   // element stride between units of y
    long long y_plane;  // element stride between the re and im planes
    int x_row;          // element stride between positions of x (>= NCOL)
    int y_row;          // element stride between bins of y (>= NCOL)
    int col_blocks;     // a sequence's columns are split into this many blocks of NCOL;
                        // blockIdx.y = sequence * col_blocks + block
};

// ---------------------------------------------------------------------------
// forward
//   grid  = (ceil(M / 32), units, tensors);  block = 256
//   rows  = rows_host, or min(rows_dev[u / rows_div], P) when rows_dev != nullptr
//   SOFTMAX_IN: x is a float32 score column; the value transformed is
//   exp(x - colmax[u*NCOL + c]) and the result is divided by its column sum
//   (softmax fused into the load; every CTA sees all rows, so each forms the
//   full sum itself).
// ---------------------------------------------------------------------------
template <typename TIn, int NCOL, bool SOFTMAX_IN>
__global__ void __launch_bounds__(kSimtThreads)
k_dft_forward_simt(DftUnitArgs a, const int32_t *__restrict__ bins, int M, uint32_t P,
                   int rows_host, const int32_t *__restrict__ rows_dev, int rows_div,
                   uint32_t pos0, float sgn, int accumulate, const float *__restrict__ colmax) {
    constexpr int CPT = NCOL / 32;  // columns per thread
    static_assert(CPT == 1 || CPT == 4, "NCOL must be 32 or 128");
    __shared__ __align__(16) float xs[kTilePos][NCOL];
    __shared__ __align__(16) float twc[kTilePos][kTileBins];
    __shared__ __align__(16) float tws[kTilePos][kTileBins];

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int u = blockIdx.y / a.col_blocks, blk = blockIdx.y % a.col_blocks, tz = blockIdx.z;
    const int k0 = blockIdx.x * kTileBins;
    const TIn *x = reinterpret_cast<const TIn *>(a.x[tz]) + (size_t)u * a.x_unit + blk * NCOL;
    float *yre = a.y[tz] + (size_t)u * a.y_unit + blk * NCOL;
    float *yim = yre + a.y_plane;
    int rows = rows_host;
    if (rows_dev != nullptr) {
        int t = rows_dev[u / rows_div];
        rows = t < (int)P ? t : (int)P;
    }

    // twiddle generator: this thread owns bin gk and positions gj..gj+3 of every tile
    const int gk = tid & 31, gj = (tid >> 5) * 4;
    uint32_t gbin = (k0 + gk < M) ? (uint32_t)bins[k0 + gk] : 0u;
    if (!FAEDKV_IN_BOUNDS(kTagDftSimt, gbin <= P / 2)) gbin = 0u;
    uint32_t ph[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) ph[i] = phase_mod(gbin, (pos0 + gj + i) % P, P);
    const uint32_t step = phase_mod(gbin, kTilePos % P, P);

    float accre[4][CPT], accim[4][CPT];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < CPT; ++j) accre[i][j] = accim[i][j] = 0.f;
    float colsum[CPT];
    float cmx[CPT];
#pragma unroll
    for (int j = 0; j < CPT; ++j) {
        colsum[j] = 0.f;
        cmx[j] = SOFTMAX_IN ? colmax[(size_t)blockIdx.y * NCOL + lane * CPT + j] : 0.f;
    }

    for (int n0 = 0; n0 < rows; n0 += kTilePos) {
        // stage x tile (zero beyond rows)
        for (int e = tid; e < kTilePos * (NCOL / CPT); e += kSimtThreads) {
            int r = e / (NCOL / CPT), cg = e % (NCOL / CPT);
            int n = n0 + r;
            if (CPT == 4) {
                float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
                if (n < rows) v = load4(x + (size_t)n * a.x_row + cg * 4);
                *reinterpret_cast<float4 *>(&xs[r][cg * 4]) = v;
            } else {
                float v = 0.f;
                if (n < rows) v = load1(x + (size_t)n * a.x_row + cg);
                xs[r][cg] = v;
            }
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            float c, s;
            twiddle(ph[i], P, c, s);
            twc[gj + i][gk] = c;
            tws[gj + i][gk] = s;
            ph[i] = add_mod(ph[i], step, P);
        }
        __syncthreads();
#pragma unroll 4
        for (int j = 0; j < kTilePos; ++j) {
            float xv[CPT];
            if (CPT == 4) {
                float4 v = *reinterpret_cast<const float4 *>(&xs[j][lane * 4]);
                xv[0] = v.x; xv[1 % CPT] = v.y; xv[2 % CPT] = v.z; xv[3 % CPT] = v.w;
            } else {
                xv[0] = xs[j][lane];
            }
            if (SOFTMAX_IN) {
                const bool live = (n0 + j) < rows;
#pragma unroll
                for (int q = 0; q < CPT; ++q) {
                    xv[q] = live ? __expf(xv[q] - cmx[q]) : 0.f;
                    colsum[q] += xv[q];
                }
            }
            const float4 c4 = *reinterpret_cast<const float4 *>(&twc[j][warp * 4]);
            const float4 s4 = *reinterpret_cast<const float4 *>(&tws[j][warp * 4]);
            const float cc[4] = {c4.x, c4.y, c4.z, c4.w};
            const float ss[4] = {s4.x, s4.y, s4.z, s4.w};
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int q = 0; q < CPT; ++q) {
                    accre[i][q] = fmaf(xv[q], cc[i], accre[i][q]);
                    accim[i][q] = fmaf(xv[q], ss[i], accim[i][q]);
                }
        }
        __syncthreads();
    }

#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int k = k0 + warp * 4 + i;
        if (k >= M) continue;
#pragma unroll
        for (int q = 0; q < CPT; ++q) {
            float inv = 1.f;
            if (SOFTMAX_IN) inv = colsum[q] > 0.f ? 1.f / colsum[q] : 0.f;   // no live row: the spectrum of nothing is zero
            const size_t o = (size_t)k * a.y_row + lane * CPT + q;
            float re = accre[i][q] * inv, im = sgn * accim[i][q] * inv;
            if (accumulate) { re += yre[o]; im += yim[o]; }
            yre[o] = re;
            yim[o] = im;
        }
    }
}

// ---------------------------------------------------------------------------
// inverse
//   grid  = (ceil(Lrows / 32), units, tensors);  block = 256
//   Rows n >= min(rows_dev[u / rows_div], P) are written as zero.
//   tile_max (optional): per (unit, row tile, column) maximum of the written
//   values over the live rows of the tile, for the softmax of decode attention.
// ---------------------------------------------------------------------------
template <typename TOut, int NCOL>
__global__ void __launch_bounds__(kSimtThreads)
k_dft_inverse_simt(DftUnitArgs a, const int32_t *__restrict__ bins, int M, uint32_t P, int Lrows,
                   const int32_t *__restrict__ rows_dev, int rows_div, float scale,
                   float *__restrict__ tile_max) {
    constexpr int CPT = NCOL / 32;
    static_assert(CPT == 1 || CPT == 4, "NCOL must be 32 or 128");
    __shared__ __align__(16) float yr[kTileBins][NCOL];
    __shared__ __align__(16) float yi[kTileBins][NCOL];
    __shared__ __align__(16) float twc[kTileBins][kTilePos];
    __shared__ __align__(16) float tws[kTileBins][kTilePos];

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int u = blockIdx.y / a.col_blocks, blk = blockIdx.y % a.col_blocks, tz = blockIdx.z;
    const int n0 = blockIdx.x * kTilePos;
    const float *yre = a.y[tz] + (size_t)u * a.y_unit + blk * NCOL;
    const float *yim = yre + a.y_plane;
    TOut *x = reinterpret_cast<TOut *>(const_cast<void *>(a.x[tz])) + (size_t)u * a.x_unit + blk * NCOL;
    int live = Lrows;
    if (rows_dev != nullptr) {
        int t = rows_dev[u / rows_div];
        live = t < (int)P ? t : (int)P;
    }

    float acc[4][CPT];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int q = 0; q < CPT; ++q) acc[i][q] = 0.f;

    if (n0 < live) {
        // twiddle generator: this thread owns bin slot gk and positions n0+gj .. +3
        const int gk = tid >> 3, gj = (tid & 7) * 4;
        for (int kt = 0; kt < M; kt += kTileBins) {
            for (int e = tid; e < kTileBins * (NCOL / CPT); e += kSimtThreads) {
                int r = e / (NCOL / CPT), cg = e % (NCOL / CPT);
                int k = kt + r;
                if (CPT == 4) {
                    float4 vr = make_float4(0.f, 0.f, 0.f, 0.f), vi = vr;
                    if (k < M) {
                        vr = load4(yre + (size_t)k * a.y_row + cg * 4);
                        vi = load4(yim + (size_t)k * a.y_row + cg * 4);
                    }
                    *reinterpret_cast<float4 *>(&yr[r][cg * 4]) = vr;
                    *reinterpret_cast<float4 *>(&yi[r][cg * 4]) = vi;
                } else {
                    float vr = 0.f, vi = 0.f;
                    if (k < M) { vr = yre[(size_t)k * a.y_row + cg]; vi = yim[(size_t)k * a.y_row + cg]; }
                    yr[r][cg] = vr;
                    yi[r][cg] = vi;
                }
            }
            {
                const int k = kt + gk;
                const uint32_t bin = k < M ? (uint32_t)bins[k] : 0u;
                const float w = (k < M ? hermitian_weight(bin, P) : 0.f) * scale;
                uint32_t ph = phase_mod(bin, (uint32_t)(n0 + gj) % P, P);
                const uint32_t st = bin % P;
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    float c, s;
                    twiddle(ph, P, c, s);
                    twc[gk][gj + i] = c * w;
                    tws[gk][gj + i] = s * w;
                    ph = add_mod(ph, st, P);
                }
            }
            __syncthreads();
#pragma unroll 4
            for (int j = 0; j < kTileBins; ++j) {
                float re[CPT], im[CPT];
                if (CPT == 4) {
                    float4 v = *reinterpret_cast<const float4 *>(&yr[j][lane * 4]);
                    float4 w = *reinterpret_cast<const float4 *>(&yi[j][lane * 4]);
                    re[0] = v.x; re[1 % CPT] = v.y; re[2 % CPT] = v.z; re[3 % CPT] = v.w;
                    im[0] = w.x; im[1 % CPT] = w.y; im[2 % CPT] = w.z; im[3 % CPT] = w.w;
                } else {
                    re[0] = yr[j][lane];
                    im[0] = yi[j][lane];
                }
                const float4 c4 = *reinterpret_cast<const float4 *>(&twc[j][warp * 4]);
                const float4 s4 = *reinterpret_cast<const float4 *>(&tws[j][warp * 4]);
                const float cc[4] = {c4.x, c4.y, c4.z, c4.w};
                const float ss[4] = {s4.x, s4.y, s4.z, s4.w};
#pragma unroll
                for (int i = 0; i < 4; ++i)
#pragma unroll
                    for (int q = 0; q < CPT; ++q)
                        acc[i][q] = fmaf(re[q], cc[i], fmaf(-im[q], ss[i], acc[i][q]));
            }
            __syncthreads();
        }
    }

    float mx[CPT];
#pragma unroll
    for (int q = 0; q < CPT; ++q) mx[q] = -INFINITY;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int n = n0 + warp * 4 + i;
        if (n >= Lrows) continue;
        const bool is_live = n < live;
        if (CPT == 4) {
            float4 v = is_live ? make_float4(acc[i][0], acc[i][1 % CPT], acc[i][2 % CPT], acc[i][3 % CPT])
                               : make_float4(0.f, 0.f, 0.f, 0.f);
            store4(x + (size_t)n * a.x_row + lane * 4, v);
        } else {
            store1(x + (size_t)n * a.x_row + lane, is_live ? acc[i][0] : 0.f);
        }
        if (is_live) {
#pragma unroll
            for (int q = 0; q < CPT; ++q) mx[q] = fmaxf(mx[q], acc[i][q]);
        }
    }
    if (tile_max != nullptr) {
        // reduce the 8 warps' maxima through shared memory (reuse twc)
        __syncthreads();
        float *red = &twc[0][0];
#pragma unroll
        for (int q = 0; q < CPT; ++q) red[warp * NCOL + lane * CPT + q] = mx[q];
        __syncthreads();
        for (int c = tid; c < NCOL; c += kSimtThreads) {
            float m = red[c];
#pragma unroll
            for (int w = 1; w < 8; ++w) m = fmaxf(m, red[w * NCOL + c]);
            tile_max[((size_t)blockIdx.y * gridDim.x + blockIdx.x) * NCOL + c] = m;
        }
    }
}

// Column maxima over the row tiles: colmax[u*ncol + c] = max_tile tile_max[u][tile][c],
// u = sequence * col_blocks + block.  (static: this header is compiled into more than one translation unit.)
static __global__ void k_colmax(const float *__restrict__ tile_max, int n_tiles, int ncol,
                         float *__restrict__ colmax) {
    const int u = blockIdx.x;
    for (int c = threadIdx.x; c < ncol; c += blockDim.x) {
        float m = -INFINITY;
        for (int t = 0; t < n_tiles; ++t) m = fmaxf(m, tile_max[((size_t)u * n_tiles + t) * ncol + c]);
        colmax[(size_t)u * ncol + c] = m;
    }
}

}  // namespace faedkv
