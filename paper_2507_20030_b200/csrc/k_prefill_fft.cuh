// FFT-shaped prefill transform (Sec. 4.2.1; Eq. 4 restricted to the retained bins by Eq. 6) for
// power-of-two grids P -- the route the paper itself names (FFT, O(N log N)), here with the two-pass
// scheme of k_fft.cuh:
//
//     C[k, c] = sum_{n < T} x[n, c] e^{-j 2 pi k n / P} = conj( W[k, c] ),   W[k] = sum_n x[n] e^{+j 2 pi k n / P}
//
// x real, so W comes from one complex transform of length N = P/2 of z[m] = x[2m] + j x[2m+1]
// (positions at or beyond T are zero; positions beyond P wrap onto n mod P, i.e. their values add).
// Columns are the channels of a run of consecutive (sequence, kv head) units of one tensor.
//
//   k_pfft_fwd_a   pass A' (per m1, over m2) + inter-pass twiddle        -> U  [N1][N2][cols]
//   k_pfft_fwd_b   pass B' (per k1', over m1)                            -> Zf [N][cols]
//   k_pfft_gather  unpack W at the retained bins, conjugate              -> coefficient planes
#pragma once
#include "common.cuh"
#include "k_fft.cuh"

namespace faedkv {

// grid = (N1 / MT, cols / 16); block = 256.  x: rows of the tensor, T rows per unit, units T_stride rows apart.
template <int LG, int LGT, typename TIn>
__global__ void __launch_bounds__(fft::kThreads)
k_pfft_fwd_a(fft::Geometry g, const TIn *__restrict__ x, int T, int T_stride, int unit0, float2 *__restrict__ U, int lgMT_rt) {
    const int lgMT = LGT >= 0 ? LGT : lgMT_rt;   // compile-time in the fast instances
    using namespace fft;
    constexpr int NF = 1 << LG;                      // = N2
    extern __shared__ float2 fft_smem[];
    const int lg_cols = lgMT + kLgCW;
    const int tile = NF << lg_cols;
    float2 *xa = fft_smem, *xb = xa + (exchange_buffers(LG) > 0 ? tile : 0);
    float2 *tw = xb + (exchange_buffers(LG) > 1 ? tile : 0);
    float2 *tab_i = tw + NF;                         // [k1'][mt]: e^{+j2pi k1' m1 / N}
    const int MT = 1 << lgMT;
    const int m1_0 = blockIdx.x << lgMT, g0 = blockIdx.y * kCW;
    fill_twiddles(tw, NF);
    for (int e = threadIdx.x; e < (NF << lgMT); e += kThreads) {
        const int mt = e & (MT - 1), r = e >> lgMT;
        tab_i[e] = unit_phasor((uint32_t)((m1_0 + mt) * r), (uint32_t)g.N);
    }
    __syncthreads();
    const TIn *xu = x + (size_t)(unit0 + (g0 >> 7)) * T_stride * kHeadDim + (g0 & (kHeadDim - 1));
    const bool wraps = T > (int)g.P;                                     // uniform: positions beyond P fold back
    auto load = [&](int m2, int cidx) {
        const int c = cidx & (kCW - 1);
        const uint32_t n = 2u * (uint32_t)(m1_0 + (cidx >> kLgCW) + g.N1 * m2);   // even position, n < P <= 2^19
        float2 z = make_float2(0.f, 0.f);
        if (!wraps) {
            const TIn *r = xu + n * (uint32_t)kHeadDim + c;
            if ((int)n < T) z.x = load1(r);
            if ((int)n + 1 < T) z.y = load1(r + kHeadDim);
        } else {
            for (long long p = n; p < T; p += g.P) {                     // P is even, so n + jP stays even
                z.x += load1(xu + (size_t)p * kHeadDim + c);
                if (p + 1 < T) z.y += load1(xu + (size_t)(p + 1) * kHeadDim + c);
            }
        }
        return z;
    };
    auto store = [&](int k1p, int cidx, float2 v) {
        const int mt = cidx >> kLgCW;
        U[y_index(g, m1_0 + mt, k1p, g0 + (cidx & (kCW - 1)))] = cmul(v, tab_i[(k1p << lgMT) + mt]);
    };
    fft_rows<LG, (LGT >= 0 ? LGT + kLgCW : -1)>(lg_cols, xa, xb, tw, load, store);
}

// grid = (N2 / KT, cols / 16); block = 256.
template <int LG, int LGT>
__global__ void __launch_bounds__(fft::kThreads)
k_pfft_fwd_b(fft::Geometry g, const float2 *__restrict__ U, float2 *__restrict__ Zf, int lgKT_rt) {
    const int lgKT = LGT >= 0 ? LGT : lgKT_rt;   // compile-time in the fast instances
    using namespace fft;
    constexpr int NF = 1 << LG;                      // = N1
    extern __shared__ float2 fft_smem[];
    const int lg_cols = lgKT + kLgCW;
    const int tile = NF << lg_cols;
    float2 *xa = fft_smem, *xb = xa + (exchange_buffers(LG) > 0 ? tile : 0);
    float2 *tw = xb + (exchange_buffers(LG) > 1 ? tile : 0);
    const int k1_0 = blockIdx.x << lgKT, g0 = blockIdx.y * kCW;
    fill_twiddles(tw, NF);
    __syncthreads();
    auto load = [&](int m1, int cidx) { return U[y_index(g, m1, k1_0 + (cidx >> kLgCW), g0 + (cidx & (kCW - 1)))]; };
    auto store = [&](int k2p, int cidx, float2 v) {
        Zf[((uint32_t)(k1_0 + (cidx >> kLgCW)) + (uint32_t)g.N2 * (uint32_t)k2p) * (uint32_t)g.Gp +
           (uint32_t)(g0 + (cidx & (kCW - 1)))] = v;
    };
    fft_rows<LG, (LGT >= 0 ? LGT + kLgCW : -1)>(lg_cols, xa, xb, tw, load, store);
}

// Coefficients at the retained bins.  grid = (ceil(M / 8), cols / 128); block = 256: a warp per bin,
// a lane per 4 channels.  coef: planes of the tensor, [units][2][M][128].
__global__ void __launch_bounds__(256)
k_pfft_gather(fft::Geometry g, const float2 *__restrict__ Zf, const int32_t *__restrict__ bins, int M, int unit0,
              float *__restrict__ coef) {
    using namespace fft;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int i = blockIdx.x * 8 + warp;
    if (i >= M) return;
    const uint32_t bin = (uint32_t)bins[i];
    const int ka = (int)bin & (g.N - 1), kb = (g.N - ka) & (g.N - 1);
    const float2 ph = unit_phasor(bin, g.P);
    const int col = blockIdx.y * kHeadDim + lane * 4;
    const float4 *za_p = reinterpret_cast<const float4 *>(Zf + (uint32_t)ka * (uint32_t)g.Gp + col);
    const float4 *zb_p = reinterpret_cast<const float4 *>(Zf + (uint32_t)kb * (uint32_t)g.Gp + col);
    const float4 a01 = za_p[0], a23 = za_p[1], b01 = zb_p[0], b23 = zb_p[1];
    const float2 za[4] = {make_float2(a01.x, a01.y), make_float2(a01.z, a01.w), make_float2(a23.x, a23.y), make_float2(a23.z, a23.w)};
    const float2 zb[4] = {make_float2(b01.x, -b01.y), make_float2(b01.z, -b01.w), make_float2(b23.x, -b23.y), make_float2(b23.z, -b23.w)};
    float re[4], im[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        const float2 A = cadd(za[q], zb[q]), D = csub(za[q], zb[q]);          // 2A, 2jB
        const float2 W = cadd(A, cmul(ph, make_float2(D.y, -D.x)));            // 2 W[k]
        re[q] = 0.5f * W.x;
        im[q] = -0.5f * W.y;                                                  // C = conj W
    }
    const bool self_conj = bin == 0u || 2u * bin == g.P;                       // real spectrum lines
    float *dst = coef + ((size_t)(unit0 + blockIdx.y) * 2 * M + i) * kHeadDim + lane * 4;
    st_stream(dst, make_float4(re[0], re[1], re[2], re[3]));
    st_stream(dst + (size_t)M * kHeadDim, self_conj ? make_float4(0.f, 0.f, 0.f, 0.f) : make_float4(im[0], im[1], im[2], im[3]));
}

inline size_t pfft_smem_a(int lg, int lgMT) {
    const size_t nf = (size_t)1 << lg, tile = nf << (lgMT + fft::kLgCW);
    return (fft::exchange_buffers(lg) * tile + nf + (nf << lgMT)) * sizeof(float2);
}
inline size_t pfft_smem_b(int lg, int lgKT) {
    const size_t nf = (size_t)1 << lg, tile = nf << (lgKT + fft::kLgCW);
    return (fft::exchange_buffers(lg) * tile + nf) * sizeof(float2);
}

}  // namespace faedkv
