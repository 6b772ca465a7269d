// FFT-shaped reconstruction (Eq. 11: Eq. 5 with every pruned bin zero) for power-of-two grids P:
//
//     x~[n, c] = (1/P) sum_k w_k (Re C[k,c] cos(w k n) - Im C[k,c] sin(w k n)),   n < min(t, P)
//
// as a real inverse FFT of the zero-filled half spectrum, per channel, with the two-pass scheme of
// k_fft.cuh.  Columns are the channels of a run of consecutive (sequence, kv head) units of one tensor:
// column = (unit - unit0) * 128 + c.
//
//   k_rfft_inv_a   gather the retained bins from the coefficient planes, pack the half spectrum,
//                  pass A (over k1) + inter-pass twiddle                      -> Y [N1][N2][cols]
//   k_rfft_inv_b   pass B (over k2); the complex result z[m] holds rows 2m and 2m+1, written in the
//                  tensor's storage type; rows at or beyond the live length are written as zero
#pragma once
#include "common.cuh"
#include "k_fft.cuh"

namespace faedkv {

// grid = (N2 / KT, cols / 16); block = 256; dynamic smem as k_afft_inv_a.
// coef: planes of the tensor, [units][2][M][128]; unit0: first unit of this launch.
template <int LG, int LGT>
__global__ void __launch_bounds__(fft::kThreads)
k_rfft_inv_a(fft::Geometry g, const int32_t *__restrict__ slot, const float *__restrict__ coef, int M, int unit0,
             float2 *__restrict__ Y, int lgKT_rt) {
    const int lgKT = LGT >= 0 ? LGT : lgKT_rt;   // compile-time in the fast instances
    using namespace fft;
    constexpr int NF = 1 << LG;                      // = N1
    extern __shared__ float2 fft_smem[];
    const int KT = 1 << lgKT, lg_cols = lgKT + kLgCW;
    const int tile = NF << lg_cols;
    float2 *xa = fft_smem, *xb = xa + (exchange_buffers(LG) > 0 ? tile : 0);
    float2 *tw = xb + (exchange_buffers(LG) > 1 ? tile : 0);
    float2 *tab_i = tw + NF;                         // [m1][kt]: e^{+j2pi k2 m1 / N}
    float2 *tab_p = tab_i + (NF << lgKT);            // [k1][kt]: e^{+j2pi (N2 k1 + k2) / P}
    int2 *tab_s = reinterpret_cast<int2 *>(tab_p + (NF << lgKT));   // [k1][kt]: plan slots of bins k and N - k (or -1)
    const int k2_0 = blockIdx.x * KT, g0 = blockIdx.y * kCW;
    fill_twiddles(tw, NF);
    for (int e = threadIdx.x; e < (NF << lgKT); e += kThreads) {
        const int kt = e & (KT - 1), r = e >> lgKT;
        tab_i[e] = unit_phasor((uint32_t)((k2_0 + kt) * r), (uint32_t)g.N);
        tab_p[e] = unit_phasor((uint32_t)(g.N2 * r + k2_0 + kt), g.P);
        tab_s[e] = make_int2(slot[g.N2 * r + k2_0 + kt], slot[g.N - (g.N2 * r + k2_0 + kt)]);
    }
    __syncthreads();
    const float inv_P = 1.0f / (float)g.P;
    const size_t plane = (size_t)M * kHeadDim;
    auto load = [&](int k1, int cidx) {
        const int c = cidx & (kCW - 1), kt = cidx >> kLgCW;
        const int col = g0 + c;
        float2 z = make_float2(0.f, 0.f);
        const int2 sl = tab_s[(k1 << lgKT) + kt];
        if ((sl.x >= 0 || sl.y >= 0) && FAEDKV_IN_BOUNDS(kTagReconFft, sl.x < M && sl.y < M)) {
            const float *u = coef + (size_t)(unit0 + (col >> 7)) * 2 * plane + (col & (kHeadDim - 1));
            float2 xk = make_float2(0.f, 0.f), xm = make_float2(0.f, 0.f);
            if (sl.x >= 0) xk = make_float2(u[(uint32_t)sl.x * kHeadDim], u[plane + (uint32_t)sl.x * kHeadDim]);
            if (sl.y >= 0) xm = make_float2(u[(uint32_t)sl.y * kHeadDim], -u[plane + (uint32_t)sl.y * kHeadDim]);   // conj X[N-k]
            if (k1 == 0 && k2_0 + kt == 0) { xk.y = 0.f; xm.y = 0.f; }   // k = 0: bins 0 and N = P/2 are their own mirrors
            xk.x *= inv_P; xk.y *= inv_P; xm.x *= inv_P; xm.y *= inv_P;
            z = cadd(cadd(xk, xm), cmulj(cmul(tab_p[(k1 << lgKT) + kt], csub(xk, xm))));
        }
        return z;
    };
    auto store = [&](int m1, int cidx, float2 v) {
        const int c = cidx & (kCW - 1), kt = cidx >> kLgCW;
        Y[y_index(g, m1, k2_0 + kt, g0 + c)] = cmul(v, tab_i[(m1 << lgKT) + kt]);
    };
    fft_rows<LG, (LGT >= 0 ? LGT + kLgCW : -1)>(lg_cols, xa, xb, tw, load, store);
}

// Where the reconstructed positions go: position n of a unit lands in row row0 + n of its unit_rows output rows;
// live positions = min(q(t_len + t_add), P), q() rounding down to a multiple of t_quant (the transformed
// segment of a windowed cache: t_add = -(S + R), t_quant = the defer block).
struct ReconRows {
    int row0, unit_rows, t_add, t_quant;
};

// grid = (N1 / MT, cols / 16); block = 256; dynamic smem = rfft_smem_b(lgN2, lgMT).
// out: rows of the tensor, [units][rows.unit_rows][128], Lrows positions written (zeros past the live ones);
// H: kv heads per sequence (t_len index = unit / H).
template <int LG, int LGT, typename TOut>
__global__ void __launch_bounds__(fft::kThreads)
k_rfft_inv_b(fft::Geometry g, const float2 *__restrict__ Y, const int32_t *__restrict__ t_len, int H, int unit0,
             int Lrows, TOut *__restrict__ out, int lgMT_rt, ReconRows rows) {
    const int lgMT = LGT >= 0 ? LGT : lgMT_rt;   // compile-time in the fast instances
    using namespace fft;
    constexpr int NF = 1 << LG;                      // = N2
    extern __shared__ float2 fft_smem[];
    const int lg_cols = lgMT + kLgCW;
    const int tile = NF << lg_cols;
    float2 *xa = fft_smem, *xb = xa + (exchange_buffers(LG) > 0 ? tile : 0);
    float2 *tw = xb + (exchange_buffers(LG) > 1 ? tile : 0);
    const int m1_0 = blockIdx.x << lgMT, g0 = blockIdx.y * kCW;
    fill_twiddles(tw, NF);
    __syncthreads();
    // the 16 columns of a CTA belong to one unit (128 channels per unit)
    const int unit = unit0 + (g0 >> 7);
    int t = t_len[unit / H] + rows.t_add;
    if (t < 0) t = 0;
    if (rows.t_quant > 1) t = t / rows.t_quant * rows.t_quant;
    const int live = t < (int)g.P ? t : (int)g.P;
    TOut *obase = out + ((size_t)unit * rows.unit_rows + rows.row0) * kHeadDim + (g0 & (kHeadDim - 1));
    auto load = [&](int k2, int cidx) {
        return Y[y_index(g, m1_0 + (cidx >> kLgCW), k2, g0 + (cidx & (kCW - 1)))];
    };
    auto store = [&](int m2, int cidx, float2 v) {
        const int n = 2 * (m1_0 + (cidx >> kLgCW) + g.N1 * m2);
        TOut *o = obase + (uint32_t)n * (uint32_t)kHeadDim + (uint32_t)(cidx & (kCW - 1));   // n < P <= 2^19
        if (n < Lrows) store1(o, n < live ? v.x : 0.f);
        if (n + 1 < Lrows) store1(o + kHeadDim, n + 1 < live ? v.y : 0.f);
    };
    fft_rows<LG, (LGT >= 0 ? LGT + kLgCW : -1)>(lg_cols, xa, xb, tw, load, store);
}

inline size_t rfft_smem_b(int lg, int lgMT) {
    const size_t nf = (size_t)1 << lg, tile = nf << (lgMT + fft::kLgCW);
    return (fft::exchange_buffers(lg) * tile + nf) * sizeof(float2);
}

}  // namespace faedkv
