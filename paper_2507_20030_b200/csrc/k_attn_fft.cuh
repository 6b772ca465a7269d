// Frequency-domain decode attention (Eq. 3 on the reconstruction of Eq. 11) with FFT-shaped transforms,
// for power-of-two grids P.  Steps as in k_attn.cuh; columns col = sequence * HQ + query head.
//
//   (1) k_attn_qs        Qs[i][col] = scale/P * sum_c q[col,c] C_K[i,c]        (one pass over C_K;
//                        with APPEND the IWDFT update of Eq. 12 is applied to C_K on the way)
//   (2) k_afft_inv_a     half-spectrum packing + pass A of the inverse transform  -> Y
//       k_afft_mid       pass B -> scores s[n]; per-tile maxima, p~ = exp(s - tile max), tile sums;
//   (3,4)                pass A' of the forward transform of p~, in place            -> Y
//       k_afft_fwd_b     rescale every tile to the column's global maximum, pass B'  -> Zf
//   (5) k_attn_out_fft   Pf at the retained bins from Zf (unpacking formula), out partials from one pass
//                        over C_V (with APPEND the update of C_V on the way); the last CTA of a kv head
//                        sums the partials and divides by P * (softmax normaliser); APPEND: t_len += 1
//
// The scores never leave shared memory; the only intermediates in (L2-resident) global memory are the
// two-pass arrays Y, Zf of P/2 complex values per column and the per-tile softmax statistics.
// For P <= 16384 the three kernels of (2)-(4) are replaced by one kernel per column (k_attn_col.cuh), which
// hands (5) ready weights Wg instead of Zf; (1) then writes Qs column-major.
#pragma once
#include "common.cuh"
#include "k_attn.cuh"
#include "k_fft.cuh"
#include "k_window.cuh"

namespace faedkv {

// ---- (1) ------------------------------------------------------------------------------------------
// grid = (ceil(M / (8 * KB)), batch * H); block = 256; KB = attn_bins_per_warp(GQ) bins per warp.
template <typename TQ, int GQ, bool APPEND>
__global__ void __launch_bounds__(kAttnWarps * 32, 3)
k_attn_qs(const TQ *__restrict__ q, float *__restrict__ coefK, const TQ *__restrict__ k_new,
          const int32_t *__restrict__ t_len, const int32_t *__restrict__ bins, float2 *__restrict__ Qs,
          int M, int H, int HQ, int Gp, uint32_t P, float scale_over_P, FoldSrc fold, int col_major) {
    constexpr int KB = attn_bins_per_warp(GQ);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int bh = blockIdx.y, b = bh / H, h = bh % H;
    const int k0 = (blockIdx.x * kAttnWarps + warp) * KB;
    if (k0 >= M) return;
    float4 qv[GQ];
#pragma unroll
    for (int g = 0; g < GQ; ++g) qv[g] = load4(q + ((size_t)b * HQ + h * GQ + g) * kHeadDim + lane * 4);
    const size_t plane = (size_t)M * kHeadDim;
    float *base = coefK + (size_t)bh * 2 * plane;
    // C_K[k, c] += x[c] * e^{-j w k t} (APPEND): same arithmetic as k_append; x is the call's new token, or with a
    // recent window the token that leaves it (k_new then points at the window tensor)
    float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
    uint32_t t = 0;
    if (APPEND) {
        size_t xrow;
        fold_locate(fold, t_len[b], bh, P, xrow, t);
        x = load4(k_new + xrow * kHeadDim + lane * 4);
    }
    // The warp's KB bins go through in groups of at most 4: rows of a group are loaded together, updated and
    // written back (APPEND), reduced to their dot products, and only those stay live.  (All 16 bins of the
    // one-query-head case at once took 158 registers with the update fused: one CTA per SM, 3.9 TB/s.)
    constexpr int GB = KB < 4 ? KB : 4;
    float v[32];
#pragma unroll
    for (int i = KB * 2 * GQ; i < 32; ++i) v[i] = 0.f;
#pragma unroll
    for (int g0 = 0; g0 < KB; g0 += GB) {
        float4 row[GB][2];
#pragma unroll
        for (int kk = 0; kk < GB; ++kk)
#pragma unroll
            for (int pl = 0; pl < 2; ++pl) {
                row[kk][pl] = make_float4(0.f, 0.f, 0.f, 0.f);
                if (g0 + kk < KB && k0 + g0 + kk < M) row[kk][pl] = ld_stream(base + pl * plane + (size_t)(k0 + g0 + kk) * kHeadDim + lane * 4);
            }
        if (APPEND) {
#pragma unroll
            for (int kk = 0; kk < GB; ++kk) {
                if (g0 + kk >= KB || k0 + g0 + kk >= M) continue;
                float c, sn;
                twiddle(phase_mod((uint32_t)bins[k0 + g0 + kk], t, P), P, c, sn);
                float4 &re = row[kk][0], &im = row[kk][1];
                re.x = fmaf(x.x, c, re.x); im.x = fmaf(-x.x, sn, im.x);
                re.y = fmaf(x.y, c, re.y); im.y = fmaf(-x.y, sn, im.y);
                re.z = fmaf(x.z, c, re.z); im.z = fmaf(-x.z, sn, im.z);
                re.w = fmaf(x.w, c, re.w); im.w = fmaf(-x.w, sn, im.w);
                float *dst = base + (size_t)(k0 + g0 + kk) * kHeadDim + lane * 4;
                st_stream(dst, re);
                st_stream(dst + plane, im);
            }
        }
#pragma unroll
        for (int kk = 0; kk < GB; ++kk)
#pragma unroll
            for (int pl = 0; pl < 2; ++pl)
#pragma unroll
                for (int g = 0; g < GQ; ++g) {
                    if (g0 + kk >= KB) continue;       // KB need not be a multiple of the group size
                    const float4 r = row[kk][pl];
                    v[((g0 + kk) * 2 + pl) * GQ + g] = r.x * qv[g].x + r.y * qv[g].y + r.z * qv[g].z + r.w * qv[g].w;
                }
    }
    const float tot = warp_transpose_reduce32(v, lane);
    const int kk = lane / (2 * GQ), pl = (lane / GQ) & 1, g = lane % GQ;
    if (kk < KB && k0 + kk < M) {
        const uint32_t bin = (uint32_t)bins[k0 + kk];
        // bins 0 and P/2 are their own mirrors: only their real part enters a real signal
        const bool self_conj = bin == 0u || 2u * bin == P;
        // Qs[bin][col] for the two-pass transforms, Qs[col][bin] for the one-kernel column transform
        const size_t col = (size_t)(b * HQ + h * GQ + g);
        if (!FAEDKV_IN_BOUNDS(kTagAttnFft, bin <= P / 2 && col < (size_t)Gp)) return;
        float *dst = reinterpret_cast<float *>(Qs + (col_major ? col * M + (k0 + kk) : (size_t)(k0 + kk) * Gp + col));
        dst[pl] = (pl == 1 && self_conj) ? 0.f : tot * scale_over_P;
    }
}

// ---- (2) pass A of the inverse transform, half-spectrum packing fused into the load ----------------
// slot[k], k in [0, N]: index of one-sided bin k in the plan, or -1.  Y: [N1][N2][Gp].
// grid = (N2 / KT, Gp / 16); block = 256; dynamic smem = afft_smem_a(lgN1, lgKT, true).
template <int LG, int LGT>
__global__ void __launch_bounds__(fft::kThreads)
k_afft_inv_a(fft::Geometry g, const int32_t *__restrict__ slot, const float2 *__restrict__ Qs,
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
        tab_i[e] = unit_phasor((uint32_t)((k2_0 + kt) * r), (uint32_t)g.N);      // k2 * m1 < N2 * N1 = N
        tab_p[e] = unit_phasor((uint32_t)(g.N2 * r + k2_0 + kt), g.P);
        tab_s[e] = make_int2(slot[g.N2 * r + k2_0 + kt], slot[g.N - (g.N2 * r + k2_0 + kt)]);
    }

    __syncthreads();
    pdl_wait();                                      // Qs comes from the previous kernel
    auto load = [&](int k1, int cidx) {
        const int c = cidx & (kCW - 1), kt = cidx >> kLgCW;
        const int col = g0 + c;
        // branch-free (see ld2_if): absent bins and padding columns read as zero
        const int2 sl = tab_s[(k1 << lgKT) + kt];
        const bool live_col = col < g.G;
        const float2 xk = ld2_if(Qs + (uint32_t)(sl.x < 0 ? 0 : sl.x) * (uint32_t)g.Gp + (uint32_t)col, sl.x >= 0 && live_col);
        float2 xm = ld2_if(Qs + (uint32_t)(sl.y < 0 ? 0 : sl.y) * (uint32_t)g.Gp + (uint32_t)col, sl.y >= 0 && live_col);
        xm.y = -xm.y;                                                // conj X[N-k]
        return cadd(cadd(xk, xm), cmulj(cmul(tab_p[(k1 << lgKT) + kt], csub(xk, xm))));
    };
    auto store = [&](int m1, int cidx, float2 v) {
        const int c = cidx & (kCW - 1), kt = cidx >> kLgCW;
        Y[y_index(g, m1, k2_0 + kt, g0 + c)] = cmul(v, tab_i[(m1 << lgKT) + kt]);
    };
    fft_rows<LG, (LGT >= 0 ? LGT + kLgCW : -1)>(lg_cols, xa, xb, tw, load, store);
}

// ---- pass B of the inverse transform, local softmax, pass A' of the forward transform ---------------
// One CTA = MT values of m1 (one "tile" of the softmax statistics) x 16 columns.
// mloc, sloc: [N1 / MT][Gp].  live length of a column = min(t_len[col / HQ] + t_add, P).
// grid = (N1 / MT, Gp / 16); block = 256; dynamic smem = afft_smem_mid(lgN2, lgMT).
template <int LG, int LGT>
__global__ void __launch_bounds__(fft::kThreads)
k_afft_mid(fft::Geometry g, float2 *__restrict__ Y, const int32_t *__restrict__ t_len, int HQ, int t_add, int t_quant,
           float *__restrict__ mloc, float *__restrict__ sloc, int lgMT_rt) {
    const int lgMT = LGT >= 0 ? LGT : lgMT_rt;   // compile-time in the fast instances
    using namespace fft;
    constexpr int NF = 1 << LG;                      // = N2
    extern __shared__ float2 fft_smem[];
    __shared__ float red[kThreads];
    __shared__ float colv[kCW];
    __shared__ int live_s[kCW];
    const int MT = 1 << lgMT, lg_cols = lgMT + kLgCW;
    const int tile = NF << lg_cols;
    float2 *T = fft_smem;                            // scores / probabilities of this tile
    float2 *xa = T + tile, *xb = xa + (exchange_buffers(LG) > 0 ? tile : 0);
    float2 *tw = xb + (exchange_buffers(LG) > 1 ? tile : 0);
    float2 *tab_i = tw + NF;                         // [k1'][mt]: e^{+j2pi k1' m1 / N}
    const int m1_0 = blockIdx.x * MT, g0 = blockIdx.y * kCW;
    fill_twiddles(tw, NF);
    for (int e = threadIdx.x; e < (NF << lgMT); e += kThreads) {
        const int mt = e & (MT - 1), r = e >> lgMT;
        tab_i[e] = unit_phasor((uint32_t)((m1_0 + mt) * r), (uint32_t)g.N);
    }
    if (threadIdx.x < kCW) {
        const int col = g0 + threadIdx.x;
        int live = 0;
        if (col < g.G) {
            long long t = (long long)t_len[col / HQ] + t_add;
            if (t_quant > 1 && t > 0) t = t / t_quant * t_quant;      // block-deferred fold: whole blocks only
            live = t < (long long)g.P ? (int)t : (int)g.P;
        }
        live_s[threadIdx.x] = live;
    }

    __syncthreads();
    pdl_wait();                                      // Y comes from the previous kernel
    // a thread always meets the same column: kThreads is a multiple of 16
    const int c = threadIdx.x & (kCW - 1);
    const int live = live_s[c];
    float mx = -INFINITY;
    {
        auto load = [&](int k2, int cidx) {
            return Y[y_index(g, m1_0 + (cidx >> kLgCW), k2, g0 + (cidx & (kCW - 1)))];
        };
        // T[m2][mt, c] = z[m1 + N1 m2] = scores of positions 2m, 2m + 1; the maximum of the live ones is
        // collected on the way out of the registers
        auto store = [&](int m2, int cidx, float2 v) {
            T[(m2 << lg_cols) + cidx] = v;
            const int n0 = 2 * (m1_0 + (cidx >> kLgCW) + g.N1 * m2);
            if (n0 < live) mx = fmaxf(mx, v.x);
            if (n0 + 1 < live) mx = fmaxf(mx, v.y);
        };
        fft_rows<LG, (LGT >= 0 ? LGT + kLgCW : -1)>(lg_cols, xa, xb, tw, load, store);
    }
    red[threadIdx.x] = mx;
    __syncthreads();                                 // also: the tile is complete
    if (threadIdx.x < kCW) {
        float m = red[threadIdx.x];
#pragma unroll
        for (int i = 1; i < kThreads / kCW; ++i) m = fmaxf(m, red[threadIdx.x + kCW * i]);
        colv[threadIdx.x] = m;
    }
    __syncthreads();
    const float mcol = colv[c];
    float sum = 0.f;
    {
        // p~ = exp(s - tile max) on the live positions, formed as the forward pass reads the tile
        auto load = [&](int m2, int cidx) {
            const float2 v = T[(m2 << lg_cols) + cidx];
            const int n0 = 2 * (m1_0 + (cidx >> kLgCW) + g.N1 * m2);
            const float pe = n0 < live ? __expf(v.x - mcol) : 0.f;
            const float po = n0 + 1 < live ? __expf(v.y - mcol) : 0.f;
            sum += pe + po;
            return make_float2(pe, po);
        };
        auto store = [&](int k1p, int cidx, float2 v) {
            const int mt = cidx >> kLgCW;
            Y[y_index(g, m1_0 + mt, k1p, g0 + (cidx & (kCW - 1)))] = cmul(v, tab_i[(k1p << lgMT) + mt]);
        };
        fft_rows<LG, (LGT >= 0 ? LGT + kLgCW : -1)>(lg_cols, xa, xb, tw, load, store);
    }
    __syncthreads();                                 // red is free again
    red[threadIdx.x] = sum;
    __syncthreads();
    if (threadIdx.x < kCW) {
        float sm = red[threadIdx.x];
#pragma unroll
        for (int i = 1; i < kThreads / kCW; ++i) sm += red[threadIdx.x + kCW * i];
        mloc[(size_t)blockIdx.x * g.Gp + g0 + threadIdx.x] = colv[threadIdx.x];
        sloc[(size_t)blockIdx.x * g.Gp + g0 + threadIdx.x] = sm;
    }
}

// ---- pass B' of the forward transform ---------------------------------------------------------------
// Every softmax tile is first brought to the column's global maximum: factor exp(mloc - max_tiles mloc).
// The CTAs with blockIdx.x == 0 also write the softmax normaliser colsum[col] = sum_tiles sloc * factor.
// Zf: [N][Gp], index k1' + N2 * k2'.
// grid = (N2 / KT, Gp / 16); block = 256; dynamic smem = afft_smem_a(lgN1, lgKT, false) + factors.
template <int LG, int LGT>
__global__ void __launch_bounds__(fft::kThreads)
k_afft_fwd_b(fft::Geometry g, const float2 *__restrict__ U, const float *__restrict__ mloc,
             const float *__restrict__ sloc, int lgMT, float2 *__restrict__ Zf, float *__restrict__ colsum, int lgKT_rt,
             int n_extra) {
    const int lgKT = LGT >= 0 ? LGT : lgKT_rt;   // compile-time in the fast instances
    using namespace fft;
    constexpr int NF = 1 << LG;                      // = N1
    extern __shared__ float2 fft_smem[];
    __shared__ float red[kThreads];
    __shared__ float mg[kCW];
    const int lg_cols = lgKT + kLgCW;
    const int tile = NF << lg_cols;
    float2 *xa = fft_smem, *xb = xa + (exchange_buffers(LG) > 0 ? tile : 0);
    float2 *tw = xb + (exchange_buffers(LG) > 1 ? tile : 0);
    float *fac = reinterpret_cast<float *>(tw + NF);  // [n_tiles][16]
    const int k1_0 = blockIdx.x << lgKT, g0 = blockIdx.y * kCW;
    const int n_tiles = NF >> lgMT;
    // n_extra = 1: row n_tiles of mloc / sloc holds the statistics of the sink + recent window, which joins
    // the softmax as one more tile; its factor is handed to the output kernel in colsum[Gp + col]
    const int n_stat = n_tiles + n_extra;
    fill_twiddles(tw, NF);

    pdl_wait();                                      // the statistics and Y come from the previous kernel
    const int c = threadIdx.x & (kCW - 1);
    {
        float mx = -INFINITY;
        for (int ti = threadIdx.x >> kLgCW; ti < n_stat; ti += kThreads / kCW) mx = fmaxf(mx, mloc[(size_t)ti * g.Gp + g0 + c]);
        red[threadIdx.x] = mx;
        __syncthreads();
        if (threadIdx.x < kCW) {
            float m = red[threadIdx.x];
#pragma unroll
            for (int i = 1; i < kThreads / kCW; ++i) m = fmaxf(m, red[threadIdx.x + kCW * i]);
            mg[threadIdx.x] = m;
        }
        __syncthreads();
        const float m = mg[c];
        float part = 0.f;
        for (int ti = threadIdx.x >> kLgCW; ti < n_stat; ti += kThreads / kCW) {
            const float ml = mloc[(size_t)ti * g.Gp + g0 + c];
            const float f = ml == -INFINITY ? 0.f : __expf(ml - m);
            fac[ti * kCW + c] = f;
            if (blockIdx.x == 0) {
                part += f * sloc[(size_t)ti * g.Gp + g0 + c];
                if (ti == n_tiles) colsum[g.Gp + g0 + c] = f;
            }
        }
        if (blockIdx.x == 0) {
            __syncthreads();
            red[threadIdx.x] = part;
            __syncthreads();
            if (threadIdx.x < kCW) {
                float s = red[threadIdx.x];
#pragma unroll
                for (int i = 1; i < kThreads / kCW; ++i) s += red[threadIdx.x + kCW * i];
                colsum[g0 + threadIdx.x] = s;
            }
        }
        __syncthreads();
    }
    auto load = [&](int m1, int cidx) {
        const int cc = cidx & (kCW - 1);
        const float f = fac[(m1 >> lgMT) * kCW + cc];
        const float2 v = U[y_index(g, m1, k1_0 + (cidx >> kLgCW), g0 + cc)];
        return make_float2(v.x * f, v.y * f);
    };
    auto store = [&](int k2p, int cidx, float2 v) {
        Zf[((uint32_t)(k1_0 + (cidx >> kLgCW)) + (uint32_t)g.N2 * (uint32_t)k2p) * (uint32_t)g.Gp + (uint32_t)(g0 + (cidx & (kCW - 1)))] = v;
    };
    fft_rows<LG, (LGT >= 0 ? LGT + kLgCW : -1)>(lg_cols, xa, xb, tw, load, store);
}

// Dynamic shared memory of the three kernels above (bytes).
inline size_t afft_smem_a(int lg, int lgKT, bool packing_table) {
    const size_t nf = (size_t)1 << lg, tile = nf << (lgKT + fft::kLgCW);
    // exchange buffers, twiddles, inter-pass twiddles (+ packing phasors and slot pairs)
    return (fft::exchange_buffers(lg) * tile + nf + (packing_table ? 3 : 1) * (nf << lgKT)) * sizeof(float2);
}
inline size_t afft_smem_mid(int lg, int lgMT) {
    const size_t nf = (size_t)1 << lg, tile = nf << (lgMT + fft::kLgCW);
    return ((1 + fft::exchange_buffers(lg)) * tile + nf + (nf << lgMT)) * sizeof(float2);
}
inline size_t afft_smem_fwd_b(int lg, int lgKT, int lgMT) {
    const size_t nf = (size_t)1 << lg, tile = nf << (lgKT + fft::kLgCW);
    return (fft::exchange_buffers(lg) * tile + nf) * sizeof(float2) + (((nf >> lgMT) + 1) * fft::kCW) * sizeof(float);
}

// ---- (5) ------------------------------------------------------------------------------------------
// One pass over C_V.  A CTA takes a slice of the bins of one (sequence, kv head) in chunks of kOutChunk:
// first the chunk's probability-spectrum weights  w_k * Pf[g, k]  are formed from Zf (the unpacking
// formula; one thread per bin) into shared memory, then the warps stream the coefficient rows, four
// bins per warp in flight.  The last CTA of a (sequence, kv head) to finish sums the slice partials in
// a fixed order, divides by P * colsum and writes the output rows.
// The partials of unit bh sit at partial[bh * slice_stride + slice]: the stride is the same for every launch of
// one call (a call cut into two runs of sequences launches twice, possibly with different slice counts, and
// the runs overlap in time), so no two units ever share a slot.
// grid = (slices, batch * H); block = 256.
constexpr int kOutChunk = 256;

template <typename TQ, int GQ, bool APPEND>
__global__ void __launch_bounds__(kAttnWarps * 32)
k_attn_out_fft(float *__restrict__ coefV, const TQ *__restrict__ v_new, int32_t *__restrict__ t_len,
               const float2 *__restrict__ Zf, const float *__restrict__ colsum, const int32_t *__restrict__ bins,
               float *__restrict__ partial, unsigned int *__restrict__ tickets, TQ *__restrict__ out,
               int M, int H, int HQ, fft::Geometry g, int bins_per_slice, float inv_P, FoldSrc fold,
               const float *__restrict__ o_win, int bump, WindowArgs commit, const float2 *__restrict__ Wg,
               int bh0, int n_units, int slice_stride) {
    using namespace fft;
    // the weights of a chunk and the final cross-warp reduction share one buffer
    constexpr size_t kWgtBytes = (size_t)kOutChunk * GQ * sizeof(float2) + (APPEND ? kOutChunk * sizeof(float2) : 0);
    constexpr size_t kRedBytes = (size_t)kAttnWarps * GQ * kHeadDim * sizeof(float);
    __shared__ __align__(16) unsigned char sbuf[kWgtBytes > kRedBytes ? kWgtBytes : kRedBytes];
    float2 (*wgt)[GQ] = reinterpret_cast<float2 (*)[GQ]>(sbuf);                         // (w Re Pf, -w Im Pf) / bin
    float2 *upd = reinterpret_cast<float2 *>(sbuf + (size_t)kOutChunk * GQ * sizeof(float2));   // APPEND: (cos, sin) of w k t
    float (*red)[GQ][kHeadDim] = reinterpret_cast<float (*)[GQ][kHeadDim]>(sbuf);
    __shared__ unsigned int last_flag;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // a launch may cover a run of whole sequences only: units [bh0, bh0 + gridDim.y) of n_units
    const int bh = bh0 + (int)blockIdx.y, b = bh / H, h = bh % H;
    const int kbeg = blockIdx.x * bins_per_slice;
    const int kend = min(M, kbeg + bins_per_slice);
    const size_t plane = (size_t)M * kHeadDim;
    float *base = coefV + (size_t)bh * 2 * plane;
    const int gcol = b * HQ + h * GQ;
    float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
    uint32_t t = 0;
    if (APPEND) {
        size_t xrow;
        fold_locate(fold, t_len[b], bh, g.P, xrow, t);
        x = load4(v_new + xrow * kHeadDim + lane * 4);
    }
    float4 acc[GQ];
#pragma unroll
    for (int q = 0; q < GQ; ++q) acc[q] = make_float4(0.f, 0.f, 0.f, 0.f);
    pdl_wait();                                      // Zf and the normalisers come from the previous kernel

    for (int c0 = kbeg; c0 < kend; c0 += kOutChunk) {
        const int cn = min(kOutChunk, kend - c0);
        __syncthreads();                             // previous chunk's weights are no longer read
        if ((int)threadIdx.x < cn && Wg != nullptr) {
            // the column transform has left the weights ready: Wg[col][bin index]
#pragma unroll
            for (int q = 0; q < GQ; ++q) wgt[threadIdx.x][q] = Wg[(size_t)(gcol + q) * M + c0 + threadIdx.x];
            if (APPEND) {
                float cs, sn;
                twiddle(phase_mod((uint32_t)bins[c0 + threadIdx.x], t, g.P), g.P, cs, sn);
                upd[threadIdx.x] = make_float2(cs, sn);
            }
        } else if ((int)threadIdx.x < cn) {
            const uint32_t bin = (uint32_t)bins[c0 + threadIdx.x];
            const float w = 0.5f * hermitian_weight(bin, g.P);
            const int ka = (int)bin & (g.N - 1), kb = (g.N - ka) & (g.N - 1);
            const float2 ph = unit_phasor(bin, g.P);
            // (checked build: a column outside the array reads column 0; no thread may leave before the barrier below)
            const int zcol = FAEDKV_IN_BOUNDS(kTagAttnFft, bin <= g.P / 2 && gcol + GQ <= g.Gp) ? gcol : 0;
            const float2 *za_p = Zf + (uint32_t)ka * (uint32_t)g.Gp + zcol, *zb_p = Zf + (uint32_t)kb * (uint32_t)g.Gp + zcol;
#pragma unroll
            for (int q = 0; q < GQ; ++q) {
                const float2 za = za_p[q];
                float2 zb = zb_p[q];
                zb.y = -zb.y;
                const float2 A = cadd(za, zb), D = csub(za, zb);                 // 2A, 2jB
                const float2 W = cadd(A, cmul(ph, make_float2(D.y, -D.x)));       // 2 Pf
                wgt[threadIdx.x][q] = make_float2(w * W.x, -w * W.y);
            }
            if (APPEND) {
                float cs, sn;
                twiddle(phase_mod(bin, t, g.P), g.P, cs, sn);
                upd[threadIdx.x] = make_float2(cs, sn);
            }
        }
        __syncthreads();
        for (int i0 = warp * 4; i0 < cn; i0 += kAttnWarps * 4) {
            float4 re[4], im[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                re[u] = im[u] = make_float4(0.f, 0.f, 0.f, 0.f);
                if (i0 + u < cn) {
                    const float *rp = base + (size_t)(c0 + i0 + u) * kHeadDim + lane * 4;
                    re[u] = ld_stream(rp);
                    im[u] = ld_stream(rp + plane);
                }
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                if (i0 + u >= cn) continue;
                if (APPEND) {
                    const float2 cs = upd[i0 + u];
                    re[u].x = fmaf(x.x, cs.x, re[u].x); im[u].x = fmaf(-x.x, cs.y, im[u].x);
                    re[u].y = fmaf(x.y, cs.x, re[u].y); im[u].y = fmaf(-x.y, cs.y, im[u].y);
                    re[u].z = fmaf(x.z, cs.x, re[u].z); im[u].z = fmaf(-x.z, cs.y, im[u].z);
                    re[u].w = fmaf(x.w, cs.x, re[u].w); im[u].w = fmaf(-x.w, cs.y, im[u].w);
                    float *wp = base + (size_t)(c0 + i0 + u) * kHeadDim + lane * 4;
                    st_stream(wp, re[u]);
                    st_stream(wp + plane, im[u]);
                }
#pragma unroll
                for (int q = 0; q < GQ; ++q) {
                    const float2 a = wgt[i0 + u][q];
                    acc[q].x = fmaf(re[u].x, a.x, fmaf(im[u].x, a.y, acc[q].x));
                    acc[q].y = fmaf(re[u].y, a.x, fmaf(im[u].y, a.y, acc[q].y));
                    acc[q].z = fmaf(re[u].z, a.x, fmaf(im[u].z, a.y, acc[q].z));
                    acc[q].w = fmaf(re[u].w, a.x, fmaf(im[u].w, a.y, acc[q].w));
                }
            }
        }
    }
    __syncthreads();                                 // the last chunk's weights are no longer read
#pragma unroll
    for (int q = 0; q < GQ; ++q) *reinterpret_cast<float4 *>(&red[warp][q][lane * 4]) = acc[q];
    __syncthreads();
    for (int e = threadIdx.x; e < GQ * kHeadDim; e += blockDim.x) {
        const int q = e / kHeadDim, c = e % kHeadDim;
        float s = 0.f;
#pragma unroll
        for (int w = 0; w < kAttnWarps; ++w) s += red[w][q][c];
        if (FAEDKV_IN_BOUNDS(kTagAttnFft, (int)blockIdx.x < slice_stride && bh < n_units))
            partial[(((size_t)bh * slice_stride + blockIdx.x) * GQ + q) * kHeadDim + c] = s;
    }
    // last CTA of this (sequence, kv head): reduce the slices in a fixed order
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
        const unsigned int prev = atomicAdd(&tickets[bh], 1u);
        last_flag = prev == gridDim.x - 1 ? 1u : 0u;
        if (last_flag) tickets[bh] = 0u;             // ready for the next call on this stream
    }
    __syncthreads();
    if (last_flag) {
        __threadfence();
        for (int e = threadIdx.x; e < GQ * kHeadDim; e += blockDim.x) {
            const int q = e / kHeadDim, c = e % kHeadDim;
            float s = 0.f;
            for (int sl = 0; sl < (int)gridDim.x; ++sl)
                s += __ldcg(partial + (((size_t)bh * slice_stride + sl) * GQ + q) * kHeadDim + c);
            s *= inv_P;
            // the sink + recent window's share of the same softmax (its factor sits behind the normalisers)
            if (o_win != nullptr) s = fmaf(o_win[(size_t)(gcol + q) * kHeadDim + c], colsum[g.Gp + gcol + q], s);
            // a sequence with no visible token (t_len = 0 and no window) has an empty softmax: its output is zero
            const float den = colsum[gcol + q];
            store1(out + (size_t)(gcol + q) * kHeadDim + c, den > 0.f ? s / den : 0.f);
        }
        if (bump) {
            // every CTA of this sequence has read t_len (and the token it folds) before taking its ticket; the
            // last CTA of the sequence's last kv head, once all H heads are through, lets the new token take
            // its ring slot (windowed step) and advances the counter
            __shared__ unsigned int seq_last;
            if (threadIdx.x == 0) {
                const unsigned int done = atomicAdd(&tickets[n_units + b], 1u);
                seq_last = done == (unsigned int)H - 1u ? 1u : 0u;
                if (seq_last) tickets[n_units + b] = 0u;
            }
            __syncthreads();
            if (seq_last) {
                const int tt = t_len[b];
                if (commit.Rc > 0) {
                    const int W = commit.S + commit.Rc, slot = commit.S + (tt - commit.S) % commit.Rc;
                    TQ *wK = static_cast<TQ *>(const_cast<void *>(commit.winK)), *wV = static_cast<TQ *>(const_cast<void *>(commit.winV));
                    const TQ *kn = static_cast<const TQ *>(commit.k_new), *vn = static_cast<const TQ *>(commit.v_new);
                    for (int e = threadIdx.x; e < H * kHeadDim; e += blockDim.x) {
                        const size_t unit = (size_t)b * H + e / kHeadDim;
                        const int c = e % kHeadDim;
                        wK[(unit * W + slot) * kHeadDim + c] = kn[unit * kHeadDim + c];
                        wV[(unit * W + slot) * kHeadDim + c] = vn[unit * kHeadDim + c];
                    }
                }
                __syncthreads();
                if (threadIdx.x == 0) t_len[b] = tt + 1;
            }
        }
    }
}

}  // namespace faedkv
