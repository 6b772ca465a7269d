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
//                        over C_V (with APPEND the update of C_V on the way)
//       k_attn_out_reduce_fft   sum partials, divide by P * (softmax normaliser); APPEND: t_len += 1
//
// The scores never leave shared memory; the only intermediates in (L2-resident) global memory are the
// two-pass arrays Y, Zf of P/2 complex values per column and the per-tile softmax statistics.
#pragma once
#include "common.cuh"
#include "k_attn.cuh"
#include "k_fft.cuh"

namespace faedkv {

// ---- (1) ------------------------------------------------------------------------------------------
// grid = (ceil(M / (8 * KB)), batch * H); block = 256; KB = 16 / GQ bins per warp.
template <typename TQ, int GQ, bool APPEND>
__global__ void __launch_bounds__(kAttnWarps * 32)
k_attn_qs(const TQ *__restrict__ q, float *__restrict__ coefK, const TQ *__restrict__ k_new,
          const int32_t *__restrict__ t_len, const int32_t *__restrict__ bins, float2 *__restrict__ Qs,
          int M, int H, int HQ, int Gp, uint32_t P, float scale_over_P) {
    constexpr int KB = 16 / GQ;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int bh = blockIdx.y, b = bh / H, h = bh % H;
    const int k0 = (blockIdx.x * kAttnWarps + warp) * KB;
    if (k0 >= M) return;
    float4 qv[GQ];
#pragma unroll
    for (int g = 0; g < GQ; ++g) qv[g] = load4(q + ((size_t)b * HQ + h * GQ + g) * kHeadDim + lane * 4);
    const size_t plane = (size_t)M * kHeadDim;
    float *base = coefK + (size_t)bh * 2 * plane;
    float4 row[KB][2];
#pragma unroll
    for (int kk = 0; kk < KB; ++kk)
#pragma unroll
        for (int pl = 0; pl < 2; ++pl) {
            row[kk][pl] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (k0 + kk < M) row[kk][pl] = ld_stream(base + pl * plane + (size_t)(k0 + kk) * kHeadDim + lane * 4);
        }
    if (APPEND) {
        // C_K[k, c] += k_new[c] * e^{-j w k t}: same arithmetic as k_append
        const uint32_t t = (uint32_t)t_len[b] % P;
        const float4 x = load4(k_new + (size_t)bh * kHeadDim + lane * 4);
#pragma unroll
        for (int kk = 0; kk < KB; ++kk) {
            if (k0 + kk >= M) continue;
            float c, s;
            twiddle(phase_mod((uint32_t)bins[k0 + kk], t, P), P, c, s);
            float4 &re = row[kk][0], &im = row[kk][1];
            re.x = fmaf(x.x, c, re.x); im.x = fmaf(-x.x, s, im.x);
            re.y = fmaf(x.y, c, re.y); im.y = fmaf(-x.y, s, im.y);
            re.z = fmaf(x.z, c, re.z); im.z = fmaf(-x.z, s, im.z);
            re.w = fmaf(x.w, c, re.w); im.w = fmaf(-x.w, s, im.w);
            float *dst = base + (size_t)(k0 + kk) * kHeadDim + lane * 4;
            st_stream(dst, re);
            st_stream(dst + plane, im);
        }
    }
    float v[32];
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
    if (k0 + kk < M) {
        const uint32_t bin = (uint32_t)bins[k0 + kk];
        // bins 0 and P/2 are their own mirrors: only their real part enters a real signal
        const bool self_conj = bin == 0u || 2u * bin == P;
        float *dst = reinterpret_cast<float *>(Qs + (size_t)(k0 + kk) * Gp + b * HQ + h * GQ + g);
        dst[pl] = (pl == 1 && self_conj) ? 0.f : tot * scale_over_P;
    }
}

// ---- (2) pass A of the inverse transform, half-spectrum packing fused into the load ----------------
// slot[k], k in [0, N]: index of one-sided bin k in the plan, or -1.  Y: [N1][N2][Gp].
// grid = (N2 / KT, Gp / 16); block = 256; dynamic smem = fft::smem_bytes(N1, KT).
__global__ void __launch_bounds__(fft::kThreads)
k_afft_inv_a(fft::Geometry g, const int32_t *__restrict__ slot, const float2 *__restrict__ Qs,
             float2 *__restrict__ Y, int lgKT) {
    using namespace fft;
    extern __shared__ float2 fft_smem[];
    const int KT = 1 << lgKT, lg_cols = lgKT + 4;
    const int tile = g.N1 << lg_cols;
    float2 *a = fft_smem, *b = fft_smem + tile, *tw = fft_smem + 2 * tile;
    fill_twiddles(tw, g.N1);
    const int k2_0 = blockIdx.x * KT, g0 = blockIdx.y * kCW;
    for (int e = threadIdx.x; e < tile; e += kThreads) {
        const int c = e & (kCW - 1), kt = (e >> 4) & (KT - 1), k1 = e >> lg_cols;
        const int k = g.N2 * k1 + k2_0 + kt;                 // 0 <= k < N
        const int col = g0 + c;
        float2 z = make_float2(0.f, 0.f);
        if (col < g.G) {
            const int sa = slot[k], sb = slot[g.N - k];
            if (sa >= 0 || sb >= 0) {
                const float2 xa = sa >= 0 ? Qs[(size_t)sa * g.Gp + col] : make_float2(0.f, 0.f);
                float2 xb = sb >= 0 ? Qs[(size_t)sb * g.Gp + col] : make_float2(0.f, 0.f);
                xb.y = -xb.y;                                            // conj X[N-k]
                const float2 s = cadd(xa, xb), d = csub(xa, xb);
                z = cadd(s, cmulj(cmul(unit_phasor((uint32_t)k, g.P), d)));
            }
        }
        a[e] = z;
    }
    __syncthreads();
    const float2 *res = fft_tile(a, b, tw, g.N1, lg_cols);
    for (int e = threadIdx.x; e < tile; e += kThreads) {
        const int c = e & (kCW - 1), kt = (e >> 4) & (KT - 1), m1 = e >> lg_cols;
        const int k2 = k2_0 + kt;
        Y[y_index(g, m1, k2, g0 + c)] = cmul(res[e], unit_phasor((uint32_t)(k2 * m1), (uint32_t)g.N));
    }
}

// ---- pass B of the inverse transform, local softmax, pass A' of the forward transform ---------------
// One CTA = MT values of m1 (one "tile" of the softmax statistics) x 16 columns.
// mloc, sloc: [N1 / MT][Gp].  live length of a column = min(t_len[col / HQ] + t_add, P).
// grid = (N1 / MT, Gp / 16); block = 256; dynamic smem = fft::smem_bytes(N2, MT).
__global__ void __launch_bounds__(fft::kThreads)
k_afft_mid(fft::Geometry g, float2 *__restrict__ Y, const int32_t *__restrict__ t_len, int HQ, int t_add,
           float *__restrict__ mloc, float *__restrict__ sloc, int lgMT) {
    using namespace fft;
    extern __shared__ float2 fft_smem[];
    __shared__ float red[kThreads];
    __shared__ float colv[kCW];
    __shared__ int live_s[kCW];
    const int MT = 1 << lgMT, lg_cols = lgMT + 4;
    const int tile = g.N2 << lg_cols;
    float2 *a = fft_smem, *b = fft_smem + tile, *tw = fft_smem + 2 * tile;
    fill_twiddles(tw, g.N2);
    const int m1_0 = blockIdx.x * MT, g0 = blockIdx.y * kCW;
    if (threadIdx.x < kCW) {
        const int col = g0 + threadIdx.x;
        int live = 0;
        if (col < g.G) {
            const long long t = (long long)t_len[col / HQ] + t_add;
            live = t < (long long)g.P ? (int)t : (int)g.P;
        }
        live_s[threadIdx.x] = live;
    }
    for (int e = threadIdx.x; e < tile; e += kThreads) {
        const int c = e & (kCW - 1), mt = (e >> 4) & (MT - 1), row = e >> lg_cols;
        a[e] = Y[y_index(g, m1_0 + mt, row, g0 + c)];
    }
    __syncthreads();
    float2 *res = fft_tile(a, b, tw, g.N2, lg_cols);        // rows are now m2; element = z[m1 + N1 m2]
    // a thread always meets the same column: kThreads is a multiple of 16
    const int c = threadIdx.x & (kCW - 1);
    const int live = live_s[c];
    float mx = -INFINITY;
    for (int e = threadIdx.x; e < tile; e += kThreads) {
        const int mt = (e >> 4) & (MT - 1), m2 = e >> lg_cols;
        const int n0 = 2 * (m1_0 + mt + g.N1 * m2);
        const float2 v = res[e];
        if (n0 < live) mx = fmaxf(mx, v.x);
        if (n0 + 1 < live) mx = fmaxf(mx, v.y);
    }
    red[threadIdx.x] = mx;
    __syncthreads();
    if (threadIdx.x < kCW) {
        float m = red[threadIdx.x];
#pragma unroll
        for (int i = 1; i < kThreads / kCW; ++i) m = fmaxf(m, red[threadIdx.x + kCW * i]);
        colv[threadIdx.x] = m;
    }
    __syncthreads();
    const float mcol = colv[c];
    float sum = 0.f;
    for (int e = threadIdx.x; e < tile; e += kThreads) {
        const int mt = (e >> 4) & (MT - 1), m2 = e >> lg_cols;
        const int n0 = 2 * (m1_0 + mt + g.N1 * m2);
        const float2 v = res[e];
        const float pe = n0 < live ? __expf(v.x - mcol) : 0.f;
        const float po = n0 + 1 < live ? __expf(v.y - mcol) : 0.f;
        sum += pe + po;
        res[e] = make_float2(pe, po);
    }
    red[threadIdx.x] = sum;
    __syncthreads();
    if (threadIdx.x < kCW) {
        float s = red[threadIdx.x];
#pragma unroll
        for (int i = 1; i < kThreads / kCW; ++i) s += red[threadIdx.x + kCW * i];
        mloc[(size_t)blockIdx.x * g.Gp + g0 + threadIdx.x] = colv[threadIdx.x];
        sloc[(size_t)blockIdx.x * g.Gp + g0 + threadIdx.x] = s;
    }
    const float2 *res2 = fft_tile(res, res == a ? b : a, tw, g.N2, lg_cols);   // rows are now k1'
    for (int e = threadIdx.x; e < tile; e += kThreads) {
        const int cc = e & (kCW - 1), mt = (e >> 4) & (MT - 1), k1p = e >> lg_cols;
        const int m1 = m1_0 + mt;
        Y[y_index(g, m1, k1p, g0 + cc)] = cmul(res2[e], unit_phasor((uint32_t)(k1p * m1), (uint32_t)g.N));
    }
}

// ---- pass B' of the forward transform ---------------------------------------------------------------
// Every softmax tile is first brought to the column's global maximum: factor exp(mloc - max_tiles mloc).
// Zf: [N][Gp], index k1' + N2 * k2'.
// grid = (N2 / KT, Gp / 16); block = 256; dynamic smem = fft::smem_bytes(N1, KT).
__global__ void __launch_bounds__(fft::kThreads)
k_afft_fwd_b(fft::Geometry g, const float2 *__restrict__ U, const float *__restrict__ mloc, int lgMT,
             float2 *__restrict__ Zf, int lgKT) {
    using namespace fft;
    extern __shared__ float2 fft_smem[];
    __shared__ float red[kThreads];
    __shared__ float mg[kCW];
    const int KT = 1 << lgKT, lg_cols = lgKT + 4;
    const int tile = g.N1 << lg_cols;
    float2 *a = fft_smem, *b = fft_smem + tile, *tw = fft_smem + 2 * tile;
    fill_twiddles(tw, g.N1);
    const int k1_0 = blockIdx.x * KT, g0 = blockIdx.y * kCW;
    const int n_tiles = g.N1 >> lgMT;
    {
        const int c = threadIdx.x & (kCW - 1);
        float mx = -INFINITY;
        for (int ti = threadIdx.x >> 4; ti < n_tiles; ti += kThreads / kCW) mx = fmaxf(mx, mloc[(size_t)ti * g.Gp + g0 + c]);
        red[threadIdx.x] = mx;
        __syncthreads();
        if (threadIdx.x < kCW) {
            float m = red[threadIdx.x];
#pragma unroll
            for (int i = 1; i < kThreads / kCW; ++i) m = fmaxf(m, red[threadIdx.x + kCW * i]);
            mg[threadIdx.x] = m;
        }
        __syncthreads();
    }
    for (int e = threadIdx.x; e < tile; e += kThreads) {
        const int c = e & (kCW - 1), kt = (e >> 4) & (KT - 1), m1 = e >> lg_cols;
        const float ml = mloc[(size_t)(m1 >> lgMT) * g.Gp + g0 + c];
        const float f = ml == -INFINITY ? 0.f : __expf(ml - mg[c]);
        const float2 v = U[y_index(g, m1, k1_0 + kt, g0 + c)];
        a[e] = make_float2(v.x * f, v.y * f);
    }
    __syncthreads();
    const float2 *res = fft_tile(a, b, tw, g.N1, lg_cols);   // rows are now k2'
    for (int e = threadIdx.x; e < tile; e += kThreads) {
        const int c = e & (kCW - 1), kt = (e >> 4) & (KT - 1), k2p = e >> lg_cols;
        Zf[((size_t)(k1_0 + kt) + (size_t)g.N2 * k2p) * g.Gp + g0 + c] = res[e];
    }
}

// ---- (5) ------------------------------------------------------------------------------------------
// grid = (slices, batch * H); block = 256.
template <typename TQ, int GQ, bool APPEND>
__global__ void __launch_bounds__(kAttnWarps * 32)
k_attn_out_fft(float *__restrict__ coefV, const TQ *__restrict__ v_new, const int32_t *__restrict__ t_len,
               const float2 *__restrict__ Zf, const int32_t *__restrict__ bins, float *__restrict__ partial,
               int M, int H, int HQ, fft::Geometry g, int bins_per_slice) {
    using namespace fft;
    __shared__ __align__(16) float red[kAttnWarps][GQ][kHeadDim];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int bh = blockIdx.y, b = bh / H, h = bh % H;
    const int kbeg = blockIdx.x * bins_per_slice;
    const int kend = min(M, kbeg + bins_per_slice);
    const size_t plane = (size_t)M * kHeadDim;
    float *base = coefV + (size_t)bh * 2 * plane;
    const int gcol = b * HQ + h * GQ;
    float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
    uint32_t t = 0;
    if (APPEND) {
        x = load4(v_new + (size_t)bh * kHeadDim + lane * 4);
        t = (uint32_t)t_len[b] % g.P;
    }
    float4 acc[GQ];
#pragma unroll
    for (int q = 0; q < GQ; ++q) acc[q] = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int k = kbeg + warp; k < kend; k += kAttnWarps) {
        float *rp = base + (size_t)k * kHeadDim + lane * 4;
        float4 re = ld_stream(rp);
        float4 im = ld_stream(rp + plane);
        const uint32_t bin = (uint32_t)bins[k];
        if (APPEND) {
            float c, s;
            twiddle(phase_mod(bin, t, g.P), g.P, c, s);
            re.x = fmaf(x.x, c, re.x); im.x = fmaf(-x.x, s, im.x);
            re.y = fmaf(x.y, c, re.y); im.y = fmaf(-x.y, s, im.y);
            re.z = fmaf(x.z, c, re.z); im.z = fmaf(-x.z, s, im.z);
            re.w = fmaf(x.w, c, re.w); im.w = fmaf(-x.w, s, im.w);
            st_stream(rp, re);
            st_stream(rp + plane, im);
        }
        const float w = hermitian_weight(bin, g.P);
        const int ka = (int)bin & (g.N - 1), kb = (g.N - ka) & (g.N - 1);
        const float2 ph = unit_phasor(bin, g.P);
#pragma unroll
        for (int q = 0; q < GQ; ++q) {
            const float2 za = Zf[(size_t)ka * g.Gp + gcol + q];
            float2 zb = Zf[(size_t)kb * g.Gp + gcol + q];
            zb.y = -zb.y;
            const float2 A = cadd(za, zb), D = csub(za, zb);             // 2A, 2jB
            const float2 W = cadd(A, cmul(ph, make_float2(D.y, -D.x)));   // 2 Pf
            const float ar = 0.5f * w * W.x, ai = -0.5f * w * W.y;
            acc[q].x = fmaf(re.x, ar, fmaf(im.x, ai, acc[q].x));
            acc[q].y = fmaf(re.y, ar, fmaf(im.y, ai, acc[q].y));
            acc[q].z = fmaf(re.z, ar, fmaf(im.z, ai, acc[q].z));
            acc[q].w = fmaf(re.w, ar, fmaf(im.w, ai, acc[q].w));
        }
    }
#pragma unroll
    for (int q = 0; q < GQ; ++q) *reinterpret_cast<float4 *>(&red[warp][q][lane * 4]) = acc[q];
    __syncthreads();
    for (int e = threadIdx.x; e < GQ * kHeadDim; e += blockDim.x) {
        const int q = e / kHeadDim, c = e % kHeadDim;
        float s = 0.f;
#pragma unroll
        for (int w = 0; w < kAttnWarps; ++w) s += red[w][q][c];
        partial[(((size_t)bh * gridDim.x + blockIdx.x) * GQ + q) * kHeadDim + c] = s;
    }
}

// Sum the slice partials; softmax normaliser = sum_tiles sloc * exp(mloc - max mloc); convert.
// With bump_batch > 0 the first block also advances the token counters (fused append).
// grid = batch * H * GQ; block = 128.
template <typename TOut>
__global__ void __launch_bounds__(kHeadDim)
k_attn_out_reduce_fft(const float *__restrict__ partial, const float *__restrict__ mloc, const float *__restrict__ sloc,
                      int n_tiles, int Gp, TOut *__restrict__ out, int slices, int GQ, float inv_P,
                      int32_t *__restrict__ t_len, int bump_batch) {
    __shared__ float red[kHeadDim];
    const int bh = blockIdx.x / GQ, q = blockIdx.x % GQ, c = threadIdx.x;
    const int col = bh * GQ + q;                 // = sequence * HQ + head
    float mx = -INFINITY;
    for (int ti = c; ti < n_tiles; ti += kHeadDim) mx = fmaxf(mx, mloc[(size_t)ti * Gp + col]);
    red[c] = mx;
    __syncthreads();
    for (int s = kHeadDim / 2; s > 0; s >>= 1) {
        if (c < s) red[c] = fmaxf(red[c], red[c + s]);
        __syncthreads();
    }
    mx = red[0];
    __syncthreads();
    float sum = 0.f;
    for (int ti = c; ti < n_tiles; ti += kHeadDim) {
        const float ml = mloc[(size_t)ti * Gp + col];
        if (ml != -INFINITY) sum += sloc[(size_t)ti * Gp + col] * __expf(ml - mx);
    }
    red[c] = sum;
    __syncthreads();
    for (int s = kHeadDim / 2; s > 0; s >>= 1) {
        if (c < s) red[c] += red[c + s];
        __syncthreads();
    }
    const float colsum = red[0];
    float s = 0.f;
    for (int sl = 0; sl < slices; ++sl) s += partial[(((size_t)bh * slices + sl) * GQ + q) * kHeadDim + c];
    store1(out + (size_t)col * kHeadDim + c, s * inv_P / colsum);
    if (blockIdx.x == 0)
        for (int i = c; i < bump_batch; i += kHeadDim) t_len[i] += 1;
}

}  // namespace faedkv
