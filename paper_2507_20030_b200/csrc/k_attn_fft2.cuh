// Steps (2)-(4) of the frequency-domain decode attention (see k_attn_fft.cuh) for grids 32768 <= P <= 2^17, whose
// columns are too long for one CTA: the same two-pass scheme and the same three kernels as k_afft_inv_a / k_afft_mid /
// k_afft_fwd_b, written on the two-columns-per-thread arithmetic of the second reconstruction engine (k_recon2.cuh).
//
//   * A thread owns two ADJACENT COLUMNS (query heads) of every point: butterflies, rotations and twiddle products
//     are packed float32x2 instructions, shared-memory exchange is one 16-byte access per point, index arithmetic
//     is paid once per two columns.  At batch 1 (32 columns) a pass is one wave of CTAs with one butterfly per
//     thread and stage, so its duration is the latency of one tile: half the instructions per point halve it.
//   * No per-CTA tables: the packing phasors e^{+j 2 pi k / P} and the inter-pass twiddles e^{+j 2 pi k2 m1 / N}
//     come from two global tables of the context (L2-resident, read through the read-only path), the plan slots
//     straight from the plan; no table-building prologue and no barrier before the first loads.
//   * The middle kernel keeps ONE tile in shared memory: scores, probabilities and both exchanges live in it, the
//     stages that overwrite what other threads still read take all their inputs into registers first
//     (stage<..., SYNC = true>).  64 KB per CTA instead of 96: every pass fits one wave at batch 1.
//
// Layouts.  Qs [M][Gp] float2 (from k_attn_qs), Zf [N][Gp] float2 (to k_attn_out_fft), statistics [tiles + 1][Gp]
// as in k_attn_fft.cuh, Gp a multiple of 32.  The array between the passes is private to these kernels:
// Y2 [Gp / 32][N1][N2][16] values of two columns each.
#pragma once
#include "common.cuh"
#include "k_fft.cuh"
#include "k_recon2.cuh"

namespace faedkv {
namespace afft2 {

using rfft2::C2;
using rfft2::cadd_j;
using rfft2::cmul;
using rfft2::padd;
using rfft2::psub;

constexpr int kThreads = 256;
constexpr int kCW = 32;              // columns per column block
constexpr int kCP = 16;              // column pairs per block
constexpr int kLgCP = 4;
constexpr int kLgTile = 12;          // 4096 two-column values (64 KB) per tile
constexpr int kMaxLg = 8;

__host__ __device__ constexpr int lg_per_tile(int lg_rows, int lg_other) {
    int lg = kLgTile - lg_rows - kLgCP;
    if (lg < 0) lg = 0;
    if (lg > lg_other) lg = lg_other;
    return lg;
}

// One Stockham stage of radix R over NF rows x (1 << LGC) column items, all butterflies of a thread held in
// registers; with SYNC every thread has read its inputs before any thread writes an output, so that the stage
// may overwrite the array it reads (the exchange tile doubling as input or output).
template <int NF, int R, int NS, int LGC, bool SYNC, typename In, typename Out>
__device__ __forceinline__ void stage(const float2 *__restrict__ tw, In in, Out out) {
    constexpr int NB = NF / R;
    constexpr int items = NB << LGC;
    constexpr int BPT = (items + kThreads - 1) / kThreads;
    C2 v[BPT][R];
#pragma unroll
    for (int b = 0; b < BPT; ++b) {
        const int it = b * kThreads + (int)threadIdx.x;
        if (items % kThreads != 0 && it >= items) continue;
        const int c = it & ((1 << LGC) - 1), j = it >> LGC;
#pragma unroll
        for (int r = 0; r < R; ++r) v[b][r] = in(j + r * NB, c);
        const int k = j & (NS - 1);
        if (NS > 1) {
#pragma unroll
            for (int r = 1; r < R; ++r) v[b][r] = cmul(v[b][r], tw[k * r * (NF / (NS * R))]);
        }
        rfft2::dft<R>(v[b]);
    }
    if (SYNC) __syncthreads();
#pragma unroll
    for (int b = 0; b < BPT; ++b) {
        const int it = b * kThreads + (int)threadIdx.x;
        if (items % kThreads != 0 && it >= items) continue;
        const int c = it & ((1 << LGC) - 1), j = it >> LGC;
        const int k = j & (NS - 1), j0 = (j - k) * R + k;
#pragma unroll
        for (int r = 0; r < R; ++r) out(j0 + fft::perm<R>(r) * NS, c, v[b][r]);
    }
}

// Length-2^LG transform over the rows of a tile; IN_XA: the inputs come out of xa itself, OUT_XA: the outputs
// go back into xa (both through load / store, which the caller writes accordingly).  One __syncthreads()
// between the stages, none before the first or after the last (beyond those SYNC stages need).
template <int LG, int LGC, bool IN_XA, bool OUT_XA, typename Load, typename Store>
__device__ __forceinline__ void fft_rows(C2 *xa, const float2 *tw, Load load, Store store) {
    constexpr int NF = 1 << LG;
    constexpr int R1 = fft::Radix<LG>::R1, R2 = fft::Radix<LG>::R2;
    static_assert(fft::Radix<LG>::R3 == 1, "two stages at most");
    auto rd = [&](int row, int c) { return xa[(row << LGC) + c]; };
    auto wr = [&](int row, int c, C2 v) { xa[(row << LGC) + c] = v; };
    if constexpr (R2 == 1) {
        stage<NF, R1, 1, LGC, IN_XA && OUT_XA>(tw, load, store);
    } else {
        stage<NF, R1, 1, LGC, IN_XA>(tw, load, wr);
        __syncthreads();
        stage<NF, R2, R1, LGC, OUT_XA>(tw, rd, store);
    }
}

__device__ __forceinline__ C2 from_aos(float4 v) { return C2{make_float2(v.x, v.z), make_float2(v.y, v.w)}; }
__device__ __forceinline__ float4 to_aos(C2 v) { return make_float4(v.re.x, v.im.x, v.re.y, v.im.y); }
// Two adjacent columns of a [rows][Gp] float2 array when pred, else zeros, without a branch.
__device__ __forceinline__ float4 ld4_if(const float2 *p, bool pred) {
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    asm("{\n\t.reg .pred q;\n\tsetp.ne.b32 q, %5, 0;\n\t@q ld.global.v4.f32 {%0, %1, %2, %3}, [%4];\n\t}"
        : "+f"(v.x), "+f"(v.y), "+f"(v.z), "+f"(v.w) : "l"(p), "r"((int)pred));
    return v;
}

struct Tables {
    const float2 *tabP;     // [N + 1]: e^{+j 2 pi k / P}
    const float2 *tabI;     // [N1 * N2]: e^{+j 2 pi k2 m1 / N} at m1 * N2 + k2
};

// ---- (2) pass A of the inverse transform, half-spectrum packing fused into the load --------------------------
// grid = (N2 / KT, Gp / 32); block = 256; dynamic smem = smem_bytes<LG1, LG2>().
template <int LG1, int LG2>
__global__ void __launch_bounds__(kThreads, 2)
k_afft2_inv_a(int Gp, const int32_t *__restrict__ slot, const float2 *__restrict__ Qs, Tables tb, C2 *__restrict__ Y2) {
    constexpr int N1 = 1 << LG1, N2 = 1 << LG2, N = N1 * N2, LGKT = lg_per_tile(LG1, LG2);
    extern __shared__ __align__(16) unsigned char smem_a2[];
    C2 *xa = reinterpret_cast<C2 *>(smem_a2);
    float2 *tw = reinterpret_cast<float2 *>(xa + (fft::exchange_buffers(LG1) > 0 ? (1 << (LG1 + LGKT + kLgCP)) : 0));
    for (int i = threadIdx.x; i < N1; i += kThreads) tw[i] = fft::unit_phasor((uint32_t)i, (uint32_t)N1);   // used after the stage barrier
    const int k2_0 = blockIdx.x << LGKT, cb = blockIdx.y;
    C2 *Yb = Y2 + (size_t)cb * N * kCP;
    pdl_wait();                                      // Qs comes from the previous kernel
    auto load = [&](int k1, int c) {
        const int cp = c & (kCP - 1), k = N2 * k1 + k2_0 + (c >> kLgCP);
        const int sa = __ldg(slot + k), sb = __ldg(slot + (N - k));
        const uint32_t col = (uint32_t)(cb * kCW + 2 * cp);
        // Z[k] = (X[k] + conj X[N-k]) + j e^{+j 2 pi k / P} (X[k] - conj X[N-k]); absent bins read as zero, branch-free
        const C2 xk = from_aos(ld4_if(Qs + (uint32_t)(sa < 0 ? 0 : sa) * (uint32_t)Gp + col, sa >= 0));
        const C2 xm = from_aos(ld4_if(Qs + (uint32_t)(sb < 0 ? 0 : sb) * (uint32_t)Gp + col, sb >= 0));
        const C2 s{padd(xk.re, xm.re), psub(xk.im, xm.im)}, d{psub(xk.re, xm.re), padd(xk.im, xm.im)};
        return cadd_j(s, cmul(d, __ldg(tb.tabP + k)));
    };
    auto store = [&](int m1, int c, C2 v) {
        Yb[((size_t)m1 * N2 + k2_0 + (c >> kLgCP)) * kCP + (c & (kCP - 1))] = v;      // the inter-pass twiddle is applied by the reader
    };
    fft_rows<LG1, LGKT + kLgCP, false, false>(xa, tw, load, store);
}

// ---- pass B of the inverse transform, local softmax, pass A' of the forward transform ------------------------
// One CTA = MT values of m1 (one "tile" of the softmax statistics) x 32 columns, in place in Y2.
// mloc, sloc: [N1 / MT][Gp].  live length of a column = min(q(t_len[col / HQ] + t_add), P).
// grid = (N1 / MT, Gp / 32); block = 256.
template <int LG1, int LG2>
__global__ void __launch_bounds__(kThreads, 2)
k_afft2_mid(int Gp, int G, C2 *__restrict__ Y2, Tables tb, const int32_t *__restrict__ t_len, int HQ, int t_add, int t_quant,
            float *__restrict__ mloc, float *__restrict__ sloc) {
    constexpr int N1 = 1 << LG1, N2 = 1 << LG2, N = N1 * N2, LGMT = lg_per_tile(LG2, LG1), LGC = LGMT + kLgCP;
    constexpr uint32_t P = 2u * N;
    extern __shared__ __align__(16) unsigned char smem_m2[];
    C2 *xa = reinterpret_cast<C2 *>(smem_m2);                        // exchange tile, then scores, then probabilities
    float2 *tw = reinterpret_cast<float2 *>(xa + (1 << (LG2 + LGC)));
    __shared__ float2 red[kThreads];
    __shared__ float2 colv[kCP];
    for (int i = threadIdx.x; i < N2; i += kThreads) tw[i] = fft::unit_phasor((uint32_t)i, (uint32_t)N2);
    const int m1_0 = blockIdx.x << LGMT, cb = blockIdx.y;
    C2 *Yb = Y2 + (size_t)cb * N * kCP;
    // a thread always meets the same column pair: kThreads is a multiple of 16
    const int cp = threadIdx.x & (kCP - 1);
    int live[2];
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        const int col = cb * kCW + 2 * cp + i;
        live[i] = 0;
        if (col < G) {
            long long t = (long long)t_len[col / HQ] + t_add;
            if (t_quant > 1 && t > 0) t = t / t_quant * t_quant;      // block-deferred fold: whole blocks only
            live[i] = t < 0 ? 0 : (t < (long long)P ? (int)t : (int)P);
        }
    }
    pdl_wait();                                      // Y2 comes from the previous kernel
    float2 mx = make_float2(-INFINITY, -INFINITY);
    {
        auto load = [&](int k2, int c) {
            const int m1 = m1_0 + (c >> kLgCP);
            const float2 w = __ldg(tb.tabI + m1 * N2 + k2);
            const float4 v = __ldcg(reinterpret_cast<const float4 *>(Yb + ((size_t)m1 * N2 + k2) * kCP + (c & (kCP - 1))));
            return cmul(C2{make_float2(v.x, v.y), make_float2(v.z, v.w)}, w);
        };
        // z[m1 + N1 m2] = scores of positions 2m (re) and 2m + 1 (im) of both columns; left in the tile, the maximum
        // of the live ones collected on the way out of the registers
        auto store = [&](int m2, int c, C2 v) {
            xa[(m2 << LGC) + c] = v;
            const int n0 = 2 * (m1_0 + (c >> kLgCP) + N1 * m2);
            if (n0 < live[0]) mx.x = fmaxf(mx.x, v.re.x);
            if (n0 + 1 < live[0]) mx.x = fmaxf(mx.x, v.im.x);
            if (n0 < live[1]) mx.y = fmaxf(mx.y, v.re.y);
            if (n0 + 1 < live[1]) mx.y = fmaxf(mx.y, v.im.y);
        };
        fft_rows<LG2, LGC, false, true>(xa, tw, load, store);
    }
    red[threadIdx.x] = mx;
    __syncthreads();                                 // also: the tile of scores is complete
    if (threadIdx.x < kCP) {
        float2 m = red[threadIdx.x];
#pragma unroll
        for (int i = 1; i < kThreads / kCP; ++i) {
            const float2 o = red[threadIdx.x + kCP * i];
            m.x = fmaxf(m.x, o.x); m.y = fmaxf(m.y, o.y);
        }
        colv[threadIdx.x] = m;
    }
    __syncthreads();
    const float2 mcol = colv[cp];
    float2 sum = make_float2(0.f, 0.f);
    {
        // p~ = exp(s - tile max) on the live positions, formed as the forward pass reads the tile
        auto load = [&](int m2, int c) {
            const C2 v = xa[(m2 << LGC) + c];
            const int n0 = 2 * (m1_0 + (c >> kLgCP) + N1 * m2);
            C2 p;
            p.re.x = n0 < live[0] ? __expf(v.re.x - mcol.x) : 0.f;
            p.im.x = n0 + 1 < live[0] ? __expf(v.im.x - mcol.x) : 0.f;
            p.re.y = n0 < live[1] ? __expf(v.re.y - mcol.y) : 0.f;
            p.im.y = n0 + 1 < live[1] ? __expf(v.im.y - mcol.y) : 0.f;
            sum.x += p.re.x + p.im.x;
            sum.y += p.re.y + p.im.y;
            return p;
        };
        auto store = [&](int k1p, int c, C2 v) {
            Yb[((size_t)(m1_0 + (c >> kLgCP)) * N2 + k1p) * kCP + (c & (kCP - 1))] = v;   // twiddle applied by the reader
        };
        fft_rows<LG2, LGC, true, false>(xa, tw, load, store);
    }
    __syncthreads();                                 // red is free again
    red[threadIdx.x] = sum;
    __syncthreads();
    if (threadIdx.x < kCP) {
        float2 sm = red[threadIdx.x];
#pragma unroll
        for (int i = 1; i < kThreads / kCP; ++i) {
            const float2 o = red[threadIdx.x + kCP * i];
            sm.x += o.x; sm.y += o.y;
        }
        const size_t o = (size_t)blockIdx.x * Gp + cb * kCW + 2 * threadIdx.x;
        *reinterpret_cast<float2 *>(mloc + o) = colv[threadIdx.x];
        *reinterpret_cast<float2 *>(sloc + o) = sm;
    }
}

// ---- pass B' of the forward transform --------------------------------------------------------------------------
// Every softmax tile is first brought to the column's global maximum (factor exp(mloc - max_tiles mloc)); the CTAs
// with blockIdx.x == 0 also write the softmax normaliser colsum[col] = sum_tiles sloc * factor and, with n_extra,
// the factor of the window tile to colsum[Gp + col].  Zf: [N][Gp] float2, index k1' + N2 * k2'.
// grid = (N2 / KT, Gp / 32); block = 256.
template <int LG1, int LG2>
__global__ void __launch_bounds__(kThreads, 2)
k_afft2_fwd_b(int Gp, const C2 *__restrict__ Y2, Tables tb, const float *__restrict__ mloc, const float *__restrict__ sloc,
              float2 *__restrict__ Zf, float *__restrict__ colsum, int n_extra) {
    constexpr int N1 = 1 << LG1, N2 = 1 << LG2, N = N1 * N2, LGKT = lg_per_tile(LG1, LG2), LGMT = lg_per_tile(LG2, LG1);
    constexpr int n_tiles = N1 >> LGMT;
    extern __shared__ __align__(16) unsigned char smem_f2[];
    C2 *xa = reinterpret_cast<C2 *>(smem_f2);
    float2 *tw = reinterpret_cast<float2 *>(xa + (fft::exchange_buffers(LG1) > 0 ? (1 << (LG1 + LGKT + kLgCP)) : 0));
    float2 *fac = tw + N1;                           // [n_tiles + 1][16] factors of the two columns of a pair
    __shared__ float2 red[kThreads];
    __shared__ float2 mg[kCP];
    for (int i = threadIdx.x; i < N1; i += kThreads) tw[i] = fft::unit_phasor((uint32_t)i, (uint32_t)N1);
    const int k1_0 = blockIdx.x << LGKT, cb = blockIdx.y;
    const C2 *Yb = Y2 + (size_t)cb * N * kCP;
    const int n_stat = n_tiles + n_extra;
    const int cp = threadIdx.x & (kCP - 1);
    const size_t c0 = (size_t)cb * kCW + 2 * cp;
    pdl_wait();                                      // the statistics and Y2 come from the previous kernel
    {
        float2 mx = make_float2(-INFINITY, -INFINITY);
        for (int ti = threadIdx.x >> kLgCP; ti < n_stat; ti += kThreads / kCP) {
            const float2 m = *reinterpret_cast<const float2 *>(mloc + (size_t)ti * Gp + c0);
            mx.x = fmaxf(mx.x, m.x); mx.y = fmaxf(mx.y, m.y);
        }
        red[threadIdx.x] = mx;
        __syncthreads();
        if (threadIdx.x < kCP) {
            float2 m = red[threadIdx.x];
#pragma unroll
            for (int i = 1; i < kThreads / kCP; ++i) {
                const float2 o = red[threadIdx.x + kCP * i];
                m.x = fmaxf(m.x, o.x); m.y = fmaxf(m.y, o.y);
            }
            mg[threadIdx.x] = m;
        }
        __syncthreads();
        const float2 m = mg[cp];
        float2 part = make_float2(0.f, 0.f);
        for (int ti = threadIdx.x >> kLgCP; ti < n_stat; ti += kThreads / kCP) {
            const float2 ml = *reinterpret_cast<const float2 *>(mloc + (size_t)ti * Gp + c0);
            const float2 f = make_float2(ml.x == -INFINITY ? 0.f : __expf(ml.x - m.x), ml.y == -INFINITY ? 0.f : __expf(ml.y - m.y));
            fac[ti * kCP + cp] = f;
            if (blockIdx.x == 0) {
                const float2 sl = *reinterpret_cast<const float2 *>(sloc + (size_t)ti * Gp + c0);
                part.x += f.x * sl.x; part.y += f.y * sl.y;
                if (ti == n_tiles) *reinterpret_cast<float2 *>(colsum + Gp + c0) = f;
            }
        }
        if (blockIdx.x == 0) {
            __syncthreads();
            red[threadIdx.x] = part;
            __syncthreads();
            if (threadIdx.x < kCP) {
                float2 s = red[threadIdx.x];
#pragma unroll
                for (int i = 1; i < kThreads / kCP; ++i) {
                    const float2 o = red[threadIdx.x + kCP * i];
                    s.x += o.x; s.y += o.y;
                }
                *reinterpret_cast<float2 *>(colsum + (size_t)cb * kCW + 2 * threadIdx.x) = s;
            }
        }
        __syncthreads();
    }
    auto load = [&](int m1, int c) {
        const int cc = c & (kCP - 1), k1p = k1_0 + (c >> kLgCP);
        const float2 f = fac[(m1 >> LGMT) * kCP + cc];
        const float2 w = __ldg(tb.tabI + m1 * N2 + k1p);
        const float4 v = __ldcg(reinterpret_cast<const float4 *>(Yb + ((size_t)m1 * N2 + k1p) * kCP + cc));
        return cmul(C2{__fmul2_rn(make_float2(v.x, v.y), f), __fmul2_rn(make_float2(v.z, v.w), f)}, w);
    };
    auto store = [&](int k2p, int c, C2 v) {
        const uint32_t row = (uint32_t)(k1_0 + (c >> kLgCP)) + (uint32_t)N2 * (uint32_t)k2p;
        *reinterpret_cast<float4 *>(Zf + row * (uint32_t)Gp + (uint32_t)(cb * kCW + 2 * (c & (kCP - 1)))) = to_aos(v);
    };
    fft_rows<LG1, LGKT + kLgCP, false, false>(xa, tw, load, store);
}

template <int LG1, int LG2> constexpr size_t smem_a() {
    return (fft::exchange_buffers(LG1) > 0 ? ((size_t)1 << (LG1 + lg_per_tile(LG1, LG2) + kLgCP)) * sizeof(C2) : 0) + ((size_t)1 << LG1) * sizeof(float2);
}
template <int LG1, int LG2> constexpr size_t smem_mid() {
    return ((size_t)1 << (LG2 + lg_per_tile(LG2, LG1) + kLgCP)) * sizeof(C2) + ((size_t)1 << LG2) * sizeof(float2);
}
template <int LG1, int LG2> constexpr size_t smem_fwd_b() {
    return smem_a<LG1, LG2>() + (size_t)(((1 << LG1) >> lg_per_tile(LG2, LG1)) + 1) * kCP * sizeof(float2);
}

// tabI[m1 * N2 + k2] = e^{+j 2 pi k2 m1 / N} (no scale; the packing table tabP is the reconstruction's).
__global__ void k_afft2_tables(float2 *__restrict__ tabI, uint32_t N, int N2) {
    for (uint32_t i = blockIdx.x * blockDim.x + threadIdx.x; i < N; i += gridDim.x * blockDim.x)
        tabI[i] = fft::unit_phasor((i / (uint32_t)N2) * (i % (uint32_t)N2), N);
}

}  // namespace afft2
}  // namespace faedkv
