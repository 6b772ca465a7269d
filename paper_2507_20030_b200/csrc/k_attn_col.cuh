// Steps (2)-(4) of the frequency-domain decode attention in ONE kernel, for grids P <= 16384: a column
// (sequence, query head) of N = P/2 packed complex points fits the shared memory of one CTA, so the inverse
// transform of the score spectrum, the softmax over the live positions and the forward transform of the
// probabilities (Eq. 3 on Eq. 11, same packing and unpacking formulas as k_fft.cuh) run without leaving it:
//
//   pack       Z[k] from the retained bins of Qs (half-spectrum packing), scattered into the zeroed column
//   inverse    z[m] = s[2m] + j s[2m+1]: in-place Stockham stages of radix 4 / 8 / 16 over the whole column
//   softmax    maximum and sum over n < live, p = exp(s - max), in place; the sink + recent window, when there
//              is one, joins here (its statistics come from k_attn_window)
//   forward    Zf = transform of p[2m] + j p[2m+1], same stages
//   unpack     w_k Pf[k] at the retained bins only -> Wg[col][i], the weights the pass over C_V consumes
//
// Against the two-pass kernels of k_attn_fft.cuh this drops two launches, the two-pass arrays in global
// memory (three round trips of N complex values per column) and the per-tile softmax statistics.
//
// A stage is "every thread reads the inputs of its butterflies into registers; barrier; every thread writes
// its outputs; barrier", which makes the autosort work in place.  Twiddles: a stage whose span NS * R is at
// most 1024 has a table of its own, laid out so that consecutive threads read consecutive entries (a shared
// table indexed k * r is read with strides and bank conflicts); the last stage of a longer column (span = N)
// takes w = e^{+j 2 pi k / N} from a table and multiplies its way through w^2, w^3, ... (15 products at most).
// The column is padded by one element per 16 so that the stride-R writes of the first stage spread over
// the banks.
#pragma once
#include "common.cuh"
#include "k_fft.cuh"

namespace faedkv {
namespace colfft {

constexpr int kLgE = 10;                             // E has 2^10 entries
constexpr int kMaxLg = 13;                           // N <= 8192: 64 KB of column per CTA

// Radices of the stages of a length-2^LGN column.
template <int LGN> struct Stages;
template <> struct Stages<5> { static constexpr int R1 = 4, R2 = 8, R3 = 1, R4 = 1; };
template <> struct Stages<6> { static constexpr int R1 = 8, R2 = 8, R3 = 1, R4 = 1; };
template <> struct Stages<7> { static constexpr int R1 = 8, R2 = 16, R3 = 1, R4 = 1; };
template <> struct Stages<8> { static constexpr int R1 = 16, R2 = 16, R3 = 1, R4 = 1; };
template <> struct Stages<9> { static constexpr int R1 = 8, R2 = 8, R3 = 8, R4 = 1; };
template <> struct Stages<10> { static constexpr int R1 = 16, R2 = 8, R3 = 8, R4 = 1; };
template <> struct Stages<11> { static constexpr int R1 = 16, R2 = 16, R3 = 8, R4 = 1; };
template <> struct Stages<12> { static constexpr int R1 = 16, R2 = 16, R3 = 16, R4 = 1; };
template <> struct Stages<13> { static constexpr int R1 = 8, R2 = 8, R3 = 8, R4 = 16; };

// One thread per 16 points, 64 to 512 threads.
template <int LGN> __host__ __device__ constexpr int threads() {
    return (1 << LGN) / 16 < 64 ? 64 : ((1 << LGN) / 16 > 512 ? 512 : (1 << LGN) / 16);
}
// Entries of the w = e^{+j 2 pi k / N} table the last stage needs (0: every stage has a table of its own).
template <int LGN> __host__ __device__ constexpr int chain_entries() {
    using S = Stages<LGN>;
    return (1 << LGN) <= (1 << kLgE) ? 0 : (1 << LGN) / (S::R4 > 1 ? S::R4 : (S::R3 > 1 ? S::R3 : S::R2));
}
// Entries of the per-stage twiddle tables tw[(r - 1) * NS + k] = e^{+j 2 pi k r / (NS * R)} of stages 2 and 3
// (stage 3: 0 when it is the chained last stage, or absent).
template <int LGN> __host__ __device__ constexpr int tw2_entries() { return (Stages<LGN>::R2 - 1) * Stages<LGN>::R1; }
template <int LGN> __host__ __device__ constexpr int tw3_entries() {
    using S = Stages<LGN>;
    return (S::R3 > 1 && S::R1 * S::R2 * S::R3 <= (1 << kLgE)) ? (S::R3 - 1) * S::R1 * S::R2 : 0;
}
__host__ __device__ constexpr int padded(int idx) { return idx + (idx >> 4); }
template <int LGN> constexpr size_t smem_bytes() {
    return (size_t)(padded(1 << LGN) + 1 + tw2_entries<LGN>() + tw3_entries<LGN>() + chain_entries<LGN>()) * sizeof(float2);
}

// One in-place stage of radix R over the N-point column z; NS = product of the radices already applied.
// OWN: the inputs are the column itself; otherwise in(index) supplies them (the gather).
// Butterfly j reads points j + r * NB and writes points j0 + perm(r) * NS.  In every stage of the plans above
// the low four bits of the base and of the offset never carry (NB and NS are multiples of 16, or base and
// offset occupy disjoint low bits), so padded(base + offset) = padded(base) + padded(offset): one padded
// base per butterfly, compile-time offsets from it.
// pre(value, index) is applied to every input read from the column, post(index, value) sees every output.
struct NoPre { __device__ __forceinline__ float2 operator()(float2 v, int) const { return v; } };
struct NoPost { __device__ __forceinline__ void operator()(int, float2) const {} };

// tw: this stage's table tw[(r - 1) * NS + k] (consecutive threads read consecutive entries), or, for the
// chained last stage of a long column, w[k] = e^{+j 2 pi k / N}.
template <int N, int NT, int R, int NS, bool OWN, typename In, typename Pre, typename Post>
__device__ __forceinline__ void stage(float2 *__restrict__ z, const float2 *__restrict__ tw, In in, Pre pre, Post post) {
    using namespace fft;
    constexpr int NB = N / R;                        // butterflies; also the stride of a butterfly's inputs
    constexpr int BPT = (NB + NT - 1) / NT;          // butterflies per thread
    constexpr int T = NS * R;                        // span of the twiddles of this stage
    float2 v[BPT][R];
#pragma unroll
    for (int b = 0; b < BPT; ++b) {
        const int j = threadIdx.x + b * NT;
        if (NB % NT != 0 && j >= NB) continue;
        if constexpr (OWN) {
            const float2 *src = z + padded(j);
#pragma unroll
            for (int r = 0; r < R; ++r) v[b][r] = pre(src[padded(r * NB)], j + r * NB);
        } else {
#pragma unroll
            for (int r = 0; r < R; ++r) v[b][r] = in(j + r * NB);
        }
        if (NS > 1) {
            const int k = j & (NS - 1);
            if constexpr (T <= (1 << kLgE)) {
#pragma unroll
                for (int r = 1; r < R; ++r) v[b][r] = cmul(v[b][r], tw[(r - 1) * NS + k]);
            } else {
                const float2 w1 = tw[k];
                float2 w = w1;
#pragma unroll
                for (int r = 1; r < R; ++r) {
                    v[b][r] = cmul(v[b][r], w);
                    if (r + 1 < R) w = cmul(w, w1);
                }
            }
        }
        dft<R>(v[b]);
    }
    __syncthreads();                                 // every input of the stage has been read
#pragma unroll
    for (int b = 0; b < BPT; ++b) {
        const int j = threadIdx.x + b * NT;
        if (NB % NT != 0 && j >= NB) continue;
        const int k = j & (NS - 1);
        float2 *dst = z + padded((j - k) * R + k);
#pragma unroll
        for (int r = 0; r < R; ++r) {
            dst[padded(perm<R>(r) * NS)] = v[b][r];
            post((j - k) * R + k + perm<R>(r) * NS, v[b][r]);
        }
    }
    __syncthreads();
}

// All stages of one transform.  The first stage reads first(index), or with OWN_FIRST the column itself
// through pre(value, index); post(index, value) sees the outputs of the last stage.
template <int LGN, bool OWN_FIRST, typename First, typename Pre, typename Post>
__device__ __forceinline__ void transform(float2 *__restrict__ z, const float2 *__restrict__ tw2, const float2 *__restrict__ tw3,
                                          const float2 *__restrict__ chain, First first, Pre pre, Post post) {
    using S = Stages<LGN>;
    constexpr int N = 1 << LGN, NT = threads<LGN>();
    constexpr int n_stages = S::R4 > 1 ? 4 : (S::R3 > 1 ? 3 : 2);
    constexpr bool chained3 = n_stages == 3 && tw3_entries<LGN>() == 0;
    stage<N, NT, S::R1, 1, OWN_FIRST>(z, tw2, first, pre, NoPost());
    if constexpr (n_stages == 2) stage<N, NT, S::R2, S::R1, true>(z, tw2, first, NoPre(), post);
    else stage<N, NT, S::R2, S::R1, true>(z, tw2, first, NoPre(), NoPost());
    if constexpr (n_stages == 3) stage<N, NT, S::R3, S::R1 * S::R2, true>(z, chained3 ? chain : tw3, first, NoPre(), post);
    else if constexpr (n_stages == 4) stage<N, NT, S::R3, S::R1 * S::R2, true>(z, tw3, first, NoPre(), NoPost());
    if constexpr (n_stages == 4) stage<N, NT, S::R4, S::R1 * S::R2 * S::R3, true>(z, chain, first, NoPre(), post);
}

// Block-wide maximum / sum of one value per thread; every thread gets the result.
template <int NT, bool MAX>
__device__ __forceinline__ float block_reduce(float v, float *red) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float u = __shfl_xor_sync(0xffffffffu, v, o);
        v = MAX ? fmaxf(v, u) : v + u;
    }
    __syncthreads();                                 // red may still be read from the previous reduction
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
    __syncthreads();
    float r = red[0];
#pragma unroll
    for (int w = 1; w < NT / 32; ++w) r = MAX ? fmaxf(r, red[w]) : r + red[w];
    return r;
}

// Tables shared by all columns: E[i] = e^{+j 2 pi i / 1024}; B[k] = e^{+j 2 pi k / N}, k < 1024;
// Pk[k] = e^{+j 2 pi k / P}, k <= N (the packing phasor of point k and the unpacking phasor of bin k).
__global__ void k_col_tables(float2 *__restrict__ E, float2 *__restrict__ Bt, float2 *__restrict__ Pk, uint32_t P) {
    const uint32_t N = P / 2;
    for (uint32_t i = blockIdx.x * blockDim.x + threadIdx.x; i <= N || i < (1u << kLgE); i += gridDim.x * blockDim.x) {
        if (i < (1u << kLgE)) {
            E[i] = fft::unit_phasor(i, 1u << kLgE);
            Bt[i] = fft::unit_phasor(i % N, N);
        }
        if (i <= N) Pk[i] = fft::unit_phasor(i, P);
    }
}

// Qs: [G][M] (column-major: a column's retained score spectrum is contiguous), already scaled by
// scale / P, imaginary part of the self-conjugate bins zero.  bins: [M] the plan's retained bins, ascending.
// live length of a column = min(q(t_len[col / HQ] + t_add), P), q() rounding down to a multiple of t_quant.
// m_w, s_w: statistics of the window tile ([G] each) or nullptr.  Out: Wg [G][M] = (w Re Pf, -w Im Pf),
// scaled to the joint maximum; colsum[col] = joint softmax normaliser, colsum[Gp + col] = the factor that
// brings the window's unnormalised output to the joint maximum.
// grid = (G); block = threads<LGN>(); dynamic smem = smem_bytes<LGN>().
template <int LGN>
__global__ void __launch_bounds__(threads<LGN>(), threads<LGN>() >= 512 ? 2 : 1)
k_afft_col(uint32_t P, int M, const int32_t *__restrict__ bins,
           const float2 *__restrict__ Qs, const float2 *__restrict__ tabE, const float2 *__restrict__ tabB,
           const float2 *__restrict__ tabP, const int32_t *__restrict__ t_len, int HQ, int t_add, int t_quant,
           const float *__restrict__ m_w, const float *__restrict__ s_w, float2 *__restrict__ Wg,
           float *__restrict__ colsum, int Gp, int col0) {
    using namespace fft;
    constexpr int N = 1 << LGN, NT = threads<LGN>(), NC = chain_entries<LGN>();
    extern __shared__ float2 col_smem[];
    __shared__ float red[NT / 32];
    using S = Stages<LGN>;
    constexpr int N2 = tw2_entries<LGN>(), N3 = tw3_entries<LGN>();
    float2 *z = col_smem;
    float2 *tw2 = z + padded(N) + 1;
    float2 *tw3 = tw2 + N2;
    float2 *Bt = tw3 + N3;
    const int col = col0 + (int)blockIdx.x;          // a launch may cover a run of columns
    // per-stage twiddle tables, entry (r - 1) * NS + k = e^{+j 2 pi k r / (NS * R)}, from E (first used after barriers)
    for (int e = threadIdx.x; e < N2; e += NT) {
        constexpr int NS = S::R1, T = S::R1 * S::R2;
        tw2[e] = tabE[(e % NS) * (e / NS + 1) * ((1 << kLgE) / T)];
    }
    for (int e = threadIdx.x; e < N3; e += NT) {
        constexpr int NS = S::R1 * S::R2, T = (N3 > 0 ? NS * S::R3 : 1);
        tw3[e] = tabE[(e % NS) * (e / NS + 1) * ((1 << kLgE) / T)];
    }
    for (int i = threadIdx.x; i < NC; i += NT) Bt[i] = tabB[i];
    long long tl = (long long)t_len[col / HQ] + t_add;
    if (t_quant > 1 && tl > 0) tl = tl / t_quant * t_quant;      // block-deferred fold: whole blocks only
    const int live = tl < 0 ? 0 : (tl < (long long)P ? (int)tl : (int)P);
    pdl_wait();                                      // Qs comes from the previous kernel
    const float2 *X = Qs + (size_t)col * M;
    // ---- half-spectrum packing, from the retained bins outwards (most of the N points are zero):
    //   Z[k] = X[k] (1 + j e^{+j2pi k/P}) + conj(X[N-k]) (1 - j e^{+j2pi k/P})
    // every retained bin b < N lands on point b, every retained bin b > 0 on point N - b; a point gets at most
    // one term of each kind, so two rounds of plain stores / read-modify-writes need no atomics
    for (int i = threadIdx.x; i < N; i += NT) z[padded(i)] = make_float2(0.f, 0.f);
    __syncthreads();
    for (int i = threadIdx.x; i < M; i += NT) {
        const int bin = bins[i];
        if (!FAEDKV_IN_BOUNDS(kTagAttnCol, bin >= 0 && bin <= N)) continue;
        if (bin < N) {
            const float2 ph = tabP[bin];
            z[padded(bin)] = cmul(X[i], make_float2(1.f - ph.y, ph.x));          // 1 + j ph
        }
    }
    __syncthreads();
    for (int i = threadIdx.x; i < M; i += NT) {
        const int bin = bins[i];
        if (!FAEDKV_IN_BOUNDS(kTagAttnCol, bin >= 0 && bin <= N)) continue;
        if (bin > 0) {
            const int k = N - bin;
            const float2 ph = tabP[k];
            const float2 x = X[i];
            const float2 t = cmul(make_float2(x.x, -x.y), make_float2(1.f + ph.y, -ph.x));   // conj(X) (1 - j ph)
            float2 &dst = z[padded(k)];
            dst = cadd(dst, t);
        }
    }
    __syncthreads();
    // ---- inverse transform in place; the last stage leaves z[m] = (s[2m], s[2m+1]) and every thread the
    // maximum of the live scores it wrote
    float mx = -INFINITY;
    transform<LGN, true>(z, tw2, tw3, Bt, [&](int) { return make_float2(0.f, 0.f); }, NoPre(), [&](int m, float2 v) {
        if (2 * m < live) mx = fmaxf(mx, v.x);
        if (2 * m + 1 < live) mx = fmaxf(mx, v.y);
    });
    const float m_col = block_reduce<NT, true>(mx, red);
    // ---- softmax over n < live, applied as the forward transform reads the column:
    // p[2m] + j p[2m+1] = exp(s - max) on the live positions, 0 elsewhere; then the transform itself
    float sum = 0.f;
    transform<LGN, true>(z, tw2, tw3, Bt, [&](int) { return make_float2(0.f, 0.f); }, [&](float2 v, int m) {
        const float pe = 2 * m < live ? __expf(v.x - m_col) : 0.f;
        const float po = 2 * m + 1 < live ? __expf(v.y - m_col) : 0.f;
        sum += pe + po;
        return make_float2(pe, po);
    }, NoPost());
    const float s_col = block_reduce<NT, false>(sum, red);
    // the window joins the softmax as one more segment: bring both to the joint maximum
    const float mw = m_w != nullptr ? m_w[col] : -INFINITY;
    const float m_all = fmaxf(m_col, mw);
    const float f_col = m_col == -INFINITY ? 0.f : __expf(m_col - m_all);
    const float f_w = mw == -INFINITY ? 0.f : __expf(mw - m_all);
    if (threadIdx.x == 0) {
        colsum[col] = s_col * f_col + (m_w != nullptr ? s_w[col] * f_w : 0.f);
        colsum[Gp + col] = f_w;
    }
    // ---- unpacking at the retained bins: W[k] = (Zf[k'] + conj Zf[-k'])/2 + e^{+j2pi k/P} (Zf[k'] - conj Zf[-k'])/(2j)
    float2 *out = Wg + (size_t)col * M;
    for (int i = threadIdx.x; i < M; i += NT) {
        const uint32_t bin = (uint32_t)bins[i];
        if (!FAEDKV_IN_BOUNDS(kTagAttnCol, bin <= (uint32_t)N)) continue;
        const float w = 0.5f * hermitian_weight(bin, P) * f_col;
        const int ka = (int)bin & (N - 1), kb = (N - ka) & (N - 1);
        const float2 za = z[padded(ka)];
        float2 zb = z[padded(kb)];
        zb.y = -zb.y;
        const float2 A = cadd(za, zb), D = csub(za, zb);                    // 2A, 2jB
        const float2 W = cadd(A, cmul(tabP[bin], make_float2(D.y, -D.x)));  // 2 Pf
        out[i] = make_float2(w * W.x, -w * W.y);
    }
}

}  // namespace colfft
}  // namespace faedkv
