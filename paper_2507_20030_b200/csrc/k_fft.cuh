// FFT-shaped evaluation of the two pruned transforms for power-of-two grids P (Eq. 5 / Eq. 11 with every
// pruned bin zero, and its adjoint), float32 throughout.
//
// A real length-P signal is handled as a complex signal of length N = P/2 (even samples in the real
// part, odd samples in the imaginary part), and the complex length-N transform with kernel e^{+j2pi km/N}
// is split as N = N1 * N2 into two passes of small FFTs with one twiddle in between:
//
//   input index  k = N2*k1 + k2,   output index  m = m1 + N1*m2
//   pass A (per k2, over k1):   Y[m1][k2] = e^{+j2pi k2 m1/N} * sum_k1 Z[N2 k1 + k2] e^{+j2pi k1 m1/N1}
//   pass B (per m1, over k2):   z[m1 + N1 m2] = sum_k2 Y[m1][k2] e^{+j2pi k2 m2/N2}
//
// Half spectrum -> packed signal (X = retained bins, zero elsewhere, X[0], X[N] real):
//   Z[k] = (X[k] + conj X[N-k]) + j e^{+j2pi k/P} (X[k] - conj X[N-k]),   z[m] = s[2m] + j s[2m+1]
// Packed signal -> half spectrum of W[k] = sum_n p[n] e^{+j2pi kn/P}, with Zf = transform of p[2m] + j p[2m+1]:
//   W[k] = (Zf[k'] + conj Zf[-k'])/2 + e^{+j2pi k/P} (Zf[k'] - conj Zf[-k'])/(2j),   k' = k mod N
//
// One small FFT (length NF = 2^LG <= 512, many independent columns side by side) is a Stockham
// autosort of one to three register-resident butterflies of radix 4, 8 or 16: the first stage reads
// its inputs straight from wherever they are (global memory, a gather, another shared-memory tile),
// the last stage hands its outputs to a store functor, and only the exchange between stages goes
// through shared memory.
#pragma once
#include "common.cuh"

namespace faedkv {
namespace fft {

constexpr int kThreads = 256;
constexpr int kCW = 16;            // independent signals (columns) per CTA
constexpr int kLgCW = 4;
constexpr int kTileMax = 4096;     // complex elements of one shared-memory tile (32 KB) when NF * 16 allows

__host__ __device__ constexpr int ilog2(int v) { return v <= 1 ? 0 : 1 + ilog2(v >> 1); }

// Geometry of one problem: N = P/2 = N1 * N2 (powers of two, N1 >= N2, both at most 512 for P <= 2^19).
struct Geometry {
    uint32_t P;
    int N, N1, N2, lgN1, lgN2;
    int Gp;        // allocated columns (multiple of 32: two column blocks of kCW, one of the two-column kernels)
    int G;         // real columns
};
inline Geometry make_geometry(int P, int G) {
    Geometry g;
    g.P = (uint32_t)P;
    g.N = P / 2;
    const int lg = ilog2(g.N);
    g.lgN1 = (lg + 1) / 2;
    g.lgN2 = lg / 2;
    g.N1 = 1 << g.lgN1;
    g.N2 = 1 << g.lgN2;
    g.G = G;
    g.Gp = (G + 31) / 32 * 32;
    return g;
}
// P is a power of two whose two passes fit the shared-memory tiles (3 <= lgN1 <= 9, 2 <= lgN2 <= 9).
inline bool supported(int P) { return P >= 64 && P <= (1 << 19) && (P & (P - 1)) == 0; }

// How many transforms of a pass one CTA takes (a power of two): fill the tile, but keep at least
// ~2 CTAs per SM (n_sm of them on the device) in the grid when the problem allows.
inline int transforms_per_cta(int rows, int n_transforms, int col_blocks, int n_sm) {
    int kt = kTileMax / (rows * kCW);
    if (kt < 1) kt = 1;
    while (kt > 1 && (kt > n_transforms || (n_transforms / kt) * col_blocks < 2 * n_sm)) kt >>= 1;
    return kt;
}

__device__ __forceinline__ float2 cmul(float2 a, float2 b) {
    return make_float2(fmaf(a.x, b.x, -a.y * b.y), fmaf(a.x, b.y, a.y * b.x));
}
__device__ __forceinline__ float2 cadd(float2 a, float2 b) { return make_float2(a.x + b.x, a.y + b.y); }
__device__ __forceinline__ float2 csub(float2 a, float2 b) { return make_float2(a.x - b.x, a.y - b.y); }
__device__ __forceinline__ float2 cmulj(float2 a) { return make_float2(-a.y, a.x); }   // j * a

// Predicated global load: the value at p when pred, else zero, WITHOUT a branch.  The gathers of the half-spectrum
// packing use it: behind branches every point of a butterfly waits for its own round trip to memory in turn;
// predicated off instead of jumped over, the loads of all its points are in flight together.
__device__ __forceinline__ float2 ld2_if(const float2 *p, bool pred) {
    float2 v = make_float2(0.f, 0.f);
    asm("{\n\t.reg .pred q;\n\tsetp.ne.b32 q, %3, 0;\n\t@q ld.global.v2.f32 {%0, %1}, [%2];\n\t}"
        : "+f"(v.x), "+f"(v.y) : "l"(p), "r"((int)pred));
    return v;
}

// e^{+j 2 pi num / den}, 0 <= num < den <= 2^24 (den a power of two: the quotient is exact).
__device__ __forceinline__ float2 unit_phasor(uint32_t num, uint32_t den) {
    float c, s;
    twiddle(num, den, c, s);
    return make_float2(c, s);
}

// tw[i] = e^{+j 2 pi i / NF}
__device__ __forceinline__ void fill_twiddles(float2 *tw, int NF) {
    for (int i = threadIdx.x; i < NF; i += kThreads) tw[i] = unit_phasor((uint32_t)i, (uint32_t)NF);
}

// ---- register butterflies: DFT of size R with kernel e^{+j 2 pi kr / R} ----------------------------------
// Output r of the DFT is left in v[perm<R>(r)] (identity except for R = 16).
// Complex additions use the packed float32x2 instructions of sm_100 (one issue slot for both components;
// these kernels are issue-bound and additions are their largest instruction class); a - b is the packed FMA
// b * (-1) + a, which rounds exactly like the subtraction.  Rotations by +-j stay scalar: they only rename
// components, which packed operands cannot do for free.
__device__ __forceinline__ float2 padd(float2 a, float2 b) { return __fadd2_rn(a, b); }
__device__ __forceinline__ float2 psub(float2 a, float2 b) { return __ffma2_rn(b, make_float2(-1.f, -1.f), a); }
__device__ __forceinline__ void dft2(float2 &a, float2 &b) {
    const float2 t = a;
    a = padd(t, b);
    b = psub(t, b);
}
__device__ __forceinline__ void dft4(float2 &v0, float2 &v1, float2 &v2, float2 &v3) {
    const float2 a0 = padd(v0, v2), a1 = psub(v0, v2), a2 = padd(v1, v3), d = psub(v1, v3);
    v0 = padd(a0, a2);
    v2 = psub(a0, a2);
    v1 = make_float2(a1.x - d.y, a1.y + d.x);        // a1 + j d
    v3 = make_float2(a1.x + d.y, a1.y - d.x);        // a1 - j d
}
template <int R> __device__ __forceinline__ void dft(float2 (&v)[R]);
template <> __device__ __forceinline__ void dft<2>(float2 (&v)[2]) { dft2(v[0], v[1]); }
template <> __device__ __forceinline__ void dft<4>(float2 (&v)[4]) { dft4(v[0], v[1], v[2], v[3]); }
template <> __device__ __forceinline__ void dft<8>(float2 (&v)[8]) {
    dft4(v[0], v[2], v[4], v[6]);      // even samples  -> E[0..3] in v[0], v[2], v[4], v[6]
    dft4(v[1], v[3], v[5], v[7]);      // odd samples   -> O[0..3] in v[1], v[3], v[5], v[7]
    const float h = 0.70710678118654752f;
    const float2 o0 = v[1];
    const float2 o1 = make_float2(h * (v[3].x - v[3].y), h * (v[3].x + v[3].y));     // * e^{+j pi/4}
    const float2 o2 = v[5];                                                           // * e^{+j pi/2}, applied below
    const float2 o3 = make_float2(-h * (v[7].x + v[7].y), h * (v[7].x - v[7].y));    // * e^{+j 3pi/4}
    const float2 e0 = v[0], e1 = v[2], e2 = v[4], e3 = v[6];
    v[0] = padd(e0, o0); v[4] = psub(e0, o0);
    v[1] = padd(e1, o1); v[5] = psub(e1, o1);
    v[2] = make_float2(e2.x - o2.y, e2.y + o2.x);    // e2 + j o2
    v[6] = make_float2(e2.x + o2.y, e2.y - o2.x);    // e2 - j o2
    v[3] = padd(e3, o3); v[7] = psub(e3, o3);
}
// 16 = 4 x 4: n = n1 + 4 n2, k = k2 + 4 k1; X[k2 + 4 k1] ends in v[k1 + 4 k2].
template <> __device__ __forceinline__ void dft<16>(float2 (&v)[16]) {
#pragma unroll
    for (int n1 = 0; n1 < 4; ++n1) dft4(v[n1], v[n1 + 4], v[n1 + 8], v[n1 + 12]);   // v[n1 + 4 k2] = A[n1][k2]
    const float c1 = 0.92387953251128674f, s1 = 0.38268343236508977f, h = 0.70710678118654752f;
    // v[n1 + 4 k2] *= e^{+j 2 pi n1 k2 / 16}
    v[5] = cmul(v[5], make_float2(c1, s1));                                   // n1 k2 = 1
    v[6] = make_float2(h * (v[6].x - v[6].y), h * (v[6].x + v[6].y));         // 2
    v[7] = cmul(v[7], make_float2(s1, c1));                                   // 3
    v[9] = make_float2(h * (v[9].x - v[9].y), h * (v[9].x + v[9].y));         // 2
    v[10] = cmulj(v[10]);                                                     // 4
    v[11] = make_float2(-h * (v[11].x + v[11].y), h * (v[11].x - v[11].y));   // 6
    v[13] = cmul(v[13], make_float2(s1, c1));                                 // 3
    v[14] = make_float2(-h * (v[14].x + v[14].y), h * (v[14].x - v[14].y));   // 6
    v[15] = cmul(v[15], make_float2(-c1, -s1));                               // 9
#pragma unroll
    for (int k2 = 0; k2 < 4; ++k2) dft4(v[4 * k2], v[4 * k2 + 1], v[4 * k2 + 2], v[4 * k2 + 3]);
}
template <int R> __device__ __forceinline__ constexpr int perm(int r) { return R == 16 ? ((r >> 2) | ((r & 3) << 2)) : r; }

// Radices of the stages of a length-2^LG transform.
template <int LG> struct Radix;
template <> struct Radix<2> { static constexpr int R1 = 4, R2 = 1, R3 = 1; };
template <> struct Radix<3> { static constexpr int R1 = 8, R2 = 1, R3 = 1; };
template <> struct Radix<4> { static constexpr int R1 = 16, R2 = 1, R3 = 1; };
template <> struct Radix<5> { static constexpr int R1 = 4, R2 = 8, R3 = 1; };
template <> struct Radix<6> { static constexpr int R1 = 8, R2 = 8, R3 = 1; };
template <> struct Radix<7> { static constexpr int R1 = 8, R2 = 16, R3 = 1; };
template <> struct Radix<8> { static constexpr int R1 = 16, R2 = 16, R3 = 1; };
template <> struct Radix<9> { static constexpr int R1 = 8, R2 = 8, R3 = 8; };
// Shared-memory exchange buffers a transform of length 2^lg needs (each rows * columns float2).
__host__ __device__ constexpr int exchange_buffers(int lg) { return lg >= 9 ? 2 : (lg >= 5 ? 1 : 0); }

// One Stockham stage of radix R over NF rows x (1 << lg_cols) columns; NS = product of the radices
// already applied.  in(row, col) -> float2, out(row, col, value).
// LGC >= 0 fixes lg_cols at compile time (index arithmetic then folds into constants: these kernels are bound
// by integer ALU work, not by the butterflies); LGC = -1 takes the run-time value.
template <int NF, int R, int NS, int LGC, typename In, typename Out>
__device__ __forceinline__ void fft_stage(int lg_cols_rt, const float2 *__restrict__ tw, In in, Out out) {
    constexpr int NB = NF / R;          // butterflies per column; also the row stride of a butterfly's inputs
    const int lg_cols = LGC >= 0 ? LGC : lg_cols_rt;
    const int items = NB << lg_cols;
#pragma unroll
    for (int it = threadIdx.x; it < items; it += kThreads) {
        const int c = it & ((1 << lg_cols) - 1), j = it >> lg_cols;
        float2 v[R];
#pragma unroll
        for (int r = 0; r < R; ++r) v[r] = in(j + r * NB, c);
        const int k = j & (NS - 1);
        if (NS > 1) {
#pragma unroll
            for (int r = 1; r < R; ++r) v[r] = cmul(v[r], tw[k * r * (NF / (NS * R))]);
        }
        dft<R>(v);
        const int j0 = (j - k) * R + k;
#pragma unroll
        for (int r = 0; r < R; ++r) out(j0 + perm<R>(r) * NS, c, v[r]);
    }
}

// Length-2^LG transform over the rows of a tile of (1 << lg_cols) columns.  load(row, col) supplies the
// inputs, store(row, col, value) takes the outputs; xa, xb are the exchange buffers (see
// exchange_buffers()), tw the NF-entry twiddle table.  All threads of the CTA must call it; it
// contains __syncthreads() between stages but none before the first or after the last stage.
template <int LG, int LGC, typename Load, typename Store>
__device__ __forceinline__ void fft_rows(int lg_cols_rt, float2 *xa, float2 *xb, const float2 *tw, Load load, Store store) {
    constexpr int NF = 1 << LG;
    const int lg_cols = LGC >= 0 ? LGC : lg_cols_rt;
    constexpr int R1 = Radix<LG>::R1, R2 = Radix<LG>::R2, R3 = Radix<LG>::R3;
    auto rd_a = [&](int row, int c) {
        if (!FAEDKV_IN_BOUNDS(kTagFftEngine, row >= 0 && row < NF && c >= 0 && c < (1 << lg_cols))) return make_float2(0.f, 0.f);
        return xa[(row << lg_cols) + c];
    };
    auto wr_a = [&](int row, int c, float2 v) {
        if (FAEDKV_IN_BOUNDS(kTagFftEngine, row >= 0 && row < NF && c >= 0 && c < (1 << lg_cols))) xa[(row << lg_cols) + c] = v;
    };
    auto rd_b = [&](int row, int c) { return xb[(row << lg_cols) + c]; };
    auto wr_b = [&](int row, int c, float2 v) { xb[(row << lg_cols) + c] = v; };
    if constexpr (R2 == 1) {
        fft_stage<NF, R1, 1, LGC>(lg_cols, tw, load, store);
    } else if constexpr (R3 == 1) {
        fft_stage<NF, R1, 1, LGC>(lg_cols, tw, load, wr_a);
        __syncthreads();
        fft_stage<NF, R2, R1, LGC>(lg_cols, tw, rd_a, store);
    } else {
        fft_stage<NF, R1, 1, LGC>(lg_cols, tw, load, wr_a);
        __syncthreads();
        fft_stage<NF, R2, R1, LGC>(lg_cols, tw, rd_a, wr_b);
        __syncthreads();
        fft_stage<NF, R3, R1 * R2, LGC>(lg_cols, tw, rd_b, store);
    }
}

// The number of transforms per CTA (lg) for which the kernels have a compile-time-indexed instance: a 4096-element
// tile where the row count allows.
__host__ __device__ constexpr int fast_lg_transforms(int lg_rows) { return lg_rows >= 8 ? 0 : (lg_rows == 7 ? 1 : 2); }

// Element (m1, row, col) of the intermediate array between the two passes: [N1][N2][Gp] float2.
// 32-bit on purpose (address arithmetic is a visible share of these kernels' instructions): the host
// only takes the FFT-shaped path while N * Gp < 2^31.
__device__ __forceinline__ uint32_t y_index(const Geometry &g, int m1, int row, int col) {
    return ((uint32_t)m1 * (uint32_t)g.N2 + (uint32_t)row) * (uint32_t)g.Gp + (uint32_t)col;
}
inline bool fits_32bit_index(int P, int G) {
    const Geometry g = make_geometry(P, G);
    return (unsigned long long)g.N * (unsigned long long)g.Gp < (1ull << 31);
}

}  // namespace fft
}  // namespace faedkv
