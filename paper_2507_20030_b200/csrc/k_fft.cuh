// FFT-shaped evaluation of the two pruned transforms for power-of-two grids P (Eq. 5 / Eq. 11 with every
// pruned bin zero, and its adjoint), float32 throughout.
//
// A real length-P signal is handled as a complex signal of length N = P/2 (even samples in the real
// part, odd samples in the imaginary part), and the complex length-N transform with kernel e^{+j2pi km/N}
// is split as N = N1 * N2 into two passes of small shared-memory FFTs with one twiddle in between:
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
// The in-shared-memory FFT is a mixed-radix (8, 4, 2) Stockham autosort over the rows of a
// [rows][columns] tile, ping-ponging between two buffers; "columns" are independent signals
// (query heads or channels) times however many transforms of the pass the CTA takes.
#pragma once
#include "common.cuh"

namespace faedkv {
namespace fft {

constexpr int kThreads = 256;
constexpr int kCW = 16;            // independent signals (columns) per CTA
constexpr int kTileMax = 4096;     // complex elements of one shared-memory tile (32 KB; two tiles ping-pong)

__host__ __device__ constexpr int ilog2(int v) { return v <= 1 ? 0 : 1 + ilog2(v >> 1); }

// Geometry of one problem: N = P/2 = N1 * N2 (powers of two, N1 >= N2, both at most 512 for P <= 2^19).
struct Geometry {
    uint32_t P;
    int N, N1, N2, lgN1, lgN2;
    int Gp;        // allocated columns (multiple of kCW)
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
    g.Gp = (G + kCW - 1) / kCW * kCW;
    return g;
}
// P is a power of two whose two passes fit the shared-memory tiles.
inline bool supported(int P) { return P >= 64 && P <= (1 << 19) && (P & (P - 1)) == 0; }

// How many transforms of a pass one CTA takes (a power of two): fill the tile, but keep at least
// ~2 CTAs per SM in the grid when the problem allows.
inline int transforms_per_cta(int rows, int n_transforms, int col_blocks) {
    int kt = kTileMax / (rows * kCW);
    if (kt < 1) kt = 1;
    while (kt > 1 && (kt > n_transforms || (n_transforms / kt) * col_blocks < 2 * 148)) kt >>= 1;
    return kt;
}
inline size_t smem_bytes(int rows, int kt) { return (size_t)(2 * rows * kt * kCW + rows) * sizeof(float2); }

__device__ __forceinline__ float2 cmul(float2 a, float2 b) {
    return make_float2(fmaf(a.x, b.x, -a.y * b.y), fmaf(a.x, b.y, a.y * b.x));
}
__device__ __forceinline__ float2 cadd(float2 a, float2 b) { return make_float2(a.x + b.x, a.y + b.y); }
__device__ __forceinline__ float2 csub(float2 a, float2 b) { return make_float2(a.x - b.x, a.y - b.y); }
__device__ __forceinline__ float2 cmulj(float2 a) { return make_float2(-a.y, a.x); }   // j * a

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

// Natural-order DFTs of size 2, 4, 8 with kernel e^{+j 2 pi kr / R}.
__device__ __forceinline__ void dft2(float2 &a, float2 &b) {
    const float2 t = a;
    a = cadd(t, b);
    b = csub(t, b);
}
__device__ __forceinline__ void dft4(float2 &v0, float2 &v1, float2 &v2, float2 &v3) {
    const float2 a0 = cadd(v0, v2), a1 = csub(v0, v2), a2 = cadd(v1, v3), a3 = cmulj(csub(v1, v3));
    v0 = cadd(a0, a2);
    v1 = cadd(a1, a3);
    v2 = csub(a0, a2);
    v3 = csub(a1, a3);
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
    const float2 o2 = cmulj(v[5]);                                                    // * e^{+j pi/2}
    const float2 o3 = make_float2(-h * (v[7].x + v[7].y), h * (v[7].x - v[7].y));    // * e^{+j 3pi/4}
    const float2 e0 = v[0], e1 = v[2], e2 = v[4], e3 = v[6];
    v[0] = cadd(e0, o0); v[4] = csub(e0, o0);
    v[1] = cadd(e1, o1); v[5] = csub(e1, o1);
    v[2] = cadd(e2, o2); v[6] = csub(e2, o2);
    v[3] = cadd(e3, o3); v[7] = csub(e3, o3);
}

// One Stockham stage of radix R over a [NF][cols] tile; Ns = product of the radices already applied.
template <int R>
__device__ __forceinline__ void fft_stage(const float2 *__restrict__ in, float2 *__restrict__ out,
                                          const float2 *__restrict__ tw, int NF, int Ns, int lg_cols) {
    const int stride = (NF / R) << lg_cols;      // elements between the R inputs of a butterfly
    const int tw_step = NF / (Ns * R);
    for (int it = threadIdx.x; it < stride; it += kThreads) {
        const int c = it & ((1 << lg_cols) - 1), j = it >> lg_cols;
        const int k = j & (Ns - 1);
        float2 v[R];
#pragma unroll
        for (int r = 0; r < R; ++r) v[r] = in[it + r * stride];
        if (Ns > 1) {
#pragma unroll
            for (int r = 1; r < R; ++r) v[r] = cmul(v[r], tw[k * r * tw_step]);
        }
        dft<R>(v);
        const int j0 = (j - k) * R + k;
#pragma unroll
        for (int r = 0; r < R; ++r) out[((j0 + r * Ns) << lg_cols) + c] = v[r];
    }
}

// FFT over the rows of the tile in `a` (scratch `b`, same size); returns the buffer holding the result.
// Every thread of the CTA must call it; it ends with a __syncthreads().
__device__ __forceinline__ float2 *fft_tile(float2 *a, float2 *b, const float2 *tw, int NF, int lg_cols) {
    const int lg = 31 - __clz(NF);
    int Ns = 1;
    const int rem = lg % 3;
    if (rem == 1) {
        fft_stage<2>(a, b, tw, NF, Ns, lg_cols);
        Ns = 2;
    } else if (rem == 2) {
        fft_stage<4>(a, b, tw, NF, Ns, lg_cols);
        Ns = 4;
    }
    if (rem != 0) {
        __syncthreads();
        float2 *t = a; a = b; b = t;
    }
    while (Ns < NF) {
        fft_stage<8>(a, b, tw, NF, Ns, lg_cols);
        Ns *= 8;
        __syncthreads();
        float2 *t = a; a = b; b = t;
    }
    return a;
}

// Element (m1, row, col) of the intermediate array between the two passes: [N1][N2][Gp] float2.
__device__ __forceinline__ size_t y_index(const Geometry &g, int m1, int row, int col) {
    return ((size_t)m1 * g.N2 + row) * g.Gp + col;
}

}  // namespace fft
}  // namespace faedkv
