// FFT-shaped reconstruction (Eq. 11: Eq. 5 with every pruned bin zero) for power-of-two grids 64 <= P <= 2^17,
// second engine: one persistent kernel per call.
//
//     x~[n, c] = (1/P) sum_k w_k (Re C[k,c] cos(w k n) - Im C[k,c] sin(w k n)),   n < min(t, P)
//
// The transform is the two-pass scheme of k_fft.cuh (real signal of length P as a complex signal of length
// N = P/2 = N1 * N2; pass A over k1 with the half-spectrum packing fused into its loads, inter-pass twiddle,
// pass B over k2 writing rows 2m and 2m + 1).  What differs from the first engine:
//
//  * A thread owns TWO ADJACENT CHANNELS of every point it touches.  Channels are the contiguous axis of the
//    coefficient planes and of the output rows, real and imaginary parts are separate planes, so the natural
//    register form is (re of channels c, c+1), (im of channels c, c+1): every butterfly addition, every +-j
//    rotation and every twiddle product is then a packed float32x2 instruction, shared-memory exchange is one
//    16-byte access per point, and all index arithmetic is paid once per two channels.
//  * Both passes run in ONE launch.  Work is cut into items -- (pass, column block of 32 channels, tile) --
//    which the CTAs claim in a fixed global order through a ticket counter: the pass-A tiles of column block i,
//    then the pass-B tiles of block i - D.  A pass-B tile waits (bounded) until a counter says that all pass-A
//    tiles of its block are done.  Every wait is on items with SMALLER tickets, and an item is only claimed by
//    a CTA that is already running, so the earliest unfinished item can always proceed: no deadlock, whatever
//    the number of CTAs resident.
//  * The array between the passes is a ring of a few column blocks (a pass-A tile of block i first waits for
//    pass B of block i - ring): it is written and read back while still in L2 and never grows with the batch.
//
// Tables (per context): tabP[k] = e^{+j 2 pi k / P}, k <= N;  tabI[m1 * N2 + k2] = e^{+j 2 pi k2 m1 / N} / P.
#pragma once
#include "common.cuh"
#include "k_fft.cuh"
#include "k_recon_fft.cuh"

namespace faedkv {
namespace rfft2 {

constexpr int kThreads = 128;         // threads per CTA
constexpr int kCW = 32;              // channels per column block
constexpr int kCP = kCW / 2;         // channel pairs per column block: one thread each
constexpr int kLgCP = 4;
constexpr int kLgTile = 11;
constexpr int kTileElems = 1 << kLgTile;   // two-channel complex values (16 bytes) in the shared exchange tile
constexpr int kMaxLg = 8;            // N1, N2 <= 256: P <= 2^17
constexpr uint32_t kErrWaitA = 0x21, kErrWaitB = 0x22;
constexpr unsigned long long kWaitLimitNs = 1000000000ull;

// One complex value of two adjacent channels.
struct __align__(16) C2 {
    float2 re, im;
};
__device__ __forceinline__ float2 p2(float v) { return make_float2(v, v); }
__device__ __forceinline__ float2 padd(float2 a, float2 b) { return __fadd2_rn(a, b); }
__device__ __forceinline__ float2 psub(float2 a, float2 b) { return __ffma2_rn(b, make_float2(-1.f, -1.f), a); }
__device__ __forceinline__ C2 cadd(C2 a, C2 b) { return C2{padd(a.re, b.re), padd(a.im, b.im)}; }
__device__ __forceinline__ C2 csub(C2 a, C2 b) { return C2{psub(a.re, b.re), psub(a.im, b.im)}; }
__device__ __forceinline__ C2 cadd_j(C2 a, C2 d) { return C2{psub(a.re, d.im), padd(a.im, d.re)}; }   // a + j d
__device__ __forceinline__ C2 csub_j(C2 a, C2 d) { return C2{padd(a.re, d.im), psub(a.im, d.re)}; }   // a - j d
// a * (w.x + j w.y), the same factor for both channels
__device__ __forceinline__ C2 cmul(C2 a, float2 w) {
    const float2 wr = p2(w.x), wi = p2(w.y), nwi = p2(-w.y);
    return C2{__ffma2_rn(a.im, nwi, __fmul2_rn(a.re, wr)), __ffma2_rn(a.im, wr, __fmul2_rn(a.re, wi))};
}

// ---- register butterflies, kernel e^{+j 2 pi k r / R}; output r in v[fft::perm<R>(r)] -----------------------
__device__ __forceinline__ void dft4(C2 &v0, C2 &v1, C2 &v2, C2 &v3) {
    const C2 a0 = cadd(v0, v2), a1 = csub(v0, v2), a2 = cadd(v1, v3), d = csub(v1, v3);
    v0 = cadd(a0, a2);
    v2 = csub(a0, a2);
    v1 = cadd_j(a1, d);
    v3 = csub_j(a1, d);
}
template <int R> __device__ __forceinline__ void dft(C2 (&v)[R]);
template <> __device__ __forceinline__ void dft<4>(C2 (&v)[4]) { dft4(v[0], v[1], v[2], v[3]); }
template <> __device__ __forceinline__ void dft<8>(C2 (&v)[8]) {
    dft4(v[0], v[2], v[4], v[6]);      // even samples -> E[0..3] in v[0], v[2], v[4], v[6]
    dft4(v[1], v[3], v[5], v[7]);      // odd samples  -> O[0..3] in v[1], v[3], v[5], v[7]
    const float2 h = p2(0.70710678118654752f), nh = p2(-0.70710678118654752f);
    const C2 e0 = v[0], e1 = v[2], e2 = v[4], e3 = v[6], o0 = v[1], o2 = v[5];
    // O1 e^{+j pi/4} = h (x - y, x + y);  O3 e^{+j 3pi/4} = h (-(x + y), x - y): the factor h rides on the final FMAs
    const float2 d1 = psub(v[3].re, v[3].im), s1 = padd(v[3].re, v[3].im);
    const float2 d3 = psub(v[7].re, v[7].im), s3 = padd(v[7].re, v[7].im);
    v[0] = cadd(e0, o0); v[4] = csub(e0, o0);
    v[1] = C2{__ffma2_rn(d1, h, e1.re), __ffma2_rn(s1, h, e1.im)};
    v[5] = C2{__ffma2_rn(d1, nh, e1.re), __ffma2_rn(s1, nh, e1.im)};
    v[2] = cadd_j(e2, o2);
    v[6] = csub_j(e2, o2);
    v[3] = C2{__ffma2_rn(s3, nh, e3.re), __ffma2_rn(d3, h, e3.im)};
    v[7] = C2{__ffma2_rn(s3, h, e3.re), __ffma2_rn(d3, nh, e3.im)};
}
// 16 = 4 x 4: n = n1 + 4 n2, k = k2 + 4 k1; X[k2 + 4 k1] ends in v[k1 + 4 k2].
template <> __device__ __forceinline__ void dft<16>(C2 (&v)[16]) {
#pragma unroll
    for (int n1 = 0; n1 < 4; ++n1) dft4(v[n1], v[n1 + 4], v[n1 + 8], v[n1 + 12]);   // v[n1 + 4 k2] = A[n1][k2]
    const float c1 = 0.92387953251128674f, s1 = 0.38268343236508977f, hh = 0.70710678118654752f;
    const float2 h = p2(hh), nh = p2(-hh);
    auto rot45 = [&](C2 &a) { const float2 d = psub(a.re, a.im), s = padd(a.re, a.im); a = C2{__fmul2_rn(d, h), __fmul2_rn(s, h)}; };
    auto rot135 = [&](C2 &a) { const float2 d = psub(a.re, a.im), s = padd(a.re, a.im); a = C2{__fmul2_rn(s, nh), __fmul2_rn(d, h)}; };
    // v[n1 + 4 k2] *= e^{+j 2 pi n1 k2 / 16}
    v[5] = cmul(v[5], make_float2(c1, s1));       // n1 k2 = 1
    rot45(v[6]);                                  // 2
    v[7] = cmul(v[7], make_float2(s1, c1));       // 3
    rot45(v[9]);                                  // 2
    v[10] = C2{__fmul2_rn(v[10].im, p2(-1.f)), v[10].re};   // 4: times j
    rot135(v[11]);                                // 6
    v[13] = cmul(v[13], make_float2(s1, c1));     // 3
    rot135(v[14]);                                // 6
    v[15] = cmul(v[15], make_float2(-c1, -s1));   // 9
#pragma unroll
    for (int k2 = 0; k2 < 4; ++k2) dft4(v[4 * k2], v[4 * k2 + 1], v[4 * k2 + 2], v[4 * k2 + 3]);
}

// One Stockham stage of radix R over NF rows x (1 << LGC) column items (see fft::fft_stage).
template <int NF, int R, int NS, int LGC, typename In, typename Out>
__device__ __forceinline__ void stage(const float2 *__restrict__ tw, In in, Out out) {
    constexpr int NB = NF / R;
    constexpr int items = NB << LGC;
#pragma unroll
    for (int it0 = 0; it0 < items; it0 += kThreads) {
        const int it = it0 + (int)threadIdx.x;
        if (items % kThreads != 0 && it >= items) break;
        const int c = it & ((1 << LGC) - 1), j = it >> LGC;
        C2 v[R];
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
        for (int r = 0; r < R; ++r) out(j0 + fft::perm<R>(r) * NS, c, v[r]);
    }
}

// Length-2^LG transform over the rows of a tile of (1 << LGC) column items; xa: exchange tile (LG >= 5);
// tw: e^{+j 2 pi i / 2^LG}.  Contains one __syncthreads() between the stages, none before or after.
template <int LG, int LGC, typename Load, typename Store>
__device__ __forceinline__ void fft_rows(C2 *xa, const float2 *tw, Load load, Store store) {
    constexpr int NF = 1 << LG;
    constexpr int R1 = fft::Radix<LG>::R1, R2 = fft::Radix<LG>::R2;
    static_assert(fft::Radix<LG>::R3 == 1, "two stages at most");
    if constexpr (R2 == 1) {
        stage<NF, R1, 1, LGC>(tw, load, store);
    } else {
        stage<NF, R1, 1, LGC>(tw, load, [&](int row, int c, C2 v) {
            if (FAEDKV_IN_BOUNDS(kTagRecon2, row >= 0 && row < NF && c >= 0 && c < (1 << LGC))) xa[(row << LGC) + c] = v;
        });
        __syncthreads();
        stage<NF, R2, R1, LGC>(tw, [&](int row, int c) { return xa[(row << LGC) + c]; }, store);
    }
}

// lg of the transforms one tile takes: fill the exchange tile, never more than there are.
__host__ __device__ constexpr int lg_per_tile(int lg_rows, int lg_other) {
    int lg = kLgTile - lg_rows - kLgCP;
    if (lg < 0) lg = 0;
    if (lg > lg_other) lg = lg_other;
    return lg;
}

// Elements of the exchange tile the two passes need (0 when both are single-stage transforms).
__host__ __device__ constexpr int xa_elems(int lg1, int lg2) {
    const int a = fft::exchange_buffers(lg1) > 0 ? 1 << (lg1 + lg_per_tile(lg1, lg2) + kLgCP) : 0;
    const int b = fft::exchange_buffers(lg2) > 0 ? 1 << (lg2 + lg_per_tile(lg2, lg1) + kLgCP) : 0;
    return a > b ? a : b;
}

struct Args {
    const float *coef[2];          // planes of up to two tensors, [units][2][M][128] each
    void *out[2];                  // rows, [units][rows.unit_rows][128] each, storage type
    int n_tensors, units, M, H, Lrows;
    const int32_t *slot;           // [N + 1]: bin -> index in the plan, or -1
    const int32_t *t_len;
    const float2 *tabP, *tabI;
    C2 *Y;                         // ring of `ring` column blocks, [ring][N1][N2][16]
    int ring, lag;                 // 1 <= lag D <= number of column blocks; D < ring when there are more blocks than ring slots
    unsigned int *sync;            // [2 + 2 * n_cb]: ticket, exits, doneA[n_cb], doneB[n_cb]; zero between calls
    unsigned int *status;
    ReconRows rows;
};

__device__ __forceinline__ unsigned int ld_acquire(const unsigned int *p) {
    unsigned int v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
// Thread 0 waits until *counter >= need (bounded: gives up after ~1 s, or at once when another wait already
// gave up, and leaves a code in the status word); then the whole CTA passes.
__device__ __forceinline__ void wait_count(const unsigned int *counter, unsigned int need, unsigned int *status, uint32_t code) {
    if (threadIdx.x == 0 && ld_acquire(counter) < need) {
        unsigned long long t0 = 0;
        for (uint32_t i = 0;; ++i) {
            if (ld_acquire(counter) >= need) break;
            __nanosleep(64);
            if ((i & 63u) == 63u) {
                if (ld_acquire(status) != 0u) break;
                unsigned long long now;
                asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(now));
                if (t0 == 0) t0 = now;
                else if (now - t0 > kWaitLimitNs) { atomicExch(status, code); break; }
            }
        }
    }
    __syncthreads();
}

// Two floats from p (evict-first) when pred, else zeros, without a branch.
__device__ __forceinline__ float2 ld_if(const float *p, bool pred) {
    float2 v = make_float2(0.f, 0.f);
    asm("{\n\t.reg .pred q;\n\tsetp.ne.b32 q, %3, 0;\n\t@q ld.global.cs.v2.f32 {%0, %1}, [%2];\n\t}"
        : "+f"(v.x), "+f"(v.y) : "l"(p), "r"((int)pred));
    return v;
}

template <typename T> __device__ __forceinline__ void store_pair(T *p, float a, float b);
template <> __device__ __forceinline__ void store_pair<float>(float *p, float a, float b) {
    __stcs(reinterpret_cast<float2 *>(p), make_float2(a, b));
}
template <> __device__ __forceinline__ void store_pair<__nv_bfloat16>(__nv_bfloat16 *p, float a, float b) {
    const __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
    __stcs(reinterpret_cast<unsigned int *>(p), *reinterpret_cast<const unsigned int *>(&v));
}

// CTAs per SM the register allocation aims at: the 128-point instances (radix 8 then 16) fit 80 registers without
// spilling, i.e. six CTAs of four warps per SM (measured best of 2 ... 6 at 128 x 128 points); the others keep 128.
__host__ __device__ constexpr int min_ctas(int lg1, int lg2) { return (lg1 == 7 && lg2 >= 6) ? 6 : 4; }

// grid = persistent CTAs (any number >= 1); block = kThreads; dynamic smem = smem_bytes<LG1, LG2>().
template <int LG1, int LG2, typename TOut>
__global__ void __launch_bounds__(kThreads, min_ctas(LG1, LG2))
k_recon2(Args a) {
    constexpr int N1 = 1 << LG1, N2 = 1 << LG2, N = N1 * N2;
    constexpr int LGKT = lg_per_tile(LG1, LG2), LGMT = lg_per_tile(LG2, LG1);
    constexpr int nA = N2 >> LGKT, nB = N1 >> LGMT;        // tiles per column block
    constexpr uint32_t P = 2u * N;
    extern __shared__ __align__(16) unsigned char smem2[];
    C2 *xa = reinterpret_cast<C2 *>(smem2);
    constexpr int kXa = xa_elems(LG1, LG2);
    float2 *tw1 = reinterpret_cast<float2 *>(xa + kXa), *tw2 = tw1 + N1;
    __shared__ unsigned int s_ticket;
    for (int i = threadIdx.x; i < N1; i += kThreads) tw1[i] = fft::unit_phasor((uint32_t)i, (uint32_t)N1);
    for (int i = threadIdx.x; i < N2; i += kThreads) tw2[i] = fft::unit_phasor((uint32_t)i, (uint32_t)N2);
    const int n_cb = a.n_tensors * a.units * (kHeadDim / kCW);
    unsigned int *ticket_ctr = a.sync, *exit_ctr = a.sync + 1, *doneA = a.sync + 2, *doneB = doneA + n_cb;
    // ticket -> item: round i holds the nA pass-A tiles of block i (i < n_cb), then the nB pass-B tiles of block i - lag
    const int D = a.lag;
    const long long n_items = (long long)n_cb * (nA + nB);
    if (threadIdx.x == 0) s_ticket = atomicAdd(ticket_ctr, 1u);
    __syncthreads();
    const size_t plane = (size_t)a.M * kHeadDim;
    for (;;) {
        const long long t = (long long)s_ticket;
        __syncthreads();                                    // everyone has read the ticket
        if (t >= n_items) break;
        if (threadIdx.x == 0) s_ticket = atomicAdd(ticket_ctr, 1u);      // the next one, fetched while this one runs
        // decode: rounds [0, D) hold nA items each, rounds [D, n_cb) nA + nB, rounds [n_cb, n_cb + D) nB
        int round, idx;
        {
            const int Dc = D < n_cb ? D : n_cb;             // rounds that start with A only
            const long long headA = (long long)Dc * nA;
            if (t < headA) {
                round = (int)(t / nA); idx = (int)(t % nA);
            } else {
                const long long u = t - headA, mid = (long long)(n_cb - Dc) * (nA + nB);
                if (u < mid) { round = Dc + (int)(u / (nA + nB)); idx = (int)(u % (nA + nB)); }
                else { round = n_cb + (int)((u - mid) / nB); idx = nA + (int)((u - mid) % nB); }
            }
        }
        const bool isA = round < n_cb && idx < nA;
        const int cb = isA ? round : round - D;
        const int tile = isA ? idx : idx - nA;
        const int tensor = cb / (a.units * (kHeadDim / kCW)), cbu = cb % (a.units * (kHeadDim / kCW));
        const int unit = cbu / (kHeadDim / kCW), ch0 = (cbu % (kHeadDim / kCW)) * kCW;
        if (!FAEDKV_IN_BOUNDS(kTagRecon2, cb >= 0 && cb < n_cb && tile >= 0 && tile < (isA ? nA : nB) && tensor < a.n_tensors)) continue;
        C2 *Yb = a.Y + (size_t)(cb % a.ring) * N * kCP;
        if (isA) {
            // the ring slot is free once pass B of the block that had it is through
            if (cb >= a.ring) wait_count(doneB + (cb - a.ring), (unsigned int)nB, a.status, kErrWaitB);
            const int k2_0 = tile << LGKT;
            const float *cu = a.coef[tensor] + (size_t)unit * 2 * plane + ch0;
            // Branch-free on purpose: with the loads of absent bins predicated off instead of jumped over, the
            // gathers of all points of a butterfly are in flight together (behind branches every point waited
            // for its own round trip to memory in turn).
            auto load = [&](int k1, int c) {
                const int cp = c & (kCP - 1), k = N2 * k1 + k2_0 + (c >> kLgCP);
                const int sa = __ldg(a.slot + k), sb = __ldg(a.slot + (N - k));
                // Z[k] = (X[k] + conj X[N-k]) + j e^{+j 2 pi k / P} (X[k] - conj X[N-k]);  bins 0 and N are real
                if (!FAEDKV_IN_BOUNDS(kTagRecon2, sa < a.M && sb < a.M && k <= N)) return C2{make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
                const float *pa = cu + (size_t)(sa < 0 ? 0 : sa) * kHeadDim + 2 * cp;
                const float *pb = cu + (size_t)(sb < 0 ? 0 : sb) * kHeadDim + 2 * cp;
                const float2 xr = ld_if(pa, sa >= 0), mr = ld_if(pb, sb >= 0);
                const float2 xi = ld_if(pa + plane, sa >= 0 && k != 0), mi = ld_if(pb + plane, sb >= 0 && k != 0);
                const C2 s{padd(xr, mr), psub(xi, mi)}, d{psub(xr, mr), padd(xi, mi)};
                return cadd_j(s, cmul(d, __ldg(a.tabP + k)));
            };
            auto store = [&](int m1, int c, C2 v) {
                const int k2 = k2_0 + (c >> kLgCP);
                Yb[((size_t)m1 * N2 + k2) * kCP + (c & (kCP - 1))] = v;
            };
            fft_rows<LG1, LGKT + kLgCP>(xa, tw1, load, store);
            __syncthreads();                                // the whole tile has been stored (and xa is free)
            if (threadIdx.x == 0) { __threadfence(); atomicAdd(doneA + cb, 1u); }   // cumulative: orders the CTA's stores
        } else {
            wait_count(doneA + cb, (unsigned int)nA, a.status, kErrWaitA);
            const int m1_0 = tile << LGMT;
            const int gunit = unit;                          // t_len index = unit / H
            int tl = a.t_len[gunit / a.H] + a.rows.t_add;
            if (tl < 0) tl = 0;
            if (a.rows.t_quant > 1) tl = tl / a.rows.t_quant * a.rows.t_quant;
            const int live = tl < (int)P ? tl : (int)P;
            const int Lrows = a.Lrows;
            TOut *obase = static_cast<TOut *>(a.out[tensor]) + ((size_t)unit * a.rows.unit_rows + a.rows.row0) * kHeadDim + ch0;
            auto load = [&](int k2, int c) {
                // the inter-pass twiddle (with the 1/P of the inverse transform) is applied here: its load is issued
                // beside the load of the value, so pass A ends in plain stores
                const int m1 = m1_0 + (c >> kLgCP);
                const float2 w = __ldg(a.tabI + m1 * N2 + k2);
                const float4 v = __ldcg(reinterpret_cast<const float4 *>(Yb + ((size_t)m1 * N2 + k2) * kCP + (c & (kCP - 1))));
                return cmul(C2{make_float2(v.x, v.y), make_float2(v.z, v.w)}, w);
            };
            auto store = [&](int m2, int c, C2 v) {
                const int n = 2 * (m1_0 + (c >> kLgCP) + N1 * m2);
                if (!FAEDKV_IN_BOUNDS(kTagRecon2, n >= 0 && n + 1 < (int)P + 1 && a.rows.row0 + (n < Lrows ? n : 0) < a.rows.unit_rows)) return;
                TOut *o = obase + (size_t)n * kHeadDim + 2 * (c & (kCP - 1));
                if (n < Lrows) { const bool lv = n < live; store_pair<TOut>(o, lv ? v.re.x : 0.f, lv ? v.re.y : 0.f); }
                if (n + 1 < Lrows) { const bool lv = n + 1 < live; store_pair<TOut>(o + kHeadDim, lv ? v.im.x : 0.f, lv ? v.im.y : 0.f); }
            };
            fft_rows<LG2, LGMT + kLgCP>(xa, tw2, load, store);
            __syncthreads();                                // every read of the ring slot has returned
            // The tile's part of the ring is dead now (pass A rewrites it whole before anyone reads it again): drop
            // its lines from L2 instead of letting them be written back to DRAM when they are evicted.
            {
                const char *dead = reinterpret_cast<const char *>(Yb + (size_t)m1_0 * N2 * kCP);
                constexpr int lines = (int)(((size_t)1 << LGMT) * N2 * kCP * sizeof(C2) / 128);
                for (int i = threadIdx.x; i < lines; i += kThreads)
                    asm volatile("discard.global.L2 [%0], 128;" ::"l"(dead + (size_t)i * 128) : "memory");
            }
            __syncthreads();
            if (threadIdx.x == 0) { __threadfence(); atomicAdd(doneB + cb, 1u); }
        }
    }
    // the last CTA out leaves the counters at zero for the next call
    if (threadIdx.x == 0) {
        __threadfence();
        const unsigned int e = atomicAdd(exit_ctr, 1u);
        s_ticket = e == gridDim.x - 1 ? 1u : 0u;
    }
    __syncthreads();
    if (s_ticket) {
        __threadfence();
        for (int i = threadIdx.x; i < 2 + 2 * n_cb; i += kThreads) a.sync[i] = 0u;
    }
}

template <int LG1, int LG2> constexpr size_t smem_bytes() {
    return (size_t)xa_elems(LG1, LG2) * sizeof(C2) + ((size_t)(1 << LG1) + (size_t)(1 << LG2)) * sizeof(float2);
}

// tabP[k] = e^{+j 2 pi k / P}, k <= N;  tabI[m1 * N2 + k2] = e^{+j 2 pi k2 m1 / N} / P.
__global__ void k_recon2_tables(float2 *__restrict__ tabP, float2 *__restrict__ tabI, uint32_t P, int N2) {
    const uint32_t N = P / 2;
    const float inv_P = 1.0f / (float)P;
    for (uint32_t i = blockIdx.x * blockDim.x + threadIdx.x; i <= N; i += gridDim.x * blockDim.x) {
        tabP[i] = fft::unit_phasor(i, P);
        if (i < N) {
            const uint32_t m1 = i / (uint32_t)N2, k2 = i % (uint32_t)N2;
            const float2 w = fft::unit_phasor(m1 * k2, N);      // m1 * k2 < N
            tabI[i] = make_float2(w.x * inv_P, w.y * inv_P);
        }
    }
}

inline bool supported(int P) { return fft::supported(P) && P <= (2 << (2 * kMaxLg)); }

}  // namespace rfft2
}  // namespace faedkv
