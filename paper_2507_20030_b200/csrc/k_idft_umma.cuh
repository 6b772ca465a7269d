// Tensor-core pruned inverse DFT (Eq. 5 on the retained bins, Eq. 11):
//
//     out[n, c] = sum_k ( cos(w k n) * Bre[k, c]  -  sin(w k n) * Bim[k, c] )
//
// where B already carries the Hermitian weight and the 1/P (and, for attention scores, the softmax
// scale): B = w_k / P * C.  Used for
//   MODE 0  faedkv_reconstruct:   B = coefficient planes (converted to f16 by k_coef_to_half),
//                                 columns = K channels | V channels of one (batch, kv head);
//                                 epilogue writes bf16 K~ / V~ rows, zero beyond the live length.
//   MODE 1  decode attention (2): B = scaled query spectrum Qf (f16), columns = (sequence, query head);
//                                 epilogue writes float32 scores and per-32-row column maxima.
//
// The twiddle operand [positions x bins] is generated on chip, never stored: a generator thread owns
// one bin row of the stage and a run of consecutive positions, exactly like the prefill kernel, and
// the same shared-memory tile (bin rows of 128-byte position runs, 128-byte swizzle) is handed to the
// tensor core as an MN-major A operand (M = positions, K = bins).  Per-bin phasor tables
// e^{jwk i}, i = 1..8, come from a table built at plan time; the run's base phasor comes from the
// exactly reduced integer phase (k * n) mod P.  Operands are f16 (11-bit significand: the scores feed
// an exponential, so bf16 twiddles would not do), accumulation float32 in TMEM.
//
// CTA = NT * 128 positions x NCOLS columns; K loop over bins in stages of 32.
#pragma once
#include <cstdio>

#include "common.cuh"
#include "umma_common.cuh"

namespace faedkv {

namespace idft {

constexpr int kBinsPerStage = 32;
constexpr int kGenWarps = 8;
constexpr int kThreads = (2 + kGenWarps) * 32;
constexpr uint32_t kATileBytes = kBinsPerStage * 128 * 2;        // [32 bins x 128 positions] f16 = 8 KB
constexpr uint32_t kBBoxBytes = kBinsPerStage * 64 * 2;          // [32 bins x 64 columns] f16 = 4 KB
constexpr int kStages = 3;
constexpr uint32_t kErrTma = 0x21, kErrGen = 0x22, kErrMma = 0x23, kErrEpi = 0x24;

template <int NCOLS, int NT> struct Cfg {
    static constexpr uint32_t kABytes = NT * 2 * kATileBytes;                 // cos and -sin tiles of NT row tiles
    static constexpr uint32_t kBBytes = 2 * (NCOLS / 64) * kBBoxBytes;        // re and im planes
    static constexpr uint32_t kStageBytes = kABytes + kBBytes;
    static constexpr uint32_t kSmemBytes = kStages * kStageBytes + 1024 + 256 + NCOLS * 4;
};

struct Args {
    const int32_t *bins;      // [M]
    const float *tab;         // [M][16]: cos, sin of w k i for i = 1..8
    const int32_t *t_len;     // [batch]
    int M;
    uint32_t P;
    int Lrows;                // rows to produce
    // MODE 0
    void *outK, *outV;        // bf16 [units][Lrows][128]
    int H;                    // kv heads per sequence (t_len index = unit / H)
    // MODE 1
    float *S;                 // [P][Gtot]
    float *tile_max;          // [ceil(P/32)][Gtot]
    int Gtot, HQ, n_seq_cols; // columns = sequence * HQ + head; n_seq_cols = batch * HQ real columns
    unsigned int *status;
};

// max-reduce 32 per-lane values across the warp; afterwards lane l holds the maximum of value l.
__device__ __forceinline__ float warp_transpose_max32(float (&v)[32], int lane) {
#pragma unroll
    for (int s = 16; s >= 1; s >>= 1) {
        const bool up = (lane & s) != 0;
#pragma unroll
        for (int i = 0; i < s; ++i) {
            float send = up ? v[i] : v[i + s];
            float keep = up ? v[i + s] : v[i];
            v[i] = fmaxf(keep, __shfl_xor_sync(0xffffffffu, send, s));
        }
    }
    return v[0];
}

}  // namespace idft

// MODE 0: grid = (ceil(Lrows / (NT*128)), units);          maps: K planes, V planes, dims {128, M, units*2}
// MODE 1: grid = (ceil(Lrows / (NT*128)), Gtot / NCOLS);   map0: Qf16, dims {Gtot, M, 2}
template <int NCOLS, int NT, int MODE>
__global__ void __launch_bounds__(idft::kThreads, 1)
k_idft_umma(const __grid_constant__ CUtensorMap map0, const __grid_constant__ CUtensorMap map1, idft::Args a) {
    using namespace umma;
    using namespace idft;
    using C = Cfg<NCOLS, NT>;
    constexpr int S = kStages;
    constexpr int NBOX = NCOLS / 64;
    constexpr uint32_t kIdescInv = make_idesc(0u, 1u, 1u, (uint32_t)NCOLS);
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    auto a_tile = [&](int s, int nt, int which) { return smem_base + s * C::kStageBytes + (nt * 2 + which) * kATileBytes; };
    auto b_tile = [&](int s, int plane) { return smem_base + s * C::kStageBytes + C::kABytes + plane * NBOX * kBBoxBytes; };
    const uint32_t bar_base = smem_base + S * C::kStageBytes;
    auto full_b = [&](int s) { return bar_base + 8 * s; };
    auto full_a = [&](int s) { return bar_base + 8 * (S + s); };
    auto empty = [&](int s) { return bar_base + 8 * (2 * S + s); };
    const uint32_t accum_bar = bar_base + 8 * (3 * S);
    const uint32_t tmem_slot = bar_base + 8 * (3 * S + 1);
    uint8_t *gen_base = smem_raw + (bar_base - smem_u32(smem_raw));
    volatile uint32_t *tmem_slot_ptr = reinterpret_cast<volatile uint32_t *>(gen_base + 8 * (3 * S + 1));
    volatile uint32_t *abort_flag = tmem_slot_ptr + 1;
    int *live_col = reinterpret_cast<int *>(gen_base + 256);     // MODE 1: live length of each column's sequence

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n0 = blockIdx.x * (NT * 128);
    const int n_steps = (a.M + kBinsPerStage - 1) / kBinsPerStage;
    constexpr uint32_t kTmemCols = (NT * NCOLS <= 32) ? 32 : (NT * NCOLS <= 64) ? 64 : (NT * NCOLS <= 128) ? 128
                                   : (NT * NCOLS <= 256) ? 256 : 512;

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(full_b(s), 1);
            mbar_init(full_a(s), kGenWarps);
            mbar_init(empty(s), 1);
        }
        mbar_init(accum_bar, 1);
        *abort_flag = 0;
        fence_barrier_init();
    }
    if (MODE == 1) {
        for (int c = threadIdx.x; c < NCOLS; c += blockDim.x) {
            const int col = blockIdx.y * NCOLS + c;
            int live = 0;
            if (col < a.n_seq_cols) {
                const int t = a.t_len[col / a.HQ];
                live = t < (int)a.P ? t : (int)a.P;
            }
            live_col[c] = live;
        }
    }
    if (warp == 0) tmem_alloc(tmem_slot, kTmemCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot_ptr;

    if (warp == 0) {
        // ---------------------------------------------------------------- TMA producer (B operand)
        if (lane == 0) {
            int issued = 0;
            bool ok = true;
            for (int it = 0; it < n_steps && ok; ++it) {
                const int s = it % S;
                const uint32_t ph = (uint32_t)(it / S) & 1u;
                if (!mbar_wait(empty(s), ph ^ 1u)) { ok = false; break; }
                if (*abort_flag) break;
                mbar_expect_tx(full_b(s), C::kBBytes);
                const int kb0 = it * kBinsPerStage;
#pragma unroll
                for (int plane = 0; plane < 2; ++plane)
#pragma unroll
                    for (int j = 0; j < NBOX; ++j) {
                        const uint32_t dst = b_tile(s, plane) + j * kBBoxBytes;
                        if (MODE == 0) {
                            const CUtensorMap *m = (j / 2 == 0) ? &map0 : &map1;
                            tma_load_3d(dst, m, full_b(s), (j & 1) * 64, kb0, (int)blockIdx.y * 2 + plane);
                        } else {
                            tma_load_3d(dst, &map0, full_b(s), (int)blockIdx.y * NCOLS + j * 64, kb0, plane);
                        }
                    }
                issued = it + 1;
            }
            if (!ok) { atomicExch(a.status, kErrTma); *abort_flag = 1; }
            if (!ok || *abort_flag)
                for (int it = max(0, issued - S); it < issued; ++it) mbar_wait(full_b(it % S), (uint32_t)(it / S) & 1u);
        }
    } else if (warp == 1) {
        // ---------------------------------------------------------------- MMA issuer
        if (lane == 0) {
            bool ok = true;
            for (int it = 0; it < n_steps && ok; ++it) {
                const int s = it % S;
                const uint32_t ph = (uint32_t)(it / S) & 1u;
                if (!mbar_wait(full_a(s), ph) || !mbar_wait(full_b(s), ph)) { ok = false; break; }
                if (*abort_flag) break;
                tc_fence_after();
#pragma unroll
                for (int ks = 0; ks < kBinsPerStage / 16; ++ks) {
                    const uint64_t bre = desc_mnmajor_sw128(b_tile(s, 0) + ks * 2048u, kBBoxBytes);
                    const uint64_t bim = desc_mnmajor_sw128(b_tile(s, 1) + ks * 2048u, kBBoxBytes);
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt) {
                        const uint32_t acc = (it > 0 || ks > 0) ? 1u : 0u;
                        // A tile: two 64-position blocks 4096 bytes apart, 8-bin groups 1024 bytes apart
                        mma_bf16(tmem + nt * NCOLS, desc_mnmajor_sw128(a_tile(s, nt, 0) + ks * 2048u, 4096u), bre, kIdescInv, acc);
                        mma_bf16(tmem + nt * NCOLS, desc_mnmajor_sw128(a_tile(s, nt, 1) + ks * 2048u, 4096u), bim, kIdescInv, 1u);
                    }
                }
                mma_commit(empty(s));
            }
            if (ok && !*abort_flag) mma_commit(accum_bar);
            if (!ok) { atomicExch(a.status, kErrMma); *abort_flag = 1; }
        }
    } else {
        // ---------------------------------------------------------------- twiddle generators
        const int g = threadIdx.x - 64;              // 0..255
        const int kb = g & 31;                        // bin row of the stage
        const int seg = g >> 5;                       // 0..7: which run of 16*NT positions
        constexpr int RUN = 16 * NT;                  // positions per thread
        const uint32_t pos_start = (uint32_t)(n0 + seg * RUN);
        const uint32_t sw = (uint32_t)(kb & 7);
        const uint32_t row_off = (uint32_t)(kb >> 3) * 1024u + sw * 128u;
        bool ok = true;
        for (int it = 0; it < n_steps; ++it) {
            const int s = it % S;
            const uint32_t ph = (uint32_t)(it / S) & 1u;
            const int k = it * kBinsPerStage + kb;
            // per-bin tables and base phasor (independent of the pipeline slot: fetch before waiting)
            float gc[8], gs[8], f1c, f1s, bc, bs;
            {
                const bool valid = k < a.M;
                const uint32_t bin = valid ? (uint32_t)a.bins[k] : 0u;
                const float4 *t4 = reinterpret_cast<const float4 *>(a.tab + (size_t)(valid ? k : 0) * 16);
                const float4 t0 = __ldg(t4), t1 = __ldg(t4 + 1), t2 = __ldg(t4 + 2), t3 = __ldg(t4 + 3);
                gc[0] = 1.f; gs[0] = 0.f;
                gc[1] = t0.x; gs[1] = t0.y; gc[2] = t0.z; gs[2] = t0.w;
                gc[3] = t1.x; gs[3] = t1.y; gc[4] = t1.z; gs[4] = t1.w;
                gc[5] = t2.x; gs[5] = t2.y; gc[6] = t2.z; gs[6] = t2.w;
                gc[7] = t3.x; gs[7] = t3.y; f1c = t3.z; f1s = t3.w;
                twiddle(phase_mod(bin, pos_start % a.P, a.P), a.P, bc, bs);
            }
            if (!mbar_wait(empty(s), ph ^ 1u)) { ok = false; break; }
            if (*abort_flag) break;
#pragma unroll
            for (int cc = 0; cc < RUN / 8; ++cc) {
                float vc[8], vs[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    vc[i] = fmaf(bc, gc[i], -bs * gs[i]);        // cos(w k n)
                    vs[i] = -fmaf(bs, gc[i], bc * gs[i]);        // -sin(w k n)
                }
                const int r = seg * RUN + cc * 8;                // position offset inside the CTA's rows
                const int nt = r >> 7, rr = r & 127;
                const uint32_t off = (uint32_t)(rr >> 6) * 4096u + row_off + ((((uint32_t)(rr & 63) >> 3) ^ sw) << 4);
                st_shared_v4(a_tile(s, nt, 0) + off, pack_f16(vc[0], vc[1]), pack_f16(vc[2], vc[3]),
                             pack_f16(vc[4], vc[5]), pack_f16(vc[6], vc[7]));
                st_shared_v4(a_tile(s, nt, 1) + off, pack_f16(vs[0], vs[1]), pack_f16(vs[2], vs[3]),
                             pack_f16(vs[4], vs[5]), pack_f16(vs[6], vs[7]));
                const float nbc = fmaf(bc, f1c, -bs * f1s);
                bs = fmaf(bs, f1c, bc * f1s);
                bc = nbc;
            }
            fence_proxy_async();
            __syncwarp();
            if (lane == 0) mbar_arrive(full_a(s));
        }
        if (!ok) { atomicExch(a.status, kErrGen); *abort_flag = 1; }

        // ---------------------------------------------------------------- epilogue
        bool have = ok && !*abort_flag;
        if (have && !mbar_wait(accum_bar, 0u)) {
            have = false;
            atomicExch(a.status, kErrEpi);
            *abort_flag = 1;
        }
        have = __all_sync(0xffffffffu, have);
        if (have) {
            tc_fence_after();
            const int q = warp & 3;
            const int half = (warp - 2) >> 2;         // which half of the columns this warp writes
            constexpr int CB = NCOLS / 2 / 32;        // 32-column chunks per half
#pragma unroll 1
            for (int nt = 0; nt < NT; ++nt) {
                const int n = n0 + nt * 128 + q * 32 + lane;
#pragma unroll 1
                for (int cb = 0; cb < CB; ++cb) {
                    const int c0 = half * (NCOLS / 2) + cb * 32;          // first column of the chunk (CTA-local)
                    uint32_t v[32];
                    tmem_ld32(tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(nt * NCOLS + c0), v);
                    tmem_ld_wait();
                    if (MODE == 0) {
                        const int unit = blockIdx.y;
                        const int t = a.t_len[unit / a.H];
                        const int live = t < (int)a.P ? t : (int)a.P;
                        if (n < a.Lrows) {
                            const int tensor = (NCOLS == 256) ? (c0 >> 7) : 0;
                            const int ch = c0 & 127;
                            __nv_bfloat16 *dst = reinterpret_cast<__nv_bfloat16 *>(tensor == 0 ? a.outK : a.outV) +
                                                 ((size_t)unit * a.Lrows + n) * kHeadDim + ch;
                            const bool lv = n < live;
#pragma unroll
                            for (int j = 0; j < 4; ++j) {
                                uint4 o;
                                o.x = lv ? pack_bf16(__uint_as_float(v[8 * j + 0]), __uint_as_float(v[8 * j + 1])) : 0u;
                                o.y = lv ? pack_bf16(__uint_as_float(v[8 * j + 2]), __uint_as_float(v[8 * j + 3])) : 0u;
                                o.z = lv ? pack_bf16(__uint_as_float(v[8 * j + 4]), __uint_as_float(v[8 * j + 5])) : 0u;
                                o.w = lv ? pack_bf16(__uint_as_float(v[8 * j + 6]), __uint_as_float(v[8 * j + 7])) : 0u;
                                *reinterpret_cast<uint4 *>(dst + 8 * j) = o;
                            }
                        }
                    } else {
                        const int gcol = blockIdx.y * NCOLS + c0;
                        if (n < a.Lrows) {
                            float *dst = a.S + (size_t)n * a.Gtot + gcol;
#pragma unroll
                            for (int j = 0; j < 8; ++j)
                                *reinterpret_cast<float4 *>(dst + 4 * j) =
                                    make_float4(__uint_as_float(v[4 * j]), __uint_as_float(v[4 * j + 1]),
                                                __uint_as_float(v[4 * j + 2]), __uint_as_float(v[4 * j + 3]));
                        }
                        float m[32];
#pragma unroll
                        for (int j = 0; j < 32; ++j) m[j] = (n < live_col[c0 + j]) ? __uint_as_float(v[j]) : -INFINITY;
                        const float cm = warp_transpose_max32(m, lane);
                        const int row_group = (n0 + nt * 128 + q * 32) >> 5;
                        if ((n0 + nt * 128 + q * 32) < a.Lrows) a.tile_max[(size_t)row_group * a.Gtot + gcol + lane] = cm;
                    }
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        tc_fence_after();
        tmem_dealloc(tmem, kTmemCols);
    }
}

// ---- small helper kernels ---------------------------------------------------------------------------

// Per-bin phasor table built at plan time: tab[k][2(i-1)], tab[k][2(i-1)+1] = cos, sin of 2*pi*bins[k]*i/P, i = 1..8.
__global__ void k_bin_tables(const int32_t *__restrict__ bins, int M, uint32_t P, float *__restrict__ tab) {
    const int e = blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= M * 8) return;
    const int k = e >> 3, i = (e & 7) + 1;
    float c, s;
    twiddle(phase_mod((uint32_t)bins[k], (uint32_t)i % P, P), P, c, s);
    tab[(size_t)k * 16 + 2 * (i - 1)] = c;
    tab[(size_t)k * 16 + 2 * (i - 1) + 1] = s;
}

// Coefficient planes -> f16 planes scaled by w_k / P (the B operand of reconstruction).
// One thread per 8 channels; grid covers units * 2 planes * M bins * 16.
__global__ void k_coef_to_half(const float *__restrict__ coef, __half *__restrict__ out, const int32_t *__restrict__ bins,
                               int M, uint32_t P, size_t n_vec) {
    const size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= n_vec) return;
    const int k = (int)((e >> 4) % (size_t)M);
    const float w = hermitian_weight((uint32_t)bins[k], P) / (float)P;
    const float4 x = ld_stream(coef + e * 8), y = ld_stream(coef + e * 8 + 4);
    uint4 o;
    o.x = umma::pack_f16(x.x * w, x.y * w); o.y = umma::pack_f16(x.z * w, x.w * w);
    o.z = umma::pack_f16(y.x * w, y.y * w); o.w = umma::pack_f16(y.z * w, y.w * w);
    *reinterpret_cast<uint4 *>(out + e * 8) = o;
}

}  // namespace faedkv
