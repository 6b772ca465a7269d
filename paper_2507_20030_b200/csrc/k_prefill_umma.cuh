// Tensor-core prefill transform (Sec. 4.2.1; Eq. 4 on the retained bins) for bf16 K/V:
//
//     [ cos(w k n) ]            [ Yre ]
//     [ sin(w k n) ] (2M x T) x  X (T x N_c)  ->  [ -Yim ]      (float32 accumulate)
//
// The twiddle matrix is never in memory: it would be [2M x T] bf16 per layer
// (gigabytes).  Generator warps write each [128 bins x 64 tokens] cos / sin
// tile straight into shared memory in the 128-byte-swizzled K-major layout
// the tensor core reads, while TMA streams the matching [64 tokens x 256
// channels] K|V tile (tokens are the strided axis of K/V, so that operand is
// declared MN-major).  One elected thread issues tcgen05.mma; two float32
// accumulators (cos rows, sin rows) of 128 x 256 fill the 512 TMEM columns.
//
// One CTA = 128 bins x one (batch, kv head) x {K, V}: a generated twiddle tile
// is reused over 256 channels and a loaded K|V tile over 256 twiddle rows.
//
// Twiddle precision: every twiddle is the product of three float32 unit
// phasors whose angles come from exactly reduced integer phases
//     e^{-jwk(n0 + 8c + i)} = e^{-jwk n0} * (e^{-jwk 8})^c * e^{-jwk i},
// where the stage base e^{-jwk n0} is re-derived from the integer phase every 16th stage and rotated by
// e^{-jwk 64} in between (absolute error < 1e-6), then rounded to bf16 once (TERMS = 1, relative
// error of a coefficient ~1e-3) or split into a bf16 hi + lo pair (TERMS = 2,
// ~1e-5, twice the MMA work).  Accumulation is float32 in TMEM.
//
// Every mbarrier wait is bounded: on a time-out the kernel records a code in
// the status word, skips the rest of its work, waits (bounded) for its own
// bulk copies, frees its TMEM and returns.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <cstdio>

#include "common.cuh"
#include "umma_common.cuh"

namespace faedkv {

namespace prefill {

constexpr int kTileBinsU = 128;   // bins per CTA (rows of each accumulator)
constexpr int kTileTok = 64;      // tokens per pipeline stage (one 128-byte swizzle row of bf16)
constexpr int kNCols = 256;       // K channels | V channels
constexpr int kGenWarps = 8;      // twiddle generator / epilogue warps
constexpr int kThreads = (2 + kGenWarps) * 32;
constexpr uint32_t kATileBytes = kTileBinsU * kTileTok * 2;   // 16 KB
constexpr uint32_t kBTileBytes = kTileTok * kNCols * 2;       // 32 KB
constexpr uint32_t kBoxBytes = kTileTok * 64 * 2;             // one TMA box: 64 tokens x 64 channels

constexpr uint32_t kErrTimeoutTma = 0x11, kErrTimeoutGen = 0x12, kErrTimeoutMma = 0x13, kErrTimeoutEpi = 0x14;

template <int TERMS> struct Cfg {
    static constexpr int kStages = TERMS == 1 ? 3 : 2;
    static constexpr uint32_t kStageBytes = 2 * TERMS * kATileBytes + kBTileBytes;
    static constexpr uint32_t kSmemBytes = kStages * kStageBytes + 1024 /*alignment slack*/ + 256 /*barriers*/;
};

// kind::f16 instruction descriptor: D float32, A and B bf16, A K-major, B MN-major, M = 128, N = 256.
constexpr uint32_t kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | (0u << 15) | (1u << 16) |
                            ((uint32_t)(kNCols >> 3) << 17) | ((uint32_t)(kTileBinsU >> 4) << 24);

}  // namespace prefill

// grid = (ceil(M / 128), batch * H); block = 320; dynamic smem = Cfg<TERMS>::kSmemBytes
// wait_limit_ns: time limit of every mbarrier wait; withhold_step: 0, or a test hook (see the generator loop)
template <int TERMS>
__global__ void __launch_bounds__(prefill::kThreads, 1)
k_prefill_umma(const __grid_constant__ CUtensorMap mapK, const __grid_constant__ CUtensorMap mapV,
               const int32_t *__restrict__ bins, int M, uint32_t P, int T, uint32_t pos0,
               float *__restrict__ coefK, float *__restrict__ coefV, unsigned int *__restrict__ status,
               unsigned long long wait_limit_ns, int withhold_step) {
    using namespace umma;
    using namespace prefill;
    using C = Cfg<TERMS>;
    constexpr int S = C::kStages;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    // stage s: [cos hi][sin hi]([cos lo][sin lo])[B: 4 boxes of 64 tokens x 64 channels]
    auto a_tile = [&](int s, int which) { return smem_base + s * C::kStageBytes + which * kATileBytes; };
    auto b_tile = [&](int s) { return smem_base + s * C::kStageBytes + 2 * TERMS * kATileBytes; };
    const uint32_t bar_base = smem_base + S * C::kStageBytes;
    auto full_b = [&](int s) { return bar_base + 8 * s; };
    auto full_a = [&](int s) { return bar_base + 8 * (S + s); };
    auto empty = [&](int s) { return bar_base + 8 * (2 * S + s); };
    const uint32_t accum_bar = bar_base + 8 * (3 * S);
    const uint32_t tmem_slot = bar_base + 8 * (3 * S + 1);
    volatile uint32_t *tmem_slot_ptr =
        reinterpret_cast<volatile uint32_t *>(smem_raw + (tmem_slot - smem_u32(smem_raw)));
    volatile uint32_t *abort_flag = tmem_slot_ptr + 1;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int k0 = blockIdx.x * kTileBinsU;
    const int unit = blockIdx.y;
    const int n_steps = (T + kTileTok - 1) / kTileTok;

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
    if (warp == 0) tmem_alloc(tmem_slot, 512);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot_ptr;

    if (warp == 0) {
        // ---------------------------------------------------------------- TMA producer
        if (lane == 0) {
            int issued = 0;
            bool ok = true;
            for (int it = 0; it < n_steps && ok; ++it) {
                const int s = it % S;
                const uint32_t ph = (uint32_t)(it / S) & 1u;
                if (!mbar_wait(empty(s), ph ^ 1u, wait_limit_ns)) { ok = false; break; }
                if (*abort_flag) break;
                mbar_expect_tx(full_b(s), kBTileBytes);
                const int n0 = it * kTileTok;
                tma_load_3d(b_tile(s) + 0 * kBoxBytes, &mapK, full_b(s), 0, n0, unit);
                tma_load_3d(b_tile(s) + 1 * kBoxBytes, &mapK, full_b(s), 64, n0, unit);
                tma_load_3d(b_tile(s) + 2 * kBoxBytes, &mapV, full_b(s), 0, n0, unit);
                tma_load_3d(b_tile(s) + 3 * kBoxBytes, &mapV, full_b(s), 64, n0, unit);
                issued = it + 1;
            }
            if (!ok) { atomicExch(status, kErrTimeoutTma); *abort_flag = 1; }
            if (!ok || *abort_flag) {
                // wait (bounded) until the bulk copies still in flight have landed
                for (int it = max(0, issued - S); it < issued; ++it)
                    mbar_wait(full_b(it % S), (uint32_t)(it / S) & 1u, wait_limit_ns);
            }
        }
    } else if (warp == 1) {
        // ---------------------------------------------------------------- MMA issuer
        if (lane == 0) {
            bool ok = true;
            for (int it = 0; it < n_steps && ok; ++it) {
                const int s = it % S;
                const uint32_t ph = (uint32_t)(it / S) & 1u;
                if (!mbar_wait(full_a(s), ph, wait_limit_ns) || !mbar_wait(full_b(s), ph, wait_limit_ns)) { ok = false; break; }
                if (*abort_flag) break;
                tc_fence_after();
#pragma unroll
                for (int ks = 0; ks < kTileTok / 16; ++ks) {
                    const uint64_t bdesc = desc_mnmajor_sw128(b_tile(s) + ks * 2048u, kBoxBytes);
#pragma unroll
                    for (int term = 0; term < TERMS; ++term) {
                        const uint32_t acc = (it > 0 || ks > 0 || term > 0) ? 1u : 0u;
                        mma_bf16(tmem + 0, desc_kmajor_sw128(a_tile(s, 2 * term + 0) + ks * 32u), bdesc, kIdesc, acc);
                        mma_bf16(tmem + kNCols, desc_kmajor_sw128(a_tile(s, 2 * term + 1) + ks * 32u), bdesc, kIdesc, acc);
                    }
                }
                mma_commit(empty(s));   // frees this stage's A and B tiles when the MMAs have read them
            }
            if (ok && !*abort_flag) mma_commit(accum_bar);
            if (!ok) { atomicExch(status, kErrTimeoutMma); *abort_flag = 1; }
        }
    } else {
        // ---------------------------------------------------------------- twiddle generators
        const int g = threadIdx.x - 64;          // 0..255
        const int r = g & 127;                    // bin row of the tile
        const int hh = g >> 7;                    // which 32-token half of the stage
        uint32_t bin = (k0 + r < M) ? (uint32_t)bins[k0 + r] : 0u;
        if (!FAEDKV_IN_BOUNDS(kTagPrefillUmma, bin <= P / 2)) bin = 0u;
        float gc[8], gs[8];                       // e^{-jwk i}, i < 8: cos and sin of w k i
#pragma unroll
        for (int i = 0; i < 8; ++i) twiddle(phase_mod(bin, (uint32_t)i % P, P), P, gc[i], gs[i]);
        // the same as pairs (i, i + 1), for the packed float32x2 form of the rotation below
        float2 gc2[4], gs2[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) { gc2[j] = make_float2(gc[2 * j], gc[2 * j + 1]); gs2[j] = make_float2(gs[2 * j], gs[2 * j + 1]); }
        float f1c, f1s;                           // cos, sin of w k 8
        twiddle(phase_mod(bin, 8u % P, P), P, f1c, f1s);
        uint32_t ph_idx = phase_mod(bin, (pos0 + (uint32_t)hh * 32u) % P, P);
        const uint32_t step_idx = phase_mod(bin, (uint32_t)kTileTok % P, P);
        const uint32_t row_off = (uint32_t)r * 128u;
        const uint32_t sw = (uint32_t)(r & 7);
        float stc, sts;                           // cos, sin of w k 64: one stage further
        twiddle(step_idx, P, stc, sts);
        float base_c = 1.f, base_s = 0.f;         // phasor of the first token this thread writes in the current stage
        bool ok = true;
        for (int it = 0; it < n_steps; ++it) {
            const int s = it % S;
            const uint32_t ph = (uint32_t)(it / S) & 1u;
            if (!mbar_wait(empty(s), ph ^ 1u, wait_limit_ns)) { ok = false; break; }
            if (*abort_flag) break;
            // every 16th stage the base phasor comes from the exactly reduced integer phase; in between it is rotated
            // one stage forward (15 float32 rotations at most: error < 1e-6, nothing accumulates beyond that)
            if ((it & 15) == 0) {
                twiddle(ph_idx, P, base_c, base_s);
            } else {
                const float nc = fmaf(base_c, stc, -base_s * sts);
                base_s = fmaf(base_s, stc, base_c * sts);
                base_c = nc;
            }
            float bc = base_c, bs = base_s;
            ph_idx = add_mod(ph_idx, step_idx, P);
#pragma unroll
            for (int cc = 0; cc < 4; ++cc) {
                // cos(a + b) = bc gc - bs gs, sin(a + b) = bs gc + bc gs for two tokens per instruction: the packed
                // FMA rounds each lane exactly like fmaf(bc, gc, -bs * gs), at half the instructions (the generator
                // warps' arithmetic is the part of this kernel's power that is not the tensor core's)
                float vc[8], vs[8];
                const float2 bc2 = make_float2(bc, bc), bs2 = make_float2(bs, bs), nbs2 = make_float2(-bs, -bs);
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const float2 c2 = __ffma2_rn(bc2, gc2[j], __fmul2_rn(nbs2, gs2[j]));
                    const float2 s2 = __ffma2_rn(bs2, gc2[j], __fmul2_rn(bc2, gs2[j]));
                    vc[2 * j] = c2.x; vc[2 * j + 1] = c2.y;
                    vs[2 * j] = s2.x; vs[2 * j + 1] = s2.y;
                }
                const uint32_t chunk = (((uint32_t)(hh * 4 + cc)) ^ sw) << 4;
                uint4 pc, psn;
                pc.x = pack_bf16(vc[0], vc[1]); pc.y = pack_bf16(vc[2], vc[3]);
                pc.z = pack_bf16(vc[4], vc[5]); pc.w = pack_bf16(vc[6], vc[7]);
                psn.x = pack_bf16(vs[0], vs[1]); psn.y = pack_bf16(vs[2], vs[3]);
                psn.z = pack_bf16(vs[4], vs[5]); psn.w = pack_bf16(vs[6], vs[7]);
                asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(a_tile(s, 0) + row_off + chunk),
                             "r"(pc.x), "r"(pc.y), "r"(pc.z), "r"(pc.w) : "memory");
                asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(a_tile(s, 1) + row_off + chunk),
                             "r"(psn.x), "r"(psn.y), "r"(psn.z), "r"(psn.w) : "memory");
                if (TERMS == 2) {
                    float lc[8], ls[8];
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        lc[i] = vc[i] - bf16_round(vc[i]);
                        ls[i] = vs[i] - bf16_round(vs[i]);
                    }
                    pc.x = pack_bf16(lc[0], lc[1]); pc.y = pack_bf16(lc[2], lc[3]);
                    pc.z = pack_bf16(lc[4], lc[5]); pc.w = pack_bf16(lc[6], lc[7]);
                    psn.x = pack_bf16(ls[0], ls[1]); psn.y = pack_bf16(ls[2], ls[3]);
                    psn.z = pack_bf16(ls[4], ls[5]); psn.w = pack_bf16(ls[6], ls[7]);
                    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(a_tile(s, 2) + row_off + chunk),
                                 "r"(pc.x), "r"(pc.y), "r"(pc.z), "r"(pc.w) : "memory");
                    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(a_tile(s, 3) + row_off + chunk),
                                 "r"(psn.x), "r"(psn.y), "r"(psn.z), "r"(psn.w) : "memory");
                }
                // advance the base phasor by 8 tokens
                const float nbc = fmaf(bc, f1c, -bs * f1s);
                bs = fmaf(bs, f1c, bc * f1s);
                bc = nbc;
            }
            fence_proxy_async();      // make the generic-proxy stores visible to the tensor core
            __syncwarp();
            // test hook (withhold_step > 0): the first generator warp skips its arrive at that step, so the tile never
            // becomes "full" and every role's bounded wait runs out: the give-up path, exercised without a fault
            if (lane == 0 && !(withhold_step > 0 && it == withhold_step - 1 && warp == 2)) mbar_arrive(full_a(s));
        }
        if (!ok) { atomicExch(status, kErrTimeoutGen); *abort_flag = 1; }

        // ---------------------------------------------------------------- epilogue (same 8 warps)
        bool have = ok && !*abort_flag;
        if (have && !mbar_wait(accum_bar, 0u, wait_limit_ns)) {
            have = false;
            atomicExch(status, kErrTimeoutEpi);
            *abort_flag = 1;
        }
        have = __all_sync(0xffffffffu, have);     // tcgen05.ld is warp-collective
        if (have) {
            tc_fence_after();
            const int q = warp & 3;                   // TMEM lane quarter this warp may read
            const int tensor = (warp - 2) >> 2;       // 0: K columns, 1: V columns
            const int row = q * 32 + lane;
            const int k = k0 + row;
            float *coef = tensor == 0 ? coefK : coefV;
            const size_t plane = (size_t)M * kHeadDim;
            float *dst_re = coef + (size_t)unit * 2 * plane + (size_t)k * kHeadDim;
            float *dst_im = dst_re + plane;
#pragma unroll 1
            for (int part = 0; part < 2; ++part) {    // 0: cos accumulator -> Re, 1: sin accumulator -> -Im
#pragma unroll 1
                for (int cb = 0; cb < 4; ++cb) {
                    uint32_t v[32];
                    const uint32_t taddr = tmem + ((uint32_t)(q * 32) << 16) +
                                           (uint32_t)(part * kNCols + tensor * 128 + cb * 32);
                    tmem_ld32(taddr, v);
                    tmem_ld_wait();
                    if (k < M) {
                        float *dst = (part == 0 ? dst_re : dst_im) + cb * 32;
                        const float sgn = part == 0 ? 1.0f : -1.0f;
#pragma unroll
                        for (int j = 0; j < 8; ++j) {
                            float4 o = make_float4(sgn * __uint_as_float(v[4 * j]), sgn * __uint_as_float(v[4 * j + 1]),
                                                   sgn * __uint_as_float(v[4 * j + 2]), sgn * __uint_as_float(v[4 * j + 3]));
                            *reinterpret_cast<float4 *>(dst + 4 * j) = o;
                        }
                    }
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        tc_fence_after();
        tmem_dealloc(tmem, 512);
    }
}

// ---- host side -----------------------------------------------------------------------------------
typedef CUresult (*PFN_encodeTiled)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                    const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                    CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                    CUtensorMapFloatOOBfill);

struct UmmaPrefillState {
    PFN_encodeTiled encode = nullptr;
    bool attr_set[3] = {false, false, false};
    unsigned long long wait_limit_ns = umma::kWaitLimitNs;   // test hooks: see faedkv_test_hooks()
    int withhold_step = 0;
};

inline bool umma_prefill_available() { return true; }

// K/V [units][T][128] bf16 as a 3-D tensor map; box = 64 channels x 64 tokens x 1 unit, 128-byte swizzle.
// Rows past T read as zero, so a ragged last stage adds nothing.
// Resolve cuTensorMapEncodeTiled through the runtime (the library does not link libcuda).
inline int umma_resolve_encode(UmmaPrefillState &st, char *msg, size_t n) {
    if (st.encode != nullptr) return 0;
    void *fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
    if (e != cudaSuccess || fn == nullptr || qres != cudaDriverEntryPointSuccess) {
        snprintf(msg, n, "cuTensorMapEncodeTiled is not available from the driver");
        return -6;
    }
    st.encode = reinterpret_cast<PFN_encodeTiled>(fn);
    return 0;
}

// T rows of each unit are transformed; consecutive units are T_stride rows apart (T_stride >= T: the
// transformed rows may be a window of a longer tensor).
inline int umma_make_map(UmmaPrefillState &st, CUtensorMap *map, const void *base, int units, int T, int T_stride, char *msg,
                         size_t n) {
    if (int r = umma_resolve_encode(st, msg, n)) return r;
    cuuint64_t dims[3] = {(cuuint64_t)kHeadDim, (cuuint64_t)T, (cuuint64_t)units};
    cuuint64_t strides[2] = {(cuuint64_t)kHeadDim * 2, (cuuint64_t)T_stride * kHeadDim * 2};
    cuuint32_t box[3] = {64, (cuuint32_t)prefill::kTileTok, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = st.encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(base), dims, strides, box, estr,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        snprintf(msg, n, "cuTensorMapEncodeTiled failed with code %d", (int)r);
        return -6;
    }
    return 0;
}

template <int TERMS>
inline int umma_launch_t(UmmaPrefillState &st, const CUtensorMap &mK, const CUtensorMap &mV, int units, int T,
                         const int32_t *d_bins, int M, int P, float *coefK, float *coefV, unsigned int *status,
                         cudaStream_t stream, char *msg, size_t n) {
    using C = prefill::Cfg<TERMS>;
    if (!st.attr_set[TERMS]) {
        cudaError_t e = cudaFuncSetAttribute(k_prefill_umma<TERMS>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)C::kSmemBytes);
        if (e != cudaSuccess) {
            snprintf(msg, n, "cannot opt in to %u bytes of shared memory: %s", C::kSmemBytes, cudaGetErrorString(e));
            return -6;
        }
        st.attr_set[TERMS] = true;
    }
    dim3 grid((M + prefill::kTileBinsU - 1) / prefill::kTileBinsU, units);
    k_prefill_umma<TERMS><<<grid, prefill::kThreads, C::kSmemBytes, stream>>>(mK, mV, d_bins, M, (uint32_t)P, T, 0u, coefK, coefV, status,
                                                                              st.wait_limit_ns, st.withhold_step);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) {
        snprintf(msg, n, "launch of k_prefill_umma failed: %s", cudaGetErrorString(e));
        return -6;
    }
    return 0;
}

inline int umma_prefill_launch(UmmaPrefillState &st, const void *K, const void *V, int batch, int H, int T, int T_stride,
                               const int32_t *d_bins, int M, int P, int terms, float *coefK, float *coefV,
                               unsigned int *status, cudaStream_t stream, char *msg, size_t n) {
    CUtensorMap mK, mV;
    const int units = batch * H;
    if (int r = umma_make_map(st, &mK, K, units, T, T_stride, msg, n)) return r;
    if (int r = umma_make_map(st, &mV, V, units, T, T_stride, msg, n)) return r;
    if (terms == 2) return umma_launch_t<2>(st, mK, mV, units, T, d_bins, M, P, coefK, coefV, status, stream, msg, n);
    return umma_launch_t<1>(st, mK, mV, units, T, d_bins, M, P, coefK, coefV, status, stream, msg, n);
}

}  // namespace faedkv
