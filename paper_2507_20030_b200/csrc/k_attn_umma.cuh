// Tensor-core pieces of frequency-domain decode attention (steps numbered as in k_attn.cuh), for bf16
// tensors.  Columns g = sequence * HQ + query head, padded to Gtot (a multiple of 64).
//
//   (1) k_attn_qf16        Qf16[plane][k][g] = f16( w_k * scale / P * sum_c q[g,c] C_K[k,c] )
//   (2) k_idft_umma<MODE 1> scores S[n][g] (float32) + per-32-row column maxima        (k_idft_umma.cuh)
//   (3) k_colmax_par, k_softmax_half: P16[n][g] = f16(exp(S - max)), zero beyond the live length;
//       per-row-block column sums of the ROUNDED values (the normaliser the tensor core actually sees)
//   (4) k_pspec_umma       Pf[split][plane][k][g] = sum_{n in split} P16[n][g] * (cos, sin)(w k n)
//   (5) k_attn_out2        out[g,c] = 1 / (P * colsum[g]) * sum_k w_k Re(C_V[k,c] * Pf[g,k])
#pragma once
#include "common.cuh"
#include "k_attn.cuh"
#include "umma_common.cuh"

namespace faedkv {

// ---- (1) ------------------------------------------------------------------------------------------
// grid = (ceil(M / (8 * KB)), batch * H); block = 256
template <typename TQ, int GQ>
__global__ void __launch_bounds__(kAttnWarps * 32)
k_attn_qf16(const TQ *__restrict__ q, const float *__restrict__ coefK, const int32_t *__restrict__ bins,
            __half *__restrict__ Qf16, int M, int H, int HQ, int Gtot, uint32_t P, float scale_over_P) {
    constexpr int KB = attn_bins_per_warp(GQ);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int bh = blockIdx.y, b = bh / H, h = bh % H;
    const int k0 = (blockIdx.x * kAttnWarps + warp) * KB;
    if (k0 >= M) return;
    float4 qv[GQ];
#pragma unroll
    for (int g = 0; g < GQ; ++g) qv[g] = load4(q + ((size_t)b * HQ + h * GQ + g) * kHeadDim + lane * 4);
    const size_t plane = (size_t)M * kHeadDim;
    const float *base = coefK + (size_t)bh * 2 * plane;
    float4 row[KB][2];
#pragma unroll
    for (int kk = 0; kk < KB; ++kk)
#pragma unroll
        for (int pl = 0; pl < 2; ++pl) {
            row[kk][pl] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (k0 + kk < M) row[kk][pl] = ld_stream(base + pl * plane + (size_t)(k0 + kk) * kHeadDim + lane * 4);
        }
    float v[32];
#pragma unroll
    for (int i = KB * 2 * GQ; i < 32; ++i) v[i] = 0.f;
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
    if (kk < KB && k0 + kk < M) {
        const float w = hermitian_weight((uint32_t)bins[k0 + kk], P) * scale_over_P;
        Qf16[((size_t)pl * M + (k0 + kk)) * Gtot + b * HQ + h * GQ + g] = __float2half_rn(tot * w);
    }
}

// ---- (3) ------------------------------------------------------------------------------------------
// Column maxima over the 32-row groups; grid = Gtot / 32, block = 256 (8 warps stride the groups).
__global__ void __launch_bounds__(256)
k_colmax_par(const float *__restrict__ tile_max, int n_groups, int Gtot, float *__restrict__ colmax) {
    __shared__ float red[8][32];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int col = blockIdx.x * 32 + lane;
    float m = -INFINITY;
    for (int t = warp; t < n_groups; t += 8) m = fmaxf(m, tile_max[(size_t)t * Gtot + col]);
    red[warp][lane] = m;
    __syncthreads();
    if (warp == 0) {
#pragma unroll
        for (int w = 1; w < 8; ++w) m = fmaxf(m, red[w][lane]);
        colmax[col] = m;
    }
}

constexpr int kSoftmaxRows = 128;   // rows per block of k_softmax_half

// P16[n][g] = f16(exp(S[n][g] - colmax[g])) for n < live(g), else 0; block partial column sums.
// grid = (ceil(P / 128), Gtot / 64); block = 256: thread = (column pair, row lane).
__global__ void __launch_bounds__(256)
k_softmax_half(const float *__restrict__ S, const float *__restrict__ colmax, const int32_t *__restrict__ t_len,
               __half *__restrict__ P16, float *__restrict__ psum, int P, int Gtot, int HQ, int n_seq_cols) {
    __shared__ float red[8][64];
    const int cp = threadIdx.x & 31, rl = threadIdx.x >> 5;       // column pair 0..31, row lane 0..7
    const int col = blockIdx.y * 64 + cp * 2;
    const int r0 = blockIdx.x * kSoftmaxRows;
    int live0 = 0, live1 = 0;
    if (col < n_seq_cols) { int t = t_len[col / HQ]; live0 = t < P ? t : P; }
    if (col + 1 < n_seq_cols) { int t = t_len[(col + 1) / HQ]; live1 = t < P ? t : P; }
    const float m0 = colmax[col], m1 = colmax[col + 1];
    float s0 = 0.f, s1 = 0.f;
    for (int r = r0 + rl; r < min(P, r0 + kSoftmaxRows); r += 8) {
        const float2 sv = *reinterpret_cast<const float2 *>(S + (size_t)r * Gtot + col);
        const float e0 = r < live0 ? __expf(sv.x - m0) : 0.f;
        const float e1 = r < live1 ? __expf(sv.y - m1) : 0.f;
        const __half2 h = __floats2half2_rn(e0, e1);
        *reinterpret_cast<__half2 *>(P16 + (size_t)r * Gtot + col) = h;
        const float2 back = __half22float2(h);
        s0 += back.x;
        s1 += back.y;
    }
    red[rl][cp * 2] = s0;
    red[rl][cp * 2 + 1] = s1;
    __syncthreads();
    if (threadIdx.x < 64) {
        float s = 0.f;
#pragma unroll
        for (int w = 0; w < 8; ++w) s += red[w][threadIdx.x];
        psum[(size_t)blockIdx.x * Gtot + blockIdx.y * 64 + threadIdx.x] = s;
    }
}

// Column sums in a fixed order: colsum[g] = sum_blocks psum[block][g].  grid = Gtot / 32, block = 32.
__global__ void k_colsum(const float *__restrict__ psum, int n_blocks, int Gtot, float *__restrict__ colsum) {
    const int col = blockIdx.x * 32 + threadIdx.x;
    float s = 0.f;
    for (int b = 0; b < n_blocks; ++b) s += psum[(size_t)b * Gtot + col];
    colsum[col] = s;
}

// ---- (4) ------------------------------------------------------------------------------------------
namespace pspec {
constexpr int kTileBinsU = 128, kTileTok = 64, kGenWarps = 8, kThreads = (2 + kGenWarps) * 32, kStages = 3;
constexpr uint32_t kATileBytes = kTileBinsU * kTileTok * 2;   // 16 KB
constexpr uint32_t kBoxBytes = kTileTok * 64 * 2;             // 64 rows x 64 columns f16 = 8 KB
constexpr uint32_t kErrTma = 0x31, kErrGen = 0x32, kErrMma = 0x33, kErrEpi = 0x34;
template <int NCOLS> struct Cfg {
    static constexpr uint32_t kBBytes = (NCOLS / 64) * kBoxBytes;
    static constexpr uint32_t kStageBytes = 2 * kATileBytes + kBBytes;
    static constexpr uint32_t kSmemBytes = kStages * kStageBytes + 1024 + 256;
};
}  // namespace pspec

// Forward transform of the probabilities on tensor cores: the prefill kernel's scheme (generated
// K-major twiddle tiles x TMA-loaded MN-major data tiles) with f16 operands, +sin, and the position
// range split over blockIdx.z so that few columns still fill the GPU; partial spectra are summed by
// the consumer in a fixed order.
// grid = (ceil(M / 128), Gtot / NCOLS, splits); map: P16 as {Gtot, P}, box {64, 64}
template <int NCOLS>
__global__ void __launch_bounds__(pspec::kThreads, 1)
k_pspec_umma(const __grid_constant__ CUtensorMap mapP, const int32_t *__restrict__ bins, int M, uint32_t P,
             int rows_per_split, int Gtot, float *__restrict__ Pf, unsigned int *__restrict__ status) {
    using namespace umma;
    using namespace pspec;
    using C = Cfg<NCOLS>;
    constexpr int S = kStages, NBOX = NCOLS / 64;
    constexpr uint32_t kIdescF = make_idesc(0u, 0u, 1u, (uint32_t)NCOLS);
    constexpr uint32_t kTmemCols = (2 * NCOLS <= 128) ? 128 : (2 * NCOLS <= 256) ? 256 : 512;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    auto a_tile = [&](int s, int which) { return smem_base + s * C::kStageBytes + which * kATileBytes; };
    auto b_tile = [&](int s) { return smem_base + s * C::kStageBytes + 2 * kATileBytes; };
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
    const int row_begin = blockIdx.z * rows_per_split;
    const int row_end = min((int)P, row_begin + rows_per_split);
    const int n_steps = max(0, (row_end - row_begin + kTileTok - 1) / kTileTok);

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
    if (warp == 0) tmem_alloc(tmem_slot, kTmemCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot_ptr;

    if (warp == 0) {
        if (lane == 0) {
            int issued = 0;
            bool ok = true;
            for (int it = 0; it < n_steps && ok; ++it) {
                const int s = it % S;
                const uint32_t ph = (uint32_t)(it / S) & 1u;
                if (!mbar_wait(empty(s), ph ^ 1u)) { ok = false; break; }
                if (*abort_flag) break;
                mbar_expect_tx(full_b(s), C::kBBytes);
#pragma unroll
                for (int j = 0; j < NBOX; ++j)
                    tma_load_3d(b_tile(s) + j * kBoxBytes, &mapP, full_b(s), (int)blockIdx.y * NCOLS + j * 64,
                                row_begin + it * kTileTok, 0);
                issued = it + 1;
            }
            if (!ok) { atomicExch(status, kErrTma); *abort_flag = 1; }
            if (!ok || *abort_flag)
                for (int it = max(0, issued - S); it < issued; ++it) mbar_wait(full_b(it % S), (uint32_t)(it / S) & 1u);
        }
    } else if (warp == 1) {
        if (lane == 0) {
            bool ok = true;
            for (int it = 0; it < n_steps && ok; ++it) {
                const int s = it % S;
                const uint32_t ph = (uint32_t)(it / S) & 1u;
                if (!mbar_wait(full_a(s), ph) || !mbar_wait(full_b(s), ph)) { ok = false; break; }
                if (*abort_flag) break;
                tc_fence_after();
#pragma unroll
                for (int ks = 0; ks < kTileTok / 16; ++ks) {
                    const uint64_t bdesc = desc_mnmajor_sw128(b_tile(s) + ks * 2048u, kBoxBytes);
                    const uint32_t acc = (it > 0 || ks > 0) ? 1u : 0u;
                    mma_bf16(tmem + 0, desc_kmajor_sw128(a_tile(s, 0) + ks * 32u), bdesc, kIdescF, acc);
                    mma_bf16(tmem + NCOLS, desc_kmajor_sw128(a_tile(s, 1) + ks * 32u), bdesc, kIdescF, acc);
                }
                mma_commit(empty(s));
            }
            if (ok && !*abort_flag) mma_commit(accum_bar);
            if (!ok) { atomicExch(status, kErrMma); *abort_flag = 1; }
        }
    } else {
        const int g = threadIdx.x - 64;
        const int r = g & 127, hh = g >> 7;
        const uint32_t bin = (k0 + r < M) ? (uint32_t)bins[k0 + r] : 0u;
        float gc[8], gs[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) twiddle(phase_mod(bin, (uint32_t)i % P, P), P, gc[i], gs[i]);
        float f1c, f1s;
        twiddle(phase_mod(bin, 8u % P, P), P, f1c, f1s);
        uint32_t ph_idx = phase_mod(bin, ((uint32_t)row_begin + (uint32_t)hh * 32u) % P, P);
        const uint32_t step_idx = phase_mod(bin, (uint32_t)kTileTok % P, P);
        const uint32_t row_off = (uint32_t)r * 128u, sw = (uint32_t)(r & 7);
        bool ok = true;
        for (int it = 0; it < n_steps; ++it) {
            const int s = it % S;
            const uint32_t ph = (uint32_t)(it / S) & 1u;
            if (!mbar_wait(empty(s), ph ^ 1u)) { ok = false; break; }
            if (*abort_flag) break;
            float bc, bs;
            twiddle(ph_idx, P, bc, bs);
            ph_idx = add_mod(ph_idx, step_idx, P);
#pragma unroll
            for (int cc = 0; cc < 4; ++cc) {
                float vc[8], vs[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    vc[i] = fmaf(bc, gc[i], -bs * gs[i]);
                    vs[i] = fmaf(bs, gc[i], bc * gs[i]);
                }
                const uint32_t chunk = (((uint32_t)(hh * 4 + cc)) ^ sw) << 4;
                st_shared_v4(a_tile(s, 0) + row_off + chunk, pack_f16(vc[0], vc[1]), pack_f16(vc[2], vc[3]),
                             pack_f16(vc[4], vc[5]), pack_f16(vc[6], vc[7]));
                st_shared_v4(a_tile(s, 1) + row_off + chunk, pack_f16(vs[0], vs[1]), pack_f16(vs[2], vs[3]),
                             pack_f16(vs[4], vs[5]), pack_f16(vs[6], vs[7]));
                const float nbc = fmaf(bc, f1c, -bs * f1s);
                bs = fmaf(bs, f1c, bc * f1s);
                bc = nbc;
            }
            fence_proxy_async();
            __syncwarp();
            if (lane == 0) mbar_arrive(full_a(s));
        }
        if (!ok) { atomicExch(status, kErrGen); *abort_flag = 1; }

        bool have = ok && !*abort_flag && n_steps > 0;
        if (have && !mbar_wait(accum_bar, 0u)) {
            have = false;
            atomicExch(status, kErrEpi);
            *abort_flag = 1;
        }
        have = __all_sync(0xffffffffu, have);
        const int q = warp & 3, half = (warp - 2) >> 2;
        const int k = k0 + q * 32 + lane;
        constexpr int CB = NCOLS / 2 / 32;            // NCOLS >= 64
        float *dst_re = Pf + (((size_t)blockIdx.z * 2 + 0) * M + k) * Gtot + blockIdx.y * NCOLS + half * (NCOLS / 2);
        float *dst_im = dst_re + (size_t)M * Gtot;
#pragma unroll 1
        for (int part = 0; part < 2; ++part)
#pragma unroll 1
            for (int cb = 0; cb < CB; ++cb) {
                uint32_t v[32];
                if (have) {
                    tmem_ld32(tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(part * NCOLS + half * (NCOLS / 2) + cb * 32), v);
                    tmem_ld_wait();
                } else {
#pragma unroll
                    for (int j = 0; j < 32; ++j) v[j] = 0u;     // an empty split contributes zero
                }
                if (k < M && (have || n_steps == 0)) {
                    float *dst = (part == 0 ? dst_re : dst_im) + cb * 32;
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        *reinterpret_cast<float4 *>(dst + 4 * j) =
                            make_float4(__uint_as_float(v[4 * j]), __uint_as_float(v[4 * j + 1]),
                                        __uint_as_float(v[4 * j + 2]), __uint_as_float(v[4 * j + 3]));
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

// ---- (5) ------------------------------------------------------------------------------------------
// grid = (slices, batch * H); block = 256.  Pf is [splits][2][M][Gtot]; the splits are summed here.
template <int GQ>
__global__ void __launch_bounds__(kAttnWarps * 32)
k_attn_out2(const float *__restrict__ coefV, const float *__restrict__ Pf, const int32_t *__restrict__ bins,
            float *__restrict__ partial, int M, int H, int HQ, int Gtot, int splits, uint32_t P, int bins_per_slice) {
    __shared__ __align__(16) float red[kAttnWarps][GQ][kHeadDim];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int bh = blockIdx.y, b = bh / H, h = bh % H;
    const int kbeg = blockIdx.x * bins_per_slice;
    const int kend = min(M, kbeg + bins_per_slice);
    const size_t plane = (size_t)M * kHeadDim;
    const float *base = coefV + (size_t)bh * 2 * plane;
    const int gcol = b * HQ + h * GQ;
    const size_t split_stride = (size_t)2 * M * Gtot, im_off = (size_t)M * Gtot;
    float4 acc[GQ];
#pragma unroll
    for (int g = 0; g < GQ; ++g) acc[g] = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int k = kbeg + warp; k < kend; k += kAttnWarps) {
        const float4 re = ld_stream(base + (size_t)k * kHeadDim + lane * 4);
        const float4 im = ld_stream(base + plane + (size_t)k * kHeadDim + lane * 4);
        const float w = hermitian_weight((uint32_t)bins[k], P);
#pragma unroll
        for (int g = 0; g < GQ; ++g) {
            float pr = 0.f, pi = 0.f;
            const float *p = Pf + (size_t)k * Gtot + gcol + g;
            for (int sp = 0; sp < splits; ++sp) {
                pr += p[sp * split_stride];
                pi += p[sp * split_stride + im_off];
            }
            const float a = w * pr, c = -w * pi;
            acc[g].x = fmaf(re.x, a, fmaf(im.x, c, acc[g].x));
            acc[g].y = fmaf(re.y, a, fmaf(im.y, c, acc[g].y));
            acc[g].z = fmaf(re.z, a, fmaf(im.z, c, acc[g].z));
            acc[g].w = fmaf(re.w, a, fmaf(im.w, c, acc[g].w));
        }
    }
#pragma unroll
    for (int g = 0; g < GQ; ++g) *reinterpret_cast<float4 *>(&red[warp][g][lane * 4]) = acc[g];
    __syncthreads();
    for (int e = threadIdx.x; e < GQ * kHeadDim; e += blockDim.x) {
        const int g = e / kHeadDim, c = e % kHeadDim;
        float s = 0.f;
#pragma unroll
        for (int w = 0; w < kAttnWarps; ++w) s += red[w][g][c];
        partial[(((size_t)bh * gridDim.x + blockIdx.x) * GQ + g) * kHeadDim + c] = s;
    }
}

// Sum the slice partials, apply 1 / (P * colsum), convert.  grid = batch * H * GQ; block = 128.
template <typename TOut>
__global__ void k_attn_out_reduce2(const float *__restrict__ partial, const float *__restrict__ colsum,
                                   TOut *__restrict__ out, int slices, int GQ, float inv_P) {
    const int bh = blockIdx.x / GQ, g = blockIdx.x % GQ, c = threadIdx.x;
    float s = 0.f;
    for (int sl = 0; sl < slices; ++sl) s += partial[(((size_t)bh * slices + sl) * GQ + g) * kHeadDim + c];
    // flat query-head index bh * GQ + g equals the column index sequence * HQ + head
    const float den = colsum[bh * GQ + g];          // zero only when the sequence has no token: output zero
    store1(out + ((size_t)bh * GQ + g) * kHeadDim + c, den > 0.f ? s * inv_P / den : 0.f);
}

}  // namespace faedkv
