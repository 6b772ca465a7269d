// faedkv_decode_attn_static: decode attention for callers that must not allocate.
//
// Some hosts of this library cannot call cudaMalloc at the point where they need
// attention: code running while a CUDA graph is being captured, a serving loop
// whose memory is handed out once by an external pool, or a plugin that is only
// given the tensors it is called with.  faedkv_decode_attn() needs a context,
// and creating or planning a context allocates.  This entry point needs no
// context: the caller passes the bin list with the other inputs, and every
// intermediate (query spectrum, scores, probability spectrum, partial sums)
// lives in one file-scope device array of fixed size that the library image
// carries.  It computes exactly what faedkv_decode_attn() computes, with the
// float32 kernels.
//
// Consequences of the fixed array:
//  * every GPU that loads the library holds kStaticScratchBytes until exit;
//  * problem sizes whose intermediates do not fit the array, or whose launch grids would exceed the
//    device's grid limits, are rejected with FAEDKV_ERR_SHAPE before anything is launched;
//  * all calls share the array and it keeps whatever the last call left in it.
//    Nothing in it has to start at zero: each region's real columns are fully written before they
//    are read.  The padding columns (query heads rounded up to 32) are read by the two transforms with
//    whatever an earlier call left there, but columns are independent and a padding column never
//    feeds an output.  So no clearing is done; but two calls that overlap on the GPU (different
//    streams, or the same call from two threads) race on the array.  Serialise them.
//  * the first call on each device looks up the array's device address
//    (cudaGetSymbolAddress); make that first call before any stream capture.
#include <cstdio>
#include <mutex>

#include "../../include/faedkv.h"
#include "common.cuh"
#include "k_attn.cuh"
#include "k_dft_simt.cuh"

using namespace faedkv;

namespace {

constexpr size_t kStaticScratchBytes = FAEDKV_STATIC_SCRATCH_BYTES;
constexpr size_t kStaticScratchFloats = kStaticScratchBytes / sizeof(float);
constexpr int kMaxDevices = 64;

// In host code this name is only a handle for cudaGetSymbolAddress, never a pointer to pass to a kernel.
static __device__ __align__(256) float g_static_scratch[kStaticScratchFloats];

std::mutex g_mutex;
float *g_scratch_addr[kMaxDevices] = {nullptr};
int g_sm_count[kMaxDevices] = {0};
// Where the current call wants its error text (caller's buffer; may be absent).
thread_local char *g_err = nullptr;
thread_local size_t g_err_len = 0;

template <typename... A>
void set_err(const char *fmt, A... args) {
    if (g_err != nullptr && g_err_len > 0) snprintf(g_err, g_err_len, fmt, args...);
}

int fail(int code, const char *msg) {
    set_err("%s", msg);
    return code;
}

// Device address of the scratch array on the current device (and the device's SM count, for grid sizing);
// resolved once per device.
int scratch_for_current_device(float **out, int *n_sm) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return fail(FAEDKV_ERR_CUDA, "cudaGetDevice failed");
    if (dev < 0 || dev >= kMaxDevices) return fail(FAEDKV_ERR_UNSUPPORTED, "device ordinal beyond the table of scratch addresses");
    std::lock_guard<std::mutex> lock(g_mutex);
    if (g_scratch_addr[dev] == nullptr) {
        float *p = nullptr;
        cudaError_t e = cudaGetSymbolAddress(reinterpret_cast<void **>(&p), g_static_scratch);
        if (e != cudaSuccess || p == nullptr) {
            set_err("cudaGetSymbolAddress(static scratch) failed: %s", cudaGetErrorString(e));
            return FAEDKV_ERR_CUDA;
        }
        int sms = 0;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1)
            return fail(FAEDKV_ERR_CUDA, "cannot read the device's multiprocessor count");
        g_sm_count[dev] = sms;
        g_scratch_addr[dev] = p;
    }
    *out = g_scratch_addr[dev];
    *n_sm = g_sm_count[dev];
    return FAEDKV_OK;
}

size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

template <typename TQ, int GQ>
int run(float *scratch, int n_sm, int P, int H, int HQ, const int32_t *bins, int M, const void *q, const float *coefK,
        const float *coefV, const int32_t *t_len, int batch, float scale, void *out, cudaStream_t st) {
    const int HQP = (HQ + 31) / 32 * 32, col_blocks = HQP / 32;
    const int n_tiles = (P + kTilePos - 1) / kTilePos;
    const int units = batch * H;
    int slices = (2 * n_sm + units - 1) / units;
    if (slices > (M + 63) / 64) slices = (M + 63) / 64;
    if (slices < 1) slices = 1;
    // every launch below puts units or batch * col_blocks in gridDim.y
    constexpr long long kMaxGridY = 65535;
    if ((long long)units > kMaxGridY || (long long)batch * col_blocks > kMaxGridY) {
        set_err("batch * n_kv_heads = %d (or batch * column blocks = %lld) exceeds the grid limit %lld", units,
                (long long)batch * col_blocks, kMaxGridY);
        return FAEDKV_ERR_SHAPE;
    }
    // carve the array (64-float granules keep every region 256-byte aligned)
    size_t off = 0;
    auto take = [&](size_t n) { float *p = scratch + off; off += round_up(n, 64); return p; };
    float *Qf = take((size_t)batch * 2 * M * HQP);
    float *Pf = take((size_t)batch * 2 * M * HQP);
    float *S = take((size_t)batch * P * HQP);
    float *tile_max = take((size_t)batch * n_tiles * HQP);
    float *colmax = take((size_t)batch * HQP);
    float *partial = take((size_t)units * slices * GQ * kHeadDim);
    if (off > kStaticScratchFloats) {
        set_err("intermediates need %zu bytes, the static scratch holds %zu (FAEDKV_STATIC_SCRATCH_BYTES)",
                off * sizeof(float), kStaticScratchBytes);
        return FAEDKV_ERR_SHAPE;
    }
    constexpr int KB = attn_bins_per_warp(GQ);
    {
        dim3 grid((M + kAttnWarps * KB - 1) / (kAttnWarps * KB), units);
        k_attn_qf<TQ, GQ><<<grid, kAttnWarps * 32, 0, st>>>(static_cast<const TQ *>(q), coefK, Qf, M, H, HQ, HQP);
    }
    DftUnitArgs a{};
    a.x[0] = S;
    a.x_unit = (long long)P * HQP;
    a.y_unit = 2LL * M * HQP;
    a.y_plane = (long long)M * HQP;
    a.x_row = HQP; a.y_row = HQP; a.col_blocks = col_blocks;
    {
        a.y[0] = Qf;
        dim3 grid(n_tiles, batch * col_blocks, 1);
        k_dft_inverse_simt<float, 32><<<grid, kSimtThreads, 0, st>>>(a, bins, M, (uint32_t)P, P, t_len, 1,
                                                                      scale / (float)P, tile_max);
        k_colmax<<<batch * col_blocks, 32, 0, st>>>(tile_max, n_tiles, 32, colmax);
    }
    {
        a.y[0] = Pf;
        dim3 grid((M + kTileBins - 1) / kTileBins, batch * col_blocks, 1);
        k_dft_forward_simt<float, 32, true><<<grid, kSimtThreads, 0, st>>>(a, bins, M, (uint32_t)P, 0, t_len, 1, 0u,
                                                                           1.0f, 0, colmax);
    }
    {
        const int per = (M + slices - 1) / slices;
        dim3 grid(slices, units);
        k_attn_out<GQ><<<grid, kAttnWarps * 32, 0, st>>>(coefV, Pf, bins, partial, M, H, HQP, (uint32_t)P, per);
        k_attn_out_reduce<TQ><<<units * GQ, kHeadDim, 0, st>>>(partial, static_cast<TQ *>(out), slices, GQ, 1.0f / (float)P);
    }
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) {
        set_err("kernel launch failed: %s", cudaGetErrorString(e));
        return FAEDKV_ERR_CUDA;
    }
    return FAEDKV_OK;
}

template <typename TQ>
int dispatch(int gq, float *scratch, int n_sm, int P, int H, int HQ, const int32_t *bins, int M, const void *q,
             const float *coefK, const float *coefV, const int32_t *t_len, int batch, float scale, void *out,
             cudaStream_t st) {
    switch (gq) {
        case 1: return run<TQ, 1>(scratch, n_sm, P, H, HQ, bins, M, q, coefK, coefV, t_len, batch, scale, out, st);
        case 2: return run<TQ, 2>(scratch, n_sm, P, H, HQ, bins, M, q, coefK, coefV, t_len, batch, scale, out, st);
        case 3: return run<TQ, 3>(scratch, n_sm, P, H, HQ, bins, M, q, coefK, coefV, t_len, batch, scale, out, st);
        case 4: return run<TQ, 4>(scratch, n_sm, P, H, HQ, bins, M, q, coefK, coefV, t_len, batch, scale, out, st);
        case 5: return run<TQ, 5>(scratch, n_sm, P, H, HQ, bins, M, q, coefK, coefV, t_len, batch, scale, out, st);
        case 6: return run<TQ, 6>(scratch, n_sm, P, H, HQ, bins, M, q, coefK, coefV, t_len, batch, scale, out, st);
        case 7: return run<TQ, 7>(scratch, n_sm, P, H, HQ, bins, M, q, coefK, coefV, t_len, batch, scale, out, st);
        case 8: return run<TQ, 8>(scratch, n_sm, P, H, HQ, bins, M, q, coefK, coefV, t_len, batch, scale, out, st);
    }
    return fail(FAEDKV_ERR_UNSUPPORTED, "query heads per kv head must be between 1 and 8");
}

}  // namespace

extern "C" {

int faedkv_decode_attn_static(int n_dft, int n_kv_heads, int n_q_heads, int kv_dtype, const int32_t *bins,
                              int n_bins, const void *q, const float *coefK, const float *coefV,
                              const int32_t *t_len, int batch, float scale, void *out, void *stream,
                              char *err_msg, size_t err_len) {
    g_err = err_msg;
    g_err_len = err_len;
    if (err_msg != nullptr && err_len > 0) err_msg[0] = 0;
    if (n_dft < 2 || n_dft > (1 << 24) || n_kv_heads < 1 || n_q_heads < 1 || batch < 1 || n_bins < 1 ||
        n_bins > n_dft / 2 + 1)
        return fail(FAEDKV_ERR_INVALID_ARG, "size argument out of range");
    if (kv_dtype != FAEDKV_F32 && kv_dtype != FAEDKV_BF16) return fail(FAEDKV_ERR_INVALID_ARG, "bad kv_dtype");
    if (n_q_heads % n_kv_heads != 0) return fail(FAEDKV_ERR_UNSUPPORTED, "n_q_heads must be a multiple of n_kv_heads");
    if (bins == nullptr || q == nullptr || coefK == nullptr || coefV == nullptr || t_len == nullptr || out == nullptr)
        return fail(FAEDKV_ERR_INVALID_ARG, "NULL pointer");
    if (!(scale >= 0.0f)) return fail(FAEDKV_ERR_INVALID_ARG, "scale must be >= 0");
    for (const void *p : {q, (const void *)coefK, (const void *)coefV, (const void *)out})
        if ((reinterpret_cast<uintptr_t>(p) & 15u) != 0) return fail(FAEDKV_ERR_ALIGN, "tensor pointer not 16-byte aligned");
    if ((reinterpret_cast<uintptr_t>(bins) & 3u) != 0 || (reinterpret_cast<uintptr_t>(t_len) & 3u) != 0)
        return fail(FAEDKV_ERR_ALIGN, "bins / t_len not 4-byte aligned");
    if (scale == 0.0f) scale = 1.0f / sqrtf((float)kHeadDim);
    float *scratch = nullptr;
    int n_sm = 0;
    if (int r = scratch_for_current_device(&scratch, &n_sm)) return r;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int gq = n_q_heads / n_kv_heads;
    if (kv_dtype == FAEDKV_BF16)
        return dispatch<__nv_bfloat16>(gq, scratch, n_sm, n_dft, n_kv_heads, n_q_heads, bins, n_bins, q, coefK, coefV, t_len,
                                       batch, scale, out, st);
    return dispatch<float>(gq, scratch, n_sm, n_dft, n_kv_heads, n_q_heads, bins, n_bins, q, coefK, coefV, t_len, batch,
                           scale, out, st);
}

}  // extern "C"
