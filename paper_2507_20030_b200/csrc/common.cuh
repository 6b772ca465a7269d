// Device helpers shared by the FAEDKV kernels: exact integer phase reduction,
// float32 twiddles, Hermitian weights, bf16 <-> float32 moves.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace faedkv {

constexpr int kHeadDim = 128;

// Checked build (-DFAEDKV_DEBUG; stands in for a memory checker): an index computed from data -- a bin, a plan slot,
// a ring slot, a row, a tile offset -- is tested against its bound before it addresses memory.  A failed test
// records (file tag << 16 | source line) in a device word, once, and the access is skipped: the kernel carries
// on and returns normally (never a trap), and the host reads the word with faedkv_debug_word().  In the normal
// build the macro is the constant `true` and leaves no code behind.
// Use:  if (!FAEDKV_IN_BOUNDS(tag, idx < n)) continue;   (or return, or skip the statement)
#ifdef FAEDKV_DEBUG
static __device__ unsigned int g_faedkv_debug_word = 0;
__device__ __forceinline__ bool debug_in_bounds(bool ok, unsigned int where) {
    if (!ok) atomicCAS(&g_faedkv_debug_word, 0u, where);
    return ok;
}
#define FAEDKV_IN_BOUNDS(tag, cond) (::faedkv::debug_in_bounds((cond), ((unsigned int)(tag) << 16) | (unsigned int)__LINE__))
#else
#define FAEDKV_IN_BOUNDS(tag, cond) (true)
#endif
// file tags of FAEDKV_IN_BOUNDS
constexpr unsigned int kTagAppend = 1, kTagAttnFft = 2, kTagAttnCol = 3, kTagRecon2 = 4, kTagPrefillUmma = 5,
                       kTagDftSimt = 6, kTagWindow = 7, kTagFftEngine = 8, kTagReconFft = 9, kTagPrefillFft = 10;

// (k * n) mod P with k, n < 2^31: the product fits 64 bits, so the reduced
// phase index is exact however long the sequence is.
__device__ __forceinline__ uint32_t phase_mod(uint32_t k, uint32_t n, uint32_t P) {
    return (uint32_t)(((uint64_t)k * (uint64_t)n) % (uint64_t)P);
}

// (a + b) mod P for a, b < P <= 2^24.
__device__ __forceinline__ uint32_t add_mod(uint32_t a, uint32_t b, uint32_t P) {
    uint32_t s = a + b;
    return s >= P ? s - P : s;
}

// cos, sin of 2*pi*ph/P for a reduced phase index ph < P <= 2^24.  The index is
// first folded to (-P/2, P/2], so the float32 argument of sincospif is exact to
// one rounding of the quotient: absolute angle error <= pi * 2^-24.
__device__ __forceinline__ void twiddle(uint32_t ph, uint32_t P, float &c, float &s) {
    int sp = (2u * ph > P) ? (int)ph - (int)P : (int)ph;
    float x = __fdiv_rn(2.0f * (float)sp, (float)P);
    sincospif(x, &s, &c);
}

// Weight of a one-sided bin in a real-signal inverse DFT: the bin and its
// mirror P-k coincide for k = 0 and (P even) k = P/2, else the mirror doubles it.
__device__ __forceinline__ float hermitian_weight(uint32_t k, uint32_t P) {
    return (k == 0u || 2u * k == P) ? 1.0f : 2.0f;
}

__device__ __forceinline__ float bf16_bits_to_float(uint32_t b16) { return __uint_as_float(b16 << 16); }

// 4 consecutive elements starting at p (16-byte aligned for float, 8-byte for bf16) as float4.
__device__ __forceinline__ float4 load4(const float *p) { return *reinterpret_cast<const float4 *>(p); }
__device__ __forceinline__ float4 load4(const __nv_bfloat16 *p) {
    uint2 r = *reinterpret_cast<const uint2 *>(p);
    return make_float4(bf16_bits_to_float(r.x & 0xffffu), __uint_as_float(r.x & 0xffff0000u),
                       bf16_bits_to_float(r.y & 0xffffu), __uint_as_float(r.y & 0xffff0000u));
}
__device__ __forceinline__ float load1(const float *p) { return *p; }
__device__ __forceinline__ float load1(const __nv_bfloat16 *p) { return __bfloat162float(*p); }

__device__ __forceinline__ void store4(float *p, float4 v) { *reinterpret_cast<float4 *>(p) = v; }
__device__ __forceinline__ void store4(__nv_bfloat16 *p, float4 v) {
    __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y);
    __nv_bfloat162 hi = __floats2bfloat162_rn(v.z, v.w);
    uint2 r;
    r.x = *reinterpret_cast<uint32_t *>(&lo);
    r.y = *reinterpret_cast<uint32_t *>(&hi);
    *reinterpret_cast<uint2 *>(p) = r;
}
__device__ __forceinline__ void store1(float *p, float v) { *p = v; }
__device__ __forceinline__ void store1(__nv_bfloat16 *p, float v) { *p = __float2bfloat16_rn(v); }

// Programmatic dependent launch: a kernel launched with the programmatic-serialisation attribute is
// scheduled while its predecessor in the stream drains, and runs its own set-up (tables in shared memory)
// at once; it must call pdl_wait() before touching anything the predecessor writes -- the wait returns when
// the predecessor has completed and its writes are visible.  Without the attribute it is a no-op.
// (Letting the predecessor release its dependents early, by griddepcontrol.launch_dependents at its start,
// was measured slower here: the waiting CTAs hold shared memory and registers the predecessor still needs.)
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// Streaming (evict-first) 16-byte global accesses for planes that are touched
// once per call and are far larger than L2.
__device__ __forceinline__ float4 ld_stream(const float *p) {
    return __ldcs(reinterpret_cast<const float4 *>(p));
}
__device__ __forceinline__ void st_stream(float *p, float4 v) {
    __stcs(reinterpret_cast<float4 *>(p), v);
}

}  // namespace faedkv
