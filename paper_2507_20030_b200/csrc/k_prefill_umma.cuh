// Tensor-core (tcgen05) prefill transform -- placeholder until the kernel lands.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>
#include <cstdio>

namespace faedkv {

struct UmmaPrefillState {};

inline bool umma_prefill_available() { return false; }

inline int umma_prefill_launch(UmmaPrefillState &, const void *, const void *, int, int, int,
                               const int32_t *, int, int, int, float *, float *, unsigned int *,
                               cudaStream_t, char *msg, size_t msg_len) {
    snprintf(msg, msg_len, "tensor-core prefill is not built in");
    return -4;
}

}  // namespace faedkv
