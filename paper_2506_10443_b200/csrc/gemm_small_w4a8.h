// Host interface of the short-prompt (M <= 64) W4A8 kernel (internal to the library).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/mnnllm.h"

namespace mnnllm {

constexpr int kGemmSmallMaxBatch = 4;
constexpr int kGemmSmallMaxTokens = 64;

struct GemmSmallArgs {
    const void* packed[kGemmSmallMaxBatch];  // device, written by mnnllm_pack_w4 (same K and group)
    void* y[kGemmSmallMaxBatch];             // device [M, N[i]] of y_dtype[i] (unused in the partials form)
    int N[kGemmSmallMaxBatch];
    int y_dtype[kGemmSmallMaxBatch];
    int count;
    const int8_t* a_q;       // device [M, K]: signed codes
    const float* a_scale;    // device fp32 [M]
    const float* a_sums_t;   // device fp32 [K / group][64]: group sums of the codes, token fastest
    int32_t* P;              // device int32 [M, N[0], G] (partials form only, count == 1)
    float* scratch;          // device, scratch_bytes (null: K is never cut into parts)
    size_t scratch_bytes;
    uint32_t* counters;      // device, n_counters words, zero when the kernel starts (null with scratch)
    int n_counters;
    int M, K, group;
};

// Enqueues the kernel on `stream` (M <= kGemmSmallMaxTokens).  With args.P set it stores every int32
// group partial instead of y.
cudaError_t gemm_small_w4a8_launch(const GemmSmallArgs& args, uint32_t* status, cudaStream_t stream);

}  // namespace mnnllm
