// Host interface of the per-channel W8A8 prefill GEMM (internal to the library).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/mnnllm.h"

namespace mnnllm {

struct GemmW8A8Args {
    const void* packed;    // device, written by mnnllm_pack_w8
    void* y;               // device [M, N] of y_dtype
    int y_dtype;
    const int8_t* a_q;     // device [M, K]: signed codes of the per-token quantiser
    const float* a_scale;  // device fp32 [M]
    const int32_t* a_sum;  // device int32 [M]: sum_k a_q[m, k]
    int M, N, K;           // K a multiple of 32
};

// Enqueues the kernel on `stream`.  Returns cudaErrorNotSupported when the driver lacks tensor-map
// encoding.
cudaError_t gemm_w8a8_launch(const GemmW8A8Args& args, uint32_t* status, cudaStream_t stream);

}  // namespace mnnllm
