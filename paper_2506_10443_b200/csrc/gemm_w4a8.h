// Host interface of the prefill W4A8 GEMM kernel (internal to the library).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/mnnllm.h"

namespace mnnllm {

struct GemmW4A8Args {
    const void* packed;    // device, written by mnnllm_pack_w4
    const int8_t* a_q;     // device int8 [M, K]
    const float* a_scale;  // device fp32 [M]
    const void* AC;        // device fp16 quadruples [M, G4] x 8 bytes (null in the partials form)
    void* y;               // device [M, N] of y_dtype (null in the partials form)
    int32_t* P;            // device int32 [M, N, G] (partials form only)
    int M, N, K, group;
    int y_dtype;
};

// Enqueues the GEMM on `stream`.  With args.P set the kernel stores every int32 group partial and
// skips the rescale; otherwise it writes y.  Returns cudaErrorNotSupported when the driver lacks
// tensor-map encoding.
cudaError_t gemm_w4a8_launch(const GemmW4A8Args& args, uint32_t* status, cudaStream_t stream);

}  // namespace mnnllm
