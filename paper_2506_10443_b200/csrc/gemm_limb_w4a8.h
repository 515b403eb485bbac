// Host interface of the integer-limb W4A8 prefill GEMM (internal to the library).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/mnnllm.h"

namespace mnnllm {

constexpr int kGemmLimbMaxBatch = 4;

struct GemmLimbArgs {
    const void* packed[kGemmLimbMaxBatch];  // device, written by mnnllm_pack_w4 (same K and group), trailer included
    void* y[kGemmLimbMaxBatch];             // device [M, N[i]] of y_dtype[i]
    int N[kGemmLimbMaxBatch];
    int y_dtype[kGemmLimbMaxBatch];
    int count;
    const int8_t* a_q;     // device [M, K]: the codes a_q + 128 as unsigned bytes
    const float* a_scale;  // device fp32 [M]
    const void* AC;        // device fp16 quadruples [M, G4] x 8 bytes (group sums for the zero-point MMA)
    int M, K, group;
};

// Tiles (128 weight rows x 128 tokens) of the launch: the kernel has no K split, so the caller uses it
// only when there are enough tiles for the GPU.
int gemm_limb_w4a8_tiles(const GemmLimbArgs& args);

// Enqueues the kernel on `stream`.  Every CTA returns at once, without writing anything, when the
// trailer of one of the packed buffers says that its scales do not fit the limbs: the caller
// launches gemm_w4a8_launch behind it with `skip_if_limb_ok` set.  Returns cudaErrorNotSupported when
// the driver lacks tensor-map encoding.
cudaError_t gemm_limb_w4a8_launch(const GemmLimbArgs& args, uint32_t* status, cudaStream_t stream);

}  // namespace mnnllm
