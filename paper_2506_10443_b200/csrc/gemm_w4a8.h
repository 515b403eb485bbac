// Host interface of the prefill W4A8 GEMM kernel (internal to the library).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/mnnllm.h"

namespace mnnllm {

constexpr int kGemmMaxBatch = 4;
// A launch with fewer tiles than SMs cuts every tile's K range into parts that run as separate
// work items; they meet through scratch memory: one 128 x 128 fp32 slot per part and sixteen
// counters per tile (the quantiser that precedes the GEMM clears the counters).
constexpr int kGemmScratchSlots = 320;
constexpr size_t kGemmScratchBytes = (size_t)kGemmScratchSlots * 128 * 128 * 4;
constexpr int kGemmCounters = 160 * 16;

// `count` weight matrices that multiply the same quantised activations (q, k, v of a layer; gate and
// up): one launch, the n-tiles of all of them in one grid.
struct GemmW4A8Args {
    const void* packed[kGemmMaxBatch];  // device, written by mnnllm_pack_w4 (same K and group)
    void* y[kGemmMaxBatch];             // device [M, N[i]] of y_dtype[i] (unused in the partials form)
    int N[kGemmMaxBatch];
    int y_dtype[kGemmMaxBatch];
    int count;
    const int8_t* a_q;     // device [M, K]: the codes a_q + 128 as unsigned bytes
    const float* a_scale;  // device fp32 [M]
    const void* AC;        // device fp16 quadruples [M, G4] x 8 bytes (null in the partials form)
    int32_t* P;            // device int32 [M, N[0], G] (partials form only, count == 1)
    float* scratch;        // device, kGemmScratchBytes (null: tiles are never split along K)
    uint32_t* counters;    // device, kGemmCounters words, zero when the kernel starts (null with scratch)
    int M, K, group;
    bool skip_if_limb_ok;  // the integer-limb kernel was launched ahead: do nothing if every matrix allowed it
};

// Enqueues the GEMM on `stream`.  With args.P set the kernel stores every int32 group partial and
// skips the rescale; otherwise it writes y.  Returns cudaErrorNotSupported when the driver lacks
// tensor-map encoding.
cudaError_t gemm_w4a8_launch(const GemmW4A8Args& args, uint32_t* status, cudaStream_t stream);

}  // namespace mnnllm
