// Launch wrapper of the per-token int8 activation quantiser (internal to the library).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/mnnllm.h"

namespace mnnllm {

// x [M, K] (fp16 or bf16) -> a_q int8 [M, K], a_scale fp32 [M], A int32 [M, K / group] (may be null)
// and, when AC is not null, the group sums as fp16 quadruples (64h, l, 64h, l), A = 64h + l,
// [M, G4] x 8 bytes with G4 = K / group rounded up to a multiple of 4 (padding written as zeros).
// With offset128 the codes are stored as unsigned bytes a_q + 128 (what the GEMM multiplies); the
// sums A and AC are those of the signed codes either way.  `clear` (may be null) is an array of
// n_clear words that the kernel sets to zero: the counters of the GEMM that follows.  `sums_t` (may be
// null; M <= 64 only) receives the group sums as fp32, transposed: [K / group][64], token fastest
// (entries of tokens >= M are left as they are).  `row_sum` (may be null) receives sum_k a_q[m, k], int32 [M].
cudaError_t act_quant_launch(const void* x, int x_dtype, int M, int K, int group, int8_t* a_q, float* a_scale,
                             int32_t* A, void* AC, bool offset128, uint32_t* clear, int n_clear, cudaStream_t stream,
                             float* sums_t = nullptr, int32_t* row_sum = nullptr);

}  // namespace mnnllm
