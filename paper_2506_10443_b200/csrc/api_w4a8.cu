// C-ABI entry points of the W4A8 prefill path.
#include "act_quant.h"
#include "common.h"
#include "layout.h"

using namespace mnnllm;

namespace {
int check_xq(const void* x, int x_dtype, int M, int K, int group) {
    if (!x || M < 1 || K < 1) return MNNLLM_ERR_INVALID_ARG;
    if (x_dtype != MNNLLM_F16 && x_dtype != MNNLLM_BF16) return MNNLLM_ERR_UNSUPPORTED;
    if ((group != 64 && group != 128) || K % group != 0) return MNNLLM_ERR_UNSUPPORTED;
    if ((uintptr_t)x & 15) return MNNLLM_ERR_ALIGNMENT;
    return MNNLLM_OK;
}
}  // namespace

extern "C" {

int mnnllm_quantize_activations(const void* x, int x_dtype, int M, int K, int group, int8_t* a_q, float* a_scale,
                                int32_t* A, void* stream) {
    const int st = check_xq(x, x_dtype, M, K, group);
    if (st != MNNLLM_OK) return st;
    if (!a_q || !a_scale || !A) return MNNLLM_ERR_INVALID_ARG;
    if (((uintptr_t)a_q & 15) || ((uintptr_t)a_scale & 3) || ((uintptr_t)A & 3)) return MNNLLM_ERR_ALIGNMENT;
    if (!device_is_supported()) return MNNLLM_ERR_UNSUPPORTED;
    if (act_quant_launch(x, x_dtype, M, K, group, a_q, a_scale, A, (cudaStream_t)stream) != cudaSuccess) {
        (void)cudaGetLastError();
        return MNNLLM_ERR_CUDA;
    }
    return MNNLLM_OK;
}

size_t mnnllm_workspace_size_w4a8(int M, int N, int K, int group) { return 0; }
int mnnllm_linear_w4a8(const void*, const void*, void*, int, int, int, int, int, int, void*, size_t, void*) {
    return MNNLLM_ERR_UNSUPPORTED;
}
int mnnllm_debug_w4a8_partials(const void*, int, const void*, int32_t*, int8_t*, float*, int32_t*, int, int, int, int,
                               void*) {
    return MNNLLM_ERR_UNSUPPORTED;
}

}  // extern "C"
