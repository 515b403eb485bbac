// C-ABI entry points of the per-channel W8A8 prefill path: argument checks, workspace carve-up, and
// the two launches (activation quantiser, then the tensor-core GEMM).
#include "act_quant.h"
#include "common.h"
#include "gemm_w8a8.h"
#include "layout.h"

using namespace mnnllm;

namespace {

size_t round256(size_t v) { return (v + 255) & ~(size_t)255; }

// workspace: a_q int8 [M, K] | a_scale fp32 [M] | a_sum int32 [M]
struct Workspace {
    size_t a_q, a_scale, a_sum, total;
};
Workspace workspace_layout(int M, int K) {
    Workspace w;
    w.a_q = 0;
    w.a_scale = round256((size_t)M * K);
    w.a_sum = w.a_scale + round256((size_t)M * 4);
    w.total = w.a_sum + round256((size_t)M * 4);
    return w;
}

}  // namespace

extern "C" {

size_t mnnllm_workspace_size_w8a8(int M, int K) {
    if (M < 1 || K < 1 || K % 32 != 0) return 0;
    return workspace_layout(M, K).total;
}

int mnnllm_linear_w8a8(const void* x, const void* packed, void* y, int M, int N, int K, int x_dtype, int y_dtype,
                       void* workspace, size_t workspace_bytes, void* stream) {
    if (!x || !packed || !y || M < 1 || N < 1 || K < 1) return MNNLLM_ERR_INVALID_ARG;
    if (x_dtype != MNNLLM_F16 && x_dtype != MNNLLM_BF16) return MNNLLM_ERR_UNSUPPORTED;
    if (y_dtype != MNNLLM_F16 && y_dtype != MNNLLM_BF16 && y_dtype != MNNLLM_F32) return MNNLLM_ERR_UNSUPPORTED;
    if (K % 32 != 0) return MNNLLM_ERR_UNSUPPORTED;
    if (((uintptr_t)x & 15) || ((uintptr_t)packed & 127) || ((uintptr_t)y & 3)) return MNNLLM_ERR_ALIGNMENT;
    const Workspace w = workspace_layout(M, K);
    if (!workspace || workspace_bytes < w.total) return MNNLLM_ERR_WORKSPACE;
    if ((uintptr_t)workspace & 255) return MNNLLM_ERR_ALIGNMENT;
    if (!device_is_supported()) return MNNLLM_ERR_UNSUPPORTED;
    uint32_t* status = status_word_ptr();
    if (!status) return MNNLLM_ERR_CUDA;
    uint8_t* base = (uint8_t*)workspace;
    int8_t* a_q = (int8_t*)(base + w.a_q);
    float* a_scale = (float*)(base + w.a_scale);
    int32_t* a_sum = (int32_t*)(base + w.a_sum);
    // signed codes (the GEMM multiplies them as signed 8-bit); the group argument only shapes sums that
    // are not asked for here
    if (act_quant_launch(x, x_dtype, M, K, 64, a_q, a_scale, nullptr, nullptr, false, nullptr, 0, (cudaStream_t)stream,
                         nullptr, a_sum) != cudaSuccess) {
        (void)cudaGetLastError();
        return MNNLLM_ERR_CUDA;
    }
    GemmW8A8Args a;
    a.packed = packed; a.y = y; a.y_dtype = y_dtype;
    a.a_q = a_q; a.a_scale = a_scale; a.a_sum = a_sum;
    a.M = M; a.N = N; a.K = K;
    const cudaError_t e = gemm_w8a8_launch(a, status, (cudaStream_t)stream);
    if (e != cudaSuccess) {
        (void)cudaGetLastError();
        return e == cudaErrorNotSupported ? MNNLLM_ERR_UNSUPPORTED : MNNLLM_ERR_CUDA;
    }
    return MNNLLM_OK;
}

}  // extern "C"
