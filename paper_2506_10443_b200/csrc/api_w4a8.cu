// C-ABI entry points of the W4A8 prefill path: argument checks, workspace carve-up, and the two
// launches (activation quantiser, then the tensor-core GEMM).
#include <cstdlib>

#include "act_quant.h"
#include "common.h"
#include "gemm_limb_w4a8.h"
#include "gemm_small_w4a8.h"
#include "gemm_w4a8.h"
#include "layout.h"

using namespace mnnllm;

namespace {

// Measured on B200 (Qwen2-1.5B shapes, graph replay): at 16 tokens the GEMV-shaped kernel takes 9-15 us per
// call against 14-26 us of the tensor-memory GEMM, at 32 tokens 11-21 against 15-26; at 64 tokens the two are
// level (17-32 against 15-27), its mma.sync main loop being latency-bound by then.
constexpr int kSmallPathDefaultMax = 32;

int check_xq(const void* x, int x_dtype, int M, int K, int group) {
    if (!x || M < 1 || K < 1) return MNNLLM_ERR_INVALID_ARG;
    if (x_dtype != MNNLLM_F16 && x_dtype != MNNLLM_BF16) return MNNLLM_ERR_UNSUPPORTED;
    if ((group != 64 && group != 128) || K % group != 0) return MNNLLM_ERR_UNSUPPORTED;
    if ((uintptr_t)x & 15) return MNNLLM_ERR_ALIGNMENT;
    return MNNLLM_OK;
}

size_t round256(size_t v) { return (v + 255) & ~(size_t)255; }

// Prompts of up to this many tokens take the GEMV-shaped kernel, longer ones the tensor-memory GEMM.
// The default can be overridden by the environment (MNNLLM_W4A8_SMALL_MAX = 0..64, read once) or by
// mnnllm_debug_set_w4a8_small_max: tuning and test knobs.
int g_small_max_override = -1;
int small_path_max_tokens() {
    if (g_small_max_override >= 0) return g_small_max_override;
    static int from_env = -2;
    if (from_env == -2) {
        from_env = -1;
        if (const char* env = std::getenv("MNNLLM_W4A8_SMALL_MAX")) {
            const int e = std::atoi(env);
            if (e >= 0 && e <= kGemmSmallMaxTokens) from_env = e;
        }
    }
    return from_env >= 0 ? from_env : kSmallPathDefaultMax;
}

// The integer-limb GEMM is an alternative that measured slower than the per-group kernel: off unless MNNLLM_W4A8_LIMB=1 (read once) or
// the debug call switches it on.
int g_limb_override = -1;
bool limb_path_forced() { return g_limb_override == 2; }   // whatever the number of tiles (tests)
bool limb_path_enabled() {
    if (g_limb_override >= 0) return g_limb_override != 0;
    static int from_env = -1;
    if (from_env < 0) {
        const char* env = std::getenv("MNNLLM_W4A8_LIMB");
        from_env = (env && env[0] == '1') ? 1 : 0;
    }
    return from_env != 0;
}

// workspace: a_q int8 [M, K] | a_scale fp32 [M] | group sums: fp16 quadruples [M, G4] x 8 bytes for the
//            tensor-memory GEMM, fp32 [G][64] for the short-prompt kernel (M <= 64)
//            | optional: counters | fp32 parts of tiles that several CTAs share
struct Workspace {
    size_t a_q, a_scale, ac, total;   // total: what every call needs
    size_t counters, scratch, total_split;   // total_split: with the scratch that lets the GEMM balance its work
};
Workspace workspace_layout(int M, int K, int group) {
    Workspace w;
    const size_t G4 = (size_t)(K / group + 3) / 4 * 4;
    w.a_q = 0;
    w.a_scale = round256((size_t)M * K);
    w.ac = w.a_scale + round256((size_t)M * 4);
    const size_t sums = (size_t)M * G4 * 8, sums_small = M <= kGemmSmallMaxTokens ? G4 * 64 * 4 : 0;
    w.total = w.ac + round256(sums > sums_small ? sums : sums_small);
    w.counters = w.total;
    w.scratch = w.counters + round256((size_t)kGemmCounters * 4);
    w.total_split = w.scratch + kGemmScratchBytes;
    return w;
}

// Scratch of mnnllm_linear_w4a8_static: lives in the library's device image, one copy on every GPU
// that loads the library, for the lifetime of the process.  Host code may not use the symbol as an
// address; static_scratch_ptr() asks the runtime for the device address once per device.
static __device__ __align__(256) unsigned char g_static_scratch[MNNLLM_STATIC_SCRATCH_BYTES];

void* static_scratch_ptr() {
    static void* ptrs[64];
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    if (!ptrs[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress((void**)&p, g_static_scratch) != cudaSuccess) {
            (void)cudaGetLastError();
            return nullptr;
        }
        ptrs[dev] = p;
    }
    return ptrs[dev];
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
    if (act_quant_launch(x, x_dtype, M, K, group, a_q, a_scale, A, nullptr, false, nullptr, 0, (cudaStream_t)stream) !=
        cudaSuccess) {
        (void)cudaGetLastError();
        return MNNLLM_ERR_CUDA;
    }
    return MNNLLM_OK;
}

size_t mnnllm_workspace_size_w4a8(int M, int N, int K, int group) {
    if (M < 1 || N < 1 || K < 1 || (group != 64 && group != 128) || K % group != 0) return 0;
    return workspace_layout(M, K, group).total_split;
}

size_t mnnllm_workspace_min_w4a8(int M, int N, int K, int group) {
    if (M < 1 || N < 1 || K < 1 || (group != 64 && group != 128) || K % group != 0) return 0;
    return workspace_layout(M, K, group).total;
}

int mnnllm_linear_w4a8_batch(const mnnllm_w4a8_problem* problems, int count, const void* x, int M, int K, int group,
                             int x_dtype, void* workspace, size_t workspace_bytes, void* stream) {
    const int st = check_xq(x, x_dtype, M, K, group);
    if (st != MNNLLM_OK) return st;
    if (!problems || count < 1 || count > MNNLLM_MAX_BATCH_W4A8) return MNNLLM_ERR_INVALID_ARG;
    for (int i = 0; i < count; ++i) {
        const mnnllm_w4a8_problem& q = problems[i];
        if (!q.packed || !q.y || q.N < 1) return MNNLLM_ERR_INVALID_ARG;
        if (q.y_dtype != MNNLLM_F16 && q.y_dtype != MNNLLM_BF16 && q.y_dtype != MNNLLM_F32) return MNNLLM_ERR_UNSUPPORTED;
        if (((uintptr_t)q.y & 15) || ((uintptr_t)q.packed & 127)) return MNNLLM_ERR_ALIGNMENT;
    }
    const Workspace w = workspace_layout(M, K, group);
    if (!workspace || workspace_bytes < w.total) return MNNLLM_ERR_WORKSPACE;
    if ((uintptr_t)workspace & 255) return MNNLLM_ERR_ALIGNMENT;
    const bool split = workspace_bytes >= w.total_split;
    if (!device_is_supported()) return MNNLLM_ERR_UNSUPPORTED;
    uint32_t* status = status_word_ptr();
    if (!status) return MNNLLM_ERR_CUDA;

    uint8_t* ws = (uint8_t*)workspace;
    int8_t* a_q = (int8_t*)(ws + w.a_q);
    float* a_scale = (float*)(ws + w.a_scale);
    void* ac = ws + w.ac;
    uint32_t* counters = split ? (uint32_t*)(ws + w.counters) : nullptr;
    if (M <= small_path_max_tokens()) {
        // short prompts: bound by HBM, not by the tensor cores; the GEMV-shaped kernel streams the weights once
        if (act_quant_launch(x, x_dtype, M, K, group, a_q, a_scale, nullptr, nullptr, false, counters, kGemmCounters,
                             (cudaStream_t)stream, (float*)ac) != cudaSuccess) {
            (void)cudaGetLastError();
            return MNNLLM_ERR_CUDA;
        }
        GemmSmallArgs a;
        a.count = count;
        for (int i = 0; i < count; ++i) {
            a.packed[i] = problems[i].packed; a.y[i] = problems[i].y; a.N[i] = problems[i].N; a.y_dtype[i] = problems[i].y_dtype;
        }
        a.a_q = a_q; a.a_scale = a_scale; a.a_sums_t = (const float*)ac; a.P = nullptr;
        a.scratch = split ? (float*)(ws + w.scratch) : nullptr;
        a.scratch_bytes = kGemmScratchBytes;
        a.counters = counters; a.n_counters = kGemmCounters;
        a.M = M; a.K = K; a.group = group;
        if (gemm_small_w4a8_launch(a, status, (cudaStream_t)stream) != cudaSuccess) {
            (void)cudaGetLastError();
            return MNNLLM_ERR_CUDA;
        }
        return MNNLLM_OK;
    }
    // the activations are quantised once for all the matrices of the batch (the same kernel clears
    // the counters of the GEMM)
    if (act_quant_launch(x, x_dtype, M, K, group, a_q, a_scale, nullptr, ac, true, counters, kGemmCounters,
                         (cudaStream_t)stream) != cudaSuccess) {
        (void)cudaGetLastError();
        return MNNLLM_ERR_CUDA;
    }
    // When the integer-limb kernel (no per-group drain) is switched on, launches with enough 128 x 128
    // tiles for the GPU try it first; the tensor-memory GEMM launched behind it returns at once unless
    // a matrix's scales do not fit the limbs (the packer's flag), in which case the limb kernel has
    // returned at once.
    bool limb = false;
    if (limb_path_enabled()) {
        GemmLimbArgs l;
        l.count = count;
        for (int i = 0; i < count; ++i) {
            l.packed[i] = problems[i].packed; l.y[i] = problems[i].y; l.N[i] = problems[i].N; l.y_dtype[i] = problems[i].y_dtype;
        }
        l.a_q = a_q; l.a_scale = a_scale; l.AC = ac; l.M = M; l.K = K; l.group = group;
        if (limb_path_forced() || gemm_limb_w4a8_tiles(l) * 5 >= device_sm_count() * 3) {   // at least 0.6 tiles per SM
            const cudaError_t e = gemm_limb_w4a8_launch(l, status, (cudaStream_t)stream);
            if (e != cudaSuccess) {
                (void)cudaGetLastError();
                return e == cudaErrorNotSupported ? MNNLLM_ERR_UNSUPPORTED : MNNLLM_ERR_CUDA;
            }
            limb = true;
        }
    }
    GemmW4A8Args a;
    a.count = count;
    a.skip_if_limb_ok = limb;
    for (int i = 0; i < count; ++i) {
        a.packed[i] = problems[i].packed; a.y[i] = problems[i].y; a.N[i] = problems[i].N; a.y_dtype[i] = problems[i].y_dtype;
    }
    a.a_q = a_q; a.a_scale = a_scale; a.AC = ac; a.P = nullptr;
    a.scratch = split ? (float*)(ws + w.scratch) : nullptr;
    a.counters = counters;
    a.M = M; a.K = K; a.group = group;
    const cudaError_t e = gemm_w4a8_launch(a, status, (cudaStream_t)stream);
    if (e != cudaSuccess) {
        (void)cudaGetLastError();
        return e == cudaErrorNotSupported ? MNNLLM_ERR_UNSUPPORTED : MNNLLM_ERR_CUDA;
    }
    return MNNLLM_OK;
}

int mnnllm_linear_w4a8(const void* x, const void* packed, void* y, int M, int N, int K, int group, int x_dtype,
                       int y_dtype, void* workspace, size_t workspace_bytes, void* stream) {
    mnnllm_w4a8_problem q;
    q.packed = packed; q.y = y; q.N = N; q.y_dtype = y_dtype;
    return mnnllm_linear_w4a8_batch(&q, 1, x, M, K, group, x_dtype, workspace, workspace_bytes, stream);
}

int mnnllm_debug_w4a8_partials(const void* x, int x_dtype, const void* packed, int32_t* P, int8_t* a_q, float* a_scale,
                               int32_t* A, int M, int N, int K, int group, void* stream) {
    const int st = check_xq(x, x_dtype, M, K, group);
    if (st != MNNLLM_OK) return st;
    if (!packed || !P || !a_q || !a_scale || !A || N < 1) return MNNLLM_ERR_INVALID_ARG;
    if (((uintptr_t)a_q & 15) || ((uintptr_t)a_scale & 3) || ((uintptr_t)A & 3) || ((uintptr_t)P & 3) ||
        ((uintptr_t)packed & 127))
        return MNNLLM_ERR_ALIGNMENT;
    if (!device_is_supported()) return MNNLLM_ERR_UNSUPPORTED;
    uint32_t* status = status_word_ptr();
    if (!status) return MNNLLM_ERR_CUDA;
    if (M <= small_path_max_tokens()) {   // the short-prompt kernel multiplies the signed codes as they are
        if (act_quant_launch(x, x_dtype, M, K, group, a_q, a_scale, A, nullptr, false, nullptr, 0, (cudaStream_t)stream) !=
            cudaSuccess) {
            (void)cudaGetLastError();
            return MNNLLM_ERR_CUDA;
        }
        GemmSmallArgs a;
        a.count = 1;
        a.packed[0] = packed; a.y[0] = nullptr; a.N[0] = N; a.y_dtype[0] = MNNLLM_F32;
        a.a_q = a_q; a.a_scale = a_scale; a.a_sums_t = nullptr; a.P = P;
        a.scratch = nullptr; a.scratch_bytes = 0; a.counters = nullptr; a.n_counters = 0;
        a.M = M; a.K = K; a.group = group;
        if (gemm_small_w4a8_launch(a, status, (cudaStream_t)stream) != cudaSuccess) {
            (void)cudaGetLastError();
            return MNNLLM_ERR_CUDA;
        }
        return MNNLLM_OK;
    }
    // the GEMM multiplies the codes in their unsigned form (a_q + 128); the caller gets the signed
    // ones, written by a second run of the quantiser once the GEMM has consumed the buffer
    if (act_quant_launch(x, x_dtype, M, K, group, a_q, a_scale, A, nullptr, true, nullptr, 0, (cudaStream_t)stream) !=
        cudaSuccess) {
        (void)cudaGetLastError();
        return MNNLLM_ERR_CUDA;
    }
    GemmW4A8Args a;
    a.count = 1;
    a.skip_if_limb_ok = false;
    a.packed[0] = packed; a.y[0] = nullptr; a.N[0] = N; a.y_dtype[0] = MNNLLM_F32;
    a.a_q = a_q; a.a_scale = a_scale; a.AC = nullptr; a.P = P;
    a.scratch = nullptr; a.counters = nullptr;
    a.M = M; a.K = K; a.group = group;
    const cudaError_t e = gemm_w4a8_launch(a, status, (cudaStream_t)stream);
    if (e != cudaSuccess) {
        (void)cudaGetLastError();
        return e == cudaErrorNotSupported ? MNNLLM_ERR_UNSUPPORTED : MNNLLM_ERR_CUDA;
    }
    if (act_quant_launch(x, x_dtype, M, K, group, a_q, a_scale, A, nullptr, false, nullptr, 0, (cudaStream_t)stream) !=
        cudaSuccess) {
        (void)cudaGetLastError();
        return MNNLLM_ERR_CUDA;
    }
    return MNNLLM_OK;
}

int mnnllm_debug_set_w4a8_limb(int enabled) {
    const int before = limb_path_enabled() ? 1 : 0;
    g_limb_override = (enabled >= 0 && enabled <= 2) ? enabled : -1;
    return before;
}

int mnnllm_debug_set_w4a8_small_max(int max_tokens) {
    const int before = small_path_max_tokens();
    g_small_max_override = (max_tokens >= 0 && max_tokens <= kGemmSmallMaxTokens) ? max_tokens : -1;
    return before;
}

int mnnllm_linear_w4a8_static(const void* x, const void* packed, void* y, int M, int N, int K, int group, int x_dtype,
                              int y_dtype, void* stream) {
    const int st = check_xq(x, x_dtype, M, K, group);
    if (st != MNNLLM_OK) return st;
    if (!packed || !y || N < 1) return MNNLLM_ERR_INVALID_ARG;
    // the activations' int8 copy, scales and group sums must fit the built-in scratch
    if (workspace_layout(M, K, group).total > (size_t)MNNLLM_STATIC_SCRATCH_BYTES) return MNNLLM_ERR_WORKSPACE;
    if (!device_is_supported()) return MNNLLM_ERR_UNSUPPORTED;
    void* scratch = static_scratch_ptr();
    if (!scratch) return MNNLLM_ERR_CUDA;
    // every byte of the scratch that the GEMM reads is written by the quantiser of the same call,
    // so nothing left over from an earlier call needs clearing
    return mnnllm_linear_w4a8(x, packed, y, M, N, K, group, x_dtype, y_dtype, scratch, MNNLLM_STATIC_SCRATCH_BYTES,
                              stream);
}

}  // extern "C"
