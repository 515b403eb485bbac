// C-ABI entry points of the decode attention over a quantised KV cache.
#include "attn_decode.h"
#include "common.h"

using namespace mnnllm;

namespace {

constexpr size_t kCounterBytes = 256;   // one uint32 per kv head (at most 64)

int check_cache(const void* k_codes, const void* k_meta, const void* v, int Hk, int S_cap, int head_dim) {
    if (!k_codes || !k_meta || !v || Hk < 1 || S_cap < 1) return MNNLLM_ERR_INVALID_ARG;
    if (head_dim != kAttnHeadDim || Hk > 64) return MNNLLM_ERR_UNSUPPORTED;
    if (((uintptr_t)k_codes & 15) || ((uintptr_t)k_meta & 3) || ((uintptr_t)v & 15)) return MNNLLM_ERR_ALIGNMENT;
    return MNNLLM_OK;
}

AttnCache cache_of(void* k_codes, void* k_meta, void* v, int Hk, int S_cap) {
    AttnCache c;
    c.k_codes = (uint8_t*)k_codes; c.k_meta = (uint32_t*)k_meta; c.v = (uint8_t*)v;
    c.Hk = Hk; c.S_cap = S_cap;
    return c;
}

}  // namespace

extern "C" {

int mnnllm_kv_append(void* k_codes, void* k_meta, void* v, int Hk, int S_cap, int head_dim, int pos, const void* k_new,
                     const void* v_new, void* stream) {
    const int st = check_cache(k_codes, k_meta, v, Hk, S_cap, head_dim);
    if (st != MNNLLM_OK) return st;
    if (!k_new || !v_new || pos < 0 || pos >= S_cap) return MNNLLM_ERR_INVALID_ARG;
    if (((uintptr_t)k_new & 1) || ((uintptr_t)v_new & 1)) return MNNLLM_ERR_ALIGNMENT;
    if (!device_is_supported()) return MNNLLM_ERR_UNSUPPORTED;
    if (attn_append_launch(cache_of(k_codes, k_meta, v, Hk, S_cap), k_new, v_new, pos, (cudaStream_t)stream) != cudaSuccess) {
        (void)cudaGetLastError();
        return MNNLLM_ERR_CUDA;
    }
    return MNNLLM_OK;
}

size_t mnnllm_attention_workspace_size(int H, int Hk, int S) {
    if (H < 1 || Hk < 1 || Hk > 64 || S < 1 || H % Hk != 0 || H / Hk > kAttnMaxRep) return 0;
    // one part per 128 tokens at most (the launch uses fewer when the sequence is long)
    return kCounterBytes + (size_t)((S + kAttnMinSplit - 1) / kAttnMinSplit) * H * (kAttnHeadDim + 2) * 4;
}

int mnnllm_attention_workspace_init(void* workspace, size_t workspace_bytes, void* stream) {
    if (!workspace || workspace_bytes < kCounterBytes) return MNNLLM_ERR_INVALID_ARG;
    if (cudaMemsetAsync(workspace, 0, kCounterBytes, (cudaStream_t)stream) != cudaSuccess) {
        (void)cudaGetLastError();
        return MNNLLM_ERR_CUDA;
    }
    return MNNLLM_OK;
}

int mnnllm_attention_decode(const void* q, const void* k_codes, const void* k_meta, const void* v, void* out, int H, int Hk,
                            int head_dim, int S, int S_cap, int out_dtype, void* workspace, size_t workspace_bytes,
                            void* stream) {
    const int st = check_cache(k_codes, k_meta, v, Hk, S_cap, head_dim);
    if (st != MNNLLM_OK) return st;
    if (!q || !out || H < 1 || S < 1 || S > S_cap) return MNNLLM_ERR_INVALID_ARG;
    if (H % Hk != 0 || H / Hk > kAttnMaxRep) return MNNLLM_ERR_UNSUPPORTED;
    if (out_dtype != MNNLLM_F16 && out_dtype != MNNLLM_F32) return MNNLLM_ERR_UNSUPPORTED;
    if (((uintptr_t)q & 1) || ((uintptr_t)out & 3)) return MNNLLM_ERR_ALIGNMENT;
    if (!device_is_supported()) return MNNLLM_ERR_UNSUPPORTED;
    if (!workspace || workspace_bytes < kCounterBytes + attn_partials_bytes(H, Hk, S)) return MNNLLM_ERR_WORKSPACE;
    if ((uintptr_t)workspace & 15) return MNNLLM_ERR_ALIGNMENT;
    uint32_t* status = status_word_ptr();
    if (!status) return MNNLLM_ERR_CUDA;
    const AttnCache c = cache_of((void*)k_codes, (void*)k_meta, (void*)v, Hk, S_cap);
    if (attn_decode_launch(c, q, out, out_dtype, H, S, (float*)((uint8_t*)workspace + kCounterBytes),
                           (unsigned int*)workspace, status, (cudaStream_t)stream) != cudaSuccess) {
        (void)cudaGetLastError();
        return MNNLLM_ERR_CUDA;
    }
    return MNNLLM_OK;
}

}  // extern "C"
