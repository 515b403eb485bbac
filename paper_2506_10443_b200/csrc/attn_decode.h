// Host interface of the decode attention over a quantised KV cache (internal to the library).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/mnnllm.h"

namespace mnnllm {

constexpr int kAttnHeadDim = 128;      // head_dim the kernels are built for
constexpr int kAttnMaxRep = 8;         // query heads per kv head at most
constexpr int kAttnChunk = 256;        // tokens a CTA handles per step
constexpr int kAttnMinSplit = 128;     // tokens per CTA at least

struct AttnCache {
    uint8_t* k_codes;    // [Hk, S_cap, 128] uint8 codes of the keys
    uint32_t* k_meta;    // [Hk, S_cap] fp16 scale | fp16 zero << 16
    uint8_t* v;          // [Hk, S_cap, 128] E4M3
    int Hk, S_cap;
};

// Quantises one new key (Eq. 1 along head_dim, codes 0..255) and value (E4M3) per kv head and stores
// them at position `pos` of the cache.  k_new, v_new: device fp16 [Hk, 128].
cudaError_t attn_append_launch(const AttnCache& c, const void* k_new, const void* v_new, int pos, cudaStream_t stream);

// out[H, 128] (fp16 or fp32) = softmax(q k_hat^T / sqrt(128)) v over positions [0, S).  partials:
// device scratch of attn_partials_bytes(H, S) bytes; counters: one uint32 per kv head, zero between calls.
size_t attn_partials_bytes(int H, int Hk, int S);
int attn_splits(int Hk, int S);
cudaError_t attn_decode_launch(const AttnCache& c, const void* q, void* out, int out_dtype, int H, int S, float* partials,
                               unsigned int* counters, uint32_t* status, cudaStream_t stream);

}  // namespace mnnllm
