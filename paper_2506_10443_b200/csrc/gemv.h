// Host/device interface of the decode GEMV kernels (internal to the library).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/mnnllm.h"
#include "layout.h"

namespace mnnllm {

constexpr int kGemvMaxWarps = 7;    // warps per CTA (7 * 32 threads leave 144 registers each at 2 CTAs per SM)
constexpr int kGemvMaxStages = 4;   // ring slots per warp
constexpr int kGemvMaxRBI = 8;      // 16-row blocks a warp walks through per k-chunk

struct GemvProblem {
    const uint8_t* packed;  // start of the packed buffer (header included)
    const __half* x;        // [M, K]
    void* y;                // [M, N]
    int N, K;
    int NB, NC, NS;         // 16-row blocks, 512-k chunks, slabs per row
    int cluster_begin;      // first cluster of this problem in the launch
    int n_clusters;         // clusters that share this problem's row blocks evenly
    int y_dtype;
    int x_dtype;            // MNNLLM_F16, or MNNLLM_BF16 (converted to fp16 as the fragments are built)
    unsigned long long row_block_bytes;
    unsigned long long table_offset;  // W8: per-row (scale, zero) table, from the buffer start
    // LoRA bypass (W4 kernel, instantiations with LORA; lora_r == 0: none):
    // y[m, n] += sum_j lora_A[n, j] * t[m, j], t[m, j] = sum_k lora_B[j, k] x[m, k].  The launch's own CTAs
    // compute t into lora_t as 8-byte {value, tag} words, tag = lora_sync[0] + 1 (the epoch); lora_sync[1]
    // counts the CTAs that are through, the last one moves the epoch on.
    const __half* lora_A;   // [N, lora_r]
    const __half* lora_B;   // [lora_r, K]
    float* lora_t;          // [M, lora_r] x 8 bytes
    unsigned int* lora_sync;
    int lora_r;
};

struct GemvLaunch {
    GemvProblem prob[MNNLLM_MAX_BATCH];
    int count;
    int M;       // tokens (<= MP of the instantiation)
    int WC, SR;  // warps per CTA = WC (k-chunk lanes) * SR (row-block lanes)
    int RBI;     // row blocks a warp walks per k-chunk and round
    int stages;
};

size_t gemv_w4a16_smem(int group, int MP, int W, int SR, int S);
// resident CTAs per SM for this configuration (queries the runtime; 0 on error)
int gemv_w4a16_occupancy(int group, int MP, int W, int SR, int S);
cudaError_t gemv_w4a16_launch(const GemvLaunch& L, int group, int MP, int n_clusters, int CS, uint32_t* status,
                              cudaStream_t stream);

size_t gemv_w8a16_smem(int W, int SR, int S);
int gemv_w8a16_occupancy(int W, int SR, int S);
cudaError_t gemv_w8a16_launch(const GemvLaunch& L, int n_clusters, int CS, uint32_t* status, cudaStream_t stream);

}  // namespace mnnllm
