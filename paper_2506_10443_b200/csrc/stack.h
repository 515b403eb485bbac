// Whole-stack W4A16 decode in ONE persistent launch: plan blob, workspace layout and the host/device
// interface of the kernel (internal to the library).
//
// A "plan" is built on the host from the caller's problem list, copied to the device by the caller
// (like packed weights) and read by every CTA.  The workspace holds the cross-CTA state:
//   word 0        epoch: number of launches that have completed on this workspace
//   word 1        CTAs of the running launch that have finished
//   flags[p]      row blocks of problem p stored so far, summed over all launches: problem p of
//                 launch number e (0-based) is complete when flags[p] == (e + 1) * NB_p (mod 2^32)
//   parts         per (problem, CTA): 16 rows x MP tokens of 8-byte words {fp32 partial sum, tag}
//                 through which the CTAs that share a 16-row block exchange their partial sums; a
//                 word is valid for launch e when its tag equals e + 1
// Nothing is ever cleared: the workspace has to be all zero before its first launch only.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/mnnllm.h"
#include "layout.h"

namespace mnnllm {

constexpr uint32_t kStackMagic = 0x4B54534Du;  // "MSTK"
constexpr int kStackMaxDeps = 4;
constexpr int kStackConsumerWarps = 14;   // + producer warp + signaller warp: 512 threads, 128 registers each
constexpr int kStackThreads = (kStackConsumerWarps + 2) * 32;

constexpr int kStackMaxSub = 4;           // weight matrices fused into one problem (q+k+v, gate+up)

// One problem of the plan: up to kStackMaxSub weight matrices that multiply the same activations and
// wait for the same predecessors; their 16-row blocks are numbered through (matrix 0 first).
struct StackProblem {            // 192 bytes, 16-byte aligned
    const uint8_t* packed[kStackMaxSub];   // packed buffers (header included)
    void* y[kStackMaxSub];                 // [M, N[i]] of the matrix's output dtype
    const void* x;                         // fp16 [M, K]
    unsigned long long row_block_bytes;
    int N[kStackMaxSub];
    int nb_end[kStackMaxSub];    // row blocks of matrices 0..i (cumulative); unused entries = NB
    int K;
    int NB, NC, NS;              // 16-row blocks (all matrices), 512-k chunks, 64-k slabs per row
    int gran;                    // CTAs receive runs of quanta that are multiples of gran (1 or NC)
    int rot;                     // CTA `cta` plays the role of virtual CTA (cta - rot) mod n_ctas
    int weff;                    // consumer warps used (a multiple of NC where NC <= the warp count)
    int y_dtypes;                // output dtype of matrix i in bits 8i .. 8i+7
    int n_deps;
    int stage_x;                 // 1: the CTA copies the k-chunks of x it needs to shared memory first
    int deps[kStackMaxDeps];     // earlier problems (of the plan) that must be complete before x is read
    int deps_nb[kStackMaxDeps];  // their row-block counts (the completion counter's increment per launch)
    int pad[2];
};
static_assert(sizeof(StackProblem) == 192, "descriptor is 192 bytes");

struct StackHeader {             // 64 bytes
    uint32_t magic, version;
    int32_t count, M, group, MP; // count = problems of the plan (after fusing matrices that share x)
    int32_t n_ctas;              // grid size the plan was made for
    int32_t ring_slots;          // quanta slots of the shared-memory ring, a multiple of the consumer warps
    int32_t max_quanta;          // most quanta one CTA holds of any one problem
    uint32_t smem_bytes;
    uint32_t xs_bytes;           // shared memory for staged activations
    uint32_t reserved[5];
};
static_assert(sizeof(StackHeader) == 64, "header is 64 bytes");

struct StackWorkspace {          // device pointers into the caller's workspace
    uint32_t* epoch;
    uint32_t* done;
    uint32_t* flags;             // [count]
    unsigned long long* parts;   // [count][n_ctas][MP][16]
};

// byte offsets inside the workspace
inline size_t stack_ws_flags_offset() { return 256; }
inline size_t stack_ws_parts_offset(int count) { return 256 + (((size_t)count * 4 + 255) & ~(size_t)255); }
inline size_t stack_ws_bytes(int count, int n_ctas, int MP) {
    return stack_ws_parts_offset(count) + (size_t)count * n_ctas * MP * 16 * 8;
}

cudaError_t stack_w4a16_launch(const StackHeader& H, const void* plan_dev, const StackWorkspace& ws, uint32_t* status,
                               cudaStream_t stream);
// shared memory of one CTA: the plan's `count` descriptors, a ring of `slots` quanta, the
// partial sums of `max_quanta` quanta and `xs_bytes` of staged activations
size_t stack_w4a16_smem(int group, int MP, int count, int slots, int max_quanta, int xs_bytes);

}  // namespace mnnllm
