// Measurement aid: the rate at which an SM retires tcgen05.mma kind::i8 when nothing else happens.
//
// The prefill path (Section 4.2: W4A8 on integer matrix instructions) is graded against the int8
// tensor rate of the GPU.  This kernel measures that rate directly: one CTA per SM keeps two
// resident 128 x 128-byte operand tiles in shared memory and one thread issues
// 128 x 128 x 32 MMAs (the shape and descriptors of the W4A8 GEMM) back to back into four
// accumulators in tensor memory.  No global memory traffic, no drain, no other warps at work: what
// comes out is the ceiling of the instruction, at the clock the GPU sustains while it runs.
#include <cuda_runtime.h>
#include <stdint.h>

#include "common.h"
#include "ptx.cuh"

namespace mnnllm {

using namespace ptx;

namespace {

constexpr int kTile = 128;                 // MMA M = N = 128, K = 32 per instruction
constexpr int kTileBytes = kTile * 128;    // 128 rows of 128 bytes (four K = 32 steps), 128B swizzle
constexpr uint32_t kCols = 512;            // four 128-column int32 accumulators
constexpr uint32_t kIdesc = (2u << 4) | (0u << 7) | (0u << 10) | ((kTile >> 3) << 17) | ((kTile >> 4) << 24);
constexpr uint32_t kBatch = 64;            // rounds of four MMAs between two bounded waits
constexpr uint32_t kMaxPolls = 1u << 15;

__global__ void __launch_bounds__(128, 1)
mma_i8_ceiling_kernel(unsigned long long rounds, unsigned long long* __restrict__ cycles, uint32_t* __restrict__ status) {
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    __shared__ uint64_t bar;
    __shared__ uint32_t tmem_slot;
    const int warp = threadIdx.x >> 5;

    // operand bytes: a cheap hash, so that the multipliers see changing data (zeros would draw less power)
    for (int i = threadIdx.x; i < 2 * kTileBytes / 4; i += blockDim.x) {
        uint32_t h = (uint32_t)i * 2654435761u + blockIdx.x * 40503u;
        h ^= h >> 15; h *= 2246822519u; h ^= h >> 13;
        reinterpret_cast<uint32_t*>(smem)[i] = h;
    }
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        fence_mbar_init();
    }
    fence_proxy_async_smem();
    if (warp == 1) {
        tmem_alloc(&tmem_slot, kCols);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = tmem_slot;

    if (warp == 0) {
        if (elect_one()) {
            const uint64_t da = desc_sw128(smem_u32(smem)), db = desc_sw128(smem_u32(smem + kTileBytes));
            const long long t0 = clock64();
            uint32_t phase = 0;
            bool ok = true;
            for (unsigned long long r = 0; r < rounds && ok; r += kBatch) {
                const unsigned long long n = rounds - r < kBatch ? rounds - r : kBatch;
                for (unsigned long long i = 0; i < n; ++i) {
                    const uint32_t acc = tmem_base + (uint32_t)(i & 3u) * kTile;
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk)   // the tile's four K = 32 steps, accumulated
                        mma_i8_ss(acc, da + (uint64_t)(kk * 2), db + (uint64_t)(kk * 2), kIdesc, kk > 0);
                }
                mma_commit(&bar);
                if (!mbar_wait_bounded_compact(&bar, phase, kMaxPolls)) {   // never expected: report, stop issuing
                    atomicOr(status, 0x4000u);
                    ok = false;
                }
                phase ^= 1u;
            }
            if (cycles) cycles[blockIdx.x] = (unsigned long long)(clock64() - t0);
        }
        __syncwarp();
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_base, kCols);
}

}  // namespace
}  // namespace mnnllm

using namespace mnnllm;

extern "C" int mnnllm_bench_mma_i8(unsigned long long mmas_per_sm, unsigned long long* cycles_out, void* stream) {
    if (mmas_per_sm < 4 || mmas_per_sm > (1ull << 40)) return MNNLLM_ERR_INVALID_ARG;
    if (!device_is_supported()) return MNNLLM_ERR_UNSUPPORTED;
    uint32_t* status = status_word_ptr();
    const int n_sms = device_sm_count();
    if (!status || n_sms < 1) return MNNLLM_ERR_CUDA;
    const size_t smem = 200 * 1024;   // far more than the two tiles need: one CTA per SM (each takes all of tensor memory)
    static PerDevice<bool> configured;
    if (configured.with([&](bool& done) {
            if (done) return cudaSuccess;
            cudaError_t e = cudaFuncSetAttribute(mma_i8_ceiling_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            done = e == cudaSuccess;
            return e;
        }) != cudaSuccess) {
        (void)cudaGetLastError();
        return MNNLLM_ERR_CUDA;
    }
    mma_i8_ceiling_kernel<<<n_sms, 128, smem, (cudaStream_t)stream>>>(mmas_per_sm / 4, cycles_out, status);
    if (cudaGetLastError() != cudaSuccess) return MNNLLM_ERR_CUDA;
    return MNNLLM_OK;
}
