// Dynamic per-token int8 activation quantisation, the first kernel of the W4A8 path
// (Section 4.2: per-token int8 activation quantisation).  For every token m:
//     amax = max_k |x[m,k]|,  a_scale = amax / 127,  a_q = clamp(rint(x * (127 / amax)), -127, 127)
// and, for the zero-point correction of the asymmetric weights, the group sums A[m,g] = sum a_q.
// One CTA per token; the row is read twice (the second read hits L2).  HBM-bound and tiny next to
// the GEMM it feeds.
//
// For the GEMM's tensor-core evaluation of the zero-point term sum_g (s z)[n,g] * A[m,g] the group
// sums are also written as fp16 quadruples (64h, l, 64h, l) with A = 64h + l, h = round(A / 64),
// l in [-32, 31]: both parts are exact in fp16 (|A| <= 127 * 128), so the term loses nothing.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "act_quant.h"
#include "common.h"
#include "ptx.cuh"

namespace mnnllm {
namespace {

constexpr int kThreads = 256;

template <typename T>
__device__ __forceinline__ void widen8(const uint4& v, float (&f)[8]);

template <>
__device__ __forceinline__ void widen8<__half>(const uint4& v, float (&f)[8]) {
    const __half2* h = reinterpret_cast<const __half2*>(&v);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float2 t = __half22float2(h[i]);
        f[2 * i] = t.x;
        f[2 * i + 1] = t.y;
    }
}
template <>
__device__ __forceinline__ void widen8<__nv_bfloat16>(const uint4& v, float (&f)[8]) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        f[2 * i] = __uint_as_float(w[i] << 16);
        f[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
    }
}

template <typename T>
__global__ void __launch_bounds__(kThreads) act_quant_kernel(const T* __restrict__ x, int K, int group,
                                                             int8_t* __restrict__ a_q, float* __restrict__ a_scale,
                                                             int32_t* __restrict__ A, uint2* __restrict__ AC, int G4,
                                                             uint32_t code_xor, uint32_t* __restrict__ clear, int n_clear,
                                                             float* __restrict__ sums_t, int32_t* __restrict__ row_sum) {
    __shared__ float warp_max[kThreads / 32];
    __shared__ int warp_tot[kThreads / 32];
    ptx::pdl_launch_dependents();
    ptx::pdl_wait();
    const int m = blockIdx.x;
    for (int i = m * kThreads + threadIdx.x; i < n_clear; i += gridDim.x * kThreads) clear[i] = 0u;
    const uint4* row = reinterpret_cast<const uint4*>(x + (size_t)m * K);
    const int nvec = K / 8;

    float amax = 0.f;
    for (int v = threadIdx.x; v < nvec; v += kThreads) {
        float f[8];
        widen8<T>(row[v], f);
#pragma unroll
        for (int i = 0; i < 8; ++i) amax = fmaxf(amax, fabsf(f[i]));
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
    if ((threadIdx.x & 31) == 0) warp_max[threadIdx.x >> 5] = amax;
    __syncthreads();
    amax = warp_max[0];
#pragma unroll
    for (int w = 1; w < kThreads / 32; ++w) amax = fmaxf(amax, warp_max[w]);

    const float inv = amax > 0.f ? __fdiv_rn(127.0f, amax) : 0.f;
    if (threadIdx.x == 0) a_scale[m] = amax > 0.f ? __fdiv_rn(amax, 127.0f) : 0.f;

    const int lanes_per_group = group / 8;  // 8 or 16 consecutive lanes share a group
    uint2* out = reinterpret_cast<uint2*>(a_q + (size_t)m * K);
    const int G = K / group;
    if (AC != nullptr)  // groups that only pad the row to a multiple of four
        for (int g = G + threadIdx.x; g < G4; g += kThreads) AC[(size_t)m * G4 + g] = make_uint2(0u, 0u);
    int total = 0;   // this thread's share of the row's sum of codes
    for (int v0 = 0; v0 < nvec; v0 += kThreads) {
        const int v = v0 + threadIdx.x;
        int sum = 0;
        if (v < nvec) {
            float f[8];
            widen8<T>(row[v], f);
            int q[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                int c = __float2int_rn(__fmul_rn(f[i], inv));
                c = max(-127, min(127, c));
                q[i] = c;
                sum += c;
            }
            uint2 pk;
            pk.x = (uint32_t)(q[0] & 0xFF) | ((uint32_t)(q[1] & 0xFF) << 8) | ((uint32_t)(q[2] & 0xFF) << 16) |
                   ((uint32_t)(q[3] & 0xFF) << 24);
            pk.y = (uint32_t)(q[4] & 0xFF) | ((uint32_t)(q[5] & 0xFF) << 8) | ((uint32_t)(q[6] & 0xFF) << 16) |
                   ((uint32_t)(q[7] & 0xFF) << 24);
            // code_xor = 0x80808080 stores a_q + 128 as unsigned bytes (the GEMM's operand form)
            pk.x ^= code_xor;
            pk.y ^= code_xor;
            out[v] = pk;
            total += sum;
        }
        // group sums: a group is 8 (or 16) consecutive vectors, i.e. consecutive lanes of one warp
        sum += __shfl_xor_sync(0xffffffffu, sum, 1);
        sum += __shfl_xor_sync(0xffffffffu, sum, 2);
        sum += __shfl_xor_sync(0xffffffffu, sum, 4);
        if (lanes_per_group == 16) sum += __shfl_xor_sync(0xffffffffu, sum, 8);
        if (v < nvec && (threadIdx.x % lanes_per_group) == 0) {
            const int g = v / lanes_per_group;
            if (g < G) {
                if (A != nullptr) A[(size_t)m * G + g] = sum;
                if (sums_t != nullptr) sums_t[(size_t)g * 64 + m] = (float)sum;   // [G][64], for at most 64 tokens
                if (AC != nullptr) {
                    const int h = (sum + 32) >> 6;  // floor((sum + 32) / 64)
                    const int l = sum - 64 * h;
                    const __half2 hl = __floats2half2_rn((float)(64 * h), (float)l);
                    const uint32_t bits = *reinterpret_cast<const uint32_t*>(&hl);
                    AC[(size_t)m * G4 + g] = make_uint2(bits, bits);
                }
            }
        }
    }
    if (row_sum != nullptr) {   // sum_k a_q[m, k]: the zero-point factor of a per-channel weight matrix
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) total += __shfl_xor_sync(0xffffffffu, total, o);
        if ((threadIdx.x & 31) == 0) warp_tot[threadIdx.x >> 5] = total;
        __syncthreads();
        if (threadIdx.x == 0) {
            int t = 0;
#pragma unroll
            for (int w = 0; w < kThreads / 32; ++w) t += warp_tot[w];
            row_sum[m] = t;
        }
    }
}

}  // namespace

cudaError_t act_quant_launch(const void* x, int x_dtype, int M, int K, int group, int8_t* a_q, float* a_scale,
                             int32_t* A, void* AC, bool offset128, uint32_t* clear, int n_clear, cudaStream_t stream,
                             float* sums_t, int32_t* row_sum) {
    if (sums_t && M > 64) return cudaErrorInvalidValue;
    if (!clear) n_clear = 0;
    static PerDevice<bool> carveout_set;
    (void)carveout_set.with([](bool& done) {
        if (!done) {
            // the GEMM that follows needs the largest shared-memory carve-out: ask for the same here, so
            // that the SMs are not re-partitioned between the two kernels of a call
            cudaFuncSetAttribute(act_quant_kernel<__half>, cudaFuncAttributePreferredSharedMemoryCarveout,
                                 (int)cudaSharedmemCarveoutMaxShared);
            cudaFuncSetAttribute(act_quant_kernel<__nv_bfloat16>, cudaFuncAttributePreferredSharedMemoryCarveout,
                                 (int)cudaSharedmemCarveoutMaxShared);
            (void)cudaGetLastError();
            done = true;
        }
        return cudaSuccess;
    });
    const uint32_t code_xor = offset128 ? 0x80808080u : 0u;
    const int G4 = (K / group + 3) / 4 * 4;
    uint2* ac = reinterpret_cast<uint2*>(AC);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)M);
    cfg.blockDim = dim3(kThreads);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (x_dtype == MNNLLM_F16)
        return cudaLaunchKernelEx(&cfg, act_quant_kernel<__half>, (const __half*)x, K, group, a_q, a_scale, A, ac,
                                  G4, code_xor, clear, n_clear, sums_t, row_sum);
    return cudaLaunchKernelEx(&cfg, act_quant_kernel<__nv_bfloat16>, (const __nv_bfloat16*)x, K, group, a_q, a_scale,
                              A, ac, G4, code_xor, clear, n_clear, sums_t, row_sum);
}

}  // namespace mnnllm
