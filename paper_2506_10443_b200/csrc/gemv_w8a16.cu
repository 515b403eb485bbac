// Decode-time W8A16 linear with per-channel int8 weights (Section 4.2: the LM head is kept in int8):
//     y[m, n] = s[n] * (sum_k q[n,k] x[m,k] - z[n] * sum_k x[m,k])
// Same streaming structure as the W4 kernel (per-warp rings of bulk copies, warp-level MMA, sums
// over k-chunks in shared / distributed shared memory).  A quantum is 16 rows x 512 k = 8 KB of
// bytes; a byte becomes the fp16 value 1024 + q with one byte permute per pair, the MMA's 8 columns
// are the tokens, and the 1024 * sum(x) offset is removed once per quantum.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "gemv.h"
#include "ptx.cuh"

namespace mnnllm {

using namespace ptx;

namespace {

constexpr uint32_t kMaxPolls = 1u << 22;
constexpr int QB = 16 * kSlabBytes;                 // bytes of a full quantum
constexpr int PART_FLOATS = kGemvMaxRBI * 8 * 16;   // [it][token][row]
constexpr int XS_FLOATS = 8;                        // per warp: sum of x over its chunks, per token

__device__ __forceinline__ float2 h2f2(uint32_t u) {
    return __half22float2(*reinterpret_cast<const __half2*>(&u));
}
__device__ __forceinline__ void store_out(void* y, int dtype, size_t idx, float v) {
    if (dtype == MNNLLM_F16) reinterpret_cast<__half*>(y)[idx] = __float2half_rn(v);
    else if (dtype == MNNLLM_BF16) reinterpret_cast<__nv_bfloat16*>(y)[idx] = __float2bfloat16_rn(v);
    else reinterpret_cast<float*>(y)[idx] = v;
}

__global__ void __launch_bounds__(kGemvMaxWarps * 32, 1)
gemv_w8a16_kernel(const __grid_constant__ GemvLaunch L, uint32_t* __restrict__ status) {
    extern __shared__ __align__(128) uint8_t smem[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int r = lane >> 2, c = lane & 3;
    const int CS = (int)cluster_nctarank(), rank = (int)cluster_ctarank();
    const int cluster_id = blockIdx.x / CS;
    const int W = L.WC * L.SR, S = L.stages;
    const GemvProblem& P = L.prob[0];
    const int cl = cluster_id;
    const int wc = warp % L.WC, sr = warp / L.WC;

    uint8_t* ring = smem + (size_t)warp * S * QB;
    float* part_all = reinterpret_cast<float*>(smem + (size_t)W * S * QB);
    float* part = part_all + warp * PART_FLOATS;
    float* xs_all = part_all + W * PART_FLOATS;      // [W][8]
    float* red = xs_all + W * XS_FLOATS;             // [SR][RBI][8][16]
    float* red_xs = red + L.SR * PART_FLOATS;        // [8]
    uint64_t* bars = reinterpret_cast<uint64_t*>(red_xs + XS_FLOATS) + warp * kGemvMaxStages;

    const int rb0 = cl * (L.SR * P.RBI) + sr;
    int rbi_eff = 0;
    if (rb0 < P.NB) {
        rbi_eff = (P.NB - rb0 + L.SR - 1) / L.SR;
        rbi_eff = rbi_eff < P.RBI ? rbi_eff : P.RBI;
    }
    const int jstride = CS * L.WC;
    const int j0 = rank * L.WC + wc;
    const int T = j0 < P.NC ? (P.NC - j0 + jstride - 1) / jstride : 0;
    const int Q = T * rbi_eff;
    const int last_ns = P.NS - 16 * (P.NC - 1);

    if (lane == 0) {
        for (int s = 0; s < S; ++s) mbar_init(&bars[s], 1);
        fence_mbar_init();
    }
    if (lane < XS_FLOATS) xs_all[warp * XS_FLOATS + lane] = 0.f;
    fence_proxy_async_smem();
    __syncwarp();

    auto issue = [&](int q) {
        const int t = q / rbi_eff, it = q - t * rbi_eff;
        const int j = j0 + t * jstride;
        const int rb = rb0 + it * L.SR;
        const int ns = (j == P.NC - 1) ? last_ns : 16;
        const uint32_t bytes = (uint32_t)(ns * kSlabBytes);
        const uint8_t* src = P.packed + kHeaderBytes + (size_t)rb * P.row_block_bytes + (size_t)j * QB;
        const int slot = q % S;
        mbar_arrive_expect_tx(&bars[slot], bytes);
        bulk_g2s(ring + (size_t)slot * QB, src, bytes, &bars[slot]);
    };

    pdl_launch_dependents();
    if (lane == 0) {
        const int pre = Q < S ? Q : S;
        for (int q = 0; q < pre; ++q) issue(q);
    }
    pdl_wait();

    uint32_t B[16][2][2];
    float X0 = 0.f, X1 = 0.f;  // sum of x over the current chunk for tokens 2c and 2c + 1
    bool dead = false;

    for (int q = 0; q < Q; ++q) {
        const int t = q / rbi_eff, it = q - t * rbi_eff;
        const int j = j0 + t * jstride;
        const int ns = (j == P.NC - 1) ? last_ns : 16;

        if (it == 0) {
            const __half* xk = P.x + (size_t)j * kChunkK;
            float xsum = 0.f;
#pragma unroll
            for (int sl = 0; sl < 16; ++sl) {
                uint4 u = make_uint4(0, 0, 0, 0);
                if (sl < ns && r < L.M)
                    u = *reinterpret_cast<const uint4*>(xk + (size_t)r * P.K + sl * kSlabK8 + 8 * c);
                B[sl][0][0] = u.x; B[sl][0][1] = u.y; B[sl][1][0] = u.z; B[sl][1][1] = u.w;
                float2 f;
                f = h2f2(u.x); xsum += f.x + f.y;
                f = h2f2(u.y); xsum += f.x + f.y;
                f = h2f2(u.z); xsum += f.x + f.y;
                f = h2f2(u.w); xsum += f.x + f.y;
            }
            xsum += __shfl_xor_sync(0xffffffffu, xsum, 1);
            xsum += __shfl_xor_sync(0xffffffffu, xsum, 2);   // lanes of row r hold sum for token r
            X0 = __shfl_sync(0xffffffffu, xsum, 4 * (2 * c));
            X1 = __shfl_sync(0xffffffffu, xsum, 4 * (2 * c + 1));
            if (sr == 0 && c == 0) xs_all[warp * XS_FLOATS + r] += xsum;  // this warp, token r
        }

        const int slot = q % S;
        if (!dead && !mbar_wait_bounded(&bars[slot], (uint32_t)((q / S) & 1), kMaxPolls)) {
            dead = true;
            if (lane == 0) atomicOr(status, 0x200u);
        }
        const uint4* slabs = reinterpret_cast<const uint4*>(ring + (size_t)slot * QB);
        float D[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int sl = 0; sl < 16; ++sl) {
            if (sl < ns) {
                const uint4 w = slabs[sl * 32 + lane];
                constexpr uint32_t MG = 0x64646464u;
                mma_m16n8k16_f16(D, __byte_perm(w.x, MG, 0x4140), __byte_perm(w.z, MG, 0x4140),
                                 __byte_perm(w.x, MG, 0x4342), __byte_perm(w.z, MG, 0x4342), B[sl][0][0], B[sl][0][1]);
                mma_m16n8k16_f16(D, __byte_perm(w.y, MG, 0x4140), __byte_perm(w.w, MG, 0x4140),
                                 __byte_perm(w.y, MG, 0x4342), __byte_perm(w.w, MG, 0x4342), B[sl][1][0], B[sl][1][1]);
            }
        }
        // D[2h + e] = sum_k (1024 + q[row r + 8h, k]) x[token 2c + e, k] over this chunk
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            float* dst0 = part + (it * 8 + 2 * c) * 16 + r + 8 * h;
            float* dst1 = dst0 + 16;
            const float v0 = D[2 * h] - 1024.f * X0, v1 = D[2 * h + 1] - 1024.f * X1;
            *dst0 = (t == 0) ? v0 : (*dst0 + v0);
            *dst1 = (t == 0) ? v1 : (*dst1 + v1);
        }
        __syncwarp();
        if (lane == 0 && q + S < Q) {
            fence_proxy_async_smem();
            issue(q + S);
        }
    }

    __syncthreads();
    const int n_out = L.SR * P.RBI * 8 * 16;
    const int wc_used = (P.NC - rank * L.WC) < L.WC ? (P.NC - rank * L.WC) : L.WC;
    const uint32_t* table = reinterpret_cast<const uint32_t*>(P.packed + P.table_offset);
    // total sum of x per token over the chunks of this CTA (sub-range 0 warps recorded them)
    if (threadIdx.x < 8) {
        float a = 0.f;
        for (int w = 0; w < wc_used; ++w) a += xs_all[w * XS_FLOATS + threadIdx.x];
        red_xs[threadIdx.x] = a;
    }
    for (int o = threadIdx.x; o < n_out; o += blockDim.x) {
        const int it = (o / 128) % P.RBI, s_r = o / (128 * P.RBI);
        const int rb = cl * (L.SR * P.RBI) + s_r + it * L.SR;
        float acc = 0.f;
        if (rb < P.NB)
            for (int w = 0; w < wc_used; ++w) acc += part_all[(s_r * L.WC + w) * PART_FLOATS + (o % (128 * P.RBI)) ];
        red[o] = acc;
    }
    __syncthreads();
    if (CS > 1) cluster_sync();
    for (int o = threadIdx.x * CS + rank; o < n_out; o += blockDim.x * CS) {
        const int row = o & 15, tok = (o >> 4) & 7, it = (o / 128) % P.RBI, s_r = o / (128 * P.RBI);
        const int rb = cl * (L.SR * P.RBI) + s_r + it * L.SR;
        const int n = rb * 16 + row;
        if (rb < P.NB && n < P.N && tok < L.M) {
            float acc = 0.f, xt = 0.f;
            if (CS == 1) {
                acc = red[o];
                xt = red_xs[tok];
            } else {
                for (int cr = 0; cr < CS; ++cr) {
                    acc += ld_dsmem_f32(red + o, (uint32_t)cr);
                    xt += ld_dsmem_f32(red_xs + tok, (uint32_t)cr);
                }
            }
            const float2 sz = h2f2(table[n]);
            store_out(P.y, P.y_dtype, (size_t)tok * P.N + n, sz.x * (acc - sz.y * xt));
        }
    }
    if (CS > 1) cluster_sync();
}

}  // namespace

size_t gemv_w8a16_smem(int W, int SR, int S) {
    return (size_t)W * S * QB + (size_t)(W * PART_FLOATS + W * XS_FLOATS + SR * PART_FLOATS + XS_FLOATS) * 4 +
           (size_t)W * kGemvMaxStages * 8;
}

cudaError_t gemv_w8a16_launch(const GemvLaunch& L, int n_clusters, int CS, uint32_t* status, cudaStream_t stream) {
    const int W = L.WC * L.SR;
    const size_t smem = gemv_w8a16_smem(W, L.SR, L.stages);
    static size_t configured = 0;
    if (smem > configured) {
        cudaError_t e = cudaFuncSetAttribute(gemv_w8a16_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        configured = smem;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(n_clusters * CS));
    cfg.blockDim = dim3((unsigned)(W * 32));
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)CS;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, gemv_w8a16_kernel, L, status);
}

}  // namespace mnnllm
