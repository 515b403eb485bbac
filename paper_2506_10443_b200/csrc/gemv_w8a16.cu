// Decode-time W8A16 linear with per-channel int8 weights (Section 4.2: the LM head is kept in int8):
//     y[m, n] = s[n] * (sum_k q[n,k] x[m,k] - z[n] * sum_k x[m,k])
// Same streaming structure as the W4 kernel (per-warp rings of bulk copies, warp-level MMA, sums
// over k-chunks in shared / distributed shared memory).  A quantum is 16 rows x 512 k = 8 KB of
// bytes; a byte becomes the fp16 value 1024 + q with one byte permute per pair, the MMA's 8 columns
// are the tokens, and the 1024 * sum(x) offset is removed once per quantum.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "common.h"
#include "gemv.h"
#include "ptx.cuh"

namespace mnnllm {

using namespace ptx;

namespace {

constexpr uint32_t kMaxPolls = 1u << 15;  // x 20 us per try: gives up after ~0.65 s
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
    const int cl = blockIdx.x / CS;
    const int W = L.WC * L.SR, S = L.stages, SR = L.SR, RBI = L.RBI;
    const GemvProblem& P = L.prob[0];
    const int wc = warp % L.WC, sr = warp / L.WC;

    uint8_t* ring = smem + (size_t)warp * S * QB;
    float* part_all = reinterpret_cast<float*>(smem + (size_t)W * S * QB);   // [W][2][RBI][8][16]
    float* xs_all = part_all + W * 2 * PART_FLOATS;                          // [W][8]
    float* red = xs_all + W * XS_FLOATS;                                     // [2][SR][RBI][8][16]
    float* red_xs = red + 2 * SR * PART_FLOATS;                              // [8]
    uint64_t* bars = reinterpret_cast<uint64_t*>(red_xs + XS_FLOATS) + warp * kGemvMaxStages;

    const int rb_begin = (int)((long long)P.NB * cl / P.n_clusters);
    const int rb_end = (int)((long long)P.NB * (cl + 1) / P.n_clusters);
    const int per_round = SR * RBI;
    const int n_rounds = (rb_end - rb_begin + per_round - 1) / per_round;
    const int jstride = CS * L.WC;
    const int j0 = rank * L.WC + wc;
    const int T = j0 < P.NC ? (P.NC - j0 + jstride - 1) / jstride : 0;
    const int last_ns = P.NS - 16 * (P.NC - 1);

    auto nit_of = [&](int rd) {
        const int first = rb_begin + rd * per_round + sr;
        if (first >= rb_end || T == 0) return 0;
        const int n = (rb_end - first + SR - 1) / SR;
        return n < RBI ? n : RBI;
    };

    if (lane == 0) {
        for (int s = 0; s < S; ++s) mbar_init(&bars[s], 1);
        fence_mbar_init();
    }
    if (lane < XS_FLOATS) xs_all[warp * XS_FLOATS + lane] = 0.f;
    fence_proxy_async_smem();
    __syncwarp();

    int i_rd = 0, i_t = 0, i_it = 0, i_nit = nit_of(0), i_slot = 0;
    while (i_rd < n_rounds && i_nit == 0) { ++i_rd; i_nit = i_rd < n_rounds ? nit_of(i_rd) : 0; }
    const uint64_t stream_policy = policy_evict_first();  // weights are read once: keep them from displacing x in L2
    bool dead = false;   // a bounded wait gave up: nothing more is copied or waited for
    auto issue_next = [&]() {
        if (i_rd >= n_rounds || dead) return;
        const int j = j0 + i_t * jstride;
        const int rb = rb_begin + i_rd * per_round + i_it * SR + sr;
        const int ns = (j == P.NC - 1) ? last_ns : 16;
        const uint32_t bytes = (uint32_t)(ns * kSlabBytes);
        const uint8_t* src = P.packed + kHeaderBytes + (size_t)rb * P.row_block_bytes + (size_t)j * QB;
        mbar_arrive_expect_tx(&bars[i_slot], bytes);
        bulk_g2s_hint(ring + (size_t)i_slot * QB, src, bytes, &bars[i_slot], stream_policy);
        i_slot = (i_slot + 1 == S) ? 0 : i_slot + 1;
        if (++i_it == i_nit) {
            i_it = 0;
            if (++i_t == T) {
                i_t = 0;
                do { ++i_rd; i_nit = i_rd < n_rounds ? nit_of(i_rd) : 0; } while (i_rd < n_rounds && i_nit == 0);
            }
        }
    };

    pdl_launch_dependents();
    if (lane == 0)
        for (int s = 0; s < S; ++s) issue_next();
    pdl_wait();

    uint32_t B[16][2][2];
    float X0 = 0.f, X1 = 0.f;  // sum of x over the current chunk for tokens 2c and 2c + 1
    int cur_j = -1, slot = 0;
    uint32_t phase = 0;
    const int wc_used = (P.NC - rank * L.WC) < L.WC ? (P.NC - rank * L.WC) : L.WC;
    const uint32_t* table = reinterpret_cast<const uint32_t*>(P.packed + P.table_offset);

    for (int rd = 0; rd < n_rounds; ++rd) {
        const int nit = nit_of(rd);
        float* part = part_all + (warp * 2 + (rd & 1)) * PART_FLOATS;
        if (nit > 0)
            for (int t = 0; t < T; ++t) {
                const int j = j0 + t * jstride;
                const int ns = (j == P.NC - 1) ? last_ns : 16;
                if (j != cur_j) {
                    const bool first_visit = (rd == 0);   // chunk sums are recorded once per chunk
                    cur_j = j;
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
                    xsum += __shfl_xor_sync(0xffffffffu, xsum, 2);   // lanes of row r: sum for token r
                    X0 = __shfl_sync(0xffffffffu, xsum, 4 * (2 * c));
                    X1 = __shfl_sync(0xffffffffu, xsum, 4 * (2 * c + 1));
                    if (first_visit && sr == 0 && c == 0) xs_all[warp * XS_FLOATS + r] += xsum;
                }
                for (int it = 0; it < nit; ++it) {
                    if (!dead && !mbar_test_wait(&bars[slot], phase) && !mbar_wait_bounded(&bars[slot], phase, kMaxPolls)) {
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
                                             __byte_perm(w.x, MG, 0x4342), __byte_perm(w.z, MG, 0x4342), B[sl][0][0],
                                             B[sl][0][1]);
                            mma_m16n8k16_f16(D, __byte_perm(w.y, MG, 0x4140), __byte_perm(w.w, MG, 0x4140),
                                             __byte_perm(w.y, MG, 0x4342), __byte_perm(w.w, MG, 0x4342), B[sl][1][0],
                                             B[sl][1][1]);
                        }
                    }
                    __syncwarp();
                    if (lane == 0) {
                        fence_proxy_async_smem();
                        issue_next();
                    }
                    slot = (slot + 1 == S) ? 0 : slot + 1;
                    phase ^= (slot == 0) ? 1u : 0u;
                    // D[2h + e] = sum_k (1024 + q[row r + 8h, k]) x[token 2c + e, k] over this chunk
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        float* dst0 = part + (it * 8 + 2 * c) * 16 + r + 8 * h;
                        float* dst1 = dst0 + 16;
                        const float v0 = D[2 * h] - 1024.f * X0, v1 = D[2 * h + 1] - 1024.f * X1;
                        *dst0 = (t == 0) ? v0 : (*dst0 + v0);
                        *dst1 = (t == 0) ? v1 : (*dst1 + v1);
                    }
                }
            }

        __syncthreads();
        // total sum of x per token over the k-chunks of this CTA (recorded during the first round)
        if (rd == 0 && threadIdx.x < 8) {
            float a = 0.f;
            for (int w = 0; w < wc_used; ++w) a += xs_all[w * XS_FLOATS + threadIdx.x];
            red_xs[threadIdx.x] = a;
        }
        const int n_out = per_round * 8 * 16;
        float* red_rd = red + (rd & 1) * SR * PART_FLOATS;
        for (int o = threadIdx.x; o < n_out; o += blockDim.x) {
            const int it = (o / 128) % RBI, s_r = o / (128 * RBI);
            const int rb = rb_begin + rd * per_round + it * SR + s_r;
            float acc = 0.f;
            if (rb < rb_end)
                for (int w = 0; w < wc_used; ++w)
                    acc += part_all[((s_r * L.WC + w) * 2 + (rd & 1)) * PART_FLOATS + (o % (128 * RBI))];
            red_rd[o] = acc;
        }
        if (CS > 1) cluster_sync(); else __syncthreads();
        for (int o = threadIdx.x * CS + rank; o < n_out; o += blockDim.x * CS) {
            const int row = o & 15, tok = (o >> 4) & 7, it = (o / 128) % RBI, s_r = o / (128 * RBI);
            const int rb = rb_begin + rd * per_round + it * SR + s_r;
            const int n = rb * 16 + row;
            if (rb < rb_end && n < P.N && tok < L.M) {
                float acc = 0.f, xt = 0.f;
                if (CS == 1) {
                    acc = red_rd[o];
                    xt = red_xs[tok];
                } else {
                    for (int cr = 0; cr < CS; ++cr) {
                        acc += ld_dsmem_f32(red_rd + o, (uint32_t)cr);
                        xt += ld_dsmem_f32(red_xs + tok, (uint32_t)cr);
                    }
                }
                const float2 sz = h2f2(table[n]);
                store_out(P.y, P.y_dtype, (size_t)tok * P.N + n, sz.x * (acc - sz.y * xt));
            }
        }
    }
    if (dead)   // copies issued before the give-up may still be in flight into this CTA's shared memory
        for (int i = 0; i < 50; ++i) __nanosleep(1000);
    if (CS > 1) cluster_sync();
}

}  // namespace

static cudaError_t ensure_smem_w8(size_t smem) {
    struct State { size_t configured; bool carveout_set; };
    static PerDevice<State> state;
    return state.with([&](State& st) {
        if (!st.carveout_set) {   // the same carve-out as every other kernel of the library
            cudaError_t e = cudaFuncSetAttribute(gemv_w8a16_kernel, cudaFuncAttributePreferredSharedMemoryCarveout,
                                                 (int)cudaSharedmemCarveoutMaxShared);
            if (e != cudaSuccess) return e;
            st.carveout_set = true;
        }
        if (smem > st.configured) {
            cudaError_t e =
                cudaFuncSetAttribute(gemv_w8a16_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            if (e != cudaSuccess) return e;
            st.configured = smem;
        }
        return cudaSuccess;
    });
}

size_t gemv_w8a16_smem(int W, int SR, int S) {
    return (size_t)W * S * QB + (size_t)(W * 2 * PART_FLOATS + W * XS_FLOATS + 2 * SR * PART_FLOATS + XS_FLOATS) * 4 +
           (size_t)W * kGemvMaxStages * 8;
}

int gemv_w8a16_occupancy(int W, int SR, int S) {
    int n = 0;
    const size_t smem = gemv_w8a16_smem(W, SR, S);
    if (ensure_smem_w8(smem) != cudaSuccess) return 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, gemv_w8a16_kernel, W * 32, smem) != cudaSuccess) return 0;
    return n;
}

cudaError_t gemv_w8a16_launch(const GemvLaunch& L, int n_clusters, int CS, uint32_t* status, cudaStream_t stream) {
    const int W = L.WC * L.SR;
    const size_t smem = gemv_w8a16_smem(W, L.SR, L.stages);
    if (cudaError_t e = ensure_smem_w8(smem); e != cudaSuccess) return e;
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
