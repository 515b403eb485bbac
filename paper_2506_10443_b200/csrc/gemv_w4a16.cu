// Decode-time W4A16 linear (M <= 8 tokens per pass): y[m, n] = sum_g s[n,g] * sum_{k in g} (q[n,k] - z[n,g]) x[m,k]
// (Section 4.2, W4A16 on GPUs).  The kernel is bound by HBM: every packed weight byte is read once.
//
// Design (one warp = one stream of "quanta", a quantum = 16 rows x 512 k of packed weights):
//   * a warp keeps ONE k-chunk of activations in registers as the B operand of the warp-level MMA
//     and streams the quanta of that chunk for a run of 16-row blocks through a private ring of
//     shared-memory slots filled by bulk (TMA) copies, each completing on its own mbarrier;
//   * codes become fp16 operands with one logic op per pair: (w & 0x000F000F) | 0x6400 is the pair
//     (1024 + q, 1024 + q') and (w & 0x00F000F0) | 0x5400 is (64 + q, 64 + q'), both exact;
//   * the MMA's 8 output columns are (token, group) pairs: a group's k only meet the activations of
//     the column that belongs to that group (the other columns hold zeros), so one accumulator
//     tile collects the raw sums of up to 8 groups and is rescaled once per quantum:
//         y += s * (D - (1024 X_lo + 64 X_hi) - z (X_lo + X_hi)),  X = sums of x over the group's k
//   * partial results of the warps (different k-chunks of the same rows) are summed in shared
//     memory, and across the CTAs of a thread-block cluster through distributed shared memory,
//     so split-K needs neither atomics nor scratch memory.
//   * programmatic dependent launch: the weight ring is filled BEFORE griddepcontrol.wait, the
//     activations are read after it, so HBM keeps streaming across dependent launches.
#include <cuda_fp16.h>
#include <cuda_bf16.h>

#include "gemv.h"
#include "ptx.cuh"

namespace mnnllm {

using namespace ptx;

namespace {

constexpr uint32_t kMaxPolls = 1u << 22;

template <int GROUP, int MP>
struct Cfg {
    static constexpr int GC = kChunkK / GROUP;           // groups per full chunk (8 or 4)
    static constexpr int SPG = GROUP / kSlabK4;          // slabs per group (1 or 2)
    static constexpr int GPS = 8 / MP;                   // group slots per accumulator tile
    static constexpr int NSETS = (GC + GPS - 1) / GPS;   // accumulator tiles per quantum
    static constexpr int QB = 8 * kSlabBytes + 16 * GC * 4;  // bytes of a full quantum
    static constexpr int CORR_FLOATS = MP * GC * 2;
    static constexpr int PART_FLOATS = kGemvMaxRBI * MP * 16;
};

__device__ __forceinline__ float2 h2f2(uint32_t u) {
    return __half22float2(*reinterpret_cast<const __half2*>(&u));
}

__device__ __forceinline__ void store_out(void* y, int dtype, size_t idx, float v) {
    if (dtype == MNNLLM_F16) reinterpret_cast<__half*>(y)[idx] = __float2half_rn(v);
    else if (dtype == MNNLLM_BF16) reinterpret_cast<__nv_bfloat16*>(y)[idx] = __float2bfloat16_rn(v);
    else reinterpret_cast<float*>(y)[idx] = v;
}

template <int GROUP, int MP>
__global__ void __launch_bounds__(kGemvMaxWarps * 32, 1)
gemv_w4a16_kernel(const __grid_constant__ GemvLaunch L, uint32_t* __restrict__ status) {
    using C = Cfg<GROUP, MP>;
    extern __shared__ __align__(128) uint8_t smem[];

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int r = lane >> 2, c = lane & 3;
    const int CS = (int)cluster_nctarank(), rank = (int)cluster_ctarank();
    const int cluster_id = blockIdx.x / CS;
    const int W = L.WC * L.SR, S = L.stages;

    int pi = 0;
    while (pi + 1 < L.count && cluster_id >= L.prob[pi + 1].cluster_begin) ++pi;
    const GemvProblem& P = L.prob[pi];
    const int cl = cluster_id - P.cluster_begin;
    const int wc = warp % L.WC, sr = warp / L.WC;

    // shared memory carve-up (all offsets multiples of 128 B)
    uint8_t* ring = smem + (size_t)warp * S * C::QB;
    float* corr = reinterpret_cast<float*>(smem + (size_t)W * S * C::QB) + warp * C::CORR_FLOATS;
    float* part_all = reinterpret_cast<float*>(smem + (size_t)W * S * C::QB) + W * C::CORR_FLOATS;
    float* part = part_all + warp * C::PART_FLOATS;
    float* red = part_all + W * C::PART_FLOATS;  // [SR][RBI][MP][16]
    uint64_t* bars = reinterpret_cast<uint64_t*>(red + L.SR * C::PART_FLOATS) + warp * kGemvMaxStages;

    // this warp's work: chunks j = rank*WC + wc + t*CS*WC, row blocks rb = rb0 + it*SR
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
    const uint32_t full_chunk_bytes = (uint32_t)C::QB;
    const int last_ns = P.NS - 8 * (P.NC - 1);  // slabs in the last chunk

    if (lane == 0) {
        for (int s = 0; s < S; ++s) mbar_init(&bars[s], 1);
        fence_mbar_init();
    }
    fence_proxy_async_smem();
    __syncwarp();

    auto issue = [&](int q) {  // lane 0 only
        const int t = q / rbi_eff, it = q - t * rbi_eff;
        const int j = j0 + t * jstride;
        const int rb = rb0 + it * L.SR;
        const int ns = (j == P.NC - 1) ? last_ns : 8;
        const uint32_t bytes = (uint32_t)(ns * kSlabBytes + 16 * (ns / C::SPG) * 4);
        const uint8_t* src = P.packed + kHeaderBytes + (size_t)rb * P.row_block_bytes + (size_t)j * full_chunk_bytes;
        const int slot = q % S;
        mbar_arrive_expect_tx(&bars[slot], bytes);
        bulk_g2s(ring + (size_t)slot * C::QB, src, bytes, &bars[slot]);
    };

    pdl_launch_dependents();
    if (lane == 0) {
        const int pre = Q < S ? Q : S;
        for (int q = 0; q < pre; ++q) issue(q);
    }
    // everything above touched only weights; the activations may come from the previous kernel
    pdl_wait();

    const int tokB = r % MP, gsB = r / MP;  // B-operand role of this lane: column r of the MMA
    uint32_t B[8][4][2];
    float C1[C::NSETS][2], C2[C::NSETS][2];
    bool dead = false;

    for (int q = 0; q < Q; ++q) {
        const int t = q / rbi_eff, it = q - t * rbi_eff;
        const int j = j0 + t * jstride;
        const int ns = (j == P.NC - 1) ? last_ns : 8;
        const int ng = ns / C::SPG;

        if (it == 0) {
            // ---- new k-chunk: activations -> B fragments, group sums -> correction terms ----
            const __half* xk = P.x + (size_t)j * kChunkK;
#pragma unroll
            for (int sl = 0; sl < 8; ++sl) {
                uint4 u0 = make_uint4(0, 0, 0, 0), u1 = u0;
                const int gi = sl / C::SPG;
                const bool mine = (sl < ns) && (tokB < L.M) && (gsB == gi % C::GPS);
                if (mine) {
                    const uint4* px = reinterpret_cast<const uint4*>(xk + (size_t)tokB * P.K + sl * kSlabK4 + 16 * c);
                    u0 = px[0];
                    u1 = px[1];
                }
                B[sl][0][0] = __byte_perm(u0.x, u0.y, 0x5410);
                B[sl][0][1] = __byte_perm(u0.z, u0.w, 0x5410);
                B[sl][1][0] = __byte_perm(u0.x, u0.y, 0x7632);
                B[sl][1][1] = __byte_perm(u0.z, u0.w, 0x7632);
                B[sl][2][0] = __byte_perm(u1.x, u1.y, 0x5410);
                B[sl][2][1] = __byte_perm(u1.z, u1.w, 0x5410);
                B[sl][3][0] = __byte_perm(u1.x, u1.y, 0x7632);
                B[sl][3][1] = __byte_perm(u1.z, u1.w, 0x7632);
            }
            __syncwarp();  // the previous chunk's correction terms are no longer read
#pragma unroll
            for (int i = 0; i < C::NSETS; ++i) {
                const int gi = gsB + C::GPS * i;
                float lo = 0.f, hi = 0.f;
                if (gi < ng && tokB < L.M) {
#pragma unroll
                    for (int sp = 0; sp < C::SPG; ++sp) {
                        const uint4* px = reinterpret_cast<const uint4*>(
                            xk + (size_t)tokB * P.K + (gi * C::SPG + sp) * kSlabK4 + 16 * c);
                        const uint4 u0 = px[0], u1 = px[1];
                        float2 f;
                        f = h2f2(u0.x); lo += f.x + f.y;
                        f = h2f2(u0.y); lo += f.x + f.y;
                        f = h2f2(u1.x); lo += f.x + f.y;
                        f = h2f2(u1.y); lo += f.x + f.y;
                        f = h2f2(u0.z); hi += f.x + f.y;
                        f = h2f2(u0.w); hi += f.x + f.y;
                        f = h2f2(u1.z); hi += f.x + f.y;
                        f = h2f2(u1.w); hi += f.x + f.y;
                    }
                }
                lo += __shfl_xor_sync(0xffffffffu, lo, 1);
                hi += __shfl_xor_sync(0xffffffffu, hi, 1);
                lo += __shfl_xor_sync(0xffffffffu, lo, 2);
                hi += __shfl_xor_sync(0xffffffffu, hi, 2);
                if (c == 0 && gi < C::GC) {
                    corr[(tokB * C::GC + gi) * 2 + 0] = 1024.f * lo + 64.f * hi;
                    corr[(tokB * C::GC + gi) * 2 + 1] = lo + hi;
                }
            }
            __syncwarp();
#pragma unroll
            for (int s = 0; s < C::NSETS; ++s)
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const int col = 2 * c + e;
                    const int gi = s * C::GPS + col / MP;
                    const bool ok = gi < C::GC;
                    C1[s][e] = ok ? corr[((col % MP) * C::GC + gi) * 2 + 0] : 0.f;
                    C2[s][e] = ok ? corr[((col % MP) * C::GC + gi) * 2 + 1] : 0.f;
                }
        }

        // ---- wait for this quantum's bulk copy ----
        const int slot = q % S;
        if (!dead && !mbar_wait_bounded(&bars[slot], (uint32_t)((q / S) & 1), kMaxPolls)) {
            dead = true;
            if (lane == 0) atomicOr(status, 0x100u | (uint32_t)pi);
        }
        const uint8_t* qp = ring + (size_t)slot * C::QB;
        const uint4* slabs = reinterpret_cast<const uint4*>(qp);

        float D[C::NSETS][4];
#pragma unroll
        for (int s = 0; s < C::NSETS; ++s) D[s][0] = D[s][1] = D[s][2] = D[s][3] = 0.f;

#pragma unroll
        for (int sl = 0; sl < 8; ++sl) {
            if (sl < ns) {
                const uint4 w = slabs[sl * 32 + lane];
                constexpr uint32_t LO = 0x000F000Fu, HI = 0x00F000F0u, M1024 = 0x64006400u, M64 = 0x54005400u;
                const int set = (sl / C::SPG) / C::GPS;
                mma_m16n8k16_f16(D[set], lop3_and_or(w.x, LO, M1024), lop3_and_or(w.z, LO, M1024),
                                 lop3_and_or(w.x, HI, M64), lop3_and_or(w.z, HI, M64), B[sl][0][0], B[sl][0][1]);
                const uint32_t x8 = w.x >> 8, z8 = w.z >> 8;
                mma_m16n8k16_f16(D[set], lop3_and_or(x8, LO, M1024), lop3_and_or(z8, LO, M1024),
                                 lop3_and_or(x8, HI, M64), lop3_and_or(z8, HI, M64), B[sl][1][0], B[sl][1][1]);
                mma_m16n8k16_f16(D[set], lop3_and_or(w.y, LO, M1024), lop3_and_or(w.w, LO, M1024),
                                 lop3_and_or(w.y, HI, M64), lop3_and_or(w.w, HI, M64), B[sl][2][0], B[sl][2][1]);
                const uint32_t y8 = w.y >> 8, w8 = w.w >> 8;
                mma_m16n8k16_f16(D[set], lop3_and_or(y8, LO, M1024), lop3_and_or(w8, LO, M1024),
                                 lop3_and_or(y8, HI, M64), lop3_and_or(w8, HI, M64), B[sl][3][0], B[sl][3][1]);
            }
        }

        // ---- rescale: column (2c + e) of tile s is (token, group) = (col % MP, s*GPS + col / MP) ----
        const uint32_t* table = reinterpret_cast<const uint32_t*>(qp + (size_t)ns * kSlabBytes);
        float out[2][2] = {{0.f, 0.f}, {0.f, 0.f}};  // [row half h][column e]
#pragma unroll
        for (int s = 0; s < C::NSETS; ++s)
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const int gi = s * C::GPS + (2 * c + e) / MP;
                if (gi < ng) {
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        const float2 sz = h2f2(table[(r + 8 * h) * ng + gi]);
                        out[h][e] += sz.x * ((D[s][2 * h + e] - C1[s][e]) - sz.y * C2[s][e]);
                    }
                }
            }
        // sum the columns that belong to the same token
        if (MP == 1) { out[0][0] += out[0][1]; out[1][0] += out[1][1]; }
#pragma unroll
        for (int h = 0; h < 2; ++h)
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                if (MP <= 2) out[h][e] += __shfl_xor_sync(0xffffffffu, out[h][e], 1);
                if (MP <= 4) out[h][e] += __shfl_xor_sync(0xffffffffu, out[h][e], 2);
            }
        // writers: MP=1: c==0 writes token 0 (e=0); MP=2: c==0 writes tokens e; MP=4: c<2 writes
        // tokens 2c+e; MP=8: every lane writes tokens 2c+e
        {
            const bool writer = (MP == 8) || (MP == 4 && c < 2) || (MP <= 2 && c == 0);
            if (writer) {
#pragma unroll
                for (int e = 0; e < (MP == 1 ? 1 : 2); ++e) {
                    const int tok = (2 * c + e) % MP;
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        float* dst = part + (it * MP + tok) * 16 + r + 8 * h;
                        *dst = (t == 0) ? out[h][e] : (*dst + out[h][e]);
                    }
                }
            }
        }

        // ---- release the slot and refill it ----
        __syncwarp();
        if (lane == 0 && q + S < Q) {
            fence_proxy_async_smem();
            issue(q + S);
        }
    }

    // ---- sum over the warps (k-chunks) of this CTA, then over the CTAs of the cluster ----
    __syncthreads();
    const int n_out = L.SR * P.RBI * MP * 16;
    const int wc_used = (P.NC - rank * L.WC) < L.WC ? (P.NC - rank * L.WC) : L.WC;  // warps that had a chunk
    for (int o = threadIdx.x; o < n_out; o += blockDim.x) {
        const int row = o & 15, tok = (o >> 4) % MP, it = (o / (16 * MP)) % P.RBI, s_r = o / (16 * MP * P.RBI);
        float acc = 0.f;
        const int rb = cl * (L.SR * P.RBI) + s_r + it * L.SR;
        if (rb < P.NB)
            for (int w = 0; w < wc_used; ++w)
                acc += part_all[(s_r * L.WC + w) * C::PART_FLOATS + (it * MP + tok) * 16 + row];
        if (CS == 1) {
            const int n = rb * 16 + row;
            if (rb < P.NB && n < P.N && tok < L.M) store_out(P.y, P.y_dtype, (size_t)tok * P.N + n, acc);
        } else {
            red[o] = acc;
        }
    }
    if (CS > 1) {
        cluster_sync();
        for (int o = threadIdx.x * CS + rank; o < n_out; o += blockDim.x * CS) {
            const int row = o & 15, tok = (o >> 4) % MP, it = (o / (16 * MP)) % P.RBI, s_r = o / (16 * MP * P.RBI);
            const int rb = cl * (L.SR * P.RBI) + s_r + it * L.SR;
            const int n = rb * 16 + row;
            if (rb < P.NB && n < P.N && tok < L.M) {
                float acc = 0.f;
                for (int cr = 0; cr < CS; ++cr) acc += ld_dsmem_f32(red + o, (uint32_t)cr);
                store_out(P.y, P.y_dtype, (size_t)tok * P.N + n, acc);
            }
        }
        cluster_sync();  // peers may still be reading this CTA's shared memory
    }
}

template <int GROUP, int MP>
size_t smem_bytes(int W, int SR, int S) {
    using C = Cfg<GROUP, MP>;
    return (size_t)W * S * C::QB + (size_t)W * C::CORR_FLOATS * 4 + (size_t)W * C::PART_FLOATS * 4 +
           (size_t)SR * C::PART_FLOATS * 4 + (size_t)W * kGemvMaxStages * 8;
}

template <int GROUP, int MP>
cudaError_t launch_one(const GemvLaunch& L, int n_clusters, int CS, uint32_t* status, cudaStream_t stream) {
    const int W = L.WC * L.SR;
    const size_t smem = smem_bytes<GROUP, MP>(W, L.SR, L.stages);
    auto kern = gemv_w4a16_kernel<GROUP, MP>;
    static size_t configured = 0;  // per instantiation
    if (smem > configured) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
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
    return cudaLaunchKernelEx(&cfg, kern, L, status);
}

}  // namespace

size_t gemv_w4a16_smem(int group, int MP, int W, int SR, int S) {
    if (group == 64) {
        switch (MP) { case 1: return smem_bytes<64, 1>(W, SR, S); case 2: return smem_bytes<64, 2>(W, SR, S);
                      case 4: return smem_bytes<64, 4>(W, SR, S); default: return smem_bytes<64, 8>(W, SR, S); }
    }
    switch (MP) { case 1: return smem_bytes<128, 1>(W, SR, S); case 2: return smem_bytes<128, 2>(W, SR, S);
                  case 4: return smem_bytes<128, 4>(W, SR, S); default: return smem_bytes<128, 8>(W, SR, S); }
}

cudaError_t gemv_w4a16_launch(const GemvLaunch& L, int group, int MP, int n_clusters, int CS, uint32_t* status,
                              cudaStream_t stream) {
#define MNN_CASE(G, P) if (group == G && MP == P) return launch_one<G, P>(L, n_clusters, CS, status, stream);
    MNN_CASE(64, 1) MNN_CASE(64, 2) MNN_CASE(64, 4) MNN_CASE(64, 8)
    MNN_CASE(128, 1) MNN_CASE(128, 2) MNN_CASE(128, 4) MNN_CASE(128, 8)
#undef MNN_CASE
    return cudaErrorInvalidValue;
}

}  // namespace mnnllm
