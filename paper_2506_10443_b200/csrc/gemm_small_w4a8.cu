// W4A8 linear for short prompts (M <= 64 tokens), bound by HBM like the decode GEMV.
//
// Section 4.2 computes the W4A8 linear from int8 activation codes and int4 weight codes with integer
// matrix instructions; at 64 tokens a weight byte meets only 4 M = 256 integer operations, far below
// the ridge of the GPU, so the job is to stream the packed weights once at the HBM rate.  The
// 128 x 128 tcgen05 tile of the prefill GEMM is the wrong tool there (half of it padding, and a
// fixed cost per call larger than the work).  This kernel is the decode GEMV's shape instead:
//   * a warp owns one 16-row block of the weights and walks its k-chunks (a contiguous run of the
//     packed buffer) through a private ring of bulk copies;
//   * the 16 warps of a CTA share the activation codes of the current k-chunk (64 tokens x 512 k,
//     int8) in shared memory, double buffered, fetched by a producer warp;
//   * per group of 64 (128) k: mma.sync m16n8k32 (u8 weights x s8 activations -> s32), eight token
//     tiles wide; the int32 partial P is exact, and y += s * P - (s z) * A in fp32 registers;
//   * a launch with too few 16-row blocks to fill the GPU cuts K into parts that meet through scratch
//     memory: the last part to arrive adds them in the order of the k ranges (a fixed sum).
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "common.h"
#include "gemm_small_w4a8.h"
#include "layout.h"
#include "ptx.cuh"

namespace mnnllm {

using namespace ptx;

namespace {

constexpr int kWarps = 16;                      // consumer warps = 16-row blocks of a CTA's tile
constexpr int kThreads = (kWarps + 1) * 32;     // + the activation producer warp
constexpr int kTok = 64;                        // tokens per launch at most (8 MMA tiles of 8)
constexpr int kPitch = kChunkK + 64;            // bytes between tokens of the activation tile: lanes of a
                                                // quarter warp (two tokens x four k pieces) hit all 32 banks
constexpr int kActBytes = kTok * kPitch;        // 36 KiB
constexpr int kAcBytes = 8 * kTok * 4;          // a chunk's group sums: up to 8 groups x 64 tokens, fp32
constexpr int kSlots = 2;                       // ring slots per warp
constexpr uint32_t kMaxPolls = 1u << 15;

template <int GROUP>
struct Geo {
    static constexpr int GC = kChunkK / GROUP;             // groups per full chunk
    static constexpr int SPG = GROUP / kSlabK4;            // slabs per group
    static constexpr int QB = 8 * kSlabBytes + 16 * GC * 4;
};

template <int GROUP>
constexpr size_t smem_bytes() {
    return (size_t)2 * kActBytes + 2 * kAcBytes + (size_t)kWarps * kSlots * Geo<GROUP>::QB + (4 + kWarps * kSlots) * 8 + 16;
}

__device__ __forceinline__ void mma_u8s8(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ void store_y(void* y, int dtype, size_t idx, float v) {
    if (dtype == MNNLLM_F16) reinterpret_cast<__half*>(y)[idx] = __float2half_rn(v);
    else if (dtype == MNNLLM_BF16) reinterpret_cast<__nv_bfloat16*>(y)[idx] = __float2bfloat16_rn(v);
    else reinterpret_cast<float*>(y)[idx] = v;
}

__device__ __forceinline__ float2 h2f2(uint32_t u) {
    return __half22float2(*reinterpret_cast<const __half2*>(&u));
}

struct Params {
    const uint8_t* packed[kGemmSmallMaxBatch];
    void* y[kGemmSmallMaxBatch];
    int N[kGemmSmallMaxBatch];
    int nb_end[kGemmSmallMaxBatch];   // 16-row blocks of matrices 0..i (cumulative)
    int y_dtype[kGemmSmallMaxBatch];
    const int8_t* a_q;                // [M, K] signed codes
    const float* a_scale;             // [M]
    const float* a_sums_t;            // [G][64] group sums of the signed codes, fp32, token fastest
    int32_t* P;                       // partials form: [M, N[0], G]
    float* scratch;
    uint32_t* counters;
    unsigned long long row_block_bytes;
    int M, K, G, NB, NC, NS;
    int parts, chunks_per_part;
};

// MT = token tiles of 8 (1, 2, 4 or 8): a compile-time bound, so that the loops over the tiles are
// straight-line code and the loads and MMAs of different tiles overlap.
template <int GROUP, bool PARTIALS, int MT>
__global__ void __launch_bounds__(kThreads, 1)
gemm_small_w4a8_kernel(const __grid_constant__ Params p, uint32_t* __restrict__ status) {
    using C = Geo<GROUP>;
    extern __shared__ __align__(128) uint8_t smem[];
    uint8_t* act = smem;                               // [2][kTok][kPitch]   activation codes of a k-chunk
    float* acs = reinterpret_cast<float*>(act + 2 * kActBytes);            // [2][GC][kTok] group sums (fp32)
    uint8_t* rings = reinterpret_cast<uint8_t*>(acs) + 2 * kAcBytes;       // [kWarps][kSlots][QB]
    uint64_t* act_full = reinterpret_cast<uint64_t*>(rings + (size_t)kWarps * kSlots * C::QB);   // [2]
    uint64_t* act_empty = act_full + 2;                                                          // [2]
    uint64_t* q_full = act_full + 4;                                                             // [kWarps][kSlots]
    volatile uint32_t* dead = reinterpret_cast<volatile uint32_t*>(q_full + kWarps * kSlots);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int r = lane >> 2, c = lane & 3;
    const int tile = blockIdx.x / p.parts, part = blockIdx.x - tile * p.parts;
    const int j0 = part * p.chunks_per_part;
    const int j1 = j0 + p.chunks_per_part < p.NC ? j0 + p.chunks_per_part : p.NC;
    const int nj = j1 - j0;
    const int n_active = p.NB - tile * kWarps < kWarps ? p.NB - tile * kWarps : kWarps;
    const int last_ns = p.NS - 8 * (p.NC - 1);

    // token rows beyond M are never copied: they must read as zero codes and zero sums
    for (int i = threadIdx.x; i < (2 * kActBytes + 2 * kAcBytes) / 16; i += kThreads)
        reinterpret_cast<uint4*>(smem)[i] = make_uint4(0, 0, 0, 0);
    if (threadIdx.x == 0) {
        for (int i = 0; i < 2; ++i) { mbar_init(&act_full[i], 1); mbar_init(&act_empty[i], (uint32_t)n_active); }
        for (int i = 0; i < kWarps * kSlots; ++i) mbar_init(&q_full[i], 1);
        *dead = 0;
        fence_mbar_init();
    }
    fence_proxy_async_smem();
    __syncthreads();
    pdl_launch_dependents();

    auto wait = [&](uint64_t* bar, uint32_t parity, uint32_t code) {
        if (*dead) return;
        if (mbar_test_wait(bar, parity) || mbar_wait_bounded_compact(bar, parity, kMaxPolls)) return;
        *dead = 1;
        atomicOr(status, 0x300u | code);
    };

    if (warp == kWarps) {
        // ---------------- producer of the activation tiles (outputs of the quantiser) ----------------
        pdl_wait();
        for (int jj = 0; jj < nj; ++jj) {
            const int j = j0 + jj, b = jj & 1;
            if (jj >= 2) wait(&act_empty[b], (uint32_t)((jj >> 1) - 1) & 1u, 1);
            if (*dead) break;
            const int ns = (j == p.NC - 1) ? last_ns : 8;
            const uint32_t tok_bytes = (uint32_t)ns * kSlabK4;               // int8 codes of one token
            const uint32_t sum_bytes = PARTIALS ? 0u : (uint32_t)(ns / C::SPG) * kTok * 4;   // ng rows of 64 fp32 sums
            if (lane == 0) mbar_arrive_expect_tx(&act_full[b], (uint32_t)p.M * tok_bytes + sum_bytes);
            __syncwarp();
            for (int m = lane; m < p.M; m += 32)
                bulk_g2s(act + (size_t)b * kActBytes + (size_t)m * kPitch, p.a_q + (size_t)m * p.K + (size_t)j * kChunkK,
                         tok_bytes, &act_full[b]);
            if (lane == 0 && !PARTIALS)
                bulk_g2s(reinterpret_cast<uint8_t*>(acs) + (size_t)b * kAcBytes,
                         p.a_sums_t + (size_t)j * C::GC * kTok, sum_bytes, &act_full[b]);
        }
    } else if (warp < n_active) {
        // ---------------- consumers: one 16-row block each ----------------
        const int grb = tile * kWarps + warp;
        int sub = 0;
        while (grb >= p.nb_end[sub]) ++sub;
        const int lrb = grb - (sub ? p.nb_end[sub - 1] : 0);
        const uint8_t* src = p.packed[sub] + kHeaderBytes + (size_t)lrb * p.row_block_bytes + (size_t)j0 * C::QB;
        uint8_t* ring = rings + (size_t)warp * kSlots * C::QB;
        uint64_t* my_full = q_full + warp * kSlots;
        const uint64_t policy = policy_evict_first();
        auto issue = [&](int jj) {   // lane 0 only
            const int ns = (j0 + jj == p.NC - 1) ? last_ns : 8;
            const uint32_t bytes = (uint32_t)(ns * kSlabBytes + 16 * (ns / C::SPG) * 4);
            const int s = jj % kSlots;
            mbar_arrive_expect_tx(&my_full[s], bytes);
            bulk_g2s_hint(ring + (size_t)s * C::QB, src + (size_t)jj * C::QB, bytes, &my_full[s], policy);
        };
        if (lane == 0)
            for (int jj = 0; jj < kSlots && jj < nj; ++jj) issue(jj);   // weights do not depend on the quantiser

        // fp32 accumulators as packed pairs: acc2[tt][0] = (row r; tokens 2c, 2c+1 of tile tt), acc2[tt][1] = row r + 8
        uint64_t acc2[MT][2];
#pragma unroll
        for (int tt = 0; tt < MT; ++tt) acc2[tt][0] = acc2[tt][1] = 0ull;
        const uint64_t kMagic2 = f32x2_pack(0x4B400000u, 0x4B400000u);   // (1.5 * 2^23, 1.5 * 2^23)
        constexpr uint32_t NIB = 0x0F0F0F0Fu;

        for (int jj = 0; jj < nj; ++jj) {
            const int j = j0 + jj, b = jj & 1, s = jj % kSlots;
            const int ns = (j == p.NC - 1) ? last_ns : 8;
            const int ng = ns / C::SPG;
            wait(&my_full[s], (uint32_t)(jj / kSlots) & 1u, 2);
            wait(&act_full[b], (uint32_t)(jj >> 1) & 1u, 3);
            const uint8_t* qp = ring + (size_t)s * C::QB;
            const uint4* slabs = reinterpret_cast<const uint4*>(qp);
            const uint32_t* table = reinterpret_cast<const uint32_t*>(qp + (size_t)ns * kSlabBytes);   // [16 rows][ng] (s, z)
            const uint8_t* at = act + (size_t)b * kActBytes + (size_t)r * kPitch + 16 * c;
            const float* st = acs + (size_t)b * (kAcBytes / 4) + 2 * c;

            for (int gi = 0; gi < ng; ++gi) {
                // this group's weight fragments: rows r and r + 8, k = 16c .. 16c+15 of each slab
                uint32_t a[C::SPG][2][4];
#pragma unroll
                for (int sp = 0; sp < C::SPG; ++sp) {
                    const uint4 w = slabs[(gi * C::SPG + sp) * 32 + lane];
                    a[sp][0][0] = w.x & NIB; a[sp][0][1] = w.z & NIB; a[sp][0][2] = (w.x >> 4) & NIB; a[sp][0][3] = (w.z >> 4) & NIB;
                    a[sp][1][0] = w.y & NIB; a[sp][1][1] = w.w & NIB; a[sp][1][2] = (w.y >> 4) & NIB; a[sp][1][3] = (w.w >> 4) & NIB;
                }
                const float2 sz0 = h2f2(table[r * ng + gi]), sz1 = h2f2(table[(r + 8) * ng + gi]);
                // (s, s) and (-s z, -s z) for the two rows; s z is exact in fp32
                const uint64_t s0 = f32x2_pack(__float_as_uint(sz0.x), __float_as_uint(sz0.x));
                const uint64_t s1 = f32x2_pack(__float_as_uint(sz1.x), __float_as_uint(sz1.x));
                const uint32_t nz0b = __float_as_uint(-sz0.x * sz0.y), nz1b = __float_as_uint(-sz1.x * sz1.y);
                const uint64_t nz0 = f32x2_pack(nz0b, nz0b), nz1 = f32x2_pack(nz1b, nz1b);
#pragma unroll
                for (int tt = 0; tt < MT; ++tt) {
                    {
                        // The accumulator starts at the bit pattern of 1.5 * 2^23: the int32 sum P then IS
                        // the float 1.5 * 2^23 + P (|P| < 2^22), and one subtraction converts it exactly:
                        // no conversion instruction, no integer add.
                        int d[4] = {PARTIALS ? 0 : 0x4B400000, PARTIALS ? 0 : 0x4B400000, PARTIALS ? 0 : 0x4B400000,
                                    PARTIALS ? 0 : 0x4B400000};
#pragma unroll
                        for (int sp = 0; sp < C::SPG; ++sp) {
                            const uint4 bq = *reinterpret_cast<const uint4*>(at + (size_t)tt * 8 * kPitch + (gi * C::SPG + sp) * kSlabK4);
                            mma_u8s8(d, a[sp][0][0], a[sp][0][1], a[sp][0][2], a[sp][0][3], bq.x, bq.y);
                            mma_u8s8(d, a[sp][1][0], a[sp][1][1], a[sp][1][2], a[sp][1][3], bq.z, bq.w);
                        }
                        if (PARTIALS) {
                            // d[0], d[1]: row r, tokens 2c, 2c+1 of the tile; d[2], d[3]: row r + 8
                            const int n0 = lrb * 16 + r, g = j * C::GC + gi;
#pragma unroll
                            for (int i = 0; i < 4; ++i) {
                                const int m = tt * 8 + 2 * c + (i & 1), n = n0 + 8 * (i >> 1);
                                if (m < p.M && n < p.N[sub]) p.P[((size_t)m * p.N[sub] + n) * p.G + g] = d[i];
                            }
                        } else {
                            const uint64_t A = *reinterpret_cast<const uint64_t*>(st + gi * kTok + tt * 8);   // sums of tokens 2c, 2c+1
                            const uint64_t f01 = f32x2_sub(f32x2_pack((uint32_t)d[0], (uint32_t)d[1]), kMagic2);
                            const uint64_t f23 = f32x2_sub(f32x2_pack((uint32_t)d[2], (uint32_t)d[3]), kMagic2);
                            acc2[tt][0] = f32x2_fma(nz0, A, f32x2_fma(s0, f01, acc2[tt][0]));
                            acc2[tt][1] = f32x2_fma(nz1, A, f32x2_fma(s1, f23, acc2[tt][1]));
                        }
                    }
                }
            }
            // both buffers have been read: hand the activation tile back, refill the ring slot
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(&act_empty[b]);
                if (jj + kSlots < nj && !*dead) issue(jj + kSlots);
            }
        }

        float acc[MT][4];
#pragma unroll
        for (int tt = 0; tt < MT; ++tt) {
            f32x2_unpack(acc2[tt][0], acc[tt][0], acc[tt][1]);
            f32x2_unpack(acc2[tt][1], acc[tt][2], acc[tt][3]);
        }
        // a_scale and the cleared counters come from the quantiser, like the tiles already consumed
        pdl_wait();
        if (!PARTIALS) {
            const int n0 = lrb * 16 + r, Ns = p.N[sub];
            bool finish = true;   // this warp writes the block's outputs
            if (p.parts > 1) {
                // this part's 16 x 64 block -> its scratch slot; the last part to arrive adds all of them
                // in the order of the k ranges, whoever it is
                float* mine = p.scratch + ((size_t)(tile * p.parts + part) * kWarps + warp) * (kTok * 16);
#pragma unroll
                for (int tt = 0; tt < MT; ++tt)
#pragma unroll
                    for (int i = 0; i < 4; ++i) __stcg(mine + (tt * 4 + i) * 32 + lane, acc[tt][i]);
                __threadfence();
                __syncwarp();
                uint32_t seen = 0;
                if (lane == 0) seen = atomicAdd(p.counters + tile * kWarps + warp, 1u);
                seen = __shfl_sync(0xffffffffu, seen, 0);
                finish = (int)seen == p.parts - 1;
                if (finish) {
                    __threadfence();
                    const float* parts0 = p.scratch + ((size_t)(tile * p.parts) * kWarps + warp) * (kTok * 16);
#pragma unroll
                    for (int tt = 0; tt < MT; ++tt)
#pragma unroll
                        for (int i = 0; i < 4; ++i) acc[tt][i] = 0.f;
                    for (int ks = 0; ks < p.parts; ++ks) {
                        const float* src_p = parts0 + (size_t)ks * kWarps * (kTok * 16);
#pragma unroll
                        for (int tt = 0; tt < MT; ++tt)
#pragma unroll
                            for (int i = 0; i < 4; ++i) acc[tt][i] += __ldcg(src_p + (tt * 4 + i) * 32 + lane);
                    }
                }
            }
#pragma unroll
            for (int tt = 0; tt < MT; ++tt) {
                if (finish) {
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int m = tt * 8 + 2 * c + (i & 1), n = n0 + 8 * (i >> 1);
                        if (m < p.M && n < Ns)
                            store_y(p.y[sub], p.y_dtype[sub], (size_t)m * Ns + n, __ldg(p.a_scale + m) * acc[tt][i]);
                    }
                }
            }
        }
    }
    if (*dead)   // copies issued before a give-up may still be in flight into this CTA's shared memory
        for (int i = 0; i < 50; ++i) __nanosleep(1000);
}

template <int GROUP, bool PARTIALS, int MT>
cudaError_t launch(const Params& p, int grid, uint32_t* status, cudaStream_t stream) {
    auto kern = gemm_small_w4a8_kernel<GROUP, PARTIALS, MT>;
    constexpr size_t smem = smem_bytes<GROUP>();
    static PerDevice<bool> configured;   // per instantiation and device
    if (cudaError_t e = configured.with([&](bool& done) {
            if (done) return cudaSuccess;
            cudaError_t err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            if (err == cudaSuccess)
                err = cudaFuncSetAttribute(kern, cudaFuncAttributePreferredSharedMemoryCarveout,
                                           (int)cudaSharedmemCarveoutMaxShared);
            done = err == cudaSuccess;
            return err;
        });
        e != cudaSuccess)
        return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // the weight side starts under the quantiser
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, p, status);
}

}  // namespace

cudaError_t gemm_small_w4a8_launch(const GemmSmallArgs& a, uint32_t* status, cudaStream_t stream) {
    if (a.M < 1 || a.M > kGemmSmallMaxTokens || a.count < 1 || a.count > kGemmSmallMaxBatch) return cudaErrorInvalidValue;
    const bool partials = a.P != nullptr;
    const W4Geometry g0 = w4_geometry(a.N[0], a.K, a.group);
    Params p;
    int nb = 0;
    for (int i = 0; i < kGemmSmallMaxBatch; ++i) {
        const int src = i < a.count ? i : a.count - 1;
        p.packed[i] = (const uint8_t*)a.packed[src];
        p.y[i] = a.y[src];
        p.N[i] = a.N[src];
        p.y_dtype[i] = a.y_dtype[src];
        if (i < a.count) nb += w4_geometry(a.N[i], a.K, a.group).n_row_blocks;
        p.nb_end[i] = nb;
    }
    p.a_q = a.a_q; p.a_scale = a.a_scale; p.a_sums_t = a.a_sums_t; p.P = a.P;
    p.scratch = a.scratch; p.counters = a.counters;
    p.row_block_bytes = g0.row_block_bytes;
    p.M = a.M; p.K = a.K; p.G = g0.G; p.NB = nb; p.NC = g0.n_chunks; p.NS = g0.n_slabs;
    const int tiles = (nb + kWarps - 1) / kWarps;
    // K may be cut into parts (whole 512-k chunks) that run as separate CTAs and meet through scratch
    // memory (64 KiB per tile and part).  The number of parts is the one with the shortest critical
    // path in units of one quantum's time per warp:
    //     waves of CTAs x (chunks per part + 1.5)  +  (parts > 1 ? 1 + 0.2 x parts : 0)
    // 1.5 standing for a CTA's prologue and epilogue, the last term for the scratch round trip and the
    // sum over the parts (fitted to graph-replay timings of the Qwen2-1.5B shapes at 16 to 64 tokens).
    p.parts = 1;
    p.chunks_per_part = p.NC;
    const int n_sm = device_sm_count();
    if (!partials && a.scratch && a.counters && tiles * kWarps <= a.n_counters && n_sm > 0) {
        const long long max_slots = (long long)(a.scratch_bytes / ((size_t)kWarps * kTok * 16 * 4));
        double best = (double)((tiles + n_sm - 1) / n_sm) * (p.NC + 1.5);
        for (int want = 2; want <= p.NC && (long long)tiles * want <= max_slots; ++want) {
            const int cpp = (p.NC + want - 1) / want;
            const int parts = (p.NC + cpp - 1) / cpp;   // no empty part
            if (parts != want) continue;
            const double cost = (double)(((long long)tiles * parts + n_sm - 1) / n_sm) * (cpp + 1.5) + 1.0 + 0.2 * parts;
            if (cost < best) {
                best = cost;
                p.parts = parts;
                p.chunks_per_part = cpp;
            }
        }
    }
    const int grid = tiles * p.parts;
    const int mt = a.M <= 8 ? 1 : (a.M <= 16 ? 2 : (a.M <= 32 ? 4 : 8));
#define MNN_CASE(G, PT, T) if (a.group == G && partials == PT && mt == T) return launch<G, PT, T>(p, grid, status, stream);
    MNN_CASE(64, false, 1) MNN_CASE(64, false, 2) MNN_CASE(64, false, 4) MNN_CASE(64, false, 8)
    MNN_CASE(128, false, 1) MNN_CASE(128, false, 2) MNN_CASE(128, false, 4) MNN_CASE(128, false, 8)
    MNN_CASE(64, true, 1) MNN_CASE(64, true, 2) MNN_CASE(64, true, 4) MNN_CASE(64, true, 8)
    MNN_CASE(128, true, 1) MNN_CASE(128, true, 2) MNN_CASE(128, true, 4) MNN_CASE(128, true, 8)
#undef MNN_CASE
    return cudaErrorInvalidValue;
}

}  // namespace mnnllm
