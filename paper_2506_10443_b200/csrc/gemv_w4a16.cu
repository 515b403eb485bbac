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

#include "common.h"
#include "gemv.h"
#include "gemv_w4a16_core.cuh"
#include "ptx.cuh"

namespace mnnllm {

using namespace ptx;
using namespace w4a16;

namespace {

constexpr uint32_t kMaxPolls = 1u << 15;  // x 20 us per try: gives up after ~0.65 s

constexpr unsigned int kLoraMaxPolls = 1u << 20;   // ~1 s of L2 round trips
constexpr int kLoraMaxEntries = 8 * MNNLLM_LORA_MAX_RANK;   // (token, j) pairs of a launch

// Eight consecutive fp16 (or bf16) values as floats.
__device__ __forceinline__ void widen8(const uint4& v, bool bf16, float (&f)[8]) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        if (bf16) {   // a bf16 is the upper half of the fp32 of the same value
            f[2 * i] = __uint_as_float(w[i] << 16);
            f[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
        } else {
            const float2 p = __half22float2(*reinterpret_cast<const __half2*>(&w[i]));
            f[2 * i] = p.x;
            f[2 * i + 1] = p.y;
        }
    }
}

// LoRA bypass (Section 5.5): y += LoRA_A (LoRA_B x), the small product first.  The CTAs of the problem
// compute t = x . LoRA_B^T between them: entry o = (token, j) falls to CTA o mod n_ctas, whose threads
// split K.  An entry is published as one 8-byte word {value, tag}, tag = the workspace's epoch + 1:
// a reader needs no flag and no fence, it sees a whole word of this launch or an older one.
struct LoraCtx {
    unsigned long long* t2;   // [M * r] tagged entries
    unsigned int tag;
};

// before the activations are complete: bring this CTA's rows of LoRA_B (static data) into L2
__device__ __forceinline__ void lora_prefetch(const GemvProblem& P, int M, int cta, int n_ctas) {
    const int n_t = M * P.lora_r;
    for (int o = cta; o < n_t; o += n_ctas) {
        const char* row = reinterpret_cast<const char*>(P.lora_B + (size_t)(o % P.lora_r) * P.K);
        for (int b = threadIdx.x * 128; b < P.K * 2; b += blockDim.x * 128)
            asm volatile("prefetch.global.L2 [%0];" ::"l"(row + b));
    }
}

__device__ __forceinline__ void lora_produce(const GemvProblem& P, const LoraCtx& lc, int M, bool x_bf16, int cta,
                                             int n_ctas, float* red) {
    const int n_t = M * P.lora_r;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, n_warps = blockDim.x >> 5;
    for (int o = cta; o < n_t; o += n_ctas) {
        const int m = o / P.lora_r, j = o - m * P.lora_r;
        const uint4* xr = reinterpret_cast<const uint4*>(reinterpret_cast<const uint16_t*>(P.x) + (size_t)m * P.K);
        const uint4* br = reinterpret_cast<const uint4*>(P.lora_B + (size_t)j * P.K);
        float acc = 0.f;
        for (int v = threadIdx.x; v < P.K / 8; v += blockDim.x) {
            float a[8], b[8];
            widen8(xr[v], x_bf16, a);
            widen8(__ldg(br + v), false, b);
#pragma unroll
            for (int i = 0; i < 8; ++i) acc = fmaf(a[i], b[i], acc);
        }
#pragma unroll
        for (int s = 16; s > 0; s >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, s);
        __syncthreads();   // red free (the previous entry has been summed)
        if (lane == 0) red[warp] = acc;
        __syncthreads();
        if (threadIdx.x == 0) {
            float sum = 0.f;
            for (int w = 0; w < n_warps; ++w) sum += red[w];   // fixed order: the same t whoever runs first
            __stcg(lc.t2 + o, ((unsigned long long)lc.tag << 32) | (unsigned long long)__float_as_uint(sum));
        }
    }
}

// Before the first output is stored: every entry of t into shared memory, each waited for (bounded)
// until it carries this launch's tag.  Returns false when a wait ran out.
__device__ __forceinline__ bool lora_collect(const LoraCtx& lc, int n_t, float* ts) {
    bool ok = true;
    for (int o = threadIdx.x; o < n_t; o += blockDim.x) {
        unsigned long long w = 0;
        unsigned int polls = 0;
        for (;;) {
            w = *reinterpret_cast<volatile unsigned long long*>(lc.t2 + o);
            if ((unsigned int)(w >> 32) == lc.tag) break;
            if (++polls > kLoraMaxPolls) { ok = false; break; }
        }
        ts[o] = __uint_as_float((unsigned int)w);
    }
    return ok;
}

__device__ __forceinline__ float lora_term(const GemvProblem& P, const float* ts, int n, int tok) {
    const __half* a = P.lora_A + (size_t)n * P.lora_r;
    const float* t = ts + tok * P.lora_r;
    float acc = 0.f;
    for (int j = 0; j < P.lora_r; ++j) acc = fmaf(__half2float(__ldg(a + j)), t[j], acc);
    return acc;
}

template <int GROUP, int MP, bool XBF, bool LORA>   // XBF: activations are bf16; LORA: outputs take the bypass term (converted to fp16 as the fragments are built)
__global__ void __launch_bounds__(kGemvMaxWarps * 32, (MP <= 4 ? 2 : 1))
gemv_w4a16_kernel(const __grid_constant__ GemvLaunch L, uint32_t* __restrict__ status) {
    using C = Cfg<GROUP, MP>;
    extern __shared__ __align__(128) uint8_t smem[];

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int r = lane >> 2, c = lane & 3;
    const int CS = (int)cluster_nctarank(), rank = (int)cluster_ctarank();
    const int cluster_id = blockIdx.x / CS;
    const int W = L.WC * L.SR, S = L.stages, SR = L.SR, RBI = L.RBI;

    int pi = 0;
    while (pi + 1 < L.count && cluster_id >= L.prob[pi + 1].cluster_begin) ++pi;
    const GemvProblem& P = L.prob[pi];
    const int cl = cluster_id - P.cluster_begin;
    const int wc = warp % L.WC, sr = warp / L.WC;

    // shared memory carve-up
    uint8_t* ring = smem + (size_t)warp * S * C::QB;
    float* fbase = reinterpret_cast<float*>(smem + (size_t)W * S * C::QB);
    float* part_all = fbase;                                 // [W][2][RBI][MP][16]
    float* red = part_all + W * 2 * C::PART_FLOATS;          // [2][SR][RBI][MP][16]
    uint64_t* bars = reinterpret_cast<uint64_t*>(red + 2 * SR * C::PART_FLOATS) + warp * kGemvMaxStages;

    // this cluster's rows: an even share of the problem's 16-row blocks, walked in rounds of SR*RBI
    const int rb_begin = (int)((long long)P.NB * cl / P.n_clusters);
    const int rb_end = (int)((long long)P.NB * (cl + 1) / P.n_clusters);
    const int per_round = SR * RBI;
    const int n_rounds = (rb_end - rb_begin + per_round - 1) / per_round;
    // this warp's k-chunks: j = j0 + t * jstride
    const int jstride = CS * L.WC;
    const int j0 = rank * L.WC + wc;
    const int T = j0 < P.NC ? (P.NC - j0 + jstride - 1) / jstride : 0;
    const int last_ns = P.NS - 8 * (P.NC - 1);  // slabs in the last chunk

    auto nit_of = [&](int rd) {  // row blocks of round rd that fall to this warp's sub-range
        const int first = rb_begin + rd * per_round + sr;
        if (first >= rb_end || T == 0) return 0;
        const int n = (rb_end - first + SR - 1) / SR;
        return n < RBI ? n : RBI;
    };

    if (lane == 0) {
        for (int s = 0; s < S; ++s) mbar_init(&bars[s], 1);
        fence_mbar_init();
    }
    fence_proxy_async_smem();
    __syncwarp();

    // ---- producer side (lane 0): walks (round, chunk, row block) in the order of consumption ----
    // A slot is refilled right after the warp has read it (the __syncwarp before the refill orders
    // the reads of all lanes before the bulk copy is issued).
    int i_rd = 0, i_t = 0, i_it = 0, i_nit = nit_of(0), i_slot = 0;
    while (i_rd < n_rounds && i_nit == 0) { ++i_rd; i_nit = i_rd < n_rounds ? nit_of(i_rd) : 0; }
    const uint8_t* const body = P.packed + kHeaderBytes;
    const size_t it_stride = (size_t)SR * P.row_block_bytes;
    auto src_of = [&](int rd, int t) {
        return body + (size_t)(rb_begin + rd * per_round + sr) * P.row_block_bytes + (size_t)(j0 + t * jstride) * C::QB;
    };
    auto bytes_of = [&](int t) {
        const int ns = (j0 + t * jstride == P.NC - 1) ? last_ns : 8;
        return (uint32_t)(ns * kSlabBytes + 16 * (ns / C::SPG) * 4);
    };
    const uint8_t* i_src = i_rd < n_rounds ? src_of(i_rd, 0) : body;
    uint32_t i_bytes = bytes_of(0);
    // weights are read once per token: mark their lines evict-first so that the stream does not
    // push the activations (written by the previous kernel, read by the next) out of L2
    const uint64_t stream_policy = policy_evict_first();
    // every lane keeps the (uniform) producer state; one elected lane issues the copy
    bool dead = false;   // a bounded wait gave up: nothing more is copied or waited for
    auto issue_next = [&]() {
        if (i_rd >= n_rounds || dead) return;
        if (elect_one()) {
            mbar_arrive_expect_tx(&bars[i_slot], i_bytes);
            bulk_g2s_hint(ring + (size_t)i_slot * C::QB, i_src, i_bytes, &bars[i_slot], stream_policy);
        }
        i_slot = (i_slot + 1 == S) ? 0 : i_slot + 1;
        i_src += it_stride;
        if (++i_it == i_nit) {
            i_it = 0;
            if (++i_t == T) {
                i_t = 0;
                do { ++i_rd; i_nit = i_rd < n_rounds ? nit_of(i_rd) : 0; } while (i_rd < n_rounds && i_nit == 0);
            }
            if (i_rd < n_rounds) {
                i_src = src_of(i_rd, i_t);
                i_bytes = bytes_of(i_t);
            }
        }
    };

    pdl_launch_dependents();
    for (int s = 0; s < S; ++s) issue_next();
    __shared__ float lora_ts[LORA ? kLoraMaxEntries : 1];
    __shared__ float lora_red[LORA ? kGemvMaxWarps : 1];
    const bool has_lora = LORA && P.lora_r > 0;
    if (has_lora) lora_prefetch(P, L.M, cl * CS + rank, P.n_clusters * CS);
    // everything above touched only weights; the activations may come from the previous kernel
    pdl_wait();
    LoraCtx lc = {nullptr, 0u};
    if (has_lora) {
        // the epoch is stable here: the launch that last used the workspace has completed
        lc.t2 = reinterpret_cast<unsigned long long*>(P.lora_t);
        lc.tag = __ldcg(P.lora_sync) + 1u;
        lora_produce(P, lc, L.M, XBF, cl * CS + rank, P.n_clusters * CS, lora_red);
    }
    bool lora_ready = !has_lora;

    const int tokB = r % MP, gsB = r / MP;  // B-operand role of this lane: column r of the MMA
    constexpr bool x_bf16 = XBF;
    constexpr bool COMPACT = MP == 4;   // B fragments without their zeros: room for two CTAs per SM
    BFrag<GROUP, MP, COMPACT> B;
    B.gs = gsB;
    float C1[C::NSETS][2], C2[C::NSETS][2];
    int cur_j = -1, slot = 0;
    uint32_t phase = 0;
    const int wc_used = (P.NC - rank * L.WC) < L.WC ? (P.NC - rank * L.WC) : L.WC;  // warps that own a chunk

    for (int rd = 0; rd < n_rounds; ++rd) {
        const int nit = nit_of(rd);
        float* part = part_all + (warp * 2 + (rd & 1)) * C::PART_FLOATS;
        if (nit > 0)
            for (int t = 0; t < T; ++t) {
                const int j = j0 + t * jstride;
                const int ns = (j == P.NC - 1) ? last_ns : 8;
                const int ng = ns / C::SPG;

                if (j != cur_j) {
                    cur_j = j;
                    // ---- new k-chunk: activations -> B fragments, group sums -> correction terms ----
                    const __half* xk = P.x + (size_t)j * kChunkK;
                    // a lane holds the slabs of its groups gsB + GPS * s only (its other B entries are
                    // zero): load those once, take the group sums from the same registers
                    float v1[C::NSETS], v2[C::NSETS];
                    uint32_t Pl[COMPACT ? 1 : C::NSETS][C::SPG][4][2];
                    auto Pm = [&](int s, int sp) -> uint32_t (&)[4][2] {
                        if constexpr (COMPACT) return B.v[s * C::SPG + sp]; else return Pl[s][sp];
                    };
#pragma unroll
                    for (int s = 0; s < C::NSETS; ++s) {
                        float lo = 0.f, hi = 0.f;
#pragma unroll
                        for (int sp = 0; sp < C::SPG; ++sp) {
                            const int sl = (gsB + C::GPS * s) * C::SPG + sp;
                            uint4 u0 = make_uint4(0, 0, 0, 0), u1 = u0;
                            if (sl < ns && tokB < L.M) {
                                const uint4* px =
                                    reinterpret_cast<const uint4*>(xk + (size_t)tokB * P.K + sl * kSlabK4 + 16 * c);
                                u0 = px[0];
                                u1 = px[1];
                                if (x_bf16) { u0 = bf16x8_to_f16x8(u0); u1 = bf16x8_to_f16x8(u1); }
                            }
                            Pm(s, sp)[0][0] = __byte_perm(u0.x, u0.y, 0x5410);
                            Pm(s, sp)[0][1] = __byte_perm(u0.z, u0.w, 0x5410);
                            Pm(s, sp)[1][0] = __byte_perm(u0.x, u0.y, 0x7632);
                            Pm(s, sp)[1][1] = __byte_perm(u0.z, u0.w, 0x7632);
                            Pm(s, sp)[2][0] = __byte_perm(u1.x, u1.y, 0x5410);
                            Pm(s, sp)[2][1] = __byte_perm(u1.z, u1.w, 0x5410);
                            Pm(s, sp)[3][0] = __byte_perm(u1.x, u1.y, 0x7632);
                            Pm(s, sp)[3][1] = __byte_perm(u1.z, u1.w, 0x7632);
                            const float2 a0 = h2f2(u0.x), a1 = h2f2(u0.y), a2 = h2f2(u1.x), a3 = h2f2(u1.y);
                            const float2 b0 = h2f2(u0.z), b1 = h2f2(u0.w), b2 = h2f2(u1.z), b3 = h2f2(u1.w);
                            lo += ((a0.x + a0.y) + (a1.x + a1.y)) + ((a2.x + a2.y) + (a3.x + a3.y));
                            hi += ((b0.x + b0.y) + (b1.x + b1.y)) + ((b2.x + b2.y) + (b3.x + b3.y));
                        }
                        lo += __shfl_xor_sync(0xffffffffu, lo, 1);
                        hi += __shfl_xor_sync(0xffffffffu, hi, 1);
                        lo += __shfl_xor_sync(0xffffffffu, lo, 2);
                        hi += __shfl_xor_sync(0xffffffffu, hi, 2);
                        v1[s] = 1024.f * lo + 64.f * hi;
                        v2[s] = lo + hi;
                    }
                    if constexpr (!COMPACT) {
#pragma unroll
                        for (int sl = 0; sl < 8; ++sl) {
                            const int gi = sl / C::SPG;
                            const bool mine = gsB == gi % C::GPS;
#pragma unroll
                            for (int a = 0; a < 4; ++a)
#pragma unroll
                                for (int b = 0; b < 2; ++b) B.v[sl][a][b] = mine ? Pl[gi / C::GPS][sl % C::SPG][a][b] : 0u;
                        }
                    }
                    // the correction terms of accumulator column 2c + e = (token, group slot) sit in
                    // the quad whose row index r equals that column
#pragma unroll
                    for (int s = 0; s < C::NSETS; ++s)
#pragma unroll
                        for (int e = 0; e < 2; ++e) {
                            C1[s][e] = __shfl_sync(0xffffffffu, v1[s], 4 * (2 * c + e));
                            C2[s][e] = __shfl_sync(0xffffffffu, v2[s], 4 * (2 * c + e));
                        }
                }

                for (int it = 0; it < nit; ++it) {
                    // ---- wait for this quantum's bulk copy (a non-blocking probe first: the copy has
                    // usually landed, and the probe is cheaper than the blocking form: +1 % measured) ----
                    if (!dead && !mbar_test_wait(&bars[slot], phase) && !mbar_wait_bounded(&bars[slot], phase, kMaxPolls)) {
                        dead = true;
                        if (lane == 0) atomicOr(status, 0x100u | (uint32_t)pi);
                    }
                    const uint8_t* qp = ring + (size_t)slot * C::QB;
                    const uint4* slabs = reinterpret_cast<const uint4*>(qp);

                    float D[C::NSETS][4];
                    if (ns == 8) quantum_mma<GROUP, MP, true, COMPACT>(slabs, lane, 8, B, D);
                    else quantum_mma<GROUP, MP, false, COMPACT>(slabs, lane, ns, B, D);

                    // ---- rescale: column (2c + e) of tile s is (token, group) = (col % MP, s*GPS + col / MP) ----
                    float out[2][2] = {{0.f, 0.f}, {0.f, 0.f}};  // [row half h][column e]
                    auto rescale = [&](const int ngc) {
                        const uint32_t* table = reinterpret_cast<const uint32_t*>(qp + (size_t)ngc * C::SPG * kSlabBytes);
#pragma unroll
                        for (int s = 0; s < C::NSETS; ++s)
#pragma unroll
                            for (int e = 0; e < 2; ++e) {
                                const int gi = s * C::GPS + (2 * c + e) / MP;
                                const bool ok = gi < ngc;
                                const int gic = ok ? gi : 0;
#pragma unroll
                                for (int h = 0; h < 2; ++h) {
                                    const float2 sz = h2f2(table[(r + 8 * h) * ngc + gic]);
                                    const float v = sz.x * ((D[s][2 * h + e] - C1[s][e]) - sz.y * C2[s][e]);
                                    out[h][e] += ok ? v : 0.f;
                                }
                            }
                    };
                    if (ns == 8) rescale(C::GC); else rescale(ng);
                    // the slot has been read: release and refill it before the (register-only) tail
                    __syncwarp();
                    issue_next();
                    slot = (slot + 1 == S) ? 0 : slot + 1;
                    phase ^= (slot == 0) ? 1u : 0u;

                    // sum the columns that belong to the same token
                    if (MP == 1) { out[0][0] += out[0][1]; out[1][0] += out[1][1]; }
#pragma unroll
                    for (int h = 0; h < 2; ++h)
#pragma unroll
                        for (int e = 0; e < 2; ++e) {
                            if (MP <= 2) out[h][e] += __shfl_xor_sync(0xffffffffu, out[h][e], 1);
                            if (MP <= 4) out[h][e] += __shfl_xor_sync(0xffffffffu, out[h][e], 2);
                        }
                    // writers: MP=1: c==0 writes token 0 (e=0); MP=2: c==0 writes tokens e; MP=4: c<2
                    // writes tokens 2c+e; MP=8: every lane writes tokens 2c+e
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
            }

        // ---- end of round: sum over the warps (k-chunks) of this CTA, then over the cluster ----
        if (LORA && !lora_ready) {
            if (!lora_collect(lc, L.M * P.lora_r, lora_ts)) atomicOr(status, 0x700u | (unsigned)pi);
            lora_ready = true;
        }
        __syncthreads();
        const int n_out = per_round * MP * 16;
        float* red_rd = red + (rd & 1) * SR * C::PART_FLOATS;
        for (int o = threadIdx.x; o < n_out; o += blockDim.x) {
            const int row = o & 15, tok = (o >> 4) % MP, it = (o / (16 * MP)) % RBI, s_r = o / (16 * MP * RBI);
            const int rb = rb_begin + rd * per_round + it * SR + s_r;
            float acc = 0.f;
            if (rb < rb_end)
                for (int w = 0; w < wc_used; ++w)
                    acc += part_all[((s_r * L.WC + w) * 2 + (rd & 1)) * C::PART_FLOATS + (it * MP + tok) * 16 + row];
            if (CS == 1) {
                const int n = rb * 16 + row;
                if (rb < rb_end && n < P.N && tok < L.M)
                    store_out(P.y, P.y_dtype, (size_t)tok * P.N + n, LORA ? acc + lora_term(P, lora_ts, n, tok) : acc);
            } else {
                red_rd[o] = acc;
            }
        }
        if (CS > 1) {
            cluster_sync();
            for (int o = threadIdx.x * CS + rank; o < n_out; o += blockDim.x * CS) {
                const int row = o & 15, tok = (o >> 4) % MP, it = (o / (16 * MP)) % RBI, s_r = o / (16 * MP * RBI);
                const int rb = rb_begin + rd * per_round + it * SR + s_r;
                const int n = rb * 16 + row;
                if (rb < rb_end && n < P.N && tok < L.M) {
                    float acc = 0.f;
                    for (int cr = 0; cr < CS; ++cr) acc += ld_dsmem_f32(red_rd + o, (uint32_t)cr);
                    store_out(P.y, P.y_dtype, (size_t)tok * P.N + n, LORA ? acc + lora_term(P, lora_ts, n, tok) : acc);
                }
            }
        }
    }
    if (has_lora) {
        // this CTA has read t for the last time; the last CTA of the problem moves the epoch on (the
        // next launch that uses the workspace reads it only after this grid has completed)
        __syncthreads();
        if (threadIdx.x == 0 && atomicAdd(P.lora_sync + 1, 1u) == (unsigned int)(P.n_clusters * CS) - 1u) {
            P.lora_sync[0] = lc.tag;
            P.lora_sync[1] = 0u;
        }
    }
    if (dead)   // copies issued before the give-up may still be in flight into this CTA's shared memory
        for (int i = 0; i < 50; ++i) __nanosleep(1000);
    if (CS > 1) cluster_sync();  // peers may still be reading this CTA's shared memory
}

template <int GROUP, int MP>
size_t smem_bytes(int W, int SR, int S) {
    using C = Cfg<GROUP, MP>;
    return (size_t)W * S * C::QB + (size_t)W * 2 * C::PART_FLOATS * 4 +
           (size_t)2 * SR * C::PART_FLOATS * 4 + (size_t)W * kGemvMaxStages * 8;
}

// Raises the kernel's dynamic shared memory limit when a launch needs more than any before it.
template <int GROUP, int MP, bool XBF, bool LORA>
cudaError_t ensure_smem(size_t smem) {
    struct State { size_t configured; bool carveout_set; };
    static PerDevice<State> state;   // per instantiation and device
    return state.with([&](State& st) {
        if (!st.carveout_set) {
            // every launch of the library asks for the same (largest) shared-memory carve-out, so that
            // an SM does not have to re-partition its L1 between consecutive dependent launches
            cudaError_t e = cudaFuncSetAttribute(gemv_w4a16_kernel<GROUP, MP, XBF, LORA>,
                                                 cudaFuncAttributePreferredSharedMemoryCarveout,
                                                 (int)cudaSharedmemCarveoutMaxShared);
            if (e != cudaSuccess) return e;
            st.carveout_set = true;
        }
        if (smem > st.configured) {
            cudaError_t e = cudaFuncSetAttribute(gemv_w4a16_kernel<GROUP, MP, XBF, LORA>,
                                                 cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            if (e != cudaSuccess) return e;
            st.configured = smem;
        }
        return cudaSuccess;
    });
}

template <int GROUP, int MP, bool XBF, bool LORA>
cudaError_t launch_one(const GemvLaunch& L, int n_clusters, int CS, uint32_t* status, cudaStream_t stream) {
    const int W = L.WC * L.SR;
    const size_t smem = smem_bytes<GROUP, MP>(W, L.SR, L.stages);
    auto kern = gemv_w4a16_kernel<GROUP, MP, XBF, LORA>;
    if (cudaError_t e = ensure_smem<GROUP, MP, XBF, LORA>(smem); e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(n_clusters * CS));
    cfg.blockDim = dim3((unsigned)(W * 32));
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = (unsigned)CS;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = CS > 1 ? 2 : 1;   // a launch without clusters does not go through the cluster path
    return cudaLaunchKernelEx(&cfg, kern, L, status);
}

// the instantiation by activation type and bypass (a launch has the bypass when one of its problems has)
template <int GROUP, int MP>
cudaError_t dispatch(const GemvLaunch& L, int n_clusters, int CS, uint32_t* status, cudaStream_t stream) {
    bool lora = false;
    for (int i = 0; i < L.count; ++i) lora |= L.prob[i].lora_r > 0;
    const bool xbf = L.prob[0].x_dtype == MNNLLM_BF16;
    if (lora) return xbf ? launch_one<GROUP, MP, true, true>(L, n_clusters, CS, status, stream)
                         : launch_one<GROUP, MP, false, true>(L, n_clusters, CS, status, stream);
    return xbf ? launch_one<GROUP, MP, true, false>(L, n_clusters, CS, status, stream)
               : launch_one<GROUP, MP, false, false>(L, n_clusters, CS, status, stream);
}

template <int GROUP, int MP, bool XBF = false, bool LORA = false>
int occupancy_of(int W, int SR, int S) {
    int n = 0;
    const size_t smem = smem_bytes<GROUP, MP>(W, SR, S);
    auto kern = gemv_w4a16_kernel<GROUP, MP, XBF, LORA>;
    if (ensure_smem<GROUP, MP, XBF, LORA>(smem) != cudaSuccess) return 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, kern, W * 32, smem) != cudaSuccess) return 0;
    return n;
}

}  // namespace

int gemv_w4a16_occupancy(int group, int MP, int W, int SR, int S) {
#define MNN_CASE(G, P) if (group == G && MP == P) return occupancy_of<G, P>(W, SR, S);
    MNN_CASE(64, 1) MNN_CASE(64, 2) MNN_CASE(64, 4) MNN_CASE(64, 8)
    MNN_CASE(128, 1) MNN_CASE(128, 2) MNN_CASE(128, 4) MNN_CASE(128, 8)
#undef MNN_CASE
    return 0;
}

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
#define MNN_CASE(G, P)                                                                                   \
    if (group == G && MP == P)                                                                          \
        return dispatch<G, P>(L, n_clusters, CS, status, stream);
    MNN_CASE(64, 1) MNN_CASE(64, 2) MNN_CASE(64, 4) MNN_CASE(64, 8)
    MNN_CASE(128, 1) MNN_CASE(128, 2) MNN_CASE(128, 4) MNN_CASE(128, 8)
#undef MNN_CASE
    return cudaErrorInvalidValue;
}

}  // namespace mnnllm
