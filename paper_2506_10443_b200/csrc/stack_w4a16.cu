// The linears of a whole decoder stack (W4A16, M <= 8 tokens) in ONE persistent launch.
//
// Decode time is the time to stream the weights (Section 2, Section 4.2), but a decoder layer's
// linears are a few megabytes each - well under a microsecond of HBM time - and every one depends
// on its predecessor.  Launched one by one, each pays a launch boundary of several microseconds.
// Here one cooperative grid (one CTA per SM) walks a list of problems in order:
//   * a producer warp streams the CTA's share of EVERY problem's packed weights, in order, through
//     one deep ring of shared-memory slots (bulk copies completing on mbarriers).  Weights depend on
//     nothing, so the ring runs ahead across problem boundaries: HBM keeps streaming while the
//     consumers sit in a dependency bubble;
//   * 14 consumer warps take the quanta (16 rows x 512 k) of the current problem round-robin,
//     multiply them with the warp-level MMA formulation of the single-launch GEMV and leave one
//     partial sum per quantum in shared memory; the CTA then adds them up in a fixed order;
//   * a 16-row block whose k-chunks are spread over several CTAs is finished by the CTA that holds
//     its first chunk: the others hand over their partial sums as 8-byte {value, tag} words that
//     the finisher polls directly (no fence, no flag: the word is the message);
//   * a problem that depends on earlier ones polls their completion counters (bounded) before it
//     reads its activations; completion = a release-ordered add after the outputs are stored.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "gemv_w4a16_core.cuh"
#include "ptx.cuh"
#include "common.h"
#include "stack.h"

namespace mnnllm {

using namespace ptx;
using namespace w4a16;

namespace {

constexpr uint32_t kMaxBarPolls = 1u << 15;    // mbarrier tries of up to 20 us each: ~0.65 s
constexpr uint32_t kMaxFlagPolls = 1u << 20;   // global-memory polls of roughly 0.5-1 us each

__device__ __forceinline__ uint32_t ld_acquire_u32(const uint32_t* p) {
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ unsigned long long ld_relaxed_u64(const unsigned long long* p) {
    unsigned long long v;
    asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_relaxed_u64(unsigned long long* p, unsigned long long v) {
    asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
// generic-address load that is not served from a stale L1 line (shared or global memory)
__device__ __forceinline__ uint4 ld_volatile_v4(const uint4* p) {
    uint4 v;
    asm volatile("ld.volatile.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ uint32_t ld_acquire_cta_u32(const uint32_t* smem_word) {
    uint32_t v;
    asm volatile("ld.acquire.cta.shared.u32 %0, [%1];" : "=r"(v) : "r"(smem_u32(smem_word)) : "memory");
    return v;
}
__device__ __forceinline__ void st_release_cta_u32(uint32_t* smem_word, uint32_t v) {
    asm volatile("st.release.cta.shared.u32 [%0], %1;" ::"r"(smem_u32(smem_word)), "r"(v) : "memory");
}
__device__ __forceinline__ void red_release_add(uint32_t* p, uint32_t v) {
    asm volatile("red.release.gpu.global.add.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

// Quanta [q0, q1) of a problem that fall to CTA `cta`, in row-block-major order (q = rb * NC + j):
// an even share of the problem's runs of `gran` quanta.
// With fewer runs than CTAs the first U virtual CTAs take one run each, so that consecutive small
// problems (rotated against each other by the plan) land on different SMs.
__device__ __forceinline__ void cta_range(int NB, int NC, int gran, int cv, int n_ctas, int& q0, int& q1) {
    const uint32_t U = (uint32_t)(NB * NC) / (uint32_t)gran;   // the plan guarantees U * n_ctas < 2^31
    if (U < (uint32_t)n_ctas) {
        q0 = (uint32_t)cv < U ? cv * gran : 0x3fffffff;   // empty, and beyond every row block
        q1 = (uint32_t)cv < U ? q0 + gran : 0x3fffffff;
    } else {
        q0 = (int)(U * (uint32_t)cv / (uint32_t)n_ctas) * gran;
        q1 = (int)(U * (uint32_t)(cv + 1) / (uint32_t)n_ctas) * gran;
    }
}
// cached read of a pointer field of the (read-only) plan
template <typename T, typename P>
__device__ __forceinline__ T* ldg_ptr(P* const* field) {
    return reinterpret_cast<T*>(__ldg(reinterpret_cast<const unsigned long long*>(field)));
}
__device__ __forceinline__ int virtual_cta(int cta, int rot, int n_ctas) {
    const int v = cta - rot;
    return v < 0 ? v + n_ctas : v;
}

template <int GROUP, int MP>
__global__ void __launch_bounds__(kStackThreads, 1)
stack_w4a16_kernel(const __grid_constant__ StackHeader H, const StackProblem* __restrict__ plan,
                   const __grid_constant__ StackWorkspace ws, uint32_t* __restrict__ status) {
    using C = Cfg<GROUP, MP>;
    extern __shared__ __align__(128) uint8_t smem[];
    constexpr int W = kStackConsumerWarps;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int cta = blockIdx.x, n_ctas = gridDim.x;
    const int S = H.ring_slots;

    const int R = S / W;                      // every consumer warp owns R slots of the ring
    uint8_t* ring = smem;
    const StackProblem* sD = plan;            // read-only for the whole launch: cached loads, prefetched ahead
    float* part = reinterpret_cast<float*>(smem + (size_t)S * C::QB);             // [max_quanta][MP][16]
    uint4* xs = reinterpret_cast<uint4*>(part + (size_t)H.max_quanta * MP * 16);   // staged activations
    // per staged (chunk, token): GC pairs (1024 X_lo + 64 X_hi, X_lo + X_hi) of the group sums of x
    float2* xsum = reinterpret_cast<float2*>(reinterpret_cast<uint8_t*>(xs) + H.xs_bytes);
    uint64_t* full = reinterpret_cast<uint64_t*>(xsum + (size_t)(H.xs_bytes / 1024) * C::GC);
    uint64_t* empty = full + S;
    volatile uint32_t* dead = reinterpret_cast<volatile uint32_t*>(empty + S);   // a bounded wait gave up
    uint32_t* finished = const_cast<uint32_t*>(dead) + 1;   // problems whose outputs this CTA has stored (mailbox)

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
        *dead = 0;
        *finished = 0;
        fence_mbar_init();
    }
    fence_proxy_async_smem();
    __syncthreads();

    const uint32_t tag = *reinterpret_cast<volatile const uint32_t*>(ws.epoch) + 1u;  // this launch's number, from 1

    if (warp == W) {
        // =================== producer: every problem's weights, in order, never waits for x ===================
        // Lane L streams the quanta of consumer warp L (quantum i of a problem goes to warp i mod weff)
        // through that warp's own R slots.  A slot is thus always filled by one lane and read by one warp,
        // both in order, so the parity waits on its barriers can never mistake one use for another; and
        // one thread could not issue the CTA's copies fast enough anyway.
        if (lane < W) {
            const uint64_t stream_policy = policy_evict_first();
            uint8_t* my_ring = ring + (size_t)lane * R * C::QB;
            uint64_t* my_full = full + lane * R;
            uint64_t* my_empty = empty + lane * R;
            int slot = 0;
            uint32_t parity = 0;      // parity of the slot's use count
            bool wrapped = false;
            int issued = 0;
            for (int p = 0; p < H.count; ++p) {
                const StackProblem& D = sD[p];
                const int weff = __ldg(&D.weff);
                if (lane >= weff) continue;
                const int NB = __ldg(&D.NB), NC = __ldg(&D.NC);
                int q0, q1;
                cta_range(NB, NC, __ldg(&D.gran), virtual_cta(cta, __ldg(&D.rot), n_ctas), n_ctas, q0, q1);
                if (q0 + lane >= q1) continue;
                const unsigned long long rbb = __ldg(&D.row_block_bytes);
                const int last_ns = __ldg(&D.NS) - 8 * (NC - 1);
                const uint32_t last_bytes = (uint32_t)(last_ns * kSlabBytes + 16 * (last_ns / C::SPG) * 4);
                for (int q = q0 + lane; q < q1; q += weff) {
                    const int rb = q / NC, j = q - rb * NC;
                    int sub = 0;
                    while (rb >= __ldg(&D.nb_end[sub])) ++sub;            // the matrix that row block rb belongs to
                    const uint8_t* src = ldg_ptr<const uint8_t>(&D.packed[sub]) + kHeaderBytes +
                                         (size_t)(rb - (sub ? __ldg(&D.nb_end[sub - 1]) : 0)) * rbb + (size_t)j * C::QB;
                    // the slot's previous occupant must have been read
                    if (wrapped && !*dead && !mbar_test_wait(&my_empty[slot], parity ^ 1u) &&
                        !mbar_wait_bounded(&my_empty[slot], parity ^ 1u, kMaxBarPolls)) {
                        *dead = 1;
                        atomicOr(status, 0x400u | (uint32_t)(p & 0xFF));
                    }
                    if (!*dead) {
                        const uint32_t bytes = (j == NC - 1) ? last_bytes : (uint32_t)C::QB;
                        mbar_arrive_expect_tx(&my_full[slot], bytes);
                        bulk_g2s_hint(my_ring + (size_t)slot * C::QB, src, bytes, &my_full[slot], stream_policy);
                        ++issued;
                    }
                    if (++slot == R) { slot = 0; parity ^= 1u; wrapped = true; }
                }
            }
            // no bulk copy may still be in flight into this CTA's shared memory when it exits: wait for
            // the last use of each of the lane's slots (after a give-up nothing more was issued: sleep
            // instead, far longer than a copy takes)
            if (!*dead) {
                for (int n = issued > R ? issued - R : 0; n < issued; ++n)
                    if (!mbar_wait_bounded_compact(&my_full[n % R], (uint32_t)(n / R) & 1u, kMaxBarPolls)) {
                        atomicOr(status, 0x800u);
                        break;
                    }
            } else {
                for (int i = 0; i < 50; ++i) __nanosleep(1000);
            }
        }
    } else if (warp == W + 1) {
        // =================== signaller: publishes "problem p complete" off the consumers' critical path ===========
        // The release-ordered add waits until the CTA's output stores are visible GPU-wide (most of a
        // microsecond); the consumers only leave a note in shared memory and move on.
        if (lane == 0) {
            uint32_t seen = 0;
            for (int p = 0; p < H.count; ++p) {
                const StackProblem& D = sD[p];
                const int NC = __ldg(&D.NC);
                int q0, q1;
                cta_range(__ldg(&D.NB), NC, __ldg(&D.gran), virtual_cta(cta, __ldg(&D.rot), n_ctas), n_ctas, q0, q1);
                if (q0 >= q1) continue;
                const int stored = (q1 + NC - 1) / NC - (q0 + NC - 1) / NC;   // row blocks whose first quantum is here
                ++seen;
                bool ok = false;
                for (uint32_t it = 0; it < (1u << 24); ++it) {
                    if (ld_acquire_cta_u32(finished) >= seen) { ok = true; break; }
                    if (*dead) break;
                    __nanosleep(20);
                }
                if (!ok) break;   // a wait elsewhere in the CTA gave up (or this one did: ~0.5 s)
                if (stored > 0) red_release_add(ws.flags + p, (uint32_t)stored);
            }
        }
    } else {
        // =================== consumers ===================
        const int r = lane >> 2, c = lane & 3;
        const int tokB = r % MP, gsB = r / MP;   // B-operand role of this lane: column r of the MMA
        BFrag<GROUP, MP, false> B;
        float C1[C::NSETS][2], C2[C::NSETS][2];
        uint32_t n_finished = 0;                  // problems this CTA has stored outputs of
        // this warp's slots of the ring, used in order across problems
        const uint8_t* my_ring = ring + (size_t)warp * R * C::QB;
        uint64_t* my_full = full + warp * R;
        uint64_t* my_empty = empty + warp * R;
        int slot = 0;
        uint32_t parity = 0;
        const int ctid = threadIdx.x;             // 0 .. W*32-1

        for (int p = 0; p < H.count; ++p) {
            // the next descriptors into L1 (192 bytes = two lines each), off the critical path
            if (ctid < 8 && p + 1 + (ctid >> 1) < H.count)
                asm volatile("prefetch.global.L1 [%0];" ::"l"(reinterpret_cast<const uint8_t*>(sD + p + 1 + (ctid >> 1)) + 128 * (ctid & 1)));
            const StackProblem& D = sD[p];
            const int NB = __ldg(&D.NB), NC = __ldg(&D.NC), K = __ldg(&D.K), gran = __ldg(&D.gran);
            int q0, q1;
            const int cv = virtual_cta(cta, __ldg(&D.rot), n_ctas);
            cta_range(NB, NC, gran, cv, n_ctas, q0, q1);
            const int n = q1 - q0;
            if (n <= 0) continue;   // uniform over the CTA
            const int weff = __ldg(&D.weff);
            const int last_ns = __ldg(&D.NS) - 8 * (NC - 1);
            const __half* xbase = ldg_ptr<const __half>(&D.x);

            // ---- dependencies: the problems whose outputs (or side effects) x depends on.  ONE thread of
            // the CTA polls their counters: a counter polled by every warp of every SM is a hot spot ----
            const int n_deps = __ldg(&D.n_deps);
            if (n_deps > 0) {
                if (ctid == 0 && !*dead) {
                    for (int d = 0; d < n_deps; ++d) {
                        const uint32_t target = tag * (uint32_t)__ldg(&D.deps_nb[d]);
                        const uint32_t* f = ws.flags + __ldg(&D.deps[d]);
                        bool ok = false;
                        for (uint32_t it = 0; it < kMaxFlagPolls; ++it) {
                            if (ld_acquire_u32(f) == target) { ok = true; break; }
                            if ((it & 255u) == 255u && *dead) break;
                        }
                        if (!ok) {
                            if (!*dead) atomicOr(status, 0x100u | (uint32_t)(p & 0xFF));
                            *dead = 1;
                            break;
                        }
                    }
                }
                bar_sync(1, W * 32);
            }
            // ---- the k-chunks of x this CTA needs -> shared memory, each 16-byte piece fetched once per
            // SM (read past L1: another SM may have written x during this launch) ----
            const int nch = n < NC ? n : NC;                 // distinct chunks among the CTA's quanta
            const int j_first = n < NC ? q0 % NC : 0;
            const bool staged = __ldg(&D.stage_x) != 0;
            if (staged) {
                // piece = 8 consecutive k (16 bytes); 8 * SPG consecutive pieces = one group, held by
                // neighbouring lanes, which add up the group's sums of x on the way
                const int pieces = nch * H.M * 64;   // a multiple of 64: whole warps run each iteration
                for (int idx = ctid; idx < pieces; idx += W * 32) {
                    const int cl = idx / (H.M * 64), rem = idx - cl * (H.M * 64);
                    const int tok = rem >> 6, piece = rem & 63;
                    int j = j_first + cl;
                    j = j >= NC ? j - NC : j;
                    const int k = j * kChunkK + piece * 8;
                    uint4 u = make_uint4(0, 0, 0, 0);
                    if (k < K) u = __ldcg(reinterpret_cast<const uint4*>(xbase + (size_t)tok * K + k));
                    xs[idx] = u;
                    const float2 a0 = h2f2(u.x), a1 = h2f2(u.y), b0 = h2f2(u.z), b1 = h2f2(u.w);
                    float lo = (a0.x + a0.y) + (a1.x + a1.y), hi = (b0.x + b0.y) + (b1.x + b1.y);
#pragma unroll
                    for (int m = 1; m < 8 * C::SPG; m <<= 1) {
                        lo += __shfl_xor_sync(0xffffffffu, lo, m);
                        hi += __shfl_xor_sync(0xffffffffu, hi, m);
                    }
                    if ((piece & (8 * C::SPG - 1)) == 0)
                        xsum[(size_t)(idx >> 6) * C::GC + piece / (8 * C::SPG)] = make_float2(1024.f * lo + 64.f * hi, lo + hi);
                }
                bar_sync(1, W * 32);
            }

            int cur_j = -1;
            {
                if (warp < weff)
                for (int i = warp; i < n; i += weff) {
                    const int q = q0 + i;
                    const int rb = q / NC, j = q - rb * NC;
                    const int ns = (j == NC - 1) ? last_ns : 8;
                    const int ng = ns / C::SPG;
                    if (j != cur_j) {
                        cur_j = j;
                        // ---- activations of k-chunk j -> B fragments and per-group sums (read past L1:
                        // another SM may have written them during this launch) ----
                        int cl = j - j_first;
                        cl = cl < 0 ? cl + NC : cl;
                        // generic pointers: the staged copy in shared memory, or x itself in global memory
                        const __half* xk = staged ? reinterpret_cast<const __half*>(xs) + (size_t)cl * H.M * kChunkK
                                                  : xbase + (size_t)j * kChunkK;
                        const size_t xrow = staged ? (size_t)kChunkK : (size_t)K;   // distance between tokens
                        // a lane holds the slabs of its groups gsB + GPS * s only (other B entries are zero)
                        float lo[C::NSETS], hi[C::NSETS];
                        uint32_t Pm[C::NSETS][C::SPG][4][2];
#pragma unroll
                        for (int s = 0; s < C::NSETS; ++s) {
                            lo[s] = hi[s] = 0.f;
#pragma unroll
                            for (int sp = 0; sp < C::SPG; ++sp) {
                                const int sl = (gsB + C::GPS * s) * C::SPG + sp;
                                uint4 u0 = make_uint4(0, 0, 0, 0), u1 = u0;
                                if (sl < ns && tokB < H.M) {
                                    const uint4* px =
                                        reinterpret_cast<const uint4*>(xk + (size_t)tokB * xrow + sl * kSlabK4 + 16 * c);
                                    u0 = ld_volatile_v4(px);
                                    u1 = ld_volatile_v4(px + 1);
                                }
                                Pm[s][sp][0][0] = __byte_perm(u0.x, u0.y, 0x5410);
                                Pm[s][sp][0][1] = __byte_perm(u0.z, u0.w, 0x5410);
                                Pm[s][sp][1][0] = __byte_perm(u0.x, u0.y, 0x7632);
                                Pm[s][sp][1][1] = __byte_perm(u0.z, u0.w, 0x7632);
                                Pm[s][sp][2][0] = __byte_perm(u1.x, u1.y, 0x5410);
                                Pm[s][sp][2][1] = __byte_perm(u1.z, u1.w, 0x5410);
                                Pm[s][sp][3][0] = __byte_perm(u1.x, u1.y, 0x7632);
                                Pm[s][sp][3][1] = __byte_perm(u1.z, u1.w, 0x7632);
                                if (!staged) {   // the staged copy comes with its group sums
                                    float2 f;
                                    f = h2f2(u0.x); lo[s] += f.x + f.y;
                                    f = h2f2(u0.y); lo[s] += f.x + f.y;
                                    f = h2f2(u1.x); lo[s] += f.x + f.y;
                                    f = h2f2(u1.y); lo[s] += f.x + f.y;
                                    f = h2f2(u0.z); hi[s] += f.x + f.y;
                                    f = h2f2(u0.w); hi[s] += f.x + f.y;
                                    f = h2f2(u1.z); hi[s] += f.x + f.y;
                                    f = h2f2(u1.w); hi[s] += f.x + f.y;
                                }
                            }
                        }
#pragma unroll
                        for (int sl = 0; sl < 8; ++sl) {
                            const int gi = sl / C::SPG;
                            const bool mine = gsB == gi % C::GPS;
#pragma unroll
                            for (int a = 0; a < 4; ++a)
#pragma unroll
                                for (int b = 0; b < 2; ++b)
                                    B.v[sl][a][b] = mine ? Pm[gi / C::GPS][sl % C::SPG][a][b] : 0u;
                        }
                        if (staged) {
                            // correction terms of accumulator column 2c + e = (token, group slot) of tile s
#pragma unroll
                            for (int s = 0; s < C::NSETS; ++s)
#pragma unroll
                                for (int e = 0; e < 2; ++e) {
                                    const int tok = (2 * c + e) % MP, gi = s * C::GPS + (2 * c + e) / MP;
                                    float2 v = make_float2(0.f, 0.f);
                                    if (tok < H.M && gi < ng) v = xsum[((size_t)cl * H.M + tok) * C::GC + gi];
                                    C1[s][e] = v.x;
                                    C2[s][e] = v.y;
                                }
                        } else
#pragma unroll
                        for (int s = 0; s < C::NSETS; ++s) {
                            float l = lo[s], h = hi[s];
                            l += __shfl_xor_sync(0xffffffffu, l, 1);
                            h += __shfl_xor_sync(0xffffffffu, h, 1);
                            l += __shfl_xor_sync(0xffffffffu, l, 2);
                            h += __shfl_xor_sync(0xffffffffu, h, 2);
                            const float v1 = 1024.f * l + 64.f * h, v2 = l + h;
                            // correction terms of accumulator column 2c + e sit in the quad with r == that column
#pragma unroll
                            for (int e = 0; e < 2; ++e) {
                                C1[s][e] = __shfl_sync(0xffffffffu, v1, 4 * (2 * c + e));
                                C2[s][e] = __shfl_sync(0xffffffffu, v2, 4 * (2 * c + e));
                            }
                        }
                    }

                    // ---- this quantum's ring slot ----
                    if (!*dead && !mbar_test_wait(&my_full[slot], parity) &&
                        !mbar_wait_bounded(&my_full[slot], parity, kMaxBarPolls)) {
                        *dead = 1;
                        if (lane == 0) atomicOr(status, 0x200u | (uint32_t)(p & 0xFF));
                    }
                    const uint8_t* qp = my_ring + (size_t)slot * C::QB;
                    const uint4* slabs = reinterpret_cast<const uint4*>(qp);
                    float Dm[C::NSETS][4];
                    if (ns == 8) quantum_mma<GROUP, MP, true, false>(slabs, lane, 8, B, Dm);
                    else quantum_mma<GROUP, MP, false, false>(slabs, lane, ns, B, Dm);

                    float out[2][2] = {{0.f, 0.f}, {0.f, 0.f}};   // [row half h][column e]
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
                                    const float v = sz.x * ((Dm[s][2 * h + e] - C1[s][e]) - sz.y * C2[s][e]);
                                    out[h][e] += ok ? v : 0.f;
                                }
                            }
                    };
                    if (ns == 8) rescale(C::GC); else rescale(ng);
                    // the slot has been read: hand it back to the producer
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&my_empty[slot]);
                    if (++slot == R) { slot = 0; parity ^= 1u; }

                    if (MP == 1) { out[0][0] += out[0][1]; out[1][0] += out[1][1]; }
#pragma unroll
                    for (int h = 0; h < 2; ++h)
#pragma unroll
                        for (int e = 0; e < 2; ++e) {
                            if (MP <= 2) out[h][e] += __shfl_xor_sync(0xffffffffu, out[h][e], 1);
                            if (MP <= 4) out[h][e] += __shfl_xor_sync(0xffffffffu, out[h][e], 2);
                        }
                    const bool writer = (MP == 8) || (MP == 4 && c < 2) || (MP <= 2 && c == 0);
                    if (writer) {
#pragma unroll
                        for (int e = 0; e < (MP == 1 ? 1 : 2); ++e) {
                            const int tok = (2 * c + e) % MP;
#pragma unroll
                            for (int h = 0; h < 2; ++h) part[((size_t)i * MP + tok) * 16 + r + 8 * h] = out[h][e];
                        }
                    }
                }
            }

            // ---- the CTA's partial sums -> outputs; row blocks shared with other CTAs go through the workspace ----
            bar_sync(1, W * 32);
            const int rb_first = q0 / NC, rb_last = (q1 - 1) / NC;
            const int n_out = (rb_last - rb_first + 1) * MP * 16;
            unsigned long long* my_parts = ws.parts + ((size_t)p * n_ctas + cv) * (MP * 16);
            for (int o = ctid; o < n_out; o += W * 32) {
                const int row = o & 15, tok = (o >> 4) % MP, rb = rb_first + o / (16 * MP);
                const int qa = rb * NC, qb = qa + NC;          // the row block's quanta
                const int lo_q = qa > q0 ? qa : q0, hi_q = qb < q1 ? qb : q1;
                float acc = 0.f;
                for (int q = lo_q; q < hi_q; ++q) acc += part[((size_t)(q - q0) * MP + tok) * 16 + row];
                if (qa < q0) {
                    // the block starts in an earlier CTA, which finishes it: hand the partial sum over
                    st_relaxed_u64(my_parts + tok * 16 + row,
                                   ((unsigned long long)tag << 32) | (unsigned long long)__float_as_uint(acc));
                    continue;
                }
                if (qb > q1) {
                    // this CTA holds the block's first quantum: add the later (virtual) CTAs' parts in order
                    for (int c2 = cv + 1; c2 < n_ctas; ++c2) {
                        int r0, r1;
                        cta_range(NB, NC, gran, c2, n_ctas, r0, r1);
                        if (r0 >= qb) break;
                        if (r0 >= r1) continue;
                        const unsigned long long* src = ws.parts + ((size_t)p * n_ctas + c2) * (MP * 16) + tok * 16 + row;
                        unsigned long long v = 0;
                        bool ok = false;
                        if (!*dead) {
                            for (uint32_t it = 0; it < kMaxFlagPolls; ++it) {
                                v = ld_relaxed_u64(src);
                                if ((uint32_t)(v >> 32) == tag) { ok = true; break; }
                                if ((it & 255u) == 255u && *dead) break;
                            }
                            if (!ok) {
                                if (!*dead) atomicOr(status, 0x1000u | (uint32_t)(p & 0xFF));
                                *dead = 1;
                            }
                        }
                        acc += __uint_as_float((uint32_t)v);
                    }
                }
                int sub = 0;
                while (rb >= __ldg(&D.nb_end[sub])) ++sub;    // the matrix that row block rb belongs to
                const int nrow = (rb - (sub ? __ldg(&D.nb_end[sub - 1]) : 0)) * 16 + row, Ns = __ldg(&D.N[sub]);
                if (nrow < Ns && tok < H.M)
                    store_out(ldg_ptr<void>(&D.y[sub]), (__ldg(&D.y_dtypes) >> (8 * sub)) & 0xFF, (size_t)tok * Ns + nrow, acc);
            }
            // ---- completion: row blocks whose first quantum this CTA holds were stored by it ----
            bar_sync(1, W * 32);
            if (ctid == 0) st_release_cta_u32(finished, ++n_finished);   // the signaller warp takes it from here
        }
    }

    // ---- end of the launch: the last CTA to finish advances the workspace's launch counter ----
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        const uint32_t old = atomicAdd(ws.done, 1u);
        if (old == (uint32_t)n_ctas - 1u) {
            *reinterpret_cast<volatile uint32_t*>(ws.done) = 0u;
            *reinterpret_cast<volatile uint32_t*>(ws.epoch) = tag;
        }
    }
}

template <int GROUP, int MP>
size_t smem_of(int count, int slots, int max_quanta, int xs_bytes) {
    using C = Cfg<GROUP, MP>;
    (void)count;   // the descriptors stay in global memory
    return (size_t)slots * C::QB + (size_t)max_quanta * MP * 16 * 4 +
           (size_t)xs_bytes + (size_t)(xs_bytes / 1024) * C::GC * 8 + (size_t)2 * slots * 8 + 16;
}

template <int GROUP, int MP>
cudaError_t launch_one(const StackHeader& H, const void* plan_dev, const StackWorkspace& ws, uint32_t* status,
                       cudaStream_t stream) {
    auto kern = stack_w4a16_kernel<GROUP, MP>;
    // function attributes belong to a device: set per device, once
    static PerDevice<bool> configured;   // per instantiation and device
    if (cudaError_t e = configured.with([&](bool& done) {
            if (done) return cudaSuccess;
            cudaError_t err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
            done = err == cudaSuccess;
            return err;
        });
        e != cudaSuccess)
        return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)H.n_ctas);
    cfg.blockDim = dim3((unsigned)kStackThreads);
    cfg.dynamicSmemBytes = H.smem_bytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeCooperative;   // all CTAs resident together, or the launch fails
    attr[0].val.cooperative = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, H, reinterpret_cast<const StackProblem*>(plan_dev), ws, status);
}

}  // namespace

size_t stack_w4a16_smem(int group, int MP, int count, int slots, int max_quanta, int xs_bytes) {
#define MNN_CASE(G, P) if (group == G && MP == P) return smem_of<G, P>(count, slots, max_quanta, xs_bytes);
    MNN_CASE(64, 1) MNN_CASE(64, 2) MNN_CASE(64, 4) MNN_CASE(64, 8)
    MNN_CASE(128, 1) MNN_CASE(128, 2) MNN_CASE(128, 4) MNN_CASE(128, 8)
#undef MNN_CASE
    return 0;
}

cudaError_t stack_w4a16_launch(const StackHeader& H, const void* plan_dev, const StackWorkspace& ws, uint32_t* status,
                               cudaStream_t stream) {
#define MNN_CASE(G, P) if (H.group == G && H.MP == P) return launch_one<G, P>(H, plan_dev, ws, status, stream);
    MNN_CASE(64, 1) MNN_CASE(64, 2) MNN_CASE(64, 4) MNN_CASE(64, 8)
    MNN_CASE(128, 1) MNN_CASE(128, 2) MNN_CASE(128, 4) MNN_CASE(128, 8)
#undef MNN_CASE
    return cudaErrorInvalidValue;
}

}  // namespace mnnllm
