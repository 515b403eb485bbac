// Prefill W4A8 linear (Section 4.2: activations quantised to int8 so that integer matrix
// instructions can be used; Section 5.1 for the operand shapes):
//     P[m,n,g] = sum_{k in g} a_q[m,k] * q[n,k]                       int32, exact
//     y[m,n]   = a_scale[m] * ( sum_g s[n,g] * P[m,n,g]  -  sum_g (s z)[n,g] * A[m,g] )
//
// The MMA multiplies the activations in their unsigned form a_u = a_q + 128 (written so by the
// quantiser), so that its result P_u = P + 128 * Q[n,g], Q = sum of the group's codes, is never
// negative.  A non-negative int32 below 2^23 IS a (denormal) float, P_u * 2^-149, bit for bit: the
// drain needs no int->float conversion at all.  It subtracts the denormal 128 Q (exact) and
// multiplies by s * 2^100 in one FMA, two instructions per partial (one per partial with the
// packed f32x2 forms); the accumulators carry
// 2^-49 * sum_g s P and the epilogue scales back.  (cvt.rn.f32.s32 runs at 16 lanes per clock per SM
// and would bound the kernel at 1024 cycles per group; adding a float bit pattern as an integer
// and subtracting it as a float is exact too but costs three instructions per partial.)
//
// One CTA computes a tile of 128 weight rows x 128 tokens.  The weights are the M side of the MMA,
// so that a tensor-memory lane is one output channel n and its per-group scale is a per-thread
// scalar in the drain.  Warp roles (23 warps):
//   warp 0      producer: TMA loads of the packed int4 codes (the packed buffer seen as a 2-D tensor
//               [row block][bytes]: one box of 8 row blocks x 1 KiB per stage; issuing one small bulk
//               copy per row block instead costs ~75 cycles each and starves the pipeline) and of
//               each 512-k chunk's (scale, zero) tables into shared-memory rings; TMA loads of the
//               int8 activation tile (128 tokens x 128 k, 128B swizzle) and of the fp16 group-sum
//               quadruples that feed the zero-point MMA
//   warp 1      allocates tensor memory, issues tcgen05.mma (kind::i8 into one of three int32
//               accumulators per group; kind::f16 for the zero-point term) and the commits
//   warps 2-5   unpack: packed int4 codes (shared-memory ring) -> int8 K-major tile in the
//               128B-swizzled layout the MMA reads; the sum Q of every (row, group)'s codes
//   warp 22     scales: each (row, group) pair of the stage: the fp32 scale for the drain; (s z)
//               split into fp16 hi + lo for the zero-point MMA (a separate warp, because these
//               conversion chains would otherwise sit on the unpack warps' critical path)
//   warps 6-21  drain (four per lane quarter, 32 token columns each: the loop is a chain of
//               latencies, so more warps per scheduler hide it better than longer warps): every
//               group's 128 x 128 int32 partial tile leaves tensor memory
//               (tcgen05.ld) and is accumulated as acc += (s 2^100) * (P_u - 128 Q) in registers
//               while the MMA fills the other accumulators; epilogue applies the zero-point term and a_scale.
// The zero-point term is a rank-G product, evaluated on the tensor cores without loss:
//   (s z) = hi + lo (fp16 each; s and z are fp16, so the product has 22 significant bits),
//   A     = 64 h + l (both exact in fp16), four fp16 products per group, fp32 accumulation in a
//   third tensor-memory region; 4 groups fill one K = 16 MMA.
// Every wait is bounded: on a time-out the CTA records a code in the status word and all roles
// leave their loops, tensor memory is released and the kernel returns.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "gemm_w4a8.h"
#include "layout.h"
#include "ptx.cuh"

namespace mnnllm {

using namespace ptx;

namespace {

constexpr int kTileN = 128;   // weight rows per CTA tile (MMA M)
constexpr int kTileT = 128;   // tokens per CTA tile (MMA N)
constexpr int kStageK = 128;  // k per pipeline stage (one 128-byte swizzle row of int8)
constexpr int kStages = 4;
constexpr int kScaleSlots = 2 * kStages + 4;  // groups whose scales may be live at once (ring + accumulators + 1)
constexpr int kPkStages = 6;                  // ring of packed-code stages (8 KiB each)
constexpr int kPkLead = 2;                    // stages the packed ring is produced ahead of the activations
constexpr int kTabSlots = 3;                  // ring of per-chunk (scale, zero) tables (8 row blocks x 512 B)
constexpr int kDrainWarps = 16;
constexpr int kUnpackWarp0 = 2, kDrainWarp0 = 6, kScaleWarp = kDrainWarp0 + kDrainWarps;
constexpr int kThreads = (kScaleWarp + 1) * 32;
constexpr uint32_t kMaxPolls = 1u << 15;  // x 20 us per try: gives up after ~0.65 s
constexpr int kAcc = 3;                       // int32 group accumulators in tensor memory (128 columns each)
constexpr uint32_t kTmemCols = 512;           // 3 x 128 int32 accumulators + 128 fp32 zero-point term
constexpr uint32_t kColCorr = kAcc * 128;

constexpr int kStageBytes = kTileN * kStageK;  // 16 KiB, int8
constexpr int kCorrBytes = 128 * 32;           // 128 rows x 16 fp16
constexpr int kPkBytes = 8 * 2 * kSlabBytes;   // packed codes of a stage: 8 row blocks x 2 slabs
constexpr int kTabBytes = 8 * 512;             // (scale, zero) tables of a chunk: 8 row blocks x 16 rows x 8 pairs

struct Smem {
    static constexpr int wq = 0;
    static constexpr int aq = wq + kStages * kStageBytes;
    static constexpr int ca = aq + kStages * kStageBytes;
    static constexpr int cb = ca + 2 * kCorrBytes;
    static constexpr int pk = cb + 2 * kCorrBytes;
    static constexpr int tab = pk + kPkStages * kPkBytes;
    static constexpr int scale = tab + kTabSlots * kTabBytes;        // per (group slot, row): {s * 2^100, 128 * Q}
    static constexpr int bars = scale + kScaleSlots * kTileN * 8;
    static constexpr int n_bars = 2 * kStages + 2 * kAcc + 2 + 2 + 2 + 2 * kPkStages + 2 * kTabSlots;
    static constexpr int misc = bars + n_bars * 8;
    static constexpr int total = misc + 16;
};
constexpr size_t kSmemBytes = Smem::total + 1024;  // slack to align the base to 1024 bytes

struct Problem {
    void* y;
    int N, n_row_blocks, y_dtype;
    int tile_begin;   // first weight-row tile of this matrix among the launch's row tiles
};
struct Params {
    const float* a_scale;
    int32_t* P;
    int M, K, G;
    int n_slabs, n_stages, count;
    int tiles_m, total_tiles;   // token tiles; all (weight tile, token tile) pairs of the launch
    unsigned long long chunk_bytes;
    Problem prob[kGemmMaxBatch];
};
struct WeightMaps {   // the packed bodies as 2-D tensors: codes box and table box per weight matrix
    CUtensorMap pk[kGemmMaxBatch], tab[kGemmMaxBatch];
};

// K-major operand tile whose rows are 128 bytes, 128B swizzle: 8-row groups are 1024 bytes apart.
__device__ __forceinline__ uint64_t desc_sw128(uint32_t smem_addr) {
    return (uint64_t)((smem_addr & 0x3FFFFu) >> 4) | (1ull << 16) | (64ull << 32) | (1ull << 46) | (2ull << 61);
}
// K-major operand tile whose rows are 32 bytes, 32B swizzle: 8-row groups are 256 bytes apart.
__device__ __forceinline__ uint64_t desc_sw32(uint32_t smem_addr) {
    return (uint64_t)((smem_addr & 0x3FFFFu) >> 4) | (1ull << 16) | (16ull << 32) | (1ull << 46) | (6ull << 61);
}
// instruction descriptors: D format (bits 4-5), A/B formats (7-9, 10-12), both K-major, N >> 3 at
// bit 17, M >> 4 at bit 24
// (kind::i8 formats: 0 = unsigned, 1 = signed 8 bit; codes 0..15 and activations a_q + 128 are both unsigned)
constexpr uint32_t kIdescI8 = (2u << 4) | (0u << 7) | (0u << 10) | ((kTileT >> 3) << 17) | ((kTileN >> 4) << 24);
constexpr uint32_t kIdescF16 = (1u << 4) | (0u << 7) | (0u << 10) | ((kTileT >> 3) << 17) | ((kTileN >> 4) << 24);

__device__ __forceinline__ void store_y(void* y, int dtype, size_t idx, float v) {
    if (dtype == MNNLLM_F16) reinterpret_cast<__half*>(y)[idx] = __float2half_rn(v);
    else if (dtype == MNNLLM_BF16) reinterpret_cast<__nv_bfloat16*>(y)[idx] = __float2bfloat16_rn(v);
    else reinterpret_cast<float*>(y)[idx] = v;
}

template <int GROUP, bool PARTIALS>
__global__ void __launch_bounds__(kThreads, 1)   // 80 registers: 84 would not spill, but 23 warps x 84 do not fit the register file's allocation units
gemm_w4a8_kernel(const __grid_constant__ CUtensorMap tm_act, const __grid_constant__ CUtensorMap tm_ac,
                 const __grid_constant__ WeightMaps wmaps, const __grid_constant__ Params p,
                 uint32_t* __restrict__ status) {
    constexpr int GPS = kStageK / GROUP;  // groups per stage (2 or 1)
    constexpr int SPB = 4 / GPS;          // stages per block of four groups (zero-point MMA cadence)
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + Smem::bars);
    uint64_t* ab_full = bars;
    uint64_t* ab_empty = ab_full + kStages;
    uint64_t* tm_full = ab_empty + kStages;
    uint64_t* tm_empty = tm_full + kAcc;
    uint64_t* c_full = tm_empty + kAcc;
    uint64_t* c_empty = c_full + 2;
    uint64_t* corr_done = c_empty + 2;
    uint64_t* corr_free = corr_done + 1;
    uint64_t* pk_full = corr_free + 1;
    uint64_t* pk_empty = pk_full + kPkStages;
    uint64_t* tab_full = pk_empty + kPkStages;
    uint64_t* tab_empty = tab_full + kTabSlots;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + Smem::misc);
    volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(smem + Smem::misc + 4);
    uint2* sq_ring = reinterpret_cast<uint2*>(smem + Smem::scale);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_stages = p.n_stages, G = p.G;
    const int n_cblk = (G + 3) >> 2;   // blocks of four groups (one zero-point MMA each) per tile
    const int total_tiles = p.total_tiles;

    // The CTA is persistent: it works through the tiles blockIdx.x, blockIdx.x + gridDim.x, ...
    // Every ring and barrier keeps running across tiles (slots and parities come from running
    // counts), so the producer, unpack, scale and MMA roles start on the next tile while the
    // drain warps are still in the epilogue of the current one.  The token tile index runs
    // fastest: CTAs that work at the same time share their weight tile.
    struct Tile { int pi, n0, m0; };
    auto tile_of = [&](int t) {
        Tile c;
        const int tn = t / p.tiles_m;
        c.m0 = (t - tn * p.tiles_m) * kTileT;
        c.pi = 0;
        while (c.pi + 1 < p.count && tn >= p.prob[c.pi + 1].tile_begin) ++c.pi;
        c.n0 = (tn - p.prob[c.pi].tile_begin) * kTileN;
        return c;
    };

    if (threadIdx.x == 0) {
        for (int i = 0; i < kStages; ++i) { mbar_init(&ab_full[i], 6); mbar_init(&ab_empty[i], 1); }
        for (int i = 0; i < kAcc; ++i) { mbar_init(&tm_full[i], 1); mbar_init(&tm_empty[i], kDrainWarps); }
        for (int i = 0; i < 2; ++i) { mbar_init(&c_full[i], 2); mbar_init(&c_empty[i], 1); }
        mbar_init(corr_done, 1);
        mbar_init(corr_free, kDrainWarps);
        for (int i = 0; i < kPkStages; ++i) { mbar_init(&pk_full[i], 1); mbar_init(&pk_empty[i], 4); }
        for (int i = 0; i < kTabSlots; ++i) { mbar_init(&tab_full[i], 1); mbar_init(&tab_empty[i], 1); }
        *abort_flag = 0;
        fence_mbar_init();
        prefetch_tensormap(&tm_act);
        for (int i = 0; i < p.count; ++i) {
            prefetch_tensormap(&wmaps.pk[i]);
            prefetch_tensormap(&wmaps.tab[i]);
        }
        if (!PARTIALS) prefetch_tensormap(&tm_ac);
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    // Programmatic dependent launch: this grid may start while the activation quantiser still runs.
    // Everything up to here and the whole weight side (packed codes, tables, unpack, scales) does
    // not depend on it; the threads that read its outputs (activation codes and group sums through
    // TMA, a_scale in the epilogue) call griddepcontrol.wait first.
    pdl_launch_dependents();

    // a failed wait marks the CTA as aborted; every role then leaves its loops
    // (every lane polls: letting one lane poll and broadcasting its verdict was measured slower)
    auto wait = [&](uint64_t* bar, uint32_t parity, uint32_t code) -> bool {
        if (mbar_wait_bounded_compact(bar, parity, kMaxPolls)) return true;
        if (*abort_flag == 0) {
            *abort_flag = 1;
            atomicOr(status, 0x200u | code);
        }
        return false;
    };

    if (warp == 0) {
        // ------------------------------------------------------------------ producer (TMA)
        // One elected thread runs the whole loop: every step is a wait and a copy by one thread.
        // Two cursors walk the same (tile, stage) sequence: the packed codes (with each 512-k
        // chunk's scale/zero tables) run kPkLead stages ahead of the activations.
        if (elect_one()) {
            int t_pk = blockIdx.x, i_pk = 0, t_ac = blockIdx.x, st = 0, lead = 0;
            uint32_t ip = 0, jc = 0, gs = 0, cb = 0;   // running counts: packed stages, chunks, stages, zero-point blocks
            Tile cp = tile_of(t_pk), ca = cp;
            bool first = true;
            while (t_ac < total_tiles) {
                if (t_pk < total_tiles) {
                    const int pslot = ip % kPkStages, j = i_pk >> 2, rb0 = cp.n0 / kRowsPerBlock;
                    if (!wait(&pk_empty[pslot], ((ip / kPkStages) & 1) ^ 1, 10)) break;
                    const int ns_chunk = (p.n_slabs - 8 * j) < 8 ? (p.n_slabs - 8 * j) : 8;
                    const unsigned long long chunk_off = (unsigned long long)j * p.chunk_bytes;
                    // boxes are counted in full even where they run past the tensor (zero fill)
                    if ((i_pk & 3) == 0) {
                        const int tslot = jc % kTabSlots;
                        if (!wait(&tab_empty[tslot], ((jc / kTabSlots) & 1) ^ 1, 12)) break;
                        mbar_arrive_expect_tx(&tab_full[tslot], kTabBytes);
                        tma_load_2d(smem + Smem::tab + tslot * kTabBytes, &wmaps.tab[cp.pi],
                                    (int)((chunk_off + (unsigned long long)ns_chunk * kSlabBytes) >> 2), rb0, &tab_full[tslot]);
                        ++jc;
                    }
                    mbar_arrive_expect_tx(&pk_full[pslot], kPkBytes);
                    tma_load_2d(smem + Smem::pk + pslot * kPkBytes, &wmaps.pk[cp.pi],
                                (int)((chunk_off + (unsigned long long)(i_pk & 3) * 2 * kSlabBytes) >> 2), rb0, &pk_full[pslot]);
                    ++ip;
                    ++lead;
                    if (++i_pk == n_stages) {
                        i_pk = 0;
                        t_pk += gridDim.x;
                        if (t_pk < total_tiles) cp = tile_of(t_pk);
                    }
                }
                if (lead > kPkLead || t_pk >= total_tiles) {
                    if (first) { pdl_wait(); first = false; }   // the quantised activations are complete from here on
                    const int slot = gs % kStages;
                    if (!wait(&ab_empty[slot], ((gs / kStages) & 1) ^ 1, 1)) break;
                    mbar_arrive_expect_tx(&ab_full[slot], kTileT * kStageK);
                    tma_load_2d(smem + Smem::aq + slot * kStageBytes, &tm_act, st * kStageK, ca.m0, &ab_full[slot]);
                    if (!PARTIALS && st % SPB == 0) {
                        const int cslot = cb & 1;
                        if (!wait(&c_empty[cslot], ((cb >> 1) & 1) ^ 1, 2)) break;
                        mbar_arrive_expect_tx(&c_full[cslot], kTileT * 32);
                        tma_load_2d(smem + Smem::cb + cslot * kCorrBytes, &tm_ac, (st / SPB) * 16, ca.m0, &c_full[cslot]);
                        ++cb;
                    }
                    ++gs;
                    --lead;
                    if (++st == n_stages) {
                        st = 0;
                        t_ac += gridDim.x;
                        if (t_ac < total_tiles) ca = tile_of(t_ac);
                    }
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issue
        // One elected thread runs the whole loop (waits, MMAs and commits are single-thread
        // operations; the issue path is a serial chain of ~50-cycle steps, so nothing is spent on
        // re-electing or re-converging the warp per stage).  A group's MMAs are issued as soon as
        // its own accumulator has been drained.
        if (elect_one()) {
            int b = 0, it = 0;
            uint32_t epar = 1;        // parity of the tm_empty phase that frees accumulator b
            uint32_t gs = 0, cb = 0;  // running counts of stages and zero-point blocks
            const uint32_t wq_addr = smem_u32(smem + Smem::wq), aq_addr = smem_u32(smem + Smem::aq);
            bool ok = true;
            for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x, ++it) {
                int gcount = 0;
                bool cfirst = true;
                for (int st = 0; st < n_stages && ok; ++st, ++gs) {
                    const int slot = gs % kStages;
                    const int ngr = (G - st * GPS) < GPS ? (G - st * GPS) : GPS;
                    if (!wait(&ab_full[slot], (gs / kStages) & 1, 3)) { ok = false; break; }
                    const uint64_t da = desc_sw128(wq_addr + slot * kStageBytes);
                    const uint64_t db = desc_sw128(aq_addr + slot * kStageBytes);
                    for (int gi = 0; gi < ngr; ++gi) {
                        if (!wait(&tm_empty[b], epar, 4)) { ok = false; break; }
                        tc_fence_after_sync();
#pragma unroll
                        for (int kk = 0; kk < GROUP / 32; ++kk) {
                            const uint64_t adv = (uint64_t)((gi * GROUP + kk * 32) >> 4);
                            mma_i8_ss(tmem_base + b * kTileT, da + adv, db + adv, kIdescI8, kk > 0);
                        }
                        mma_commit(&tm_full[b]);
                        if (++b == kAcc) { b = 0; epar ^= 1u; }
                    }
                    if (!ok) break;
                    mma_commit(&ab_empty[slot]);
                    gcount += ngr;
                    if (!PARTIALS && ((gcount & 3) == 0 || st == n_stages - 1)) {
                        const int cslot = cb & 1;
                        if (!wait(&c_full[cslot], (cb >> 1) & 1, 5)) { ok = false; break; }
                        // the previous tile's zero-point term must have left tensor memory
                        if (cfirst && it > 0 && !wait(corr_free, (it - 1) & 1, 15)) { ok = false; break; }
                        tc_fence_after_sync();
                        mma_f16_ss(tmem_base + kColCorr, desc_sw32(smem_u32(smem + Smem::ca + cslot * kCorrBytes)),
                                   desc_sw32(smem_u32(smem + Smem::cb + cslot * kCorrBytes)), kIdescF16, !cfirst);
                        mma_commit(&c_empty[cslot]);
                        cfirst = false;
                        ++cb;
                    }
                }
                if (!PARTIALS && ok) mma_commit(corr_done);
            }
        }
        __syncwarp();
    } else if (warp < kDrainWarp0) {
        // ------------------------------------------------------------------ unpack
        const int wu = warp - kUnpackWarp0;
        const int r = lane >> 2, c = lane & 3;
        // Lanes of odd rows take the two slabs of a row block in the other order: the 16-byte
        // stores of rows 2p and 2p + 1 (one shared-memory wavefront) then fall into different
        // halves of the 128-byte swizzle row instead of colliding two-way.
        const int odd = r & 1;
        uint32_t ip = 0, gs = 0, gg = 0;   // running counts: packed stages, stages, groups (at the tile's start)
        bool ok = true;
        for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x, gg += G) {
            const Tile tc = tile_of(t);
            const Problem& q = p.prob[tc.pi];
            const int nrb = (q.n_row_blocks - tc.n0 / kRowsPerBlock) < 8 ? (q.n_row_blocks - tc.n0 / kRowsPerBlock) : 8;
            for (int st = 0; st < n_stages; ++st, ++ip, ++gs) {
                const int slot = gs % kStages, pslot = ip % kPkStages, j = st >> 2;
                const int ns_chunk = (p.n_slabs - 8 * j) < 8 ? (p.n_slabs - 8 * j) : 8;
                if (!wait(&pk_full[pslot], (ip / kPkStages) & 1, 11)) { ok = false; break; }
                // this thread's four 16-byte entries of the stage (zero where the tile or K runs out)
                uint4 cur[4];
                {
                    const uint4* pk = reinterpret_cast<const uint4*>(smem + Smem::pk + pslot * kPkBytes);
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int sidx = wu * 4 + (i ^ odd);   // row blocks 2 wu and 2 wu + 1, both slabs of each
                        const bool valid = (sidx >> 1) < nrb && (st & 3) * 2 + (sidx & 1) < ns_chunk;
                        cur[i] = valid ? pk[sidx * 32 + lane] : make_uint4(0, 0, 0, 0);
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&pk_empty[pslot]);
                // codes -> int8 (registers) before the stage's slot is waited for; then only the stores
                // (doing the conversion after the wait instead was measured 8 % slower end to end)
                constexpr uint32_t M4 = 0x0F0F0F0Fu;
                uint4 lo8[4], hi8[4];
                uint32_t q0[4], q1[4];   // sums of the codes of rows R0 and R0 + 8 over the slab (after the lane reduction)
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const uint4 w = cur[i];
                    lo8[i] = make_uint4(w.x & M4, (w.x >> 4) & M4, w.y & M4, (w.y >> 4) & M4);   // row R0
                    hi8[i] = make_uint4(w.z & M4, (w.z >> 4) & M4, w.w & M4, (w.w >> 4) & M4);   // row R0 + 8
                    uint32_t a = __dp4a(lo8[i].x, 0x01010101u, 0u), b = __dp4a(hi8[i].x, 0x01010101u, 0u);
                    a = __dp4a(lo8[i].y, 0x01010101u, a); b = __dp4a(hi8[i].y, 0x01010101u, b);
                    a = __dp4a(lo8[i].z, 0x01010101u, a); b = __dp4a(hi8[i].z, 0x01010101u, b);
                    a = __dp4a(lo8[i].w, 0x01010101u, a); b = __dp4a(hi8[i].w, 0x01010101u, b);
                    // the four lanes 4r .. 4r+3 hold the four 16-k pieces of the same rows
                    a += __shfl_xor_sync(0xffffffffu, a, 1); b += __shfl_xor_sync(0xffffffffu, b, 1);
                    a += __shfl_xor_sync(0xffffffffu, a, 2); b += __shfl_xor_sync(0xffffffffu, b, 2);
                    q0[i] = a; q1[i] = b;
                }
                if (!wait(&ab_empty[slot], ((gs / kStages) & 1) ^ 1, 6)) { ok = false; break; }
                // 128B-swizzled K-major rows
                uint8_t* wq = smem + Smem::wq + slot * kStageBytes;
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int sidx = wu * 4 + (i ^ odd);
                    const int R0 = (sidx >> 1) * 16 + r;          // rows R0 and R0 + 8 of the tile
                    const int kc = (sidx & 1) * 4 + c;            // 16-byte chunk of the 128-byte row
                    const uint32_t off = (uint32_t)(R0 >> 3) * 1024u + (uint32_t)r * 128u + (uint32_t)((kc ^ r) << 4);
                    *reinterpret_cast<uint4*>(wq + off) = lo8[i];
                    *reinterpret_cast<uint4*>(wq + off + 1024u) = hi8[i];
                }
                // 128 * Q per (row, group) for the drain: a slab is a group of 64, two slabs a group of 128
                if (c == 0) {
                    const uint32_t gslot0 = (gg + (uint32_t)st * GPS) % kScaleSlots;
#pragma unroll
                    for (int i = 0; i < 4; i += (GROUP == 64 ? 1 : 2)) {
                        const int gl = GROUP == 64 ? ((i ^ odd) & 1) : 0;   // group of the stage
                        if (st * GPS + gl < G) {
                            const uint32_t gslot = (gslot0 + gl == kScaleSlots) ? 0u : gslot0 + gl;
                            const int R0 = (wu * 2 + (i >> 1)) * 16 + r;
                            const uint32_t s0 = GROUP == 64 ? q0[i] : q0[i] + q0[i + 1];
                            const uint32_t s1 = GROUP == 64 ? q1[i] : q1[i] + q1[i + 1];
                            sq_ring[gslot * kTileN + R0].y = 128u * s0;
                            sq_ring[gslot * kTileN + R0 + 8].y = 128u * s1;
                        }
                    }
                }
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) mbar_arrive(&ab_full[slot]);
            }
        }
    } else if (warp == kScaleWarp) {
        // ------------------------------------------------------------------ scales and (s z) halves
        uint32_t gs = 0, jc = 0, gg = 0, cbase = 0;   // running counts: stages, chunks, groups and zero-point blocks (at the tile's start)
        bool ok = true;
        for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x, gg += G, cbase += n_cblk) {
            const Tile tc = tile_of(t);
            const Problem& q = p.prob[tc.pi];
            const int nrb = (q.n_row_blocks - tc.n0 / kRowsPerBlock) < 8 ? (q.n_row_blocks - tc.n0 / kRowsPerBlock) : 8;
            uint32_t tslot = 0;
            for (int st = 0; st < n_stages && ok; ++st, ++gs) {
                const int slot = gs % kStages;
                const int j = st >> 2;
                const int ns_chunk = (p.n_slabs - 8 * j) < 8 ? (p.n_slabs - 8 * j) : 8;
                const int ng = ns_chunk * kSlabK4 / GROUP;
                if ((st & 3) == 0) {
                    tslot = jc % kTabSlots;
                    if (!wait(&tab_full[tslot], (jc / kTabSlots) & 1, 13)) { ok = false; break; }
                    ++jc;
                }
                // this lane's rows: lane, lane + 32, lane + 64, lane + 96
                uint32_t zc[4][GPS];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int row = lane + 32 * i;
                    const uint32_t* tab = reinterpret_cast<const uint32_t*>(smem + Smem::tab + tslot * kTabBytes + (row >> 4) * 512);
#pragma unroll
                    for (int gi = 0; gi < GPS; ++gi) {
                        const int gc = (st & 3) * GPS + gi;
                        zc[i][gi] = ((row >> 4) < nrb && gc < ng) ? tab[(row & 15) * ng + gc] : 0u;
                    }
                }
                if ((st & 3) == 3 || st == n_stages - 1) {  // the chunk's table has been read in full
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&tab_empty[tslot]);
                }
                // The conversion chains and the zero-point tile (which has its own flow control) come
                // first; only the cheap publication of the scales waits for the stage's slot, so that
                // this warp is never what the MMA waits for.
                float sreg[4][GPS];
#pragma unroll
                for (int gi = 0; gi < GPS; ++gi) {
                    const int g = st * GPS + gi;
                    if (g >= G) break;
                    const int pos = g & 3;
                    const uint32_t cb = cbase + (uint32_t)(g >> 2);
                    const int cslot = cb & 1;
                    if (!PARTIALS && pos == 0 && !wait(&c_empty[cslot], ((cb >> 1) & 1) ^ 1, 7)) { ok = false; break; }
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int row = lane + 32 * i;
                        const __half2 h2 = *reinterpret_cast<const __half2*>(&zc[i][gi]);
                        const float s = __low2float(h2), z = __high2float(h2);
                        sreg[i][gi] = s;
                        if (!PARTIALS) {
                            const float szf = s * z;  // exact: 11-bit x 11-bit significands
                            const __half hi = __float2half_rn(szf);
                            const __half lo = __float2half_rn(szf - __half2float(hi));
                            const uint32_t hh = (uint32_t)__half_as_ushort(hi) * 0x00010001u;
                            const uint32_t ll = (uint32_t)__half_as_ushort(lo) * 0x00010001u;
                            uint8_t* tile = smem + Smem::ca + cslot * kCorrBytes;
                            const int rowoff = (row >> 3) * 256 + (row & 7) * 32, sw = (row & 7) >> 2;
                            *reinterpret_cast<uint2*>(tile + rowoff + (((pos >> 1) ^ sw) << 4) + (pos & 1) * 8) = make_uint2(hh, ll);
                            if (g == G - 1)
                                for (int e = pos + 1; e < 4; ++e)
                                    *reinterpret_cast<uint2*>(tile + rowoff + (((e >> 1) ^ sw) << 4) + (e & 1) * 8) = make_uint2(0u, 0u);
                        }
                    }
                    if (!PARTIALS && (pos == 3 || g == G - 1)) {
                        fence_proxy_async_smem();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(&c_full[cslot]);
                    }
                }
                if (!ok) break;
                if (!wait(&ab_empty[slot], ((gs / kStages) & 1) ^ 1, 14)) { ok = false; break; }
                const uint32_t gslot0 = (gg + (uint32_t)st * GPS) % kScaleSlots;
#pragma unroll
                for (int gi = 0; gi < GPS; ++gi) {
                    if (st * GPS + gi >= G) break;
                    const uint32_t gslot = (gslot0 + gi == kScaleSlots) ? 0u : gslot0 + gi;
#pragma unroll
                    for (int i = 0; i < 4; ++i)   // s * 2^100 (the drain's operand is the denormal P * 2^-149)
                        sq_ring[gslot * kTileN + lane + 32 * i].x = __float_as_uint(__fmul_rn(sreg[i][gi], 0x1p100f));
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&ab_full[slot]);
            }
        }
    } else {
        // ------------------------------------------------------------------ drain + epilogue
        const int q4 = warp & 3;                      // tensor-memory lane quarter this warp may read
        const int part = (warp - kDrainWarp0) >> 2;   // which 32 token columns
        const int nl = q4 * 32 + lane;
        const uint32_t lane_base = tmem_base + ((uint32_t)(q4 * 32) << 16) + part * 32;
        // The loop is a chain of latencies, so everything that can be started early is: ring
        // positions are counters (no divisions), the group's scale and 128 Q come in one load, and
        // the next group's barrier is probed (non-blocking) while this group's partials are in
        // flight, so that the usual case enters the next iteration without waiting at all.
        // One counter of groups modulo 12 gives the scale slot (ss), the accumulator (ss % 3) and the
        // parity of its barrier ((ss / 3) & 1): 12 is a multiple of both rings' periods (3 and 6).
        uint32_t ss = 0;
        bool ready = false;
        const uint2* sq_lane = sq_ring + nl;
        for (int t = blockIdx.x; t < total_tiles; t += gridDim.x) {
            uint64_t acc2[16];   // 32 fp32 accumulators as packed pairs (columns 2j, 2j + 1)
#pragma unroll
            for (int i = 0; i < 16; ++i) acc2[i] = 0ull;
            bool ok = true;
            for (int g = 0; g < G; ++g) {
                const uint32_t b = (0x924924u >> (2 * ss)) & 3u;   // ss % 3
                const uint32_t par = (0xE38u >> ss) & 1u;          // (ss / 3) & 1
                if (!ready && !wait(&tm_full[b], par, 8)) { ok = false; break; }
                tc_fence_after_sync();
                uint32_t v[32];
                tmem_ld_x32(lane_base + b * kTileT, v);
                const uint2 sq = sq_lane[ss * kTileN];
                const float sf = __uint_as_float(sq.x);
                const uint32_t qb_bits = sq.y;   // 128 Q, also the float 128 Q 2^-149
                const uint32_t sn = (ss + 1 == kScaleSlots) ? 0u : ss + 1;
                ready = __all_sync(0xffffffffu, mbar_test_wait(&tm_full[(0x924924u >> (2 * sn)) & 3u], (0xE38u >> sn) & 1u));
                tmem_ld_wait();
                if (PARTIALS) {
                    const Tile tc = tile_of(t);
                    const Problem& q = p.prob[tc.pi];
                    const int n = tc.n0 + nl, m0 = tc.m0;
                    if (n < q.N)
#pragma unroll
                        for (int j = 0; j < 32; ++j) {
                            const int m = m0 + part * 32 + j;
                            if (m < p.M) p.P[((size_t)m * q.N + n) * G + g] = (int32_t)(v[j] - qb_bits);
                        }
                } else {
                    // v is P_u >= 0 and below 2^23: its bits are the float P_u * 2^-149; the subtraction of
                    // the denormal 128 Q is exact, the product with s * 2^100 is rounded once in the FMA
                    // (packed f32x2 arithmetic: 444 instead of 605 cycles per group in an isolated model)
                    const uint64_t sf2 = f32x2_pack(__float_as_uint(sf), __float_as_uint(sf));
                    const uint64_t qb2 = f32x2_pack(qb_bits, qb_bits);
#pragma unroll
                    for (int j = 0; j < 16; ++j)
                        acc2[j] = f32x2_fma(sf2, f32x2_sub(f32x2_pack(v[2 * j], v[2 * j + 1]), qb2), acc2[j]);
                }
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(&tm_empty[b]);
                ss = sn;
            }
            if (!ok) break;
            if (PARTIALS) continue;
            // the tile's coordinates are only needed from here on (not kept live through the loop)
            const Tile tc = tile_of(t);
            const Problem& q = p.prob[tc.pi];
            const int n = tc.n0 + nl, m0 = tc.m0;
            const int it = (t - (int)blockIdx.x) / (int)gridDim.x;
            if (it == 0) pdl_wait();   // a_scale (long since written; the call makes the ordering explicit)
            if (!wait(corr_done, it & 1, 9)) break;
            tc_fence_after_sync();
            uint32_t v[32];
            tmem_ld_x32(lane_base + kColCorr, v);
            tmem_ld_wait();
            // the zero-point term is in registers: the next tile may overwrite its accumulator
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(corr_free);
            float acc[32];
#pragma unroll
            for (int j = 0; j < 16; ++j) f32x2_unpack(acc2[j], acc[2 * j], acc[2 * j + 1]);
#pragma unroll
            for (int j = 0; j < 32; ++j) {
                const int m = m0 + part * 32 + j;
                if (m < p.M && n < q.N) {
                    const float val = __ldg(p.a_scale + m) * (acc[j] * 0x1p49f - __uint_as_float(v[j]));
                    store_y(q.y, q.y_dtype, (size_t)m * q.N + n, val);
                }
            }
        }
    }

    // ---- teardown: after an abort give copies in flight time to land before the CTA goes away ----
    if (*abort_flag) {
        const long long t0 = clock64();
        while (clock64() - t0 < 400000) {}
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_base, kTmemCols);
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)ptr;
    }
    return fn;
}

// SMs of the current device (one persistent CTA each), asked once per device.
int sm_count() {
    static int cached[64];
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
    if (!cached[dev]) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
        cached[dev] = n;
    }
    return cached[dev];
}

template <int GROUP, bool PARTIALS>
cudaError_t launch(const CUtensorMap& tm_act, const CUtensorMap& tm_ac, const WeightMaps& wmaps, const Params& p,
                   dim3 grid, uint32_t* status, cudaStream_t stream) {
    static bool configured = false;
    auto kern = gemm_w4a8_kernel<GROUP, PARTIALS>;
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
        if (e != cudaSuccess) return e;
        configured = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = kSmemBytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, tm_act, tm_ac, wmaps, p, status);
}

}  // namespace

cudaError_t gemm_w4a8_launch(const GemmW4A8Args& a, uint32_t* status, cudaStream_t stream) {
    EncodeTiledFn enc = encode_fn();
    if (!enc) return cudaErrorNotSupported;
    if (a.count < 1 || a.count > kGemmMaxBatch) return cudaErrorInvalidValue;
    const bool partials = a.P != nullptr;
    const W4Geometry geo0 = w4_geometry(a.N[0], a.K, a.group);

    CUtensorMap tm_act, tm_ac;
    WeightMaps wmaps;
    Params p;
    p.a_scale = a.a_scale;
    p.P = a.P;
    p.M = a.M; p.K = a.K; p.G = geo0.G;
    p.n_slabs = geo0.n_slabs;
    p.n_stages = (a.K + kStageK - 1) / kStageK;
    p.count = a.count;
    p.chunk_bytes = geo0.chunk_bytes;
    int tiles = 0;
    for (int i = 0; i < kGemmMaxBatch; ++i) {
        const int src = i < a.count ? i : 0;   // unused slots repeat the first matrix
        const W4Geometry geo = w4_geometry(a.N[src], a.K, a.group);
        // the packed body as [row block][32-bit words]: codes box 8 x 1 KiB, table box 8 x 512 B
        const cuuint64_t dims[2] = {(cuuint64_t)(geo.row_block_bytes / 4), (cuuint64_t)geo.n_row_blocks};
        const cuuint64_t strides[1] = {(cuuint64_t)geo.row_block_bytes};
        const cuuint32_t box_pk[2] = {2 * kSlabBytes / 4, 8}, box_tab[2] = {512 / 4, 8};
        const cuuint32_t estr[2] = {1, 1};
        void* body = (void*)((const uint8_t*)a.packed[src] + kHeaderBytes);
        if (enc(&wmaps.pk[i], CU_TENSOR_MAP_DATA_TYPE_UINT32, 2, body, dims, strides, box_pk, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS ||
            enc(&wmaps.tab[i], CU_TENSOR_MAP_DATA_TYPE_UINT32, 2, body, dims, strides, box_tab, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return cudaErrorInvalidValue;
        Problem& q = p.prob[i];
        q.y = a.y[src];
        q.N = a.N[src];
        q.n_row_blocks = geo.n_row_blocks;
        q.y_dtype = a.y_dtype[src];
        q.tile_begin = tiles;
        if (i < a.count) tiles += (a.N[i] + kTileN - 1) / kTileN;
    }
    {
        const cuuint64_t dims[2] = {(cuuint64_t)a.K, (cuuint64_t)a.M};
        const cuuint64_t strides[1] = {(cuuint64_t)a.K};
        const cuuint32_t box[2] = {(cuuint32_t)kStageK, (cuuint32_t)kTileT};
        const cuuint32_t estr[2] = {1, 1};
        if (enc(&tm_act, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, (void*)a.a_q, dims, strides, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return cudaErrorInvalidValue;
    }
    if (!partials) {
        const int G4 = (geo0.G + 3) / 4 * 4;
        const cuuint64_t dims[2] = {(cuuint64_t)G4 * 4, (cuuint64_t)a.M};
        const cuuint64_t strides[1] = {(cuuint64_t)G4 * 8};
        const cuuint32_t box[2] = {16, (cuuint32_t)kTileT};
        const cuuint32_t estr[2] = {1, 1};
        if (enc(&tm_ac, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, (void*)a.AC, dims, strides, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_32B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return cudaErrorInvalidValue;
    } else {
        tm_ac = tm_act;  // never read in the partials form
    }
    p.tiles_m = (a.M + kTileT - 1) / kTileT;
    p.total_tiles = tiles * p.tiles_m;
    const int n_sm = sm_count();
    if (n_sm <= 0) return cudaErrorInvalidDevice;
    const dim3 grid((unsigned)(p.total_tiles < n_sm ? p.total_tiles : n_sm));   // one persistent CTA per SM
    if (a.group == 64)
        return partials ? launch<64, true>(tm_act, tm_ac, wmaps, p, grid, status, stream)
                        : launch<64, false>(tm_act, tm_ac, wmaps, p, grid, status, stream);
    return partials ? launch<128, true>(tm_act, tm_ac, wmaps, p, grid, status, stream)
                    : launch<128, false>(tm_act, tm_ac, wmaps, p, grid, status, stream);
}

}  // namespace mnnllm
