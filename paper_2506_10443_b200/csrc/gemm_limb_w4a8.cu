// W4A8 prefill GEMM without a per-group drain: the integer-limb form.
//
// y[m,n] = a_scale[m] * ( sum_g s[n,g] P[m,n,g]  -  sum_g (s z)[n,g] A[m,g] )          (Section 4.2, W4A8)
//
// The tensor-memory GEMM of gemm_w4a8.cu takes every group's int32 partial P out of tensor memory to
// multiply it with its scale: 16384 partials per group and tile through the CUDA cores, which is
// what bounds it.  Here the scale goes INTO the integer operand instead.  The packer writes, per
// weight row, an exponent e[n] such that every group scale of the row is an integer multiple
// S[n,g] * 2^e[n] (fp16 scales: an 11-bit significand shifted by the row's exponent spread).  Then
//     sum_g s[n,g] P[m,n,g] = 2^e[n] * sum_k a_q[m,k] * (q[n,k] * S[n,g(k)]),
// one integer dot product over ALL of K.  The product q * S (up to 20 bits when S < 2^16) is cut
// into three unsigned byte "limbs" with weights 1, 256 and 4096; each limb is a u8 operand of
// tcgen05.mma kind::i8 and owns one int32 accumulator in tensor memory for the whole tile:
//     T = L0 + 256 L1 + 4096 L2,   L_i = sum_k a_q * limb_i     (exact, |L_i| < 2^31 up to K = 18944)
// Three times the MMA work, which the tensor cores have to spare, and no drain: tensor memory is
// read once per tile.  The activations keep their unsigned form a_q + 128 (one quantiser for both
// GEMM kernels); the excess 128 * sum_k limb_i[n,k] is a per-row constant from the packer.
// The zero-point term is the fp16 tensor-core product of gemm_w4a8.cu, unchanged.
// A weight matrix whose packer flag says that some row's scales span too many binades (S >= 2^16)
// does not take this kernel: every CTA returns at once and gemm_w4a8.cu's kernel, launched behind
// it, does the work (and returns at once in the other case).
//
// Measured (Qwen2-1.5B layer, 1024 tokens): 250 TOP/s against 390 for gemm_w4a8.cu.  The drain is gone,
// but its work has moved rather than vanished: the unpack costs ~2.5 instructions per code (eight
// multiplies and six byte permutes per packed word) against one AND per four codes there, the tile
// count of instructions is only 20 % lower (4600 against 5700 warp instructions per tile and 128-k
// stage), the tensor pipe is busy three times as long, and the epilogue cannot overlap the next
// tile (four 128-column regions fill tensor memory).  The kernel is therefore off by default and
// kept as a checked alternative.
//
// Roles (15 warps): TMA producer | MMA issue | 8 unpack warps (packed int4 -> three limb tiles) |
// zero-point operand warp | 4 epilogue warps.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "common.h"
#include "gemm_limb_w4a8.h"
#include "layout.h"
#include "ptx.cuh"

namespace mnnllm {

using namespace ptx;

namespace {

constexpr int kTileN = 128;    // weight rows per tile (MMA M)
constexpr int kTileT = 128;    // tokens per tile (MMA N)
constexpr int kStageK = 128;   // k per pipeline stage (one 128-byte swizzle row of int8)
constexpr int kStages = 2;     // ring of limb-tile stages (3 x 16 KiB each)
constexpr int kActStages = 4;  // ring of activation stages (16 KiB each): deeper, their loads have HBM/L2 latency to hide
constexpr int kLimbs = 3;
constexpr int kPkStages = 4;   // ring of packed-code stages (8 KiB each)
constexpr int kPkLead = 2;     // stages the packed ring runs ahead of the activations
constexpr int kTabSlots = 3;   // ring of per-chunk (scale, zero) tables
constexpr int kUnpackWarps = 8, kUnpackWarp0 = 2, kScaleWarp = 10, kEpiWarp0 = 11, kEpiWarps = 4;
constexpr int kThreads = (kEpiWarp0 + kEpiWarps) * 32;
constexpr uint32_t kMaxPolls = 1u << 15;
constexpr uint32_t kTmemCols = 512;            // three int32 accumulators + the fp32 zero-point term, 128 columns each
constexpr uint32_t kColCorr = kLimbs * 128;

constexpr int kStageBytes = kTileN * kStageK;  // 16 KiB
constexpr int kCorrBytes = 128 * 32;
constexpr int kPkBytes = 8 * 2 * kSlabBytes;
constexpr int kTabBytes = 8 * 512;

struct Smem {
    static constexpr int act = 0;                                          // [kActStages] activations (a_q + 128)
    static constexpr int limb = act + kActStages * kStageBytes;            // [kStages][kLimbs] limb tiles
    static constexpr int ca = limb + kStages * kLimbs * kStageBytes;       // [2] (s z) halves
    static constexpr int cb = ca + 2 * kCorrBytes;                         // [2] group sums of the activations
    static constexpr int pk = cb + 2 * kCorrBytes;
    static constexpr int tab = pk + kPkStages * kPkBytes;
    static constexpr int bars = tab + kTabSlots * kTabBytes;
    static constexpr int n_bars = 2 * kStages + 2 * kActStages + 2 * 2 + 2 + 2 * kPkStages + 2 * kTabSlots;
    static constexpr int misc = bars + n_bars * 8;
    static constexpr int total = misc + 16;
};
constexpr size_t kSmemBytes = Smem::total + 1024;

constexpr uint32_t kIdescI8 = (2u << 4) | (0u << 7) | (0u << 10) | ((kTileT >> 3) << 17) | ((kTileN >> 4) << 24);
constexpr uint32_t kIdescF16 = (1u << 4) | (0u << 7) | (0u << 10) | ((kTileT >> 3) << 17) | ((kTileN >> 4) << 24);

struct Problem {
    void* y;
    const W4RowInfo* info;      // the packed buffer's trailer: per padded row {sum_k q S, exponent}
    const uint32_t* limb_ok;    // the trailer's flag
    int N, n_row_blocks, y_dtype, tile_begin;
};
struct Params {
    const float* a_scale;
    int M, K, G, n_slabs, n_stages, count, tiles_m, total_tiles;
    unsigned long long chunk_bytes;
    Problem prob[kGemmLimbMaxBatch];
};
struct WeightMaps {
    CUtensorMap pk[kGemmLimbMaxBatch], tab[kGemmLimbMaxBatch];
};

// 32 lanes x 16 consecutive 32-bit columns of tensor memory (thread i receives lane base + i)
__device__ __forceinline__ void tmem_ld_x16(uint32_t taddr, uint32_t (&v)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
          "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
        : "r"(taddr)
        : "memory");
}

__device__ __forceinline__ void store_y(void* y, int dtype, size_t idx, float v) {
    if (dtype == MNNLLM_F16) reinterpret_cast<__half*>(y)[idx] = __float2half_rn(v);
    else if (dtype == MNNLLM_BF16) reinterpret_cast<__nv_bfloat16*>(y)[idx] = __float2bfloat16_rn(v);
    else reinterpret_cast<float*>(y)[idx] = v;
}

template <int GROUP>
__global__ void __launch_bounds__(kThreads, 1)
gemm_limb_w4a8_kernel(const __grid_constant__ CUtensorMap tm_act, const __grid_constant__ CUtensorMap tm_ac,
                      const __grid_constant__ WeightMaps wmaps, const __grid_constant__ Params p,
                      uint32_t* __restrict__ status) {
    // not this kernel's turn: some matrix of the launch needs scales wider than the limbs hold
    for (int i = 0; i < p.count; ++i)
        if (__ldg(p.prob[i].limb_ok) == 0u) return;

    constexpr int GPS = kStageK / GROUP;  // groups per stage (2 or 1)
    constexpr int SPB = 4 / GPS;          // stages per block of four groups (zero-point MMA cadence)
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + Smem::bars);
    uint64_t* ab_full = bars;                    // [kStages] limb tiles written
    uint64_t* ab_empty = ab_full + kStages;      // [kStages] the stage's MMAs have completed
    uint64_t* act_full = ab_empty + kStages;     // [kActStages] activations landed
    uint64_t* act_empty = act_full + kActStages; // [kActStages] the stage's MMAs have completed
    uint64_t* c_full = act_empty + kActStages;   // [2] zero-point operands ready
    uint64_t* c_empty = c_full + 2;              // [2]
    uint64_t* acc_full = c_empty + 2;            // the tile's accumulators are complete
    uint64_t* acc_empty = acc_full + 1;          // ... and have been read
    uint64_t* pk_full = acc_empty + 1;
    uint64_t* pk_empty = pk_full + kPkStages;
    uint64_t* tab_full = pk_empty + kPkStages;
    uint64_t* tab_empty = tab_full + kTabSlots;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + Smem::misc);
    volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(smem + Smem::misc + 4);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_stages = p.n_stages, G = p.G, total_tiles = p.total_tiles;

    // The CTA is persistent: tiles blockIdx.x, blockIdx.x + gridDim.x, ...; the token tile index runs
    // fastest, so CTAs that work at the same time share their weight tile (L2).
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
        for (int i = 0; i < kStages; ++i) { mbar_init(&ab_full[i], kUnpackWarps); mbar_init(&ab_empty[i], 1); }
        for (int i = 0; i < kActStages; ++i) { mbar_init(&act_full[i], 1); mbar_init(&act_empty[i], 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(&c_full[i], 2); mbar_init(&c_empty[i], 1); }
        mbar_init(acc_full, 1);
        mbar_init(acc_empty, kEpiWarps);
        for (int i = 0; i < kPkStages; ++i) { mbar_init(&pk_full[i], 1); mbar_init(&pk_empty[i], kUnpackWarps); }
        for (int i = 0; i < kTabSlots; ++i) { mbar_init(&tab_full[i], 1); mbar_init(&tab_empty[i], kUnpackWarps + 1); }
        *abort_flag = 0;
        fence_mbar_init();
        prefetch_tensormap(&tm_act);
        prefetch_tensormap(&tm_ac);
        for (int i = 0; i < p.count; ++i) {
            prefetch_tensormap(&wmaps.pk[i]);
            prefetch_tensormap(&wmaps.tab[i]);
        }
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    // the weight side (packed codes, tables, unpack) does not depend on the quantiser that precedes
    // this grid; the threads that read its outputs call griddepcontrol.wait first
    pdl_launch_dependents();

    auto wait = [&](uint64_t* bar, uint32_t parity, uint32_t code) -> bool {
        if (mbar_wait_bounded_compact(bar, parity, kMaxPolls)) return true;
        if (*abort_flag == 0) {
            *abort_flag = 1;
            atomicOr(status, 0x500u | code);
        }
        return false;
    };

    if (warp == 0) {
        // ------------------------------------------------------------------ producer (TMA)
        // Two cursors over the same (tile, stage) sequence: the packed codes (with each 512-k chunk's
        // scale/zero tables) run kPkLead stages ahead of the activations.
        if (elect_one()) {
            int t_pk = blockIdx.x, t_ac = blockIdx.x, lead = 0;
            uint32_t ip = 0, jc = 0, gs = 0, cb = 0;   // running counts: packed stages, chunks, stages, zero-point blocks
            Tile cp = tile_of(t_pk), ca = cp;
            int i_pk = 0, st = 0;
            bool first = true;
            while (t_ac < total_tiles) {
                if (t_pk < total_tiles) {
                    const int pslot = ip % kPkStages, j = i_pk >> 2, rb0 = cp.n0 / kRowsPerBlock;
                    if (!wait(&pk_empty[pslot], ((ip / kPkStages) & 1) ^ 1, 10)) break;
                    const int ns_chunk = (p.n_slabs - 8 * j) < 8 ? (p.n_slabs - 8 * j) : 8;
                    const unsigned long long chunk_off = (unsigned long long)j * p.chunk_bytes;
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
                        t_pk += gridDim.x;
                        if (t_pk < total_tiles) cp = tile_of(t_pk);
                        i_pk = 0;
                    }
                }
                if (lead > kPkLead || t_pk >= total_tiles) {
                    if (first) { pdl_wait(); first = false; }   // the quantised activations are complete from here on
                    const int slot = gs % kActStages;
                    if (!wait(&act_empty[slot], ((gs / kActStages) & 1) ^ 1, 1)) break;
                    mbar_arrive_expect_tx(&act_full[slot], kTileT * kStageK);
                    tma_load_2d(smem + Smem::act + slot * kStageBytes, &tm_act, st * kStageK, ca.m0, &act_full[slot]);
                    if (st % SPB == 0) {
                        const int cslot = cb & 1;
                        if (!wait(&c_empty[cslot], ((cb >> 1) & 1) ^ 1, 2)) break;
                        mbar_arrive_expect_tx(&c_full[cslot], kTileT * 32);
                        tma_load_2d(smem + Smem::cb + cslot * kCorrBytes, &tm_ac, (st / SPB) * 16, ca.m0, &c_full[cslot]);
                        ++cb;
                    }
                    ++gs;
                    --lead;
                    if (++st == n_stages) {
                        t_ac += gridDim.x;
                        if (t_ac < total_tiles) ca = tile_of(t_ac);
                        st = 0;
                    }
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issue
        // Per stage and 32-k step three MMAs, one per limb, each into its own accumulator that runs
        // over the whole tile; the zero-point MMA (fp16, K = 16 = four groups) joins whenever a block
        // of four groups is complete.  Tensor memory is handed to the epilogue once per tile.
        if (elect_one()) {
            uint32_t gs = 0, cb = 0;
            int it = 0;
            const uint32_t act_addr = smem_u32(smem + Smem::act), limb_addr = smem_u32(smem + Smem::limb);
            bool ok = true;
            for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x, ++it) {
                // the previous tile's accumulators must have been read
                if (it > 0 && !wait(acc_empty, (uint32_t)(it - 1) & 1u, 4)) { ok = false; break; }
                tc_fence_after_sync();
                int gcount = 0;
                bool cfirst = true;
                for (int st = 0; st < n_stages && ok; ++st, ++gs) {
                    const int slot = gs % kStages, aslot = gs % kActStages;
                    const int ngr = (G - st * GPS) < GPS ? (G - st * GPS) : GPS;
                    if (!wait(&act_full[aslot], (gs / kActStages) & 1, 8)) { ok = false; break; }
                    if (!wait(&ab_full[slot], (gs / kStages) & 1, 3)) { ok = false; break; }
                    tc_fence_after_sync();
                    const uint64_t db = desc_sw128(act_addr + aslot * kStageBytes);
                    const int ksteps = ngr * GROUP / 32;   // a last stage may hold fewer groups
#pragma unroll 1
                    for (int kk = 0; kk < ksteps; ++kk) {
                        const uint64_t adv = (uint64_t)((kk * 32) >> 4);
#pragma unroll
                        for (int l = 0; l < kLimbs; ++l)
                            mma_i8_ss(tmem_base + l * kTileT, desc_sw128(limb_addr + (slot * kLimbs + l) * kStageBytes) + adv,
                                      db + adv, kIdescI8, (st > 0 || kk > 0) ? 1u : 0u);
                    }
                    mma_commit(&ab_empty[slot]);
                    mma_commit(&act_empty[aslot]);
                    gcount += ngr;
                    if ((gcount & 3) == 0 || st == n_stages - 1) {
                        const int cslot = cb & 1;
                        if (!wait(&c_full[cslot], (cb >> 1) & 1, 5)) { ok = false; break; }
                        tc_fence_after_sync();
                        mma_f16_ss(tmem_base + kColCorr, desc_sw32(smem_u32(smem + Smem::ca + cslot * kCorrBytes)),
                                   desc_sw32(smem_u32(smem + Smem::cb + cslot * kCorrBytes)), kIdescF16, !cfirst);
                        mma_commit(&c_empty[cslot]);
                        cfirst = false;
                        ++cb;
                    }
                }
                if (ok) mma_commit(acc_full);
            }
        }
        __syncwarp();
    } else if (warp < kUnpackWarp0 + kUnpackWarps) {
        // ------------------------------------------------------------------ unpack: int4 codes -> three limb tiles
        // Warp wu owns row block wu of the tile (rows 16 wu .. 16 wu + 15) and both 64-k slabs of a
        // stage.  Two codes are multiplied at once: (q_a + 2^16 q_b) * S_lo keeps both 16-bit products
        // apart (q S_lo < 2^16), likewise for S_hi; byte permutes then gather each limb's four
        // consecutive k into one register.
        const int wu = warp - kUnpackWarp0;
        const int r = lane >> 2, c = lane & 3;
        const int odd = r & 1;   // odd rows take the two slabs in the other order (shared-memory banks, see gemm_w4a8)
        uint32_t ip = 0, gs = 0, jc = 0;
        bool ok = true;
        for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x) {
            const Tile tc = tile_of(t);
            const Problem& q = p.prob[tc.pi];
            const int rb = tc.n0 / kRowsPerBlock + wu;
            const bool rb_valid = rb < q.n_row_blocks;
            // the rows' exponents (trailer of the packed buffer: static data, no dependency)
            int e0 = 0, e1 = 0;
            if (rb_valid) {
                e0 = __ldg(&q.info[rb * 16 + r].row_exp);
                e1 = __ldg(&q.info[rb * 16 + r + 8].row_exp);
            }
            uint32_t tslot = 0;
            for (int st = 0; st < n_stages; ++st, ++ip, ++gs) {
                const int slot = gs % kStages, pslot = ip % kPkStages, j = st >> 2;
                const int ns_chunk = (p.n_slabs - 8 * j) < 8 ? (p.n_slabs - 8 * j) : 8;
                const int ng = ns_chunk * kSlabK4 / GROUP;
                if ((st & 3) == 0) {
                    tslot = jc % kTabSlots;
                    if (!wait(&tab_full[tslot], (jc / kTabSlots) & 1, 13)) { ok = false; break; }
                    ++jc;
                }
                if (!wait(&pk_full[pslot], (ip / kPkStages) & 1, 11)) { ok = false; break; }
                uint4 cur[2];
                uint32_t S[2][2];   // [slab][row half]: integer scale of the slab's group for rows r and r + 8
                {
                    const uint4* pk = reinterpret_cast<const uint4*>(smem + Smem::pk + pslot * kPkBytes);
                    const uint32_t* tab = reinterpret_cast<const uint32_t*>(smem + Smem::tab + tslot * kTabBytes + wu * 512);
#pragma unroll
                    for (int i = 0; i < 2; ++i) {
                        const int sl = i ^ odd;
                        const bool valid = rb_valid && (st & 3) * 2 + sl < ns_chunk;
                        cur[i] = valid ? pk[(wu * 2 + sl) * 32 + lane] : make_uint4(0, 0, 0, 0);
                        const int gc = (st & 3) * GPS + (GROUP == 64 ? sl : 0);
                        int M, x;
                        w4_scale_parts(valid ? (tab[r * ng + gc] & 0xFFFFu) : 0u, M, x);
                        S[i][0] = M ? (uint32_t)M << (x - e0) : 0u;
                        w4_scale_parts(valid ? (tab[(r + 8) * ng + gc] & 0xFFFFu) : 0u, M, x);
                        S[i][1] = M ? (uint32_t)M << (x - e1) : 0u;
                    }
                }
                __syncwarp();
                if (lane == 0) {
                    mbar_arrive(&pk_empty[pslot]);
                    if ((st & 3) == 3 || st == n_stages - 1) mbar_arrive(&tab_empty[tslot]);
                }
                // limbs of the 16 codes of a row's 16-k piece: words w0 (k 0..7) and w1 (k 8..15)
                uint4 L[2][2][kLimbs];   // [slab][row half][limb]
#pragma unroll
                for (int i = 0; i < 2; ++i)
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        const uint32_t s_lo = S[i][h] & 4095u, s_hi = S[i][h] >> 12;
                        const uint32_t w0 = h ? cur[i].z : cur[i].x, w1 = h ? cur[i].w : cur[i].y;
                        uint32_t out[kLimbs][4];
#pragma unroll
                        for (int wd = 0; wd < 2; ++wd) {
                            const uint32_t w = wd ? w1 : w0;
                            constexpr uint32_t PM = 0x000F000Fu;
                            // code pairs (k0,k2) (k4,k6) (k1,k3) (k5,k7) of the word (nibble order of the packed layout)
                            const uint32_t c02 = w & PM, c46 = (w >> 4) & PM, c13 = (w >> 8) & PM, c57 = (w >> 12) & PM;
                            const uint32_t a02 = c02 * s_lo, a46 = c46 * s_lo, a13 = c13 * s_lo, a57 = c57 * s_lo;
                            const uint32_t b02 = c02 * s_hi, b46 = c46 * s_hi, b13 = c13 * s_hi, b57 = c57 * s_hi;
                            out[0][2 * wd] = __byte_perm(a02, a13, 0x6240);       // low bytes, k0 k1 k2 k3
                            out[0][2 * wd + 1] = __byte_perm(a46, a57, 0x6240);   // k4 k5 k6 k7
                            out[1][2 * wd] = __byte_perm(a02, a13, 0x7351);       // high bytes
                            out[1][2 * wd + 1] = __byte_perm(a46, a57, 0x7351);
                            out[2][2 * wd] = __byte_perm(b02, b13, 0x6240);       // q * (S >> 12)
                            out[2][2 * wd + 1] = __byte_perm(b46, b57, 0x6240);
                        }
#pragma unroll
                        for (int l = 0; l < kLimbs; ++l) L[i][h][l] = make_uint4(out[l][0], out[l][1], out[l][2], out[l][3]);
                    }
                if (!wait(&ab_empty[slot], ((gs / kStages) & 1) ^ 1, 6)) { ok = false; break; }
                // 128B-swizzled K-major rows: row R of the tile at (R >> 3) * 1024 + (R & 7) * 128, 16-byte
                // chunk kc of the row at ((kc ^ (R & 7)) << 4)
                uint8_t* base = smem + Smem::limb + slot * kLimbs * kStageBytes;
#pragma unroll
                for (int i = 0; i < 2; ++i) {
                    const int sl = i ^ odd;
                    const int R0 = wu * 16 + r;               // rows R0 and R0 + 8 (same swizzle phase r)
                    const int kc = sl * 4 + c;
                    const uint32_t off = (uint32_t)(R0 >> 3) * 1024u + (uint32_t)r * 128u + (uint32_t)((kc ^ r) << 4);
#pragma unroll
                    for (int l = 0; l < kLimbs; ++l) {
                        *reinterpret_cast<uint4*>(base + l * kStageBytes + off) = L[i][0][l];
                        *reinterpret_cast<uint4*>(base + l * kStageBytes + off + 1024u) = L[i][1][l];
                    }
                }
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) mbar_arrive(&ab_full[slot]);
            }
        }
    } else if (warp == kScaleWarp) {
        // ------------------------------------------------------------------ (s z) halves for the zero-point MMA
        uint32_t jc = 0, cbase = 0;
        bool ok = true;
        for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x) {
            const Tile tc = tile_of(t);
            const Problem& q = p.prob[tc.pi];
            const int nrb = (q.n_row_blocks - tc.n0 / kRowsPerBlock) < 8 ? (q.n_row_blocks - tc.n0 / kRowsPerBlock) : 8;
            uint32_t tslot = 0;
            for (int st = 0; st < n_stages && ok; ++st) {
                const int j = st >> 2;
                const int ns_chunk = (p.n_slabs - 8 * j) < 8 ? (p.n_slabs - 8 * j) : 8;
                const int ng = ns_chunk * kSlabK4 / GROUP;
                if ((st & 3) == 0) {
                    tslot = jc % kTabSlots;
                    if (!wait(&tab_full[tslot], (jc / kTabSlots) & 1, 14)) { ok = false; break; }
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
                if ((st & 3) == 3 || st == n_stages - 1) {
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&tab_empty[tslot]);
                }
#pragma unroll
                for (int gi = 0; gi < GPS; ++gi) {
                    const int g = st * GPS + gi;
                    if (g >= G) break;
                    const int pos = g & 3;
                    const uint32_t cb = cbase + (uint32_t)(g >> 2);
                    const int cslot = cb & 1;
                    if (pos == 0 && !wait(&c_empty[cslot], ((cb >> 1) & 1) ^ 1, 7)) { ok = false; break; }
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int row = lane + 32 * i;
                        const __half2 h2 = *reinterpret_cast<const __half2*>(&zc[i][gi]);
                        const float s = __low2float(h2), z = __high2float(h2);
                        // 2^8 s z as fp16 hi + lo (see gemm_w4a8: keeps lo a normal number; undone in the epilogue)
                        const float szf = s * z * 0x1p8f;
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
                    if (pos == 3 || g == G - 1) {
                        fence_proxy_async_smem();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(&c_full[cslot]);
                    }
                }
            }
            cbase += (uint32_t)((G + 3) >> 2);
        }
    } else {
        // ------------------------------------------------------------------ epilogue: once per tile
        const int q4 = warp & 3;                       // tensor-memory lane quarter this warp may read
        const int nl = q4 * 32 + lane;                 // this thread's weight row of the tile
        const uint32_t lane_base = tmem_base + ((uint32_t)(q4 * 32) << 16);
        int it = 0;
        for (int t = blockIdx.x; t < total_tiles; t += gridDim.x, ++it) {
            const Tile tc = tile_of(t);
            const Problem& q = p.prob[tc.pi];
            const int n = tc.n0 + nl, m0 = tc.m0;
            // this row's constants: 128 * sum_k limb_i (the activations carry + 128) and 2^row_exp
            int rs0 = 0, rs1 = 0, rs2 = 0;
            float two_e = 0.f;
            if (n < q.n_row_blocks * 16) {
                const int4 inf = __ldg(reinterpret_cast<const int4*>(q.info + n));
                rs0 = 128 * inf.x; rs1 = 128 * inf.y; rs2 = 128 * inf.z;
                two_e = __int_as_float((inf.w + 127) << 23);   // 2^row_exp, exactly (row_exp in [-24, 5])
            }
            if (it == 0) pdl_wait();   // a_scale comes from the quantiser
            if (!wait(acc_full, (uint32_t)it & 1u, 9)) break;
            tc_fence_after_sync();
#pragma unroll 1
            for (int cq = 0; cq < 8; ++cq) {   // sixteen token columns at a time
                uint32_t v0[16], v1[16], v2[16], vc[16];
                tmem_ld_x16(lane_base + 0 * kTileT + cq * 16, v0);
                tmem_ld_x16(lane_base + 1 * kTileT + cq * 16, v1);
                tmem_ld_x16(lane_base + 2 * kTileT + cq * 16, v2);
                tmem_ld_x16(lane_base + kColCorr + cq * 16, vc);
                tmem_ld_wait();
                if (cq == 7) {   // everything is in registers: the next tile may overwrite tensor memory
                    tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(acc_empty);
                }
#pragma unroll
                for (int jx = 0; jx < 16; ++jx) {
                    const int m = m0 + cq * 16 + jx;
                    // exact: T = L0 + 256 L1 + 4096 L2 with the + 128 excess of the unsigned activations removed
                    const long long T = (long long)((int)v0[jx] - rs0) + 256ll * (long long)((int)v1[jx] - rs1) +
                                        4096ll * (long long)((int)v2[jx] - rs2);
                    const float val = fmaf(__uint_as_float(vc[jx]), -0x1p-8f, two_e * (float)T);
                    if (m < p.M && n < q.N) store_y(q.y, q.y_dtype, (size_t)m * q.N + n, __ldg(p.a_scale + m) * val);
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

template <int GROUP>
cudaError_t launch(const CUtensorMap& tm_act, const CUtensorMap& tm_ac, const WeightMaps& wmaps, const Params& p,
                   dim3 grid, uint32_t* status, cudaStream_t stream) {
    static PerDevice<bool> configured;   // per instantiation and device
    auto kern = gemm_limb_w4a8_kernel<GROUP>;
    if (cudaError_t e = configured.with([&](bool& done) {
            if (done) return cudaSuccess;
            cudaError_t err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
            done = err == cudaSuccess;
            return err;
        });
        e != cudaSuccess)
        return e;
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

int gemm_limb_w4a8_tiles(const GemmLimbArgs& a) {
    int tiles = 0;
    for (int i = 0; i < a.count; ++i) tiles += (a.N[i] + kTileN - 1) / kTileN;
    return tiles * ((a.M + kTileT - 1) / kTileT);
}

cudaError_t gemm_limb_w4a8_launch(const GemmLimbArgs& a, uint32_t* status, cudaStream_t stream) {
    EncodeTiledFn enc = encode_fn();
    if (!enc) return cudaErrorNotSupported;
    if (a.count < 1 || a.count > kGemmLimbMaxBatch) return cudaErrorInvalidValue;
    const W4Geometry geo0 = w4_geometry(a.N[0], a.K, a.group);

    CUtensorMap tm_act, tm_ac;
    WeightMaps wmaps;
    Params p;
    p.a_scale = a.a_scale;
    p.M = a.M; p.K = a.K; p.G = geo0.G;
    p.n_slabs = geo0.n_slabs;
    p.n_stages = (a.K + kStageK - 1) / kStageK;
    p.count = a.count;
    p.chunk_bytes = geo0.chunk_bytes;
    int tiles = 0;
    const cuuint32_t estr[2] = {1, 1};
    for (int i = 0; i < kGemmLimbMaxBatch; ++i) {
        if (i >= a.count) {   // unused slots repeat the first matrix (never read)
            wmaps.pk[i] = wmaps.pk[0];
            wmaps.tab[i] = wmaps.tab[0];
            p.prob[i] = p.prob[0];
            continue;
        }
        const W4Geometry geo = w4_geometry(a.N[i], a.K, a.group);
        // the packed body as [row block][32-bit words]: codes box 8 x 1 KiB, table box 8 x 512 B
        const cuuint64_t dims[2] = {(cuuint64_t)(geo.row_block_bytes / 4), (cuuint64_t)geo.n_row_blocks};
        const cuuint64_t strides[1] = {(cuuint64_t)geo.row_block_bytes};
        const cuuint32_t box_pk[2] = {2 * kSlabBytes / 4, 8}, box_tab[2] = {512 / 4, 8};
        const uint8_t* base = (const uint8_t*)a.packed[i];
        void* body = (void*)(base + kHeaderBytes);
        if (enc(&wmaps.pk[i], CU_TENSOR_MAP_DATA_TYPE_UINT32, 2, body, dims, strides, box_pk, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS ||
            enc(&wmaps.tab[i], CU_TENSOR_MAP_DATA_TYPE_UINT32, 2, body, dims, strides, box_tab, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return cudaErrorInvalidValue;
        Problem& q = p.prob[i];
        q.y = a.y[i];
        q.limb_ok = (const uint32_t*)(base + geo.trailer_offset);
        q.info = (const W4RowInfo*)(base + geo.trailer_offset + kTrailerHeadBytes);
        q.N = a.N[i];
        q.n_row_blocks = geo.n_row_blocks;
        q.y_dtype = a.y_dtype[i];
        q.tile_begin = tiles;
        tiles += (a.N[i] + kTileN - 1) / kTileN;
    }
    {
        const cuuint64_t dims[2] = {(cuuint64_t)a.K, (cuuint64_t)a.M};
        const cuuint64_t strides[1] = {(cuuint64_t)a.K};
        const cuuint32_t box[2] = {(cuuint32_t)kStageK, (cuuint32_t)kTileT};
        if (enc(&tm_act, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, (void*)a.a_q, dims, strides, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return cudaErrorInvalidValue;
    }
    {
        const int G4 = (geo0.G + 3) / 4 * 4;
        const cuuint64_t dims[2] = {(cuuint64_t)G4 * 4, (cuuint64_t)a.M};
        const cuuint64_t strides[1] = {(cuuint64_t)G4 * 8};
        const cuuint32_t box[2] = {16, (cuuint32_t)kTileT};
        if (enc(&tm_ac, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, (void*)a.AC, dims, strides, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_32B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return cudaErrorInvalidValue;
    }
    p.tiles_m = (a.M + kTileT - 1) / kTileT;
    p.total_tiles = tiles * p.tiles_m;
    const int n_sm = device_sm_count();
    if (n_sm <= 0) return cudaErrorInvalidDevice;
    const dim3 grid((unsigned)(p.total_tiles < n_sm ? p.total_tiles : n_sm));   // one persistent CTA per SM
    return a.group == 64 ? launch<64>(tm_act, tm_ac, wmaps, p, grid, status, stream)
                         : launch<128>(tm_act, tm_ac, wmaps, p, grid, status, stream);
}

}  // namespace mnnllm
