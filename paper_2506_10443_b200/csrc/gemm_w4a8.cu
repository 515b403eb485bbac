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
// A tile is 128 weight rows x 128 tokens.  The weights are the M side of the MMA, so that a
// tensor-memory lane is one output channel n and its per-group scale is a per-thread scalar in the
// drain.  The kernel is persistent: one CTA per SM walks the work items (tiles; or, when a launch
// has fewer tiles than SMs, K ranges of tiles that meet through scratch memory: the kernel source
// in gemm_w4a8_kernel.inc is expanded once for each form).  Rings and barriers run across work
// items.  Warp roles (23 warps):
//   warp 0      producer, one elected thread: TMA loads of the packed int4 codes (the packed buffer
//               seen as a 2-D tensor [row block][words]: one box of 8 row blocks x 1 KiB per stage;
//               issuing one small bulk copy per row block instead costs ~75 cycles each and
//               starves the pipeline) and of each 512-k chunk's (scale, zero) tables into
//               shared-memory rings; TMA loads of the int8 activation tile (128 tokens x 128 k,
//               128B swizzle) and of the fp16 group-sum quadruples that feed the zero-point MMA
//   warp 1      allocates tensor memory; one elected thread issues tcgen05.mma (kind::i8 into one of
//               three int32 accumulators per group; kind::f16 for the zero-point term) and the commits
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

#include "common.h"
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
    int split, split_stages;    // K ranges per tile (1: whole tiles) and stages per range (a multiple of 4)
    float* scratch;             // split > 1: [total_tiles * split][kTileT][kTileN] fp32 parts of the tiles
    uint32_t* counters;         // split > 1: [total_tiles][kDrainWarps], zero when the kernel starts
    unsigned long long chunk_bytes;
    const uint32_t* limb_ok[kGemmMaxBatch];   // null, or the packed buffers' limb flags: return at once if all are set
    Problem prob[kGemmMaxBatch];
};
struct WeightMaps {   // the packed bodies as 2-D tensors: codes box and table box per weight matrix
    CUtensorMap pk[kGemmMaxBatch], tab[kGemmMaxBatch];
};

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

#define MNNLLM_GEMM_SPLIT 0
#define MNNLLM_GEMM_KERNEL gemm_w4a8_kernel
#include "gemm_w4a8_kernel.inc"
#undef MNNLLM_GEMM_SPLIT
#undef MNNLLM_GEMM_KERNEL
#define MNNLLM_GEMM_SPLIT 1
#define MNNLLM_GEMM_KERNEL gemm_w4a8_split_kernel
#include "gemm_w4a8_kernel.inc"
#undef MNNLLM_GEMM_SPLIT
#undef MNNLLM_GEMM_KERNEL

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
    return device_sm_count();
}

template <int GROUP, bool PARTIALS, bool SPLIT>
cudaError_t launch(const CUtensorMap& tm_act, const CUtensorMap& tm_ac, const WeightMaps& wmaps, const Params& p,
                   dim3 grid, uint32_t* status, cudaStream_t stream) {
    static PerDevice<bool> configured;   // per instantiation and device
    void (*kern)(CUtensorMap, CUtensorMap, WeightMaps, Params, uint32_t*) =
        SPLIT ? gemm_w4a8_split_kernel<GROUP, PARTIALS> : gemm_w4a8_kernel<GROUP, PARTIALS>;
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
    for (int i = 0; i < kGemmMaxBatch; ++i) {
        const int src = i < a.count ? i : 0;
        p.limb_ok[i] = a.skip_if_limb_ok
            ? (const uint32_t*)((const uint8_t*)a.packed[src] + w4_geometry(a.N[src], a.K, a.group).trailer_offset) : nullptr;
    }
    int tiles = 0;
    for (int i = 0; i < kGemmMaxBatch; ++i) {
        const int src = i < a.count ? i : 0;   // unused slots repeat the first matrix
        const W4Geometry geo = w4_geometry(a.N[src], a.K, a.group);
        if (i >= a.count) {   // ... without encoding its tensor maps again
            wmaps.pk[i] = wmaps.pk[0];
            wmaps.tab[i] = wmaps.tab[0];
            p.prob[i] = p.prob[0];
            continue;
        }
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
    // With fewer tiles than SMs the K range of every tile is cut into `split` parts (whole 512-k
    // chunks) that run as separate work items and meet through scratch memory.  The split is the
    // one with the shortest critical path, in units of one group's time (~0.5 us):
    //     whole tiles:  groups per tile
    //     split:        waves of work items x (groups per item + 11) + 0.6 x split
    // where 11 stands for what a part costs beyond a whole tile's epilogue (scratch round trip,
    // fences, counter) and 0.6 for each part that the last arrival adds up (fitted to graph-replay
    // timings of 64 to 1024 tokens, K from 512 to 8960).
    const int n_chunks = (p.n_stages + 3) / 4;
    p.split = 1;
    p.split_stages = 4 * n_chunks;
    p.scratch = a.scratch;
    p.counters = a.counters;
    if (!partials && a.scratch && a.counters && p.total_tiles < n_sm && p.total_tiles * kDrainWarps <= kGemmCounters) {
        const int groups_per_chunk = 512 / a.group;
        long long best = 10ll * n_chunks * groups_per_chunk;   // tenths of a group
        for (int s = 2; s <= n_chunks && (long long)p.total_tiles * s <= kGemmScratchSlots; ++s) {
            const int cps = (n_chunks + s - 1) / s;
            if ((s - 1) * cps >= n_chunks) continue;   // a range would be empty
            const long long waves = ((long long)p.total_tiles * s + n_sm - 1) / n_sm;
            const long long cost = waves * (10ll * cps * groups_per_chunk + 110) + 6 * s;
            if (cost < best) {
                best = cost;
                p.split = s;
                p.split_stages = 4 * cps;
            }
        }
    }
    const int work = p.total_tiles * p.split;
    const dim3 grid((unsigned)(work < n_sm ? work : n_sm));   // one persistent CTA per SM
    if (a.group == 64) {
        if (partials) return launch<64, true, false>(tm_act, tm_ac, wmaps, p, grid, status, stream);
        return p.split > 1 ? launch<64, false, true>(tm_act, tm_ac, wmaps, p, grid, status, stream)
                           : launch<64, false, false>(tm_act, tm_ac, wmaps, p, grid, status, stream);
    }
    if (partials) return launch<128, true, false>(tm_act, tm_ac, wmaps, p, grid, status, stream);
    return p.split > 1 ? launch<128, false, true>(tm_act, tm_ac, wmaps, p, grid, status, stream)
                       : launch<128, false, false>(tm_act, tm_ac, wmaps, p, grid, status, stream);
}

}  // namespace mnnllm
