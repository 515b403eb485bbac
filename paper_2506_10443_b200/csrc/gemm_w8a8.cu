// Per-channel W8A8 prefill GEMM (Section 4.2: int8 weights, int8 activations) on tcgen05.
//
//   y[m, n] = a_scale[m] * ( s[n] * P[m, n]  -  (s z)[n] * A[m] ),   P = sum_k a_q[m, k] q[n, k],  A[m] = sum_k a_q[m, k]
//
// One scale and zero point per weight row: the integer dot product runs over all of K in one int32
// accumulator in tensor memory and is rescaled once, in the epilogue.  Nothing is taken out of
// tensor memory per group, which is what bounds the W4A8 kernel (gemm_w4a8.cu).
//
// Tile: 128 weight rows (MMA M) x TT tokens (MMA N; 256, or 128 for short prompts), tcgen05.mma
// kind::i8 with unsigned weight codes and signed activation codes, K = 32 per instruction.  Tensor
// memory holds two accumulators (2 x TT columns): the epilogue of a tile overlaps the main loop of
// the next.  The CTA is persistent, one per SM; tiles blockIdx.x, + gridDim.x, ..., token tile
// fastest (CTAs that run together share their weight tile in L2).
//
// Operands.  Activations [M, K] int8 are loaded by TMA straight into the 128B-swizzled K-major form.
// Weights are in the packed W8 layout that the decode GEMV streams (slabs of 16 rows x 32 k, 16 bytes
// per lane: 8 bytes of row r, 8 bytes of row r + 8): TMA brings a stage's slabs as they are, and four
// warps move them into the swizzled K-major tile with one 16-byte load and two 8-byte stores per
// lane and slab.  Row r's lanes take the stage's four slabs in the order i ^ (r & 3): the sixteen
// lanes of a store wavefront then write eight different 16-byte columns (no bank conflict), and
// the loads are conflict-free in any order.
//
// Measured on B200: 1.2-1.7 POP/s (17920 x 1536 at 1024 tokens: 1.5; K = 6144: 1.7), three to four
// times the W4A8 kernel.  The main loop takes ~0.7 us per 128-k stage whatever the tile count, i.e.
// every SM takes in its 48 KiB of operands per stage at ~67 GB/s, ~10 TB/s over the GPU: the operand
// feed from L2, not the tensor pipe (0.29 us per stage), sets the pace.  A variant that copied the
// slabs with 8-byte cp.async straight into the swizzled tile (no staging buffer, four stages
// instead of three) was 15 % slower: twice the requests for the same bytes.
//
// Roles (14 warps): TMA producer | MMA issue | 4 rearranging warps | 8 epilogue warps (two per
// tensor-memory lane quarter, half of the token columns each).
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include <type_traits>

#include "common.h"
#include "gemm_w8a8.h"
#include "layout.h"
#include "ptx.cuh"

namespace mnnllm {

using namespace ptx;

namespace {

constexpr int kTileN = 128;    // weight rows per tile (MMA M)
constexpr int kStageK = 128;   // k per pipeline stage (one 128-byte swizzle row of int8): four W8 slabs
constexpr int kStages = 3;
constexpr int kMoveWarps = 4, kMoveWarp0 = 2, kEpiWarp0 = 6, kEpiWarps = 8;
constexpr int kThreads = (kEpiWarp0 + kEpiWarps) * 32;
constexpr uint32_t kMaxPolls = 1u << 15;
constexpr uint32_t kTmemCols = 512;

constexpr int kTileBytes = kTileN * kStageK;     // 16 KiB: the swizzled weight tile of a stage
constexpr int kRawBytes = 8 * 4 * kSlabBytes;    // 16 KiB: the same codes as packed (8 row blocks x 4 slabs)

template <int TT>
struct Smem {
    static constexpr int act_bytes = TT * kStageK;
    static constexpr int act = 0;                                  // [kStages] activations
    static constexpr int tile = act + kStages * act_bytes;         // [kStages] weight tiles (swizzled K-major)
    static constexpr int raw = tile + kStages * kTileBytes;        // [kStages] packed slabs
    static constexpr int tok = raw + kStages * kRawBytes;          // [kEpiWarps][TT / 2] per-token {a_scale, a_scale * A}
    static constexpr int bars = tok + kEpiWarps * (TT / 2) * 8;
    static constexpr int n_bars = 5 * kStages + 4;
    static constexpr int misc = bars + n_bars * 8;
    static constexpr int total = misc + 16;
    static constexpr size_t bytes = total + 1024;
};

// D int32, A (weights) unsigned 8-bit, B (activations) signed 8-bit, both K-major
template <int TT>
constexpr uint32_t idesc_i8() {
    return (2u << 4) | (0u << 7) | (1u << 10) | ((uint32_t)(TT >> 3) << 17) | ((uint32_t)(kTileN >> 4) << 24);
}

struct Params {
    void* y;
    const uint32_t* table;   // per padded weight row: fp16 scale | fp16 zero << 16
    const float* a_scale;
    const int32_t* a_sum;
    int M, N, K, n_stages, tiles_m, total_tiles, y_dtype;
};

template <typename T>
__device__ __forceinline__ T to_out(float v);
template <>
__device__ __forceinline__ __half to_out<__half>(float v) { return __float2half_rn(v); }
template <>
__device__ __forceinline__ __nv_bfloat16 to_out<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }
template <>
__device__ __forceinline__ float to_out<float>(float v) { return v; }

template <int TT>
__global__ void __launch_bounds__(kThreads, 1)
gemm_w8a8_kernel(const __grid_constant__ CUtensorMap tm_act, const __grid_constant__ CUtensorMap tm_raw,
                 const __grid_constant__ Params p, uint32_t* __restrict__ status) {
    using S = Smem<TT>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + S::bars);
    uint64_t* raw_full = bars;                  // [kStages] packed slabs landed
    uint64_t* raw_empty = raw_full + kStages;   // [kStages] ... and are in the moving warps' registers
    uint64_t* tile_full = raw_empty + kStages;  // [kStages] swizzled weight tile written
    uint64_t* act_full = tile_full + kStages;   // [kStages] activations landed
    uint64_t* st_free = act_full + kStages;     // [kStages] the stage's MMAs have completed (tile and activations)
    uint64_t* acc_full = st_free + kStages;     // [2] a tile's accumulator is complete
    uint64_t* acc_empty = acc_full + 2;         // [2] ... and has been read
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + S::misc);
    volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(smem + S::misc + 4);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_stages = p.n_stages, total_tiles = p.total_tiles;

    if (threadIdx.x == 0) {
        for (int i = 0; i < kStages; ++i) {
            mbar_init(&raw_full[i], 1);
            mbar_init(&raw_empty[i], kMoveWarps);
            mbar_init(&tile_full[i], kMoveWarps);
            mbar_init(&act_full[i], 1);
            mbar_init(&st_free[i], 1);
        }
        for (int i = 0; i < 2; ++i) { mbar_init(&acc_full[i], 1); mbar_init(&acc_empty[i], kEpiWarps); }
        *abort_flag = 0;
        fence_mbar_init();
        prefetch_tensormap(&tm_act);
        prefetch_tensormap(&tm_raw);
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    // the weight side does not depend on the quantiser that precedes this grid; the threads that read
    // its outputs call griddepcontrol.wait first
    pdl_launch_dependents();

    auto wait = [&](uint64_t* bar, uint32_t parity, uint32_t code) -> bool {
        if (mbar_wait_bounded_compact(bar, parity, kMaxPolls)) return true;
        if (*abort_flag == 0) {
            *abort_flag = 1;
            atomicOr(status, 0x600u | code);
        }
        return false;
    };

    if (warp == 0) {
        // ------------------------------------------------------------------ producer (TMA)
        // Two cursors over the same (tile, stage) sequence: the packed weights run kStages stages ahead
        // of the activations (their slots are free at the start, and they do not wait for the quantiser).
        if (elect_one()) {
            int t_r = blockIdx.x, st_r = 0, t_a = blockIdx.x, st_a = 0;
            uint32_t gr = 0, ga = 0;   // running stage counts of the two cursors
            bool first = true;
            while (t_a < total_tiles) {
                while (t_r < total_tiles && gr < ga + kStages) {
                    const int slot = gr % kStages;
                    if (!wait(&raw_empty[slot], ((gr / kStages) & 1) ^ 1, 1)) { t_a = total_tiles; break; }
                    const int tn = t_r / p.tiles_m;
                    mbar_arrive_expect_tx(&raw_full[slot], kRawBytes);
                    // x in 8-byte elements: four slabs of 512 bytes per stage
                    tma_load_2d(smem + S::raw + slot * kRawBytes, &tm_raw, st_r * (4 * kSlabBytes / 8), tn * 8, &raw_full[slot]);
                    ++gr;
                    if (++st_r == n_stages) { st_r = 0; t_r += gridDim.x; }
                }
                if (t_a >= total_tiles) break;
                if (first) { pdl_wait(); first = false; }   // the quantised activations are complete from here on
                const int slot = ga % kStages;
                if (!wait(&st_free[slot], ((ga / kStages) & 1) ^ 1, 2)) break;
                const int tn = t_a / p.tiles_m, m0 = (t_a - tn * p.tiles_m) * TT;
                mbar_arrive_expect_tx(&act_full[slot], S::act_bytes);
                tma_load_2d(smem + S::act + slot * S::act_bytes, &tm_act, st_a * kStageK, m0, &act_full[slot]);
                ++ga;
                if (++st_a == n_stages) { st_a = 0; t_a += gridDim.x; }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issue
        if (elect_one()) {
            uint32_t gs = 0;
            int it = 0;
            const uint32_t act_addr = smem_u32(smem + S::act), tile_addr = smem_u32(smem + S::tile);
            bool ok = true;
            for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x, ++it) {
                const int buf = it & 1;
                // the accumulator's previous tile (two tiles ago) must have been read
                if (!wait(&acc_empty[buf], (((uint32_t)it >> 1) & 1u) ^ 1u, 3)) break;
                tc_fence_after_sync();
                for (int st = 0; st < n_stages; ++st, ++gs) {
                    const int slot = gs % kStages;
                    const uint32_t par = (gs / kStages) & 1;
                    if (!wait(&act_full[slot], par, 4) || !wait(&tile_full[slot], par, 5)) { ok = false; break; }
                    tc_fence_after_sync();
                    const uint64_t da = desc_sw128(tile_addr + slot * kTileBytes);
                    const uint64_t db = desc_sw128(act_addr + slot * S::act_bytes);
#pragma unroll
                    for (int kk = 0; kk < kStageK / 32; ++kk) {
                        const uint64_t adv = (uint64_t)((kk * 32) >> 4);
                        mma_i8_ss(tmem_base + buf * TT, da + adv, db + adv, idesc_i8<TT>(), (st > 0 || kk > 0) ? 1u : 0u);
                    }
                    mma_commit(&st_free[slot]);
                }
                if (ok) mma_commit(&acc_full[buf]);
            }
        }
        __syncwarp();
    } else if (warp < kEpiWarp0) {
        // ------------------------------------------------------------------ packed slabs -> swizzled K-major tile
        const int wu = warp - kMoveWarp0;   // row blocks 2 wu and 2 wu + 1 of the tile
        const int r = lane >> 2, c = lane & 3;
        uint32_t gs = 0;
        bool ok = true;
        for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x) {
            for (int st = 0; st < n_stages; ++st, ++gs) {
                const int slot = gs % kStages;
                const uint32_t par = (gs / kStages) & 1;
                if (!wait(&raw_full[slot], par, 6)) { ok = false; break; }
                const uint4* raw = reinterpret_cast<const uint4*>(smem + S::raw + slot * kRawBytes);
                uint4 v[2][4];
#pragma unroll
                for (int b = 0; b < 2; ++b)
#pragma unroll
                    for (int i = 0; i < 4; ++i) v[b][i] = raw[((wu * 2 + b) * 4 + (i ^ (r & 3))) * 32 + lane];
                __syncwarp();
                if (lane == 0) mbar_arrive(&raw_empty[slot]);
                if (!wait(&st_free[slot], par ^ 1, 7)) { ok = false; break; }
                // row R of the tile at (R >> 3) * 1024 + (R & 7) * 128, its 16-byte chunk kc at ((kc ^ (R & 7)) << 4)
                uint8_t* tile = smem + S::tile + slot * kTileBytes;
#pragma unroll
                for (int b = 0; b < 2; ++b)
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int sl = i ^ (r & 3);
                        const int kc = sl * 2 + (c >> 1);
                        const uint32_t off = (uint32_t)((wu * 2 + b) * 2) * 1024u + (uint32_t)r * 128u +
                                             (uint32_t)((kc ^ r) << 4) + (uint32_t)(c & 1) * 8u;
                        *reinterpret_cast<uint2*>(tile + off) = make_uint2(v[b][i].x, v[b][i].y);            // row r
                        *reinterpret_cast<uint2*>(tile + off + 1024u) = make_uint2(v[b][i].z, v[b][i].w);    // row r + 8
                    }
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) mbar_arrive(&tile_full[slot]);
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue: once per tile
        const int ew = warp - kEpiWarp0;
        const int q4 = warp & 3;          // tensor-memory lane quarter this warp may read
        const int half = ew >> 2;         // which half of the token columns
        const int nl = q4 * 32 + lane;    // this thread's weight row of the tile
        constexpr int kCols = TT / 2;
        const uint32_t lane_base = tmem_base + ((uint32_t)(q4 * 32) << 16) + half * kCols;
        float2* tok = reinterpret_cast<float2*>(smem + S::tok) + ew * kCols;
        const int n_pad = ((p.N + 15) / 16) * 16;
        int it = 0;
        for (int t = blockIdx.x; t < total_tiles; t += gridDim.x, ++it) {
            const int tn = t / p.tiles_m;
            const int m0 = (t - tn * p.tiles_m) * TT + half * kCols, n = tn * kTileN + nl;
            const int buf = it & 1;
            float s = 0.f, sz = 0.f;
            if (n < n_pad) {
                const uint32_t e = __ldg(p.table + n);
                const __half2 h2 = *reinterpret_cast<const __half2*>(&e);
                s = __low2float(h2);
                sz = s * __high2float(h2);   // exact in fp32 (two 11-bit significands)
            }
            if (it == 0) pdl_wait();   // a_scale and a_sum come from the quantiser
            __syncwarp();              // the previous tile's reads of tok are done
#pragma unroll
            for (int c4 = 0; c4 < kCols / 32; ++c4) {
                const int m = m0 + c4 * 32 + lane;
                float as = 0.f, asum = 0.f;
                if (m < p.M) {
                    as = __ldg(p.a_scale + m);
                    asum = (float)__ldg(p.a_sum + m);   // |sum| <= 127 K: exact
                }
                tok[c4 * 32 + lane] = make_float2(as, as * asum);
            }
            __syncwarp();
            if (!wait(&acc_full[buf], ((uint32_t)it >> 1) & 1u, 8)) break;
            tc_fence_after_sync();
            auto run = [&](auto* yout) {
                using T = typename std::remove_pointer<decltype(yout)>::type;
#pragma unroll 1
                for (int c4 = 0; c4 < kCols / 32; ++c4) {
                    uint32_t v[32];
                    tmem_ld_x32(lane_base + buf * TT + c4 * 32, v);
                    tmem_ld_wait();
                    if (c4 == kCols / 32 - 1) {   // everything is in registers: the accumulator may be overwritten
                        tc_fence_before_sync();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(&acc_empty[buf]);
                    }
                    if (n < p.N) {
                        T* col = yout + (size_t)(m0 + c4 * 32) * p.N + n;
                        const int mrem = p.M - (m0 + c4 * 32);
#pragma unroll
                        for (int j = 0; j < 32; ++j) {
                            const float2 tk = tok[c4 * 32 + j];
                            const float val = fmaf(s * tk.x, (float)(int32_t)v[j], -(sz * tk.y));
                            if (j < mrem) col[(size_t)j * p.N] = to_out<T>(val);
                        }
                    }
                }
            };
            if (p.y_dtype == MNNLLM_F16) run(reinterpret_cast<__half*>(p.y));
            else if (p.y_dtype == MNNLLM_BF16) run(reinterpret_cast<__nv_bfloat16*>(p.y));
            else run(reinterpret_cast<float*>(p.y));
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

template <int TT>
cudaError_t launch(const GemmW8A8Args& a, uint32_t* status, cudaStream_t stream) {
    EncodeTiledFn enc = encode_fn();
    if (!enc) return cudaErrorNotSupported;
    const W8Geometry geo = w8_geometry(a.N, a.K);
    const uint8_t* base = (const uint8_t*)a.packed;
    CUtensorMap tm_act, tm_raw;
    const cuuint32_t estr[2] = {1, 1};
    {
        // the packed body as [row block][8-byte words]: a stage is 8 row blocks x 2 KiB (four slabs);
        // rows past the last row block and words past a row block's end read as zeros
        const cuuint64_t dims[2] = {(cuuint64_t)(geo.row_block_bytes / 8), (cuuint64_t)geo.n_row_blocks};
        const cuuint64_t strides[1] = {(cuuint64_t)geo.row_block_bytes};
        const cuuint32_t box[2] = {4 * kSlabBytes / 8, 8};
        if (enc(&tm_raw, CU_TENSOR_MAP_DATA_TYPE_UINT64, 2, (void*)(base + kHeaderBytes), dims, strides, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return cudaErrorInvalidValue;
    }
    {
        const cuuint64_t dims[2] = {(cuuint64_t)a.K, (cuuint64_t)a.M};
        const cuuint64_t strides[1] = {(cuuint64_t)a.K};
        const cuuint32_t box[2] = {(cuuint32_t)kStageK, (cuuint32_t)TT};
        if (enc(&tm_act, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, (void*)a.a_q, dims, strides, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return cudaErrorInvalidValue;
    }
    Params p;
    p.y = a.y;
    p.table = (const uint32_t*)(base + geo.table_offset);
    p.a_scale = a.a_scale;
    p.a_sum = a.a_sum;
    p.M = a.M; p.N = a.N; p.K = a.K;
    p.n_stages = (a.K + kStageK - 1) / kStageK;
    p.tiles_m = (a.M + TT - 1) / TT;
    p.total_tiles = ((a.N + kTileN - 1) / kTileN) * p.tiles_m;
    p.y_dtype = a.y_dtype;

    static PerDevice<bool> configured;   // per instantiation and device
    auto kern = gemm_w8a8_kernel<TT>;
    if (cudaError_t e = configured.with([&](bool& done) {
            if (done) return cudaSuccess;
            cudaError_t err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Smem<TT>::bytes);
            done = err == cudaSuccess;
            return err;
        });
        e != cudaSuccess)
        return e;
    const int n_sm = device_sm_count();
    if (n_sm <= 0) return cudaErrorInvalidDevice;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(p.total_tiles < n_sm ? p.total_tiles : n_sm));   // one persistent CTA per SM
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = Smem<TT>::bytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, tm_act, tm_raw, p, status);
}

}  // namespace

cudaError_t gemm_w8a8_launch(const GemmW8A8Args& a, uint32_t* status, cudaStream_t stream) {
    // 256-token tiles halve the weight-side work per MAC; prompts that would leave SMs idle with
    // them (or fit one 128-token tile) take 128-token tiles
    const int n_sm = device_sm_count();
    const long long tiles256 = (long long)((a.N + kTileN - 1) / kTileN) * ((a.M + 255) / 256);
    if (a.M > 128 && tiles256 >= n_sm) return launch<256>(a, status, stream);
    return launch<128>(a, status, stream);
}

}  // namespace mnnllm
