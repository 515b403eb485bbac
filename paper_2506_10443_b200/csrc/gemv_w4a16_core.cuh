// Building blocks shared by the W4A16 decode kernels: quantum geometry, the warp-level MMAs of one
// quantum (16 rows x 512 k of packed int4 codes against fp16 activation fragments) and output stores.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "gemv.h"
#include "ptx.cuh"

namespace mnnllm {
namespace w4a16 {

using namespace ptx;

template <int GROUP, int MP>
struct Cfg {
    static constexpr int GC = kChunkK / GROUP;           // groups per full chunk (8 or 4)
    static constexpr int SPG = GROUP / kSlabK4;          // slabs per group (1 or 2)
    static constexpr int GPS = 8 / MP;                   // group slots per accumulator tile
    static constexpr int NSETS = (GC + GPS - 1) / GPS;   // accumulator tiles per quantum
    static constexpr int QB = 8 * kSlabBytes + 16 * GC * 4;  // bytes of a full quantum
    static constexpr int PART_FLOATS = kGemvMaxRBI * MP * 16;
};

__device__ __forceinline__ float2 h2f2(uint32_t u) {
    return __half22float2(*reinterpret_cast<const __half2*>(&u));
}

// Eight bf16 values -> eight fp16 values.  Exact for every bf16 value whose magnitude lies in
// [2^-17, 65504] (8 significant bits fit fp16's 11; below, fp16 runs out of exponent; above, it saturates).
__device__ __forceinline__ uint32_t bf16x2_to_f16x2(uint32_t v) {
    const float2 f = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&v));
    const __half2 h = __floats2half2_rn(fminf(fmaxf(f.x, -65504.f), 65504.f), fminf(fmaxf(f.y, -65504.f), 65504.f));
    return *reinterpret_cast<const uint32_t*>(&h);
}
__device__ __forceinline__ uint4 bf16x8_to_f16x8(uint4 u) {
    return make_uint4(bf16x2_to_f16x2(u.x), bf16x2_to_f16x2(u.y), bf16x2_to_f16x2(u.z), bf16x2_to_f16x2(u.w));
}

__device__ __forceinline__ void store_out(void* y, int dtype, size_t idx, float v) {
    if (dtype == MNNLLM_F16) reinterpret_cast<__half*>(y)[idx] = __float2half_rn(v);
    else if (dtype == MNNLLM_BF16) reinterpret_cast<__nv_bfloat16*>(y)[idx] = __float2bfloat16_rn(v);
    else reinterpret_cast<float*>(y)[idx] = v;
}

// MMAs of one quantum.  FULL: the chunk has all 8 slabs, so the loop is branch-free and the loads
// and logic ops of different slabs can be interleaved.  Accumulator tile `set` collects GPS groups;
// with few tiles the four MMAs of a slab go to separate banks (summed afterwards) to keep the
// dependent-MMA chains short.
// B operand of slab sl, MMA a: either the full array (zeros stored for the groups that are not this
// lane's), or, in the compact form, only the lane's own slabs Pm[set][slab of the group], with the
// zeros made by a select where they are needed (half the registers at MP = 4, two selects per MMA).
template <int GROUP, int MP, bool COMPACT>
struct BFrag {
    using C = Cfg<GROUP, MP>;
    uint32_t v[COMPACT ? C::NSETS * C::SPG : 8][4][2];
    int gs;   // this lane's group slot (compact form)
    __device__ __forceinline__ uint32_t get(int sl, int a, int b) const {
        if (!COMPACT) return v[sl][a][b];
        const int gi = sl / C::SPG;
        return gs == gi % C::GPS ? v[(gi / C::GPS) * C::SPG + sl % C::SPG][a][b] : 0u;
    }
};

template <int GROUP, int MP, bool FULL, bool COMPACT>
__device__ __forceinline__ void quantum_mma(const uint4* __restrict__ slabs, int lane, int ns,
                                            const BFrag<GROUP, MP, COMPACT>& B, float (&D)[Cfg<GROUP, MP>::NSETS][4]) {
    using C = Cfg<GROUP, MP>;
    constexpr int NBANK = C::NSETS == 1 ? 2 : 1;  // four banks spill at the 128-register cap and run slower
    constexpr uint32_t LO = 0x000F000Fu, HI = 0x00F000F0u, M1024 = 0x64006400u, M64 = 0x54005400u;
    float acc[C::NSETS][NBANK][4];
#pragma unroll
    for (int s = 0; s < C::NSETS; ++s)
#pragma unroll
        for (int b = 0; b < NBANK; ++b) acc[s][b][0] = acc[s][b][1] = acc[s][b][2] = acc[s][b][3] = 0.f;
#pragma unroll
    for (int sl = 0; sl < 8; ++sl) {
        if (FULL || sl < ns) {
            const uint4 w = slabs[sl * 32 + lane];
            const int set = (sl / C::SPG) / C::GPS;
            const uint32_t x8 = w.x >> 8, z8 = w.z >> 8, y8 = w.y >> 8, w8 = w.w >> 8;
            mma_m16n8k16_f16(acc[set][0 % NBANK], lop3_and_or(w.x, LO, M1024), lop3_and_or(w.z, LO, M1024),
                             lop3_and_or(w.x, HI, M64), lop3_and_or(w.z, HI, M64), B.get(sl, 0, 0), B.get(sl, 0, 1));
            mma_m16n8k16_f16(acc[set][1 % NBANK], lop3_and_or(x8, LO, M1024), lop3_and_or(z8, LO, M1024),
                             lop3_and_or(x8, HI, M64), lop3_and_or(z8, HI, M64), B.get(sl, 1, 0), B.get(sl, 1, 1));
            mma_m16n8k16_f16(acc[set][2 % NBANK], lop3_and_or(w.y, LO, M1024), lop3_and_or(w.w, LO, M1024),
                             lop3_and_or(w.y, HI, M64), lop3_and_or(w.w, HI, M64), B.get(sl, 2, 0), B.get(sl, 2, 1));
            mma_m16n8k16_f16(acc[set][3 % NBANK], lop3_and_or(y8, LO, M1024), lop3_and_or(w8, LO, M1024),
                             lop3_and_or(y8, HI, M64), lop3_and_or(w8, HI, M64), B.get(sl, 3, 0), B.get(sl, 3, 1));
        }
    }
#pragma unroll
    for (int s = 0; s < C::NSETS; ++s)
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            float v = acc[s][0][i];
#pragma unroll
            for (int b = 1; b < NBANK; ++b) v += acc[s][b][i];
            D[s][i] = v;
        }
}

}  // namespace w4a16
}  // namespace mnnllm
