// Attention of one decoded token over a quantised KV cache (Section 4.2: keys int8, quantised per
// key vector along head_dim when they are stored; values fp8, stored as they come; Section 5.4:
// softmax in fp32, the query divided by sqrt(head_dim) before the product with the keys).
//
// Cache layout (per layer; head_dim = 128): k_codes [Hk][S_cap][128] uint8, k_meta [Hk][S_cap]
// (fp16 scale | fp16 zero << 16), v [Hk][S_cap][128] E4M3.  A key or value row is one 128-byte line:
// the cache is read in the order it is stored and never re-tiled (Section 5.1).
//
// Decode is bound by the bytes of the cache (256 B + 4 B per token and kv head): the grid splits the
// sequence so that every SM streams a share (flash-decoding), each CTA serves all query heads of its
// kv head from one pass over its tokens, and the last CTA of a kv head to finish merges the parts.
#include <cuda_fp16.h>

#include <cstdlib>

#include "attn_decode.h"
#include "common.h"
#include "ptx.cuh"

namespace mnnllm {

namespace {

constexpr int kD = kAttnHeadDim;
constexpr int kThreads = 256;
constexpr int kTile = 128;   // tokens per stage of the row buffers (two stages)
constexpr size_t kRowBytes = 2 * 2 * (size_t)kTile * 128;   // two stages of key and value rows

// fp16 bits of v, saturating at +-65504 instead of infinity
__device__ __forceinline__ uint16_t f16_sat_bits(float v) {
    uint16_t h = __half_as_ushort(__float2half_rn(v));
    if ((h & 0x7FFFu) == 0x7C00u) h = (uint16_t)((h & 0x8000u) | 0x7BFFu);
    return h;
}

// E4M3 (bias 7, no infinities, largest finite 448): round to nearest even, saturating.  x is exact
// in fp32 (it comes from fp16), so every step below is exact until the one rounding.
__device__ __forceinline__ uint8_t e4m3_from_f32(float x) {
    if (x != x) return 0x7F;
    const uint8_t sign = (__float_as_uint(x) >> 31) ? 0x80 : 0;
    const float a = fabsf(x);
    if (a >= 448.f) return sign | 0x7E;
    if (a < 0x1p-6f) return sign | (uint8_t)__float2int_rn(a * 0x1p9f);   // subnormals: multiples of 2^-9 (8 -> 2^-6)
    int e = (int)((__float_as_uint(a) >> 23) & 0xFF) - 127;
    const float mant = __uint_as_float((__float_as_uint(a) & 0x007FFFFFu) | 0x3F800000u);   // in [1, 2)
    int m = __float2int_rn((mant - 1.f) * 8.f);
    if (m == 8) { m = 0; ++e; }
    const int code = ((e + 7) << 3) | m;
    return sign | (uint8_t)(code > 0x7E ? 0x7E : code);
}

// One warp per kv head: the new key by Eq. 1 over its 128 entries (codes 0..255, fp16 scale and zero
// point, the arithmetic of the weight packer), the new value entry by entry to E4M3.
__global__ void __launch_bounds__(32) attn_append_kernel(AttnCache c, const __half* __restrict__ k_new,
                                                         const __half* __restrict__ v_new, int pos) {
    const int hk = blockIdx.x, lane = threadIdx.x;
    float w[4], vv[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        w[i] = __half2float(k_new[hk * kD + lane * 4 + i]);
        vv[i] = __half2float(v_new[hk * kD + lane * 4 + i]);
    }
    float mn = fminf(fminf(w[0], w[1]), fminf(w[2], w[3])), mx = fmaxf(fmaxf(w[0], w[1]), fmaxf(w[2], w[3]));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, o));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    }
    uint16_t sb = f16_sat_bits(__fdiv_rn(__fsub_rn(mx, mn), 255.f));
    float s = __half2float(__ushort_as_half(sb));
    uint32_t codes = 0;
    if (!(s > 0.f)) {   // constant key, or a range too small for fp16
        sb = 0x3C00u;
        s = 1.f;
    } else {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            int q = __float2int_rn(__fdiv_rn(__fsub_rn(w[i], mn), s));
            q = q < 0 ? 0 : (q > 255 ? 255 : q);
            codes |= (uint32_t)q << (8 * i);
        }
    }
    const size_t row = (size_t)hk * c.S_cap + pos;
    reinterpret_cast<uint32_t*>(c.k_codes + row * kD)[lane] = codes;
    if (lane == 0) c.k_meta[row] = (uint32_t)sb | ((uint32_t)f16_sat_bits(__fdiv_rn(-mn, s)) << 16);
    uint32_t vb = 0;
#pragma unroll
    for (int i = 0; i < 4; ++i) vb |= (uint32_t)e4m3_from_f32(vv[i]) << (8 * i);
    reinterpret_cast<uint32_t*>(c.v + row * kD)[lane] = vb;
}

}  // namespace

namespace {

// four E4M3 bytes of a word as floats TIMES 2^-8: a byte's bits placed in an fp16 give exactly that
// (subnormals included); the factor 2^8 goes on once, where a CTA's part is written
__device__ __forceinline__ void e4m3x4_to_f32_scaled(uint32_t w, float (&f)[4]) {
    // bytes 0, 1 and 2, 3 as two half2: sign to bit 15, the other seven bits to bits 7..13
    const uint32_t lo = __byte_perm(w, 0u, 0x1404), hi = __byte_perm(w, 0u, 0x3424);   // [0, b0, 0, b1], [0, b2, 0, b3]
    const uint32_t hl = (lo & 0x80008000u) | ((lo & 0x7F007F00u) >> 1);
    const uint32_t hh = (hi & 0x80008000u) | ((hi & 0x7F007F00u) >> 1);
    const float2 a = __half22float2(*reinterpret_cast<const __half2*>(&hl));
    const float2 b = __half22float2(*reinterpret_cast<const __half2*>(&hh));
    f[0] = a.x; f[1] = a.y; f[2] = b.x; f[3] = b.y;
}

// grid (splits, Hk), 256 threads = 8 warps.  Tokens [t0, t1) of kv head hk in chunks of up to 256:
//   1. scores on the tensor cores: mma.sync m16n8k16 with the kv head's query heads as rows (fp16,
//      unscaled: exact) and eight tokens as columns; the codes enter as the fp16 numbers 1024 + code
//      (a byte permute), head_dim is walked in an order that lets a lane take its two 16-byte pieces
//      of a key row as they are (the same order on the query side); the excess 1024 and the zero
//      point come off with the row sum of the query, the scale and 1/sqrt(128) go on in fp32;
//   2. warp h: the chunk's maximum for head h, the new running maximum and the factor that rescales
//      what has been accumulated so far; then every score becomes its weight exp(score - max);
//   3. weighted values: warp w takes tokens w, w + 8, ..., a lane four value entries of the row
//      (one 128-byte row per load instruction), REP x 4 accumulators per thread.
template <int REP>
__global__ void __launch_bounds__(kThreads) attn_decode_kernel(AttnCache c, const __half* __restrict__ q, void* out,
                                                               int out_dtype, int S, int per_split, float* partials,
                                                               unsigned int* counters, uint32_t* status) {
    __shared__ float m_run[REP], l_run[REP];
    __shared__ __align__(16) float ps[kThreads / 32][REP * 16 + 8];   // per warp: weights of its 16 tokens, rescale factors
    __shared__ float wm[kThreads / 32][REP], wl[kThreads / 32][REP];  // the warps' maxima and sums, merged at the end
    __shared__ unsigned int last_flag;
    __shared__ uint32_t meta_s[2][kTile];    // a tile's (scale, zero) pairs
    __shared__ __align__(8) uint64_t bar[2];  // a tile's key and value rows have landed
    extern __shared__ __align__(128) uint8_t dyn[];   // two stages of [kTile][128] key codes | [kTile][128] values

    const int split = blockIdx.x, hk = blockIdx.y, n_splits = gridDim.x;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int g = lane >> 2, cq = lane & 3;
    const int t0 = split * per_split, t1 = min(S, t0 + per_split);
    if (tid == 0) {
        ptx::mbar_init(&bar[0], 1);
        ptx::mbar_init(&bar[1], 1);
        ptx::fence_mbar_init();
        ptx::fence_proxy_async_smem();
    }
    // A tile's rows are contiguous in the cache: two bulk copies put all of its bytes in flight at once
    // (with loads issued by the warps as they go, the kernel ran at a tenth of the memory rate).  Rows
    // before position S - 1 were stored by earlier decode steps; only the newest row (and q) can come
    // from the kernels just before this one, so the first tile is requested BEFORE the wait for them
    // and its last row, when that is the newest one, after it.
    auto issue_rows = [&](int stage, int first, int count, int dst_row) {   // thread 0
        const size_t row0 = ((size_t)hk * c.S_cap + first) * kD;
        uint8_t* kb = dyn + (size_t)stage * 2 * kTile * kD + (size_t)dst_row * kD;
        ptx::bulk_g2s(kb, c.k_codes + row0, (uint32_t)count * kD, &bar[stage]);
        ptx::bulk_g2s(kb + kTile * kD, c.v + row0, (uint32_t)count * kD, &bar[stage]);
    };
    const int n0 = min(kTile, t1 - t0);
    const int n0_early = max(0, min(n0, S - 1 - t0));   // rows of the first tile that are older than the newest
    if (tid == 0 && n0 > 0) {
        ptx::mbar_arrive_expect_tx(&bar[0], 2u * (uint32_t)n0 * kD);
        if (n0_early > 0) issue_rows(0, t0, n0_early, 0);
    }
    ptx::pdl_wait();   // q and the newest cache row come from kernels before
    if (tid == 0 && n0 > n0_early) issue_rows(0, t0 + n0_early, n0 - n0_early, n0_early);
    if (tid < n0) meta_s[0][tid] = __ldg(c.k_meta + (size_t)hk * c.S_cap + t0 + tid);

    // query fragments: k-step s covers head_dim entries 16 (cq + 4 (s >> 2)) + 4 (s & 3) + {0, 1 | 2, 3}
    uint32_t qa0[8], qa2[8];
    float qs;   // sum_d q[g, d] of this lane's head
    {
        const __half* qr = q + (size_t)(hk * REP + (g < REP ? g : 0)) * kD;
        float sum = 0.f;
#pragma unroll
        for (int s = 0; s < 8; ++s) {
            const uint2 w = *reinterpret_cast<const uint2*>(qr + 16 * (cq + 4 * (s >> 2)) + 4 * (s & 3));
            qa0[s] = g < REP ? w.x : 0u;
            qa2[s] = g < REP ? w.y : 0u;
            const float2 a = __half22float2(*reinterpret_cast<const __half2*>(&w.x));
            const float2 b = __half22float2(*reinterpret_cast<const __half2*>(&w.y));
            sum += (a.x + a.y) + (b.x + b.y);
        }
        sum += __shfl_xor_sync(0xffffffffu, sum, 1);
        sum += __shfl_xor_sync(0xffffffffu, sum, 2);
        qs = sum;
    }
    __syncthreads();
    bool dead = false;   // a bounded wait gave up

    // Every warp keeps its own online softmax over the tokens it is dealt (16 of each tile): its
    // scores, weights and weighted values need no barrier of the CTA; the warps' states are merged
    // once, after the last tile.
    uint64_t acc2[REP][2];   // packed pairs of fp32: this lane's four value entries per head
#pragma unroll
    for (int h = 0; h < REP; ++h) acc2[h][0] = acc2[h][1] = 0ull;
    float m_w = -INFINITY, l_w = 0.f;   // head g of this lane's quad: running maximum, this lane's share of the sum
    float* pw = &ps[warp][0];           // [REP][16] weights of the warp's tokens, then [8] rescale factors

    for (int c0 = t0, it = 0; c0 < t1; c0 += kTile, ++it) {
        const int n = min(kTile, t1 - c0), st = it & 1;
        const uint8_t* kbuf = dyn + (size_t)st * 2 * kTile * kD;
        const uint8_t* vbuf = kbuf + kTile * kD;
        const uint32_t* meta_t = meta_s[st];
        // one barrier per tile: every warp is through with the previous tile (so the other stage may be
        // refilled and its scale/zero pairs rewritten), and a wait that gave up is known to all
        dead = __syncthreads_or(dead);
        if (dead) break;
        const int c1 = c0 + kTile;
        if (c1 < t1) {
            const int n1 = min(kTile, t1 - c1);
            if (tid == 0) {
                ptx::mbar_arrive_expect_tx(&bar[st ^ 1], 2u * (uint32_t)n1 * kD);
                issue_rows(st ^ 1, c1, n1, 0);
            }
            if (tid < n1) meta_s[st ^ 1][tid] = __ldg(c.k_meta + (size_t)hk * c.S_cap + c1 + tid);
        }
        if (!ptx::mbar_wait_bounded(&bar[st], (uint32_t)(it >> 1) & 1u, 1u << 22)) {
            dead = true;
            if (lane == 0) atomicOr(status, 0x800u);
        }
        const int w0 = warp * 16;         // this warp's tokens of the tile: w0 .. w0 + 15
        if (w0 >= n) continue;            // (uniform per warp)
        // ---- 1. scores of two groups of eight tokens; lane (g, cq) gets head g, tokens 2 cq, 2 cq + 1
        float sv[4];
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            const int tok = w0 + j * 8 + g;   // this lane's B-operand column
            uint4 u0 = make_uint4(0, 0, 0, 0), u1 = u0;
            if (tok < n) {
                const uint4* kr = reinterpret_cast<const uint4*>(kbuf + tok * kD);
                u0 = kr[cq];
                u1 = kr[cq + 4];
            }
            const uint32_t w[8] = {u0.x, u0.y, u0.z, u0.w, u1.x, u1.y, u1.z, u1.w};
            float d[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int s = 0; s < 8; ++s)
                ptx::mma_m16n8k16_f16(d, qa0[s], 0u, qa2[s], 0u, __byte_perm(w[s], 0x64646464u, 0x4140),
                                      __byte_perm(w[s], 0x64646464u, 0x4342));
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const int t = w0 + j * 8 + 2 * cq + e;
                float v = -INFINITY;
                if (t < n) {
                    const uint32_t meta = meta_t[t];
                    const __half2 sz = *reinterpret_cast<const __half2*>(&meta);
                    v = (__low2float(sz) * 0.08838834764831845f) * (d[e] - (1024.f + __high2float(sz)) * qs);
                }
                sv[2 * j + e] = v;
            }
        }
        // ---- 2. the quad's new maximum for head g, the factor for what is accumulated, the weights
        float mx = fmaxf(fmaxf(sv[0], sv[1]), fmaxf(sv[2], sv[3]));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
        const float m_new = fmaxf(m_w, mx);             // finite: token w0 is below n
        const float r = expf(m_w - m_new);              // 0 on the warp's first tile (m_w = -inf)
        float psum = 0.f;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            sv[i] = expf(sv[i] - m_new);                // 0 for a token past the end (-inf)
            psum += sv[i];
        }
        l_w = l_w * r + psum;
        m_w = m_new;
        if (g < REP) {
            *reinterpret_cast<float2*>(pw + g * 16 + 2 * cq) = make_float2(sv[0], sv[1]);
            *reinterpret_cast<float2*>(pw + g * 16 + 8 + 2 * cq) = make_float2(sv[2], sv[3]);
            if (cq == 0) pw[REP * 16 + g] = r;
        }
        __syncwarp();
        // ---- 3. weighted values: a lane holds four entries of a value row, for every head
        {
            const float4 r0 = *reinterpret_cast<const float4*>(pw + REP * 16);
            const float4 r1 = *reinterpret_cast<const float4*>(pw + REP * 16 + 4);
            const float rr[8] = {r0.x, r0.y, r0.z, r0.w, r1.x, r1.y, r1.z, r1.w};
#pragma unroll
            for (int h = 0; h < REP; ++h) {
                const uint64_t r2 = ptx::f32x2_pack(__float_as_uint(rr[h]), __float_as_uint(rr[h]));
                acc2[h][0] = ptx::f32x2_fma(acc2[h][0], r2, 0ull);   // + (+0, +0)
                acc2[h][1] = ptx::f32x2_fma(acc2[h][1], r2, 0ull);
            }
        }
        const uint32_t* vr = reinterpret_cast<const uint32_t*>(vbuf) + (size_t)w0 * (kD / 4) + lane;
#pragma unroll
        for (int t4 = 0; t4 < 4; ++t4) {
            if (w0 + 4 * t4 >= n) break;
            float4 p4[REP];
#pragma unroll
            for (int h = 0; h < REP; ++h) p4[h] = *reinterpret_cast<const float4*>(pw + h * 16 + 4 * t4);
#pragma unroll
            for (int tt = 0; tt < 4; ++tt) {
                if (w0 + 4 * t4 + tt < n) {   // rows past the end hold whatever the buffer held before
                    float val[4];
                    e4m3x4_to_f32_scaled(vr[(4 * t4 + tt) * (kD / 4)], val);
                    const uint64_t v01 = ptx::f32x2_pack(__float_as_uint(val[0]), __float_as_uint(val[1]));
                    const uint64_t v23 = ptx::f32x2_pack(__float_as_uint(val[2]), __float_as_uint(val[3]));
#pragma unroll
                    for (int h = 0; h < REP; ++h) {
                        const float pv = tt == 0 ? p4[h].x : (tt == 1 ? p4[h].y : (tt == 2 ? p4[h].z : p4[h].w));
                        const uint64_t pp = ptx::f32x2_pack(__float_as_uint(pv), __float_as_uint(pv));
                        acc2[h][0] = ptx::f32x2_fma(pp, v01, acc2[h][0]);
                        acc2[h][1] = ptx::f32x2_fma(pp, v23, acc2[h][1]);
                    }
                }
            }
        }
        __syncwarp();   // pw is rewritten for the next tile
    }
    dead = __syncthreads_or(dead);
    if (dead)   // give copies in flight time to land; this CTA's part is not counted (the status word says why)
        for (int i = 0; i < 50; ++i) __nanosleep(1000);

    ptx::pdl_launch_dependents();   // the next kernel's CTAs come in (and request their rows) while the parts are merged
    // ---- the warps' states brought to the CTA's maximum per head
    l_w += __shfl_xor_sync(0xffffffffu, l_w, 1);
    l_w += __shfl_xor_sync(0xffffffffu, l_w, 2);
    if (cq == 0 && g < REP) {
        wm[warp][g] = m_w;
        wl[warp][g] = l_w;
    }
    __syncthreads();
    // every warp scales its accumulators to the CTA's maximum and leaves them in the row buffers
    // (all tiles have been consumed); then each (head, four entries) is summed over the warps in warp
    // order by one thread: two CTA barriers in all
    float* wacc = reinterpret_cast<float*>(dyn);   // [warps][REP][128]
#pragma unroll
    for (int h = 0; h < REP; ++h) {
        float M = -INFINITY;
#pragma unroll
        for (int w = 0; w < kThreads / 32; ++w) M = fmaxf(M, wm[w][h]);
        const float mine_m = wm[warp][h];
        const float f = mine_m == -INFINITY ? 0.f : expf(mine_m - M) * 256.f;   // a warp without tokens carries nothing; 2^8: the values' scale
        float a0, a1, a2, a3;
        ptx::f32x2_unpack(acc2[h][0], a0, a1);
        ptx::f32x2_unpack(acc2[h][1], a2, a3);
        *reinterpret_cast<float4*>(wacc + (size_t)(warp * REP + h) * kD + lane * 4) = make_float4(a0 * f, a1 * f, a2 * f, a3 * f);
    }
    if (tid < REP) {
        float M = -INFINITY, l = 0.f;
        for (int w = 0; w < kThreads / 32; ++w) M = fmaxf(M, wm[w][tid]);
        for (int w = 0; w < kThreads / 32; ++w)   // warp order: the same sum whatever the timing
            l += wm[w][tid] == -INFINITY ? 0.f : wl[w][tid] * expf(wm[w][tid] - M);
        m_run[tid] = M;
        l_run[tid] = l;
    }
    __syncthreads();
    // ---- this CTA's part: {m, l, acc[128]} per query head.  In a cluster every CTA stores its part
    // into the shared memory of the CTA of rank 0 (distributed shared memory), which merges them in
    // rank order (the same sum whatever the timing): the final merge reads an eighth of the parts.
    constexpr int kPart = kD + 2;
    constexpr int kPitch = kD + 4;   // in shared memory {m, l, -, -, acc[128]}: the accumulators on a 16-byte boundary
    const int CS = (int)ptx::cluster_nctarank(), crank = (int)ptx::cluster_ctarank();
    const int n_parts = n_splits / CS;
    float* mine = partials + ((size_t)(hk * n_parts + split / CS) * REP) * kPart;
    float* cbuf = reinterpret_cast<float*>(dyn + kRowBytes);   // [8 ranks][REP][kPitch], written by the peers
    for (int idx = tid; idx < REP * 32; idx += kThreads) {
        const int h = idx >> 5;
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int w = 0; w < kThreads / 32; ++w) {
            const float4 o = *reinterpret_cast<const float4*>(wacc + (size_t)(w * REP + h) * kD + lane * 4);
            v.x += o.x; v.y += o.y; v.z += o.z; v.w += o.w;
        }
        if (CS == 1) {
            __stcg(reinterpret_cast<float2*>(mine + h * kPart + 2 + lane * 4), make_float2(v.x, v.y));
            __stcg(reinterpret_cast<float2*>(mine + h * kPart + 4 + lane * 4), make_float2(v.z, v.w));
            if (lane == 0) __stcg(reinterpret_cast<float2*>(mine + h * kPart), make_float2(m_run[h], l_run[h]));
        } else {
            float* slot = cbuf + (size_t)(crank * REP + h) * kPitch;
            ptx::st_dsmem_f32x4(slot + 4 + lane * 4, 0u, v);
            if (lane == 0) ptx::st_dsmem_f32x2(slot, 0u, make_float2(m_run[h], l_run[h]));
        }
    }
    if (CS > 1) {
        ptx::cluster_arrive_release();   // this CTA's stores into rank 0 are ordered before the arrival
        if (crank != 0) return;          // nothing reads a peer's shared memory: it may go
        ptx::cluster_wait_acquire();
        for (int idx = tid; idx < REP * 32; idx += kThreads) {
            const int h = idx >> 5;
            float2 ml[8];
            float4 av[8];
#pragma unroll
            for (int r = 0; r < 8; ++r) {
                ml[r] = make_float2(-INFINITY, 0.f);
                av[r] = make_float4(0.f, 0.f, 0.f, 0.f);
                if (r < CS) {
                    const float* slot = cbuf + (size_t)(r * REP + h) * kPitch;
                    ml[r] = *reinterpret_cast<const float2*>(slot);
                    av[r] = *reinterpret_cast<const float4*>(slot + 4 + lane * 4);
                }
            }
            float m = -INFINITY;
#pragma unroll
            for (int r = 0; r < 8; ++r) m = fmaxf(m, ml[r].x);
            float l = 0.f, a4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int r = 0; r < 8; ++r) {   // rank order
                const float w = ml[r].x == -INFINITY ? 0.f : expf(ml[r].x - m);   // a CTA without tokens carries nothing
                l = fmaf(ml[r].y, w, l);
                a4[0] = fmaf(av[r].x, w, a4[0]); a4[1] = fmaf(av[r].y, w, a4[1]);
                a4[2] = fmaf(av[r].z, w, a4[2]); a4[3] = fmaf(av[r].w, w, a4[3]);
            }
            __stcg(reinterpret_cast<float2*>(mine + h * kPart + 2 + lane * 4), make_float2(a4[0], a4[1]));
            __stcg(reinterpret_cast<float2*>(mine + h * kPart + 4 + lane * 4), make_float2(a4[2], a4[3]));
            if (lane == 0) __stcg(reinterpret_cast<float2*>(mine + h * kPart), make_float2(m, l));
        }
    }
    __threadfence();
    __syncthreads();
    if (tid == 0) last_flag = !dead && atomicAdd(counters + hk, 1u) == (unsigned int)n_parts - 1u;
    __syncthreads();
    if (!last_flag) return;
    // ---- the last CTA of the kv head merges the parts, in the order of the parts (the same sum
    // whoever comes last), and clears the counter for the next call.  One thread per (head, four
    // entries): all of its loads are issued before any is used, 16 parts at a time, so the merge is
    // one round trip to L2; no shared memory, no barrier.
    __threadfence();
    if (tid == 0) counters[hk] = 0u;
    const float* parts = partials + ((size_t)hk * n_parts * REP) * kPart;
    for (int idx = tid; idx < REP * 32; idx += kThreads) {
        const int h = idx >> 5;
        float m = -INFINITY, l = 0.f, a4[4] = {0.f, 0.f, 0.f, 0.f};
        for (int s0 = 0; s0 < n_parts; s0 += 16) {
            float2 ml[16], lo[16], hi[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                ml[i] = make_float2(-INFINITY, 0.f);
                lo[i] = hi[i] = make_float2(0.f, 0.f);
                if (s0 + i < n_parts) {
                    const float* ps_ = parts + ((size_t)(s0 + i) * REP + h) * kPart;
                    ml[i] = __ldcg(reinterpret_cast<const float2*>(ps_));
                    lo[i] = __ldcg(reinterpret_cast<const float2*>(ps_ + 2 + lane * 4));
                    hi[i] = __ldcg(reinterpret_cast<const float2*>(ps_ + 4 + lane * 4));
                }
            }
            float m_new = m;
#pragma unroll
            for (int i = 0; i < 16; ++i) m_new = fmaxf(m_new, ml[i].x);
            const float r = m == -INFINITY ? 0.f : expf(m - m_new);   // what has been summed so far
            l *= r;
#pragma unroll
            for (int i = 0; i < 4; ++i) a4[i] *= r;
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                const float w = ml[i].x == -INFINITY ? 0.f : expf(ml[i].x - m_new);   // a part without tokens carries nothing
                l = fmaf(ml[i].y, w, l);
                a4[0] = fmaf(lo[i].x, w, a4[0]); a4[1] = fmaf(lo[i].y, w, a4[1]);
                a4[2] = fmaf(hi[i].x, w, a4[2]); a4[3] = fmaf(hi[i].y, w, a4[3]);
            }
            m = m_new;
        }
        const size_t o = (size_t)(hk * REP + h) * kD + lane * 4;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float r = a4[i] / l;
            if (out_dtype == MNNLLM_F32) reinterpret_cast<float*>(out)[o + i] = r;
            else reinterpret_cast<__half*>(out)[o + i] = __float2half_rn(r);
        }
    }
    (void)status;
}

}  // namespace

constexpr size_t kDynSmem = kRowBytes + (size_t)8 * kAttnMaxRep * (kD + 4) * sizeof(float);   // row stages, then the parts of a cluster's CTAs

template <int REP>
static cudaError_t ensure_smem() {
    static PerDevice<bool> configured;   // per instantiation and device
    return configured.with([&](bool& done) {
        if (done) return cudaSuccess;
        cudaError_t e = cudaFuncSetAttribute(attn_decode_kernel<REP>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kDynSmem);
        done = e == cudaSuccess;
        return e;
    });
}

// Tokens per CTA: the sequence over about two CTAs per SM, in multiples of 32 and at least 128 (a part
// costs a merge step: short sequences are not cut finer than that).
constexpr int kClusterSize = 8;

// CTAs that can be resident at once when they come in clusters of eight (clusters do not straddle
// GPCs, so this is less than two per SM); asked of the runtime once per device for the instantiation
// with the most registers.  0: the query failed.
static int resident_cluster_ctas() {
    static PerDevice<int> cached;
    int out = 0;
    (void)cached.with([&](int& v) {
        if (v == 0) {
            v = -1;
            if (ensure_smem<kAttnMaxRep>() == cudaSuccess) {
                cudaLaunchConfig_t cfg = {};
                cfg.gridDim = dim3(kClusterSize * 64);
                cfg.blockDim = dim3(kThreads);
                cfg.dynamicSmemBytes = kDynSmem;
                cudaLaunchAttribute attr[1];
                attr[0].id = cudaLaunchAttributeClusterDimension;
                attr[0].val.clusterDim.x = kClusterSize;
                attr[0].val.clusterDim.y = 1;
                attr[0].val.clusterDim.z = 1;
                cfg.attrs = attr;
                cfg.numAttrs = 1;
                int n = 0;
                if (cudaOccupancyMaxActiveClusters(&n, attn_decode_kernel<kAttnMaxRep>, &cfg) == cudaSuccess && n > 0)
                    v = n * kClusterSize;
                else
                    (void)cudaGetLastError();
            }
        }
        out = v > 0 ? v : 0;
        return cudaSuccess;
    });
    return out;
}

static int tokens_per_split(int Hk, int S) {
    const int n_sm = device_sm_count() > 0 ? device_sm_count() : 148;
    int ctas = 2 * n_sm;
    if (const int rc = resident_cluster_ctas(); rc > 0 && rc < ctas) ctas = rc;   // one wave of clusters
    int want = ctas / Hk;
    if (want >= 2 * kClusterSize) want = want / kClusterSize * kClusterSize;   // the grid is padded to whole clusters
    if (want < 1) want = 1;
    if (want > kAttnChunk) want = kAttnChunk;   // the merge keeps one weight per part in a chunk-sized array
    int per = ((S + want - 1) / want + 31) / 32 * 32;
    if (const char* env = std::getenv("MNNLLM_ATTN_SPLIT_TOKENS")) {   // tuning override (multiples of 32, never finer than the default's limits)
        const int v = std::atoi(env);
        if (v >= kAttnMinSplit && v % 32 == 0 && (S + v - 1) / v <= kAttnChunk) per = v;
    }
    return per < kAttnMinSplit ? kAttnMinSplit : per;
}

int attn_splits(int Hk, int S) {
    const int per = tokens_per_split(Hk, S);
    return (S + per - 1) / per;
}

size_t attn_partials_bytes(int H, int Hk, int S) {
    return (size_t)attn_splits(Hk, S) * H * (kD + 2) * sizeof(float);
}

cudaError_t attn_append_launch(const AttnCache& c, const void* k_new, const void* v_new, int pos, cudaStream_t stream) {
    attn_append_kernel<<<c.Hk, 32, 0, stream>>>(c, (const __half*)k_new, (const __half*)v_new, pos);
    return cudaGetLastError();
}

cudaError_t attn_decode_launch(const AttnCache& c, const void* q, void* out, int out_dtype, int H, int S, float* partials,
                               unsigned int* counters, uint32_t* status, cudaStream_t stream) {
    const int rep = H / c.Hk, splits = attn_splits(c.Hk, S), per_split = tokens_per_split(c.Hk, S);
    // clusters of eight CTAs merge their parts on chip; the grid is padded to whole clusters (a CTA
    // past the end of the sequence contributes an empty part)
    const int CS = splits >= 2 * kClusterSize ? kClusterSize : 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)((splits + CS - 1) / CS * CS), (unsigned)c.Hk);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = kDynSmem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = (unsigned)CS;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    // A grid of clusters is launched in plain stream order: as a programmatic dependent launch its
    // CTAs took their places before the grid ahead had finished and every launch then lost ~7 us
    // (measured at 32768 tokens, where a grid fills the GPU: 23.5 against 17.6 us per layer).
    cfg.attrs = CS > 1 ? attr + 1 : attr;
    cfg.numAttrs = 1;
    const __half* qh = (const __half*)q;
#define MNN_CASE(R)                                                                                                      \
    case R:                                                                                                             \
        if (cudaError_t e = ensure_smem<R>(); e != cudaSuccess) return e;                                               \
        return cudaLaunchKernelEx(&cfg, attn_decode_kernel<R>, c, qh, out, out_dtype, S, per_split, partials, counters, status);
    switch (rep) {
        MNN_CASE(1) MNN_CASE(2) MNN_CASE(3) MNN_CASE(4) MNN_CASE(5) MNN_CASE(6) MNN_CASE(7) MNN_CASE(8)
    }
#undef MNN_CASE
    return cudaErrorInvalidValue;
}

}  // namespace mnnllm
