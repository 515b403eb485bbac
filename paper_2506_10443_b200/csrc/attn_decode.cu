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

#include "attn_decode.h"
#include "common.h"
#include "ptx.cuh"

namespace mnnllm {

namespace {

constexpr int kD = kAttnHeadDim;
constexpr int kThreads = 256;

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

// an E4M3 byte as float: its bits placed in an fp16 give the value * 2^-8, exactly (subnormals too)
__device__ __forceinline__ float e4m3_to_f32(uint32_t b) {
    const uint16_t h = (uint16_t)(((b & 0x80u) << 8) | ((b & 0x7Fu) << 7));
    return __half2float(__ushort_as_half(h)) * 256.f;
}

struct Part {   // what a CTA leaves per query head: running maximum, sum of weights, weighted values
    float m, l;
};

// grid (splits, Hk), 256 threads.  Tokens [t0, t1) of kv head hk in chunks of 256:
//   1. thread t: scores of token t for the kv head's `rep` query heads (the key row is 8 x 16 bytes
//      per thread, the scaled queries come from shared memory as broadcasts);
//   2. warp h: the chunk's maximum for head h, the new running maximum and the factor that rescales
//      what has been accumulated so far; then every score becomes its weight exp(score - max);
//   3. thread (d, half): value entry d of the tokens of its half of the chunk, rep accumulators.
template <int REP>
__global__ void __launch_bounds__(kThreads) attn_decode_kernel(AttnCache c, const __half* __restrict__ q, void* out,
                                                               int out_dtype, int S, int per_split, float* partials,
                                                               unsigned int* counters, uint32_t* status) {
    __shared__ float qs[REP][kD];          // q / sqrt(128)
    __shared__ float qsum[REP];            // sum_d of the scaled query (zero-point term)
    __shared__ float sc[REP][kAttnChunk];  // scores, then weights
    __shared__ float m_run[REP], l_run[REP], rescale[REP];
    __shared__ float acc_half[REP][kD];    // second half's accumulators for the final sum
    __shared__ unsigned int last_flag;

    const int split = blockIdx.x, hk = blockIdx.y, n_splits = gridDim.x;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int t0 = split * per_split, t1 = min(S, t0 + per_split);
    ptx::pdl_launch_dependents();
    ptx::pdl_wait();   // q (and the newest cache row) come from kernels before
    for (int i = tid; i < REP * kD; i += kThreads)
        qs[i / kD][i % kD] = __half2float(q[(size_t)(hk * REP) * kD + i]) * 0.08838834764831845f;   // 1 / sqrt(128)
    if (tid < REP) { m_run[tid] = -INFINITY; l_run[tid] = 0.f; }
    __syncthreads();
    if (warp < REP) {
        float a = qs[warp][lane] + qs[warp][lane + 32] + qs[warp][lane + 64] + qs[warp][lane + 96];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
        if (lane == 0) qsum[warp] = a;
    }
    __syncthreads();

    const int d = tid & (kD - 1), half = tid >> 7;
    float acc[REP];
#pragma unroll
    for (int h = 0; h < REP; ++h) acc[h] = 0.f;

    for (int c0 = t0; c0 < t1; c0 += kAttnChunk) {
        const int n = min(kAttnChunk, t1 - c0);
        // ---- 1. scores
        if (tid < n) {
            const size_t row = (size_t)hk * c.S_cap + c0 + tid;
            const uint4* kr = reinterpret_cast<const uint4*>(c.k_codes + row * kD);
            const uint32_t meta = __ldg(c.k_meta + row);
            const __half2 sz = *reinterpret_cast<const __half2*>(&meta);
            const float s = __low2float(sz), z = __high2float(sz);
            float dot[REP];
#pragma unroll
            for (int h = 0; h < REP; ++h) dot[h] = 0.f;
#pragma unroll
            for (int v = 0; v < kD / 16; ++v) {
                const uint4 w = __ldg(kr + v);
                const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    const float code = (float)((ww[j >> 2] >> (8 * (j & 3))) & 0xFFu);
#pragma unroll
                    for (int h = 0; h < REP; ++h) dot[h] = fmaf(qs[h][v * 16 + j], code, dot[h]);
                }
            }
#pragma unroll
            for (int h = 0; h < REP; ++h) sc[h][tid] = s * (dot[h] - z * qsum[h]);
        }
        __syncthreads();
        // ---- 2. running maximum and weights
        if (warp < REP) {
            float mx = -INFINITY;
            for (int t = lane; t < n; t += 32) mx = fmaxf(mx, sc[warp][t]);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
            const float m_new = fmaxf(m_run[warp], mx);
            float sum = 0.f;
            for (int t = lane; t < n; t += 32) {
                const float p = expf(sc[warp][t] - m_new);
                sc[warp][t] = p;
                sum += p;
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
            if (lane == 0) {
                const float r = expf(m_run[warp] - m_new);   // 0 on the first chunk (m_run = -inf)
                rescale[warp] = r;
                l_run[warp] = l_run[warp] * r + sum;
                m_run[warp] = m_new;
            }
        }
        __syncthreads();
        // ---- 3. weighted values
#pragma unroll
        for (int h = 0; h < REP; ++h) acc[h] *= rescale[h];
        const uint8_t* vr = c.v + ((size_t)hk * c.S_cap + c0) * kD + d;
        for (int t = half; t < n; t += 2) {
            const float val = e4m3_to_f32(__ldg(vr + (size_t)t * kD));
#pragma unroll
            for (int h = 0; h < REP; ++h) acc[h] = fmaf(sc[h][t], val, acc[h]);
        }
        __syncthreads();   // sc and rescale are rewritten by the next chunk
    }

    // ---- this CTA's part: {m, l, acc[128]} per query head (the two halves of the threads summed)
    if (half == 1)
#pragma unroll
        for (int h = 0; h < REP; ++h) acc_half[h][d] = acc[h];
    __syncthreads();
    constexpr int kPart = kD + 2;
    float* mine = partials + ((size_t)(hk * n_splits + split) * REP) * kPart;
    if (half == 0)
#pragma unroll
        for (int h = 0; h < REP; ++h) __stcg(mine + h * kPart + 2 + d, acc[h] + acc_half[h][d]);
    if (tid < REP) {
        __stcg(mine + tid * kPart, m_run[tid]);
        __stcg(mine + tid * kPart + 1, l_run[tid]);
    }
    __threadfence();
    __syncthreads();
    if (tid == 0) last_flag = atomicAdd(counters + hk, 1u) == (unsigned int)n_splits - 1u;
    __syncthreads();
    if (!last_flag) return;
    // ---- the last CTA of the kv head merges the parts, in the order of the splits (the same sum
    // whoever comes last), and clears the counter for the next call
    __threadfence();
    if (tid == 0) counters[hk] = 0u;
    const float* parts = partials + ((size_t)hk * n_splits * REP) * kPart;
    for (int o = tid; o < REP * kD; o += kThreads) {
        const int h = o / kD, dd = o - h * kD;
        float m = -INFINITY;
        for (int s = 0; s < n_splits; ++s) m = fmaxf(m, __ldcg(parts + ((size_t)s * REP + h) * kPart));
        float l = 0.f, a = 0.f;
        for (int s = 0; s < n_splits; ++s) {
            const float* ps = parts + ((size_t)s * REP + h) * kPart;
            const float ms = __ldcg(ps);
            const float w = ms == -INFINITY ? 0.f : expf(ms - m);   // a split without tokens carries nothing
            l = fmaf(__ldcg(ps + 1), w, l);
            a = fmaf(__ldcg(ps + 2 + dd), w, a);
        }
        const float r = a / l;
        const size_t idx = (size_t)(hk * REP + h) * kD + dd;
        if (out_dtype == MNNLLM_F32) reinterpret_cast<float*>(out)[idx] = r;
        else reinterpret_cast<__half*>(out)[idx] = __float2half_rn(r);
    }
    (void)status;
}

}  // namespace

int attn_splits(int Hk, int S) {
    // enough CTAs for every SM twice over, each with at least one chunk of tokens
    const int n_sm = device_sm_count() > 0 ? device_sm_count() : 148;
    int want = (2 * n_sm + Hk - 1) / Hk;
    const int chunks = (S + kAttnChunk - 1) / kAttnChunk;
    if (want > chunks) want = chunks;
    return want < 1 ? 1 : want;
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
    const int rep = H / c.Hk, splits = attn_splits(c.Hk, S);
    // whole chunks per split, so that only the last split of the sequence is ragged
    const int chunks = (S + kAttnChunk - 1) / kAttnChunk;
    const int per_split = ((chunks + splits - 1) / splits) * kAttnChunk;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)splits, (unsigned)c.Hk);
    cfg.blockDim = dim3(kThreads);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const __half* qh = (const __half*)q;
#define MNN_CASE(R) \
    case R: return cudaLaunchKernelEx(&cfg, attn_decode_kernel<R>, c, qh, out, out_dtype, S, per_split, partials, counters, status);
    switch (rep) {
        MNN_CASE(1) MNN_CASE(2) MNN_CASE(3) MNN_CASE(4) MNN_CASE(5) MNN_CASE(6) MNN_CASE(7) MNN_CASE(8)
    }
#undef MNN_CASE
    return cudaErrorInvalidValue;
}

}  // namespace mnnllm
