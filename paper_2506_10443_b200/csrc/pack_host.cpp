// Host-side weight packer: Eq. 1 quantisation (Section 4.2) and the reorder of codes and
// (scale, zero) pairs into the bulk-copy friendly layout of layout.h.  Runs once at model load
// (packing happens once, at model load, Section 5.1); no GPU involved.
//
// Built with floating-point contraction off: each fp32 operation below rounds once, as written.
#include <cmath>
#include <cstring>
#include <vector>

#include "../../include/mnnllm.h"
#include "layout.h"

namespace {

using namespace mnnllm;

// fp32 -> fp16 bits, round to nearest even, by integer manipulation of the fp32 encoding.
inline uint16_t half_bits_rn(float f) {
    uint32_t u;
    std::memcpy(&u, &f, 4);
    const uint32_t sign = (u >> 16) & 0x8000u;
    u &= 0x7FFFFFFFu;
    if (u >= 0x7F800000u) return (uint16_t)(sign | (u > 0x7F800000u ? 0x7E00u : 0x7C00u));
    if (u >= 0x477FF000u) return (uint16_t)(sign | 0x7C00u);  // >= 65520 rounds to infinity
    if (u < 0x38800000u) {                                    // below 2^-14: subnormal half
        if (u < 0x33000000u) return (uint16_t)sign;           // below 2^-25: zero
        const int e = (int)(u >> 23);                         // biased fp32 exponent, 102..112
        const uint32_t man = (u & 0x7FFFFFu) | 0x800000u;     // 24-bit significand
        const int shift = 126 - e;                            // result = man >> shift, 14..24
        uint32_t r = man >> shift;
        const uint32_t rem = man & ((1u << shift) - 1u);
        const uint32_t half = 1u << (shift - 1);
        if (rem > half || (rem == half && (r & 1u))) ++r;
        return (uint16_t)(sign | r);
    }
    uint32_t r = (u - 0x38000000u) >> 13;  // rebias exponent, drop 13 fraction bits
    const uint32_t rem = u & 0x1FFFu;
    if (rem > 0x1000u || (rem == 0x1000u && (r & 1u))) ++r;  // a carry moves into the exponent
    return (uint16_t)(sign | r);
}

inline float half_bits_to_float(uint16_t h) {
    const uint32_t sign = (uint32_t)(h & 0x8000u) << 16;
    uint32_t e = (h >> 10) & 0x1Fu, f = h & 0x3FFu, u;
    if (e == 0) {
        if (f == 0) {
            u = sign;
        } else {  // normalise the subnormal
            int sh = 0;
            while (!(f & 0x400u)) { f <<= 1; ++sh; }
            u = sign | ((uint32_t)(113 - sh) << 23) | ((f & 0x3FFu) << 13);
        }
    } else if (e == 31) {
        u = sign | 0x7F800000u | (f << 13);
    } else {
        u = sign | ((e + 112u) << 23) | (f << 13);
    }
    float out;
    std::memcpy(&out, &u, 4);
    return out;
}

inline uint16_t half_bits_sat(float f) {
    uint16_t h = half_bits_rn(f);
    if ((h & 0x7FFFu) == 0x7C00u) h = (uint16_t)((h & 0x8000u) | 0x7BFFu);
    return h;
}

// Eq. 1 for one group; codes written to q[0..len).
inline void quantize_group(const float* w, int len, int clip_max, uint8_t* q, uint16_t* s_bits,
                           uint16_t* z_bits) {
    float mn = w[0], mx = w[0];
    for (int k = 1; k < len; ++k) {
        mn = w[k] < mn ? w[k] : mn;
        mx = w[k] > mx ? w[k] : mx;
    }
    const float s32 = (mx - mn) / (float)clip_max;
    uint16_t sb = half_bits_sat(s32);
    float s = half_bits_to_float(sb);
    if (!(s > 0.0f)) {
        sb = 0x3C00u;
        s = 1.0f;
        for (int k = 0; k < len; ++k) q[k] = 0;
    } else {
        for (int k = 0; k < len; ++k) {
            int c = (int)std::rintf((w[k] - mn) / s);
            c = c < 0 ? 0 : (c > clip_max ? clip_max : c);
            q[k] = (uint8_t)c;
        }
    }
    *s_bits = sb;
    *z_bits = half_bits_sat(-mn / s);
}

constexpr int kNibbleK[8] = {0, 4, 1, 5, 2, 6, 3, 7};  // k offset stored in nibble i of a word

bool header_ok(const PackedHeader& h, uint32_t bits) {
    return h.magic == kMagic && h.version == kVersion && h.bits == bits && h.N > 0 && h.K > 0;
}

}  // namespace

extern "C" {

size_t mnnllm_packed_size_w4(int N, int K, int group) {
    if (N < 1 || K < 1 || (group != 64 && group != 128) || K % group != 0) return 0;
    return w4_geometry(N, K, group).total_bytes;
}

int mnnllm_pack_w4(const float* W, int N, int K, int group, void* packed_out) {
    if (!W || !packed_out || N < 1 || K < 1) return MNNLLM_ERR_INVALID_ARG;
    if ((group != 64 && group != 128) || K % group != 0) return MNNLLM_ERR_UNSUPPORTED;
    const W4Geometry geo = w4_geometry(N, K, group);
    uint8_t* out = (uint8_t*)packed_out;

    PackedHeader h;
    std::memset(&h, 0, sizeof(h));
    h.magic = kMagic; h.version = kVersion; h.bits = 4;
    h.N = N; h.K = K; h.group = group;
    h.n_row_blocks = geo.n_row_blocks; h.n_chunks = geo.n_chunks;
    h.row_block_bytes = geo.row_block_bytes; h.chunk_bytes = geo.chunk_bytes;
    h.body_bytes = geo.total_bytes - kHeaderBytes;
    std::memcpy(out, &h, sizeof(h));
    // padding between the last row block and the trailer, and the trailer's head
    std::memset(out + kHeaderBytes + (size_t)geo.n_row_blocks * geo.row_block_bytes, 0,
                geo.total_bytes - (kHeaderBytes + (size_t)geo.n_row_blocks * geo.row_block_bytes));
    W4RowInfo* info = (W4RowInfo*)(out + geo.trailer_offset + kTrailerHeadBytes);
    int limb_ok = 1;

#pragma omp parallel reduction(&& : limb_ok)
    {
        std::vector<uint8_t> q((size_t)16 * K);        // codes of the 16 rows of this block
        std::vector<uint16_t> sb((size_t)16 * geo.G), zb((size_t)16 * geo.G);
#pragma omp for schedule(dynamic, 4)
        for (int rb = 0; rb < geo.n_row_blocks; ++rb) {
            for (int r = 0; r < 16; ++r) {
                const int n = rb * 16 + r;
                if (n < N) {
                    for (int g = 0; g < geo.G; ++g)
                        quantize_group(W + (size_t)n * K + (size_t)g * group, group, 15,
                                       &q[(size_t)r * K + (size_t)g * group], &sb[(size_t)r * geo.G + g],
                                       &zb[(size_t)r * geo.G + g]);
                } else {  // padding rows decode to exactly zero
                    std::memset(&q[(size_t)r * K], 0, K);
                    for (int g = 0; g < geo.G; ++g) sb[(size_t)r * geo.G + g] = zb[(size_t)r * geo.G + g] = 0;
                }
            }
            // trailer: the row's scales as integers S * 2^row_exp, and sum_k q * S (integer-limb GEMM)
            for (int r = 0; r < 16; ++r) {
                int emin = 1 << 20;
                for (int g = 0; g < geo.G; ++g) {
                    int M, x;
                    w4_scale_parts(sb[(size_t)r * geo.G + g], M, x);
                    if (M && x < emin) emin = x;
                }
                if (emin == (1 << 20)) emin = 0;   // a row of zero scales (padding)
                long long sums[3] = {0, 0, 0};
                for (int g = 0; g < geo.G; ++g) {
                    int M, x;
                    w4_scale_parts(sb[(size_t)r * geo.G + g], M, x);
                    const int sh = x - emin;
                    if (M && sh > kLimbMaxShift) { limb_ok = 0; continue; }
                    const long long S = M ? ((long long)M << sh) : 0;
                    for (int k = 0; k < group; ++k) {
                        const long long qq = q[(size_t)r * K + (size_t)g * group + k];
                        const long long lo = qq * (S & 4095);
                        sums[0] += lo & 255;
                        sums[1] += lo >> 8;
                        sums[2] += qq * (S >> 12);
                    }
                }
                for (int i = 0; i < 3; ++i) info[rb * 16 + r].limb_sum[i] = (int32_t)sums[i];   // < 255 K
                info[rb * 16 + r].row_exp = emin;
            }
            for (int j = 0; j < geo.n_chunks; ++j) {
                uint8_t* chunk = out + w4_chunk_offset(geo, rb, j);
                const int ns = w4_chunk_slabs(geo, j), ng = w4_chunk_groups(geo, j);
                for (int sl = 0; sl < ns; ++sl) {
                    const int k0 = (j * 8 + sl) * kSlabK4;
                    uint32_t* slab = (uint32_t*)(chunk + (size_t)sl * kSlabBytes);
                    for (int lane = 0; lane < 32; ++lane) {
                        const int r = lane >> 2, c = lane & 3;
                        for (int wd = 0; wd < 4; ++wd) {
                            const int row = r + (wd >> 1) * 8;
                            const uint8_t* src = &q[(size_t)row * K + k0 + 16 * c + (wd & 1) * 8];
                            uint32_t v = 0;
                            for (int i = 0; i < 8; ++i) v |= (uint32_t)src[kNibbleK[i]] << (4 * i);
                            slab[lane * 4 + wd] = v;
                        }
                    }
                }
                uint16_t* tab = (uint16_t*)(chunk + (size_t)ns * kSlabBytes);
                const int g0 = j * geo.groups_per_chunk;
                for (int r = 0; r < 16; ++r)
                    for (int g = 0; g < ng; ++g) {
                        tab[(r * ng + g) * 2 + 0] = sb[(size_t)r * geo.G + g0 + g];
                        tab[(r * ng + g) * 2 + 1] = zb[(size_t)r * geo.G + g0 + g];
                    }
            }
        }
    }
    *(uint32_t*)(out + geo.trailer_offset) = (uint32_t)limb_ok;
    return MNNLLM_OK;
}

int mnnllm_packed_info(const void* packed, int* N, int* K, int* group, int* bits) {
    if (!packed) return MNNLLM_ERR_INVALID_ARG;
    PackedHeader h;
    std::memcpy(&h, packed, sizeof(h));
    if (h.magic != kMagic || h.version != kVersion) return MNNLLM_ERR_INVALID_ARG;
    if (N) *N = h.N;
    if (K) *K = h.K;
    if (group) *group = h.group;
    if (bits) *bits = (int)h.bits;
    return MNNLLM_OK;
}

int mnnllm_unpack_w4(const void* packed, uint8_t* q, uint16_t* scale_bits, uint16_t* zero_bits) {
    if (!packed || !q || !scale_bits || !zero_bits) return MNNLLM_ERR_INVALID_ARG;
    PackedHeader h;
    std::memcpy(&h, packed, sizeof(h));
    if (!header_ok(h, 4)) return MNNLLM_ERR_INVALID_ARG;
    if ((h.group != 64 && h.group != 128) || h.K % h.group != 0) return MNNLLM_ERR_UNSUPPORTED;
    const W4Geometry geo = w4_geometry(h.N, h.K, h.group);
    const uint8_t* in = (const uint8_t*)packed;
    const int N = h.N, K = h.K;
    for (int rb = 0; rb < geo.n_row_blocks; ++rb)
        for (int j = 0; j < geo.n_chunks; ++j) {
            const uint8_t* chunk = in + w4_chunk_offset(geo, rb, j);
            const int ns = w4_chunk_slabs(geo, j), ng = w4_chunk_groups(geo, j);
            for (int sl = 0; sl < ns; ++sl) {
                const int k0 = (j * 8 + sl) * kSlabK4;
                const uint32_t* slab = (const uint32_t*)(chunk + (size_t)sl * kSlabBytes);
                for (int lane = 0; lane < 32; ++lane)
                    for (int wd = 0; wd < 4; ++wd) {
                        const int n = rb * 16 + (lane >> 2) + (wd >> 1) * 8;
                        if (n >= N) continue;
                        const uint32_t v = slab[lane * 4 + wd];
                        uint8_t* dst = q + (size_t)n * K + k0 + 16 * (lane & 3) + (wd & 1) * 8;
                        for (int i = 0; i < 8; ++i) dst[kNibbleK[i]] = (uint8_t)((v >> (4 * i)) & 0xFu);
                    }
            }
            const uint16_t* tab = (const uint16_t*)(chunk + (size_t)ns * kSlabBytes);
            const int g0 = j * geo.groups_per_chunk;
            for (int r = 0; r < 16; ++r) {
                const int n = rb * 16 + r;
                if (n >= N) continue;
                for (int g = 0; g < ng; ++g) {
                    scale_bits[(size_t)n * geo.G + g0 + g] = tab[(r * ng + g) * 2 + 0];
                    zero_bits[(size_t)n * geo.G + g0 + g] = tab[(r * ng + g) * 2 + 1];
                }
            }
        }
    return MNNLLM_OK;
}

size_t mnnllm_packed_size_w8(int N, int K) {
    if (N < 1 || K < 1 || K % kSlabK8 != 0) return 0;
    return w8_geometry(N, K).total_bytes;
}

int mnnllm_pack_w8(const float* W, int N, int K, void* packed_out) {
    if (!W || !packed_out || N < 1 || K < 1) return MNNLLM_ERR_INVALID_ARG;
    if (K % kSlabK8 != 0) return MNNLLM_ERR_UNSUPPORTED;
    const W8Geometry geo = w8_geometry(N, K);
    uint8_t* out = (uint8_t*)packed_out;
    PackedHeader h;
    std::memset(&h, 0, sizeof(h));
    h.magic = kMagic; h.version = kVersion; h.bits = 8;
    h.N = N; h.K = K; h.group = K;
    h.n_row_blocks = geo.n_row_blocks; h.n_chunks = geo.n_chunks;
    h.row_block_bytes = geo.row_block_bytes; h.chunk_bytes = geo.chunk_bytes;
    h.body_bytes = geo.total_bytes - kHeaderBytes;
    h.table_offset = geo.table_offset;
    std::memcpy(out, &h, sizeof(h));
    uint16_t* table = (uint16_t*)(out + geo.table_offset);

#pragma omp parallel
    {
        std::vector<uint8_t> q((size_t)16 * K);
#pragma omp for schedule(dynamic, 4)
        for (int rb = 0; rb < geo.n_row_blocks; ++rb) {
            for (int r = 0; r < 16; ++r) {
                const int n = rb * 16 + r;
                uint16_t sb = 0, zb = 0;
                if (n < N) quantize_group(W + (size_t)n * K, K, 255, &q[(size_t)r * K], &sb, &zb);
                else std::memset(&q[(size_t)r * K], 0, K);
                table[(size_t)(rb * 16 + r) * 2 + 0] = sb;
                table[(size_t)(rb * 16 + r) * 2 + 1] = zb;
            }
            uint8_t* block = out + kHeaderBytes + (size_t)rb * geo.row_block_bytes;
            for (int sl = 0; sl < geo.n_slabs; ++sl)
                for (int lane = 0; lane < 32; ++lane)
                    for (int half = 0; half < 2; ++half) {
                        const int row = (lane >> 2) + half * 8;
                        std::memcpy(block + (size_t)sl * kSlabBytes + lane * 16 + half * 8,
                                    &q[(size_t)row * K + sl * kSlabK8 + 8 * (lane & 3)], 8);
                    }
        }
    }
    return MNNLLM_OK;
}

int mnnllm_unpack_w8(const void* packed, uint8_t* q, uint16_t* scale_bits, uint16_t* zero_bits) {
    if (!packed || !q || !scale_bits || !zero_bits) return MNNLLM_ERR_INVALID_ARG;
    PackedHeader h;
    std::memcpy(&h, packed, sizeof(h));
    if (!header_ok(h, 8) || h.K % kSlabK8 != 0) return MNNLLM_ERR_INVALID_ARG;
    const W8Geometry geo = w8_geometry(h.N, h.K);
    const uint8_t* in = (const uint8_t*)packed;
    const uint16_t* table = (const uint16_t*)(in + geo.table_offset);
    for (int n = 0; n < h.N; ++n) {
        scale_bits[n] = table[(size_t)n * 2];
        zero_bits[n] = table[(size_t)n * 2 + 1];
        const uint8_t* block = in + kHeaderBytes + (size_t)(n / 16) * geo.row_block_bytes;
        const int r = n % 16;
        for (int sl = 0; sl < geo.n_slabs; ++sl)
            for (int c = 0; c < 4; ++c)
                std::memcpy(q + (size_t)n * h.K + sl * kSlabK8 + 8 * c,
                            block + (size_t)sl * kSlabBytes + ((r & 7) * 4 + c) * 16 + (r >> 3) * 8, 8);
    }
    return MNNLLM_OK;
}

const char* mnnllm_status_string(int status) {
    switch (status) {
        case MNNLLM_OK: return "ok";
        case MNNLLM_ERR_INVALID_ARG: return "invalid argument";
        case MNNLLM_ERR_UNSUPPORTED: return "unsupported configuration or device";
        case MNNLLM_ERR_ALIGNMENT: return "misaligned pointer";
        case MNNLLM_ERR_CUDA: return "CUDA runtime error";
        case MNNLLM_ERR_TIMEOUT: return "a bounded device-side wait gave up";
        case MNNLLM_ERR_WORKSPACE: return "workspace missing or too small";
        default: return "unknown status";
    }
}

}  // extern "C"
