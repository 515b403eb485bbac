// Packed weight layout shared by the host packer and the kernels (product code only).
//
// W4 (bits = 4), group in {64, 128}:
//   header (128 B) | row block 0 | row block 1 | ...            row block = 16 consecutive rows n
//   row block      = chunk 0 | chunk 1 | ...                     chunk = 512 consecutive k (8 slabs);
//                                                                 the last chunk may hold fewer slabs
//   chunk          = slab 0 .. slab ns-1 | scale/zero table
//   slab           = 16 rows x 64 k = 512 B = 32 lanes x 16 B.  Lane L = 4r + c (r = 0..7, c = 0..3)
//                    holds words w0 w1 (row r, k = 16c .. 16c+15 of the slab) and w2 w3 (row r + 8).
//                    Nibble i (bits 4i..4i+3) of w0 holds k offset kNibbleK[i] = {0,4,1,5,2,6,3,7};
//                    w1 the same + 8.  Hence (w & 0x0F0F0F0F) is k 0..3 as bytes and
//                    ((w >> 4) & 0x0F0F0F0F) is k 4..7: the int8 expansion needs no shuffle, and
//                    (w & 0x000F000F), (w & 0x00F000F0) are (k0,k2), (k4,k6) as fp16 mantissa bits.
//   scale/zero     = [row 0..15][group 0..ng-1] pairs of fp16 (scale, zero), 4 B each.
//   trailer        (after the last row block, 128-byte aligned) = 16 bytes {uint32 limb_ok, reserved} followed by
//                    one {int32 limb_sum[3], int32 row_exp} per padded row.  It serves the integer-limb form of
//                    the prefill GEMM: every scale of row n is S[n,g] * 2^row_exp[n] with an integer S; the product
//                    q * S = b0 + 256 b1 + 4096 c0 with the byte limbs b0 = (q (S & 4095)) & 255,
//                    b1 = (q (S & 4095)) >> 8, c0 = q (S >> 12); limb_sum[i] = sum_k limb_i[n,k];
//                    limb_ok = 1 when S < 2^16 for every group of every row (a row's scales span at most five
//                    binades beyond the 11 bits of their significands).
//
// W8 (bits = 8), per channel: same blocking with slabs of 16 rows x 32 k (lane L = 4r + c holds
//   bytes k = 8c .. 8c+7 of row r in w0 w1 and of row r + 8 in w2 w3, natural byte order), 16 slabs
//   per 512-k chunk, no per-chunk table; one [N_padded] table of (scale, zero) pairs follows the
//   last row block.
#pragma once
#include <stddef.h>
#include <stdint.h>

#if defined(__CUDACC__)
#define MNN_HD __host__ __device__ __forceinline__
#else
#define MNN_HD inline
#endif

namespace mnnllm {

constexpr uint32_t kMagic = 0x34574E4Du;  // "MNW4" little endian
constexpr uint32_t kVersion = 1;
constexpr int kHeaderBytes = 128;
constexpr int kRowsPerBlock = 16;
constexpr int kChunkK = 512;
constexpr int kSlabBytes = 512;
constexpr int kSlabK4 = 64;  // k per slab, 4-bit codes
constexpr int kSlabK8 = 32;  // k per slab, 8-bit codes

struct PackedHeader {
    uint32_t magic, version, bits;
    int32_t N, K, group;
    int32_t n_row_blocks, n_chunks;
    uint64_t row_block_bytes;  // distance between consecutive row blocks
    uint64_t chunk_bytes;      // size of a full 512-k chunk (codes + table)
    uint64_t body_bytes;       // everything after the header
    uint64_t table_offset;     // W8: offset of the per-row (scale, zero) table from the buffer start
    uint8_t reserved[128 - 64];
};
static_assert(sizeof(PackedHeader) == kHeaderBytes, "header is 128 bytes");

struct W4Geometry {
    int N, K, group;
    int n_row_blocks;  // ceil(N / 16)
    int n_slabs;       // K / 64
    int n_chunks;      // ceil(n_slabs / 8)
    int groups_per_chunk;  // 512 / group
    int G;                 // K / group
    size_t chunk_bytes;      // full chunk: 8 slabs + 16 * groups_per_chunk * 4
    size_t row_block_bytes;  // n_slabs * 512 + 16 * G * 4
    size_t trailer_offset;   // header + n_row_blocks * row_block_bytes, rounded up to 128
    size_t total_bytes;
};
constexpr int kTrailerHeadBytes = 16;
struct W4RowInfo { int32_t limb_sum[3]; int32_t row_exp; };
constexpr int kLimbMaxShift = 5;   // S = M << shift with M < 2048: S < 2^16

// A scale's fp16 bit pattern as integer significand M and exponent x: value = M * 2^x (M = 0 for zero).
MNN_HD void w4_scale_parts(uint32_t bits, int& M, int& x) {
    const int e = (int)((bits >> 10) & 31u), m = (int)(bits & 1023u);
    M = e ? 1024 + m : m;
    x = e ? e - 25 : -24;
}

MNN_HD W4Geometry w4_geometry(int N, int K, int group) {
    W4Geometry g;
    g.N = N; g.K = K; g.group = group;
    g.n_row_blocks = (N + kRowsPerBlock - 1) / kRowsPerBlock;
    g.n_slabs = K / kSlabK4;
    g.n_chunks = (g.n_slabs + 7) / 8;
    g.groups_per_chunk = kChunkK / group;
    g.G = K / group;
    g.chunk_bytes = (size_t)8 * kSlabBytes + (size_t)16 * g.groups_per_chunk * 4;
    g.row_block_bytes = (size_t)g.n_slabs * kSlabBytes + (size_t)16 * g.G * 4;
    g.trailer_offset = (kHeaderBytes + (size_t)g.n_row_blocks * g.row_block_bytes + 127) & ~(size_t)127;
    g.total_bytes = g.trailer_offset +
                    (((size_t)kTrailerHeadBytes + (size_t)g.n_row_blocks * kRowsPerBlock * sizeof(W4RowInfo) + 127) & ~(size_t)127);
    return g;
}

// slabs / groups held by chunk j
MNN_HD int w4_chunk_slabs(const W4Geometry& g, int j) {
    int left = g.n_slabs - 8 * j;
    return left < 8 ? left : 8;
}
MNN_HD int w4_chunk_groups(const W4Geometry& g, int j) { return w4_chunk_slabs(g, j) * kSlabK4 / g.group; }
MNN_HD size_t w4_chunk_size(const W4Geometry& g, int j) {
    return (size_t)w4_chunk_slabs(g, j) * kSlabBytes + (size_t)16 * w4_chunk_groups(g, j) * 4;
}
MNN_HD size_t w4_chunk_offset(const W4Geometry& g, int row_block, int j) {
    return kHeaderBytes + (size_t)row_block * g.row_block_bytes + (size_t)j * g.chunk_bytes;
}

struct W8Geometry {
    int N, K;
    int n_row_blocks;
    int n_slabs;   // ceil(K / 32)  (K is padded with code 0 up to a multiple of 32)
    int n_chunks;  // ceil(n_slabs / 16)
    size_t chunk_bytes;      // 16 slabs
    size_t row_block_bytes;  // n_slabs * 512
    size_t table_offset;     // header + n_row_blocks * row_block_bytes
    size_t total_bytes;      // + n_row_blocks * 16 * 4
};

MNN_HD W8Geometry w8_geometry(int N, int K) {
    W8Geometry g;
    g.N = N; g.K = K;
    g.n_row_blocks = (N + kRowsPerBlock - 1) / kRowsPerBlock;
    g.n_slabs = (K + kSlabK8 - 1) / kSlabK8;
    g.n_chunks = (g.n_slabs + 15) / 16;
    g.chunk_bytes = (size_t)16 * kSlabBytes;
    g.row_block_bytes = (size_t)g.n_slabs * kSlabBytes;
    g.table_offset = kHeaderBytes + (size_t)g.n_row_blocks * g.row_block_bytes;
    g.total_bytes = g.table_offset + (size_t)g.n_row_blocks * kRowsPerBlock * 4;
    return g;
}

}  // namespace mnnllm
