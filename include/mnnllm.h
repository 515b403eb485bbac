/*
 * mnnllm.h - C ABI of the B200 (sm_100a) weight-quantised linear layer.
 *
 * The operation is the Linear operator of Section 5.1: activations x [M, K] ("[e, l]") times
 * weights W [N, K] ("[h, l]") give y [M, N] ("[e, h]"), with W stored as asymmetric int4 (or int8)
 * codes produced by Eq. 1 of Section 4.2 and dequantised inside the kernel.  On a GPU the
 * activations stay floating point (W4A16 / W8A16); the W4A8 path first quantises them to int8 per
 * token so that integer matrix instructions can be used (Section 4.2).
 *
 * Conventions shared by every entry point
 *   - Pointers marked "host" are ordinary CPU memory, pointers marked "device" are CUDA global
 *     memory of the current device.  The caller owns every buffer; the library never allocates or
 *     frees device memory and keeps no reference after a call returns.
 *   - Matrices are dense row-major.  W is [N, K]; groups are `group` consecutive k of one row,
 *     G = K / group groups per row.
 *   - GPU entry points only enqueue work on `stream` (a cudaStream_t passed as void*) and return at
 *     once; errors reported are argument and launch errors.  Results are ready when the stream
 *     reaches that point.
 *   - Device pointers must be 16-byte aligned; the packed weight buffer must be 128-byte aligned.
 *   - There is no CPU fallback: on a device that is not compute capability 10.x the GPU entry
 *     points return MNNLLM_ERR_UNSUPPORTED.
 *   - Every function returns MNNLLM_OK (0) on success; nothing is written on an argument error.
 */
#ifndef MNNLLM_H_
#define MNNLLM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    MNNLLM_OK = 0,
    MNNLLM_ERR_INVALID_ARG = 1, /* null pointer, non-positive size, bad header */
    MNNLLM_ERR_UNSUPPORTED = 2, /* group size, dtype, shape or device not supported */
    MNNLLM_ERR_ALIGNMENT = 3,   /* a pointer breaks the alignment rules above */
    MNNLLM_ERR_CUDA = 4,        /* a CUDA runtime call failed (launch, attribute, ...) */
    MNNLLM_ERR_TIMEOUT = 5,     /* a bounded device-side wait gave up (see mnnllm_read_status) */
    MNNLLM_ERR_WORKSPACE = 6    /* workspace pointer null or too small */
} mnnllm_status;

typedef enum { MNNLLM_F16 = 0, MNNLLM_BF16 = 1, MNNLLM_F32 = 2 } mnnllm_dtype;

const char* mnnllm_status_string(int status);

/* ------------------------------------------------------------------------------------------------
 * Weight packing (host only, done once when the model is loaded).
 *
 * Eq. 1 (Section 4.2) with clip_min = 0 and clip_max = 15, applied to every group of one row:
 *     scale = fp16((w_max - w_min) / 15),   q = clamp(round((w - w_min) / scale), 0, 15),
 *     zero  = fp16(-w_min / scale),         so that  w ~ scale * (q - zero).
 * round() is fp32 round-half-to-even and the division uses the fp16-rounded scale.  A group whose
 * range is zero (or rounds to a zero scale) gets scale = 1, q = 0, zero = fp16(-w_min); scale and
 * zero saturate at +-65504.
 *
 * The packed buffer is position independent (it may be copied anywhere, to the device as is).
 * Layout: a 128-byte header (magic, version, bits, N, K, group, counts, strides), then one record
 * per block of 16 rows, each record a run of chunks of 512 k (the last chunk of a row may be
 * shorter).  A chunk holds its codes as 512-byte slabs of 16 rows x 64 k - 16 bytes for each of the
 * 32 threads of a warp: thread 4r+c owns k = 16c..16c+15 of rows r and r+8, nibbles interleaved so
 * that `word & 0x0F0F0F0F` and `(word >> 4) & 0x0F0F0F0F` are four consecutive k each - followed by
 * the chunk's (scale, zero) fp16 pairs ordered [row][group].  Every chunk is a contiguous,
 * 16-byte-aligned run, i.e. one bulk copy.  Rows beyond N in the last block are stored as q = 0,
 * scale = 0, zero = 0.
 * ---------------------------------------------------------------------------------------------- */

/* Bytes needed for the packed form of an [N, K] matrix; 0 if the arguments are not supported
 * (N, K >= 1, group in {64, 128}, K a multiple of group). */
size_t mnnllm_packed_size_w4(int N, int K, int group);

/* W: host, fp32 [N, K].  packed_out: host, mnnllm_packed_size_w4(N, K, group) bytes, written in full. */
int mnnllm_pack_w4(const float* W, int N, int K, int group, void* packed_out);

/* Inverse of the reorder, for parity checks: reads a packed buffer (host) and writes the codes
 * q [N, K] (one per byte, 0..15) and the fp16 bit patterns of scale and zero, each [N, G].
 * N, K and group are taken from the header. */
int mnnllm_unpack_w4(const void* packed, uint8_t* q, uint16_t* scale_bits, uint16_t* zero_bits);

/* Reads N, K and group of a packed buffer (host); any output pointer may be null.  (A helper of this
 * library's buffer format; the paper has no counterpart.) */
int mnnllm_packed_info(const void* packed, int* N, int* K, int* group, int* bits);

/* int8 per-channel variant (Section 4.2: the LM head is kept in int8): Eq. 1 with clip_max = 255,
 * one group per row (group = K), codes stored as unsigned bytes, scale and zero fp16 per row. */
size_t mnnllm_packed_size_w8(int N, int K);
int mnnllm_pack_w8(const float* W, int N, int K, void* packed_out);
int mnnllm_unpack_w8(const void* packed, uint8_t* q, uint16_t* scale_bits, uint16_t* zero_bits);

/* ------------------------------------------------------------------------------------------------
 * W4A16: y[m, n] = sum_g scale[n, g] * sum_{k in g} (q[n, k] - zero[n, g]) * x[m, k]
 * (Section 4.2: the weight-only floating-point pairing that the paper assigns to GPUs; Section 5.1 for
 * the operand shapes).  Accumulation is fp32.
 *
 *   x       device, fp16 [M, K]
 *   packed  device, a buffer written by mnnllm_pack_w4 for the same N, K, group
 *   y       device, fp16 [M, N] (or the dtype given to the _ex form), overwritten
 *   M >= 1  any M is accepted; the kernel is built for decode (M <= 8 per pass over the weights)
 *
 * The header of `packed` lives in device memory and is not read by the host: N, K and group are
 * the caller's statement of what was packed.
 * ---------------------------------------------------------------------------------------------- */
int mnnllm_linear_w4a16(const void* x, const void* packed, void* y, int M, int N, int K, int group,
                        void* stream);

/* Same with explicit dtypes (Section 4.2: floating-point activations on GPUs): x_dtype MNNLLM_F16 or
 * MNNLLM_BF16; y_dtype MNNLLM_F16, MNNLLM_BF16 or MNNLLM_F32 (fp32 logits for the LM head).  bf16
 * activations are converted to fp16 as the kernel loads them, which is exact for magnitudes in
 * [2^-17, 65504]; larger values saturate at +-65504, smaller ones lose low bits. */
int mnnllm_linear_w4a16_ex(const void* x, const void* packed, void* y, int M, int N, int K, int group,
                           int x_dtype, int y_dtype, void* stream);

/* Several independent W4A16 problems that share M (for example q, k, v of one layer, or gate and
 * up) in ONE launch: each computes exactly what mnnllm_linear_w4a16_ex computes (Section 4.2, W4A16);
 * putting them in one launch is this library's, as the paper's GPU path adjusts its parallelism to
 * the problem's dimensions (Section 5.1).  `problems` is a host array of `count` (1..MNNLLM_MAX_BATCH) descriptors; it
 * is copied into the launch and may be reused when the call returns. */
#define MNNLLM_MAX_BATCH 8
typedef struct {
    const void* x;      /* device fp16 [M, K] */
    const void* packed; /* device */
    void* y;            /* device [M, N] of y_dtype */
    int N, K, group;
    int y_dtype;
} mnnllm_w4a16_problem;
int mnnllm_linear_w4a16_batch(const mnnllm_w4a16_problem* problems, int count, int M, void* stream);

/* W4A16 linear with a LoRA bypass (Section 5.5, Table 3):
 *   y[m, n] = (W4A16 linear of x)[m, n] + sum_j lora_A[n, j] * t[m, j],   t[m, j] = sum_k lora_B[j, k] * x[m, k]
 * i.e. A' = W A + LoRA_A (LoRA_B A) in the order the paper chooses: the rank-r product first, so that
 * the bypass costs 2 r (N + K) operations and r (N + K) fp16 values per token instead of an N x K
 * matrix.  lora_A device fp16 [N, rank] (row n contiguous), lora_B device fp16 [rank, K] (16-byte
 * aligned), 1 <= rank <= MNNLLM_LORA_MAX_RANK; the other arguments as for mnnllm_linear_w4a16_ex.
 * workspace: device, 16-byte aligned, at least mnnllm_workspace_size_lora(M, rank) bytes (0 for
 * invalid arguments), owned by the caller and cleared ONCE with mnnllm_lora_workspace_init before
 * its first use; calls on one stream may share it (it is free for reuse when the stream has passed
 * the call), calls that can overlap on the GPU may not.  It holds an epoch, a counter and the entries
 * of t as {fp32 value, epoch tag} words.  ONE launch on `stream`: the GEMV's own CTAs compute the
 * entries of t between them once the activations are complete (while their weights are already
 * streaming in) and publish each as one tagged word; every CTA waits (bounded) for the words of this
 * launch before it stores its first outputs, to which it adds the second product; y is written
 * once, both products accumulate in fp32.  A
 * separate launch for t would put another dependent stage in front of every linear, which costs
 * more than the whole bypass.
 * Errors: as mnnllm_linear_w4a16_ex, plus INVALID_ARG (null LoRA pointer, rank out of range),
 * WORKSPACE (null or too small); a wait that ran out shows as MNNLLM_ERR_TIMEOUT (detail 0x700 |
 * problem) in mnnllm_read_status. */
#define MNNLLM_LORA_MAX_RANK 64
size_t mnnllm_workspace_size_lora(int M, int rank);
int mnnllm_lora_workspace_init(void* workspace, size_t workspace_bytes, void* stream);
int mnnllm_linear_w4a16_lora(const void* x, const void* packed, const void* lora_A, const void* lora_B, void* y,
                             int M, int N, int K, int group, int rank, int x_dtype, int y_dtype, void* workspace,
                             size_t workspace_bytes, void* stream);

/* ------------------------------------------------------------------------------------------------
 * A whole decoder stack of W4A16 linears in ONE launch (decode, M <= 8 tokens).
 *
 * Decode time is the time to read the weights (Section 2; Section 4.2: decode is memory-bound), but
 * one linear of a small model is well under a microsecond of memory time and each depends on its
 * predecessor, so a launch per linear spends most of its time at launch boundaries.  This entry
 * point runs a list of up to MNNLLM_STACK_MAX_PROBLEMS linears (each computing exactly what
 * mnnllm_linear_w4a16_ex computes) as one persistent grid that keeps streaming weights while a
 * dependent problem waits for its input.  (The operation is the paper's; the single launch, the
 * plan and the dependency list are this library's.)
 *
 *   problems   host array.  Problem p reads x only after the problems listed in deps[0..n_deps-1]
 *              (indices < p) have stored all their outputs; a problem without deps may start at once.
 *              Problems run in index order on every SM, so list them in execution order.
 *   plan       built once on the host by mnnllm_stack_plan_w4a16 (mnnllm_stack_plan_size bytes),
 *              then copied by the caller to device memory (16-byte aligned), like packed weights.
 *              n_sms = 0 takes the SM count of the current device (needs a GPU); a positive value
 *              plans for that many SMs without touching a device.  The plan holds the device
 *              pointers of the problems: rebuild it when a buffer moves.
 *   workspace  device, 256-byte aligned, mnnllm_stack_workspace_size(plan) bytes, ALL ZERO before
 *              its first use (mnnllm_stack_workspace_init enqueues that memset).  The launch keeps
 *              its completion counters there; it never needs clearing again, but after a launch that
 *              reported MNNLLM_ERR_TIMEOUT it must be zeroed before it is reused.  Two launches
 *              that may overlap on the GPU need separate workspaces.
 *   The launch is cooperative (every CTA resident at once): it fails with MNNLLM_ERR_CUDA if the GPU
 *   cannot hold the grid, e.g. under a partitioning that hides SMs.  x is fp16; accumulation fp32.
 * ---------------------------------------------------------------------------------------------- */
#define MNNLLM_STACK_MAX_PROBLEMS 256
#define MNNLLM_STACK_MAX_DEPS 4
typedef struct {
    const void* x;      /* device fp16 [M, K] */
    const void* packed; /* device, from mnnllm_pack_w4 for [N, K] and the plan's group */
    void* y;            /* device [M, N] of y_dtype, overwritten */
    int N, K;
    int y_dtype;
    int n_deps;
    int deps[MNNLLM_STACK_MAX_DEPS];
} mnnllm_stack_problem;
size_t mnnllm_stack_plan_size(int count);
int mnnllm_stack_plan_w4a16(const mnnllm_stack_problem* problems, int count, int M, int group, int n_sms,
                            void* plan_out);
size_t mnnllm_stack_workspace_size(const void* plan_host);
int mnnllm_stack_workspace_init(void* workspace, size_t workspace_bytes, void* stream);
/* plan_host: the plan in host memory (only its header is read); plan_dev: the same bytes on the device. */
int mnnllm_linear_w4a16_stack(const void* plan_host, const void* plan_dev, void* workspace, size_t workspace_bytes,
                              void* stream);

/* W8A16 with per-channel int8 weights packed by mnnllm_pack_w8. */
int mnnllm_linear_w8a16(const void* x, const void* packed, void* y, int M, int N, int K, int y_dtype,
                        void* stream);

/* ------------------------------------------------------------------------------------------------
 * W4A8 (Section 4.2: per-token int8 activation quantisation in front of integer matrix instructions):
 *   per token m:   amax = max_k |x[m, k]|,  a_scale[m] = amax / 127,
 *                  a_q[m, k] = clamp(round(x[m, k] * (127 / amax)), -127, 127)   (0 if amax == 0)
 *   per group g:   P[m, n, g] = sum_{k in g} a_q[m, k] * q[n, k]      (int32, exact)
 *                  A[m, g]    = sum_{k in g} a_q[m, k]
 *   y[m, n] = a_scale[m] * sum_g scale[n, g] * (P[m, n, g] - zero[n, g] * A[m, g])    (fp32)
 *
 *   x          device [M, K] of x_dtype (MNNLLM_F16 or MNNLLM_BF16)
 *   y          device [M, N] of y_dtype, overwritten
 *   M          prompts of up to 32 tokens are memory-bound (Section 2) and run on a GEMV-shaped kernel
 *              (warp-level u8 x s8 MMAs on the streamed weights), longer ones on the tensor-memory GEMM
 *   weights    the zero-point term sum_g scale*zero*A is evaluated on the tensor cores from a two-term
 *              fp16 split of scale*zero (about the group's |w_min|): every group needs |w_min| < 256,
 *              and the term is carried to 2^-33 absolute, i.e. without loss for weights whose typical
 *              magnitude is above ~1e-5 (the W4A16 path has neither limit)
 *   workspace  device scratch, 256-byte aligned; holds a_q, a_scale, A between the two kernels.
 *              mnnllm_workspace_size_w4a8(M, N, K, group) is the size to allocate.  It includes
 *              about 20 MB in which a problem with fewer 128 x 128 output tiles than the GPU has
 *              SMs is split along K (the parts of a tile are summed there in fp32, in a fixed
 *              order: results do not depend on timing).  A workspace of at least
 *              mnnllm_workspace_min_w4a8(M, N, K, group) bytes is accepted too: such problems
 *              then keep some SMs idle; the results are the same up to the fp32 summation order.
 *              Smaller: MNNLLM_ERR_WORKSPACE.  Contents are undefined afterwards; two calls that
 *              may overlap on the GPU need separate workspaces.  Both sizes are 0 for arguments
 *              the call would reject.
 * ---------------------------------------------------------------------------------------------- */
size_t mnnllm_workspace_size_w4a8(int M, int N, int K, int group);
/* Smallest workspace mnnllm_linear_w4a8 accepts (no room for splitting tiles along K); a sizing
 * helper of this library, the paper has no counterpart. */
size_t mnnllm_workspace_min_w4a8(int M, int N, int K, int group);
int mnnllm_linear_w4a8(const void* x, const void* packed, void* y, int M, int N, int K, int group,
                       int x_dtype, int y_dtype, void* workspace, size_t workspace_bytes, void* stream);

/* Several weight matrices that multiply the SAME activations (q, k, v of a layer; gate and up) in
 * one call: the activations are quantised once and one GEMM launch covers all the matrices
 * (Section 4.2; the fusion itself is this library's).  All problems share M, K, group and x; the
 * workspace is that of a single problem (the workspace sizes do not depend on N). */
#define MNNLLM_MAX_BATCH_W4A8 4
typedef struct {
    const void* packed; /* device, from mnnllm_pack_w4 for [N, K], the call's group */
    void* y;            /* device [M, N] of y_dtype, overwritten */
    int N;
    int y_dtype;
} mnnllm_w4a8_problem;
int mnnllm_linear_w4a8_batch(const mnnllm_w4a8_problem* problems, int count, const void* x, int M, int K, int group,
                             int x_dtype, void* workspace, size_t workspace_bytes, void* stream);

/* Same computation as mnnllm_linear_w4a8 for callers that cannot allocate device memory.  (The paper
 * has no counterpart; this is a convenience of this library.)  Some users of this code run where
 * cudaMalloc is off limits: inside a plugin whose host application owns every allocation, in a
 * latency-critical serving loop that forbids allocator calls after start-up, or in a process whose
 * memory pool was sized and handed out before the library was loaded.  Such callers have nowhere
 * to get the workspace from, so this entry point brings its own: a fixed array of
 * MNNLLM_STATIC_SCRATCH_BYTES that is part of the library's device image.  Every GPU on which the
 * library is loaded holds that array until the process exits.
 *
 *   - x, packed, y and the other arguments are exactly those of mnnllm_linear_w4a8; the caller
 *     still owns inputs and outputs.  The call itself allocates and frees nothing.
 *   - Limit: the activations' int8 copy (M*K bytes), their scales (4*M) and the fp16 group sums
 *     (8 * M * ceil(K/group/4)*4), each rounded up to 256 bytes, must fit the array; a larger
 *     problem returns MNNLLM_ERR_WORKSPACE and nothing is launched.  8 MiB covers, for example,
 *     M = 1024 tokens at K = 3584 or M = 512 at K = 8960.  The array has no room for the scratch
 *     in which mnnllm_linear_w4a8 splits small problems along K: this entry point never does.
 *   - The first call on each device looks up the array's device address (one runtime query, the
 *     device must be current); make that first call before starting any stream capture.
 *   - All calls on a device share the one array and it keeps whatever the last call left there.
 *     Nothing in it has to start at zero (each call rewrites all it reads), but two calls that can
 *     overlap on the GPU - different streams without an ordering between them - race on it and
 *     corrupt each other's results.  Calls on one stream are safe. */
#define MNNLLM_STATIC_SCRATCH_BYTES (8u << 20)
int mnnllm_linear_w4a8_static(const void* x, const void* packed, void* y, int M, int N, int K, int group,
                              int x_dtype, int y_dtype, void* stream);

/* ------------------------------------------------------------------------------------------------
 * W8A8 (Section 4.2 names W4A8 and W8A8 as the integer paths): per-channel int8 weights packed by
 * mnnllm_pack_w8 (one fp16 scale s[n] and zero point z[n] per weight row, codes 0..255) and the
 * per-token int8 activations defined above:
 *   y[m, n] = a_scale[m] * s[n] * ( sum_k a_q[m, k] q[n, k]  -  z[n] * sum_k a_q[m, k] )
 * The integer sum runs over all of K in one int32 tensor-memory accumulator (|sum| <= 127 * 255 * K:
 * K <= 66048) and is rescaled once, in fp32.  x device [M, K] fp16/bf16 (16-byte aligned), packed
 * device (128-byte aligned), y device [M, N] fp16/bf16/fp32, K a multiple of 32.  workspace: device,
 * 256-byte aligned, at least mnnllm_workspace_size_w8a8(M, K) bytes (0 for invalid arguments), owned
 * by the caller, free for reuse when the stream has passed the call; it holds a_q, a_scale and the
 * row sums of a_q.  Two launches (quantiser, GEMM) on `stream`; nothing is allocated or synchronised.
 * Built for prompts (hundreds of tokens); any M >= 1 is computed correctly.
 * Errors: INVALID_ARG (null pointer, size < 1), UNSUPPORTED (dtype, K % 32 != 0, device),
 * ALIGNMENT, WORKSPACE (null or too small), CUDA (launch failure; the sticky error is cleared). */
size_t mnnllm_workspace_size_w8a8(int M, int K);
int mnnllm_linear_w8a8(const void* x, const void* packed, void* y, int M, int N, int K, int x_dtype, int y_dtype,
                       void* workspace, size_t workspace_bytes, void* stream);

/* ------------------------------------------------------------------------------------------------
 * Attention of one decoded token over a quantised KV cache (Section 4.2: keys are quantised to int8
 * along head_dim when they are stored, one Eq. 1 scale and zero point per key vector; values are
 * stored as fp8, entry by entry, so that nothing already in the cache changes when a token is added;
 * Section 5.4: softmax in full precision, the query divided by sqrt(head_dim) before the product):
 *   k_hat[t, :] = s[t] * (codes[t, :] - z[t]);  score[h, t] = (q[h, :] / sqrt(D)) . k_hat[t, :]
 *   out[h, :] = sum_t softmax_t(score[h, .])[t] * v[t, :]         query head h reads kv head h / (H / Hk)
 * Cache of one layer, device memory owned by the caller, head_dim = 128 only:
 *   k_codes  uint8 [Hk, S_cap, 128]  (16-byte aligned)     k_meta  uint32 [Hk, S_cap]: fp16 scale | fp16 zero << 16
 *   v        E4M3  [Hk, S_cap, 128]  (1 sign, 4 exponent bits with bias 7, 3 fraction bits, no infinities, max 448)
 * mnnllm_kv_append quantises one new key and value per kv head (k_new, v_new: device fp16 [Hk, 128];
 * round to nearest even; E4M3 saturates at +-448) and stores them at position pos < S_cap.
 * mnnllm_attention_decode: q device fp16 [H, 128], out device fp16 or fp32 [H, 128], positions [0, S),
 * 1 <= S <= S_cap, H a multiple of Hk with H / Hk <= 8, Hk <= 64.  workspace: device, 16-byte aligned,
 * at least mnnllm_attention_workspace_size(H, Hk, S) bytes (0 for invalid arguments), cleared ONCE
 * with mnnllm_attention_workspace_init before its first use (every call leaves it cleared); calls on
 * one stream may share it.  One launch each; nothing is allocated or synchronised.  The sequence is
 * split over the SMs; the last CTA of a kv head merges the parts in the order of the splits.
 * Errors: INVALID_ARG (null pointer, size < 1, pos or S outside the cache), UNSUPPORTED (head_dim,
 * head counts, dtype, device), ALIGNMENT, WORKSPACE, CUDA. */
int mnnllm_kv_append(void* k_codes, void* k_meta, void* v, int Hk, int S_cap, int head_dim, int pos,
                     const void* k_new, const void* v_new, void* stream);
size_t mnnllm_attention_workspace_size(int H, int Hk, int S);
int mnnllm_attention_workspace_init(void* workspace, size_t workspace_bytes, void* stream);
int mnnllm_attention_decode(const void* q, const void* k_codes, const void* k_meta, const void* v, void* out,
                            int H, int Hk, int head_dim, int S, int S_cap, int out_dtype, void* workspace,
                            size_t workspace_bytes, void* stream);

/* The activation quantiser alone (first kernel of the W4A8 path), writing caller-owned outputs:
 * a_q int8 [M, K], a_scale fp32 [M], A int32 [M, G]. */
int mnnllm_quantize_activations(const void* x, int x_dtype, int M, int K, int group, int8_t* a_q,
                                float* a_scale, int32_t* A, void* stream);

/* Parity/debug form of the W4A8 path: runs the same tensor-core main loop and stores every int32
 * group partial, P device int32 [M, N, G], together with a_q, a_scale and A as above. */
int mnnllm_debug_w4a8_partials(const void* x, int x_dtype, const void* packed, int32_t* P, int8_t* a_q,
                               float* a_scale, int32_t* A, int M, int N, int K, int group, void* stream);

/* Device-side waits in the kernels are bounded; one that gives up records a code in a status word
 * instead of spinning.  This call synchronises `stream`, reads the word, clears it and returns
 * MNNLLM_OK or MNNLLM_ERR_TIMEOUT (detail, if not null, receives the raw word). */
int mnnllm_read_status(void* stream, uint32_t* detail);

/* mnnllm_linear_w4a8 has two kernels: prompts of up to 32 tokens go to a GEMV-shaped kernel that
 * streams the weights once (such prompts are bound by memory, Section 2), longer ones to the
 * tensor-memory GEMM.  This call moves the boundary for the whole process (0..64 tokens; anything
 * else restores the default) and returns the value in force before: a tuning and test knob.  Both
 * kernels compute the same int32 group partials; their fp32 sums differ in order only. */
int mnnllm_debug_set_w4a8_small_max(int max_tokens);

/* Long prompts have a second tensor-core kernel, off by default.  It folds every group scale into
 * the integer weight operand (three byte "limbs" of code x integer scale, one int32 accumulator each
 * over all of K: no per-group rescale; Section 4.2's W4A8 evaluated exactly in integers) and needs
 * every row's scales within five binades of each other, which the packer records; where that does
 * not hold the kernel that rescales every group's partial does the work.  Its unpack
 * costs what the rescale saved, and it measured slower than the default kernel (250 against 390
 * TOP/s on a Qwen2-1.5B layer at 1024 tokens); it is kept as a checked alternative.  This
 * call switches it off (0), on for launches with at least 0.6 tiles per SM (1) or on whatever the
 * number of tiles (2); anything else restores the default (off, or on with MNNLLM_W4A8_LIMB=1 in the
 * environment); returns 1 if it was on before, else 0: a tuning and test knob. */
int mnnllm_debug_set_w4a8_limb(int enabled);

/* Exercises the time-out path without any of the library's kernels having to fail: enqueues a
 * one-warp kernel that waits, with the kernels' own bounded wait, on a barrier nobody arrives at
 * (max_polls tries of at most 20 microseconds each, 1..1000), records MNNLLM_DEBUG_TIMEOUT_DETAIL in
 * the status word and ends normally.  mnnllm_read_status then reports MNNLLM_ERR_TIMEOUT once.
 * (Failure reporting is this library's; the paper has no counterpart.) */
#define MNNLLM_DEBUG_TIMEOUT_DETAIL 0x2000u
int mnnllm_debug_wait_timeout(int max_polls, void* stream);

/* Measurement aid for the prefill roofline (Section 4.2 puts W4A8 on integer matrix instructions;
 * the measurement itself is this library's): one CTA per SM issues mmas_per_sm (rounded down to a
 * multiple of 4) back-to-back 128 x 128 x 32 tcgen05.mma kind::i8 on operand tiles resident in
 * shared memory, nothing else.  Integer operations performed = SMs * mmas * 2 * 128 * 128 * 32; time
 * it with events on `stream`.  cycles_out: device, one entry per SM (the issuing thread's elapsed SM
 * clock cycles), or null. */
int mnnllm_bench_mma_i8(unsigned long long mmas_per_sm, unsigned long long* cycles_out, void* stream);

/* 1 if the current CUDA device can run the kernels (compute capability 10.x), else 0. */
int mnnllm_device_supported(void);

#ifdef __cplusplus
}
#endif
#endif /* MNNLLM_H_ */
