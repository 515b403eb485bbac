// CPU oracle for the weight-quantised linear layer (int4/int8 asymmetric, group-quantised along K).
//
// THIS FILE IS TEST INFRASTRUCTURE.  It defines what the CUDA library must compute and is timed as
// the CPU baseline; the product never calls it.  It shares no code, header, table or helper with
// the CUDA path: every conversion (fp16 rounding included) is written out here a second time.
//
// Style: plain scalar loops in the order of the definitions, fp64 accumulation, no blocking, no
// fusion.  The only parallelism is an optional OpenMP "for" over independent output rows.
//
// Pins (tests that hold each function to something other than itself):
//   orc_quantize_w4 / w8   Eq. 1 end points and monotonicity, a hand-worked group, lossless
//                          round-trip of exactly representable weights.
//   orc_dequant            the same lossless round-trip (w_hat == w exactly).
//   orc_linear_wa16        long-double triple loop over dequantised weights; subset-sum and
//                          constant-q closed forms.
//   orc_act_quant          hand-worked rows; a_q exact for integer-valued rows with amax = 127.
//   orc_group_partials     Python-integer brute force.
//   orc_linear_w4a8        the per-group identity  sum_k a*s*(q-z) = s*(sum a*q - z*sum a)  in
//                          exact rational arithmetic; equality with orc_linear_wa16 when the
//                          activations are exactly representable in int8.
//   orc_linear_w8a8        Python-integer brute force of its one dot product per output; equality
//                          with orc_linear_wa16 on int8-exact activations; the closed form for
//                          constant codes (y = a_scale s (c - z) sum_k a_q).
//   orc_lora_bypass        equality with the other association (LoRA_A LoRA_B) x in exact rationals
//                          on small integers; rank-1 closed form; Table 3's operation and memory
//                          counts for both orders (tests/golden/table3_lora.txt).
//   orc_f32_to_e4m3 / back the 256 bit patterns written out from the format's definition in the test,
//                          round trip, ties to even, saturation at 448.
//   orc_attention_decode   equal keys -> mean of the values; one key far ahead -> its value; softmax
//                          shift invariance; Python brute force of a tiny case; group-query mapping.
//   fp16 conversions       exhaustive round trip over all 65536 bit patterns and comparison with
//                          numpy's float16 on random and boundary values.
//
// Readings of the paper taken here (the paper states Eq. 1 with symbols only):
//   * clip_min = 0, clip_max = 15 (int4) or 255 (int8); codes are unsigned.
//   * groups are `group` consecutive k of one weight row; per-channel means group == K.
//   * scale s = fp16((w_max - w_min) / (clip_max - clip_min)); the code q is computed against the
//     rounded s; the zero point is the real number z = fp16(-w_min / s), so w_hat = s * (q - z).
//   * round() is round-half-to-even in fp32.
//   * a group with w_max == w_min (or whose scale rounds to 0 in fp16) gets s = 1, q = 0,
//     z = fp16(-w_min).  A scale or zero that overflows fp16 saturates at +-65504.
//   * activations: per token, symmetric, a_q in [-127, 127], a_scale = amax / 127 in fp32.

#include <cmath>
#include <cstdint>
#include <cstring>
#ifdef _OPENMP
#include <omp.h>
#endif

extern "C" {

// ---------------------------------------------------------------------------------------------
// IEEE binary16 <-> binary32, written from the format definition (1 sign, 5 exponent, 10 fraction
// bits, bias 15, subnormals below 2^-14).  Round to nearest, ties to even.
// ---------------------------------------------------------------------------------------------
float orc_f16_to_f32(uint16_t h) {
    const int sign = (h >> 15) & 1;
    const int e = (h >> 10) & 0x1F;
    const int f = h & 0x3FF;
    double v;
    if (e == 0) {
        v = std::ldexp((double)f, -24);  // subnormal: f * 2^-10 * 2^-14
    } else if (e == 31) {
        v = f ? (double)NAN : (double)INFINITY;
    } else {
        v = std::ldexp(1.0 + (double)f / 1024.0, e - 15);
    }
    return (float)(sign ? -v : v);
}

uint16_t orc_f32_to_f16(float x) {
    uint32_t u;
    std::memcpy(&u, &x, 4);
    const uint16_t sign = (uint16_t)((u >> 16) & 0x8000u);
    if (std::isnan(x)) return (uint16_t)(sign | 0x7E00u);
    double a = std::fabs((double)x);
    if (std::isinf(x)) return (uint16_t)(sign | 0x7C00u);
    if (a == 0.0) return sign;
    int ex;  // a = m * 2^ex with m in [0.5, 1)
    (void)std::frexp(a, &ex);
    int e = ex - 1;          // floor(log2 a)
    if (e < -14) e = -14;    // subnormal range shares the exponent of the smallest normal
    // spacing of representable numbers in this binade is 2^(e-10); nearbyint is half-to-even
    double n = std::nearbyint(std::ldexp(a, 10 - e));
    if (n >= 2048.0) {  // rounded up into the next binade
        n = 1024.0;
        e += 1;
    }
    if (e > 15) return (uint16_t)(sign | 0x7C00u);  // overflow -> infinity
    if (n < 1024.0) return (uint16_t)(sign | (uint16_t)n);  // subnormal (e == -14) or zero
    return (uint16_t)(sign | ((uint16_t)(e + 15) << 10) | ((uint16_t)n - 1024u));
}

static inline uint16_t f16_saturating(float v) {
    uint16_t h = orc_f32_to_f16(v);
    if ((h & 0x7FFFu) == 0x7C00u) h = (uint16_t)((h & 0x8000u) | 0x7BFFu);  // +-65504
    return h;
}

// ---------------------------------------------------------------------------------------------
// Eq. 1 (asymmetric quantisation), applied per (row n, group g of `group` consecutive k).
// q: [N, K] codes in [0, clip_max]; scale_bits / zero_bits: [N, K/group] fp16 bit patterns.
// ---------------------------------------------------------------------------------------------
static void quantize_rows(const float* W, int N, int K, int group, int clip_max, uint8_t* q,
                          uint16_t* scale_bits, uint16_t* zero_bits) {
    const int G = K / group;
#pragma omp parallel for schedule(static)
    for (int n = 0; n < N; ++n) {
        for (int g = 0; g < G; ++g) {
            const float* w = W + (size_t)n * K + (size_t)g * group;
            float mn = w[0], mx = w[0];
            for (int k = 1; k < group; ++k) {
                if (w[k] < mn) mn = w[k];
                if (w[k] > mx) mx = w[k];
            }
            const float s32 = (mx - mn) / (float)clip_max;
            uint16_t sb = f16_saturating(s32);
            float s = orc_f16_to_f32(sb);
            uint8_t* qo = q + (size_t)n * K + (size_t)g * group;
            if (!(s > 0.0f)) {  // constant group, or a range too small for fp16
                sb = 0x3C00u;   // 1.0
                s = 1.0f;
                for (int k = 0; k < group; ++k) qo[k] = 0;
            } else {
                for (int k = 0; k < group; ++k) {
                    const float t = (w[k] - mn) / s;
                    int c = (int)std::rintf(t);
                    if (c < 0) c = 0;
                    if (c > clip_max) c = clip_max;
                    qo[k] = (uint8_t)c;
                }
            }
            scale_bits[(size_t)n * G + g] = sb;
            zero_bits[(size_t)n * G + g] = f16_saturating(-mn / s);
        }
    }
}

void orc_quantize_w4(const float* W, int N, int K, int group, uint8_t* q, uint16_t* scale_bits,
                     uint16_t* zero_bits) {
    quantize_rows(W, N, K, group, 15, q, scale_bits, zero_bits);
}

// int8 per-channel variant (the LM head): one group per row, codes in [0, 255].
void orc_quantize_w8(const float* W, int N, int K, uint8_t* q, uint16_t* scale_bits,
                     uint16_t* zero_bits) {
    quantize_rows(W, N, K, K, 255, q, scale_bits, zero_bits);
}

// w_hat[n, k] = s[n, g] * (q[n, k] - z[n, g]) in fp64.
void orc_dequant(const uint8_t* q, const uint16_t* scale_bits, const uint16_t* zero_bits, int N,
                 int K, int group, double* w_hat) {
    const int G = K / group;
#pragma omp parallel for schedule(static)
    for (int n = 0; n < N; ++n)
        for (int k = 0; k < K; ++k) {
            const double s = (double)orc_f16_to_f32(scale_bits[(size_t)n * G + k / group]);
            const double z = (double)orc_f16_to_f32(zero_bits[(size_t)n * G + k / group]);
            w_hat[(size_t)n * K + k] = s * ((double)q[(size_t)n * K + k] - z);
        }
}

// Weight-only path (W4A16 / W8A16): y[m, n] = sum_k x[m, k] * w_hat[n, k], fp64, natural k order.
// x holds the activation values already widened (exactly) to fp32.
void orc_linear_wa16(const float* x, const uint8_t* q, const uint16_t* scale_bits,
                     const uint16_t* zero_bits, int M, int N, int K, int group, double* y) {
    const int G = K / group;
#pragma omp parallel for schedule(static)
    for (int n = 0; n < N; ++n) {
        for (int m = 0; m < M; ++m) {
            double acc = 0.0;
            for (int k = 0; k < K; ++k) {
                const double s = (double)orc_f16_to_f32(scale_bits[(size_t)n * G + k / group]);
                const double z = (double)orc_f16_to_f32(zero_bits[(size_t)n * G + k / group]);
                const double w_hat = s * ((double)q[(size_t)n * K + k] - z);
                acc += (double)x[(size_t)m * K + k] * w_hat;
            }
            y[(size_t)m * N + n] = acc;
        }
    }
}

// Dynamic per-token symmetric int8 activation quantisation.
//   amax = max_k |x[m, k]|;  a_q = clamp(rint(x * (127 / amax)), -127, 127);  a_scale = amax / 127
//   A_g[m, g] = sum_{k in g} a_q[m, k]   (the factor of the zero-point correction)
void orc_act_quant(const float* x, int M, int K, int group, int8_t* a_q, float* a_scale,
                   int32_t* A_g) {
    const int G = K / group;
#pragma omp parallel for schedule(static)
    for (int m = 0; m < M; ++m) {
        const float* xr = x + (size_t)m * K;
        float amax = 0.0f;
        for (int k = 0; k < K; ++k) {
            const float a = std::fabs(xr[k]);
            if (a > amax) amax = a;
        }
        if (amax == 0.0f) {
            for (int k = 0; k < K; ++k) a_q[(size_t)m * K + k] = 0;
            for (int g = 0; g < G; ++g) A_g[(size_t)m * G + g] = 0;
            a_scale[m] = 0.0f;
            continue;
        }
        const float inv = 127.0f / amax;
        for (int k = 0; k < K; ++k) {
            int c = (int)std::rintf(xr[k] * inv);
            if (c < -127) c = -127;
            if (c > 127) c = 127;
            a_q[(size_t)m * K + k] = (int8_t)c;
        }
        for (int g = 0; g < G; ++g) {
            int32_t s = 0;
            for (int k = 0; k < group; ++k) s += a_q[(size_t)m * K + (size_t)g * group + k];
            A_g[(size_t)m * G + g] = s;
        }
        a_scale[m] = amax / 127.0f;
    }
}

// Integer group partials: P[m, n, g] = sum_{k in g} a_q[m, k] * q[n, k]   (exact, int32).
void orc_group_partials(const int8_t* a_q, const uint8_t* q, int M, int N, int K, int group,
                        int32_t* P) {
    const int G = K / group;
#pragma omp parallel for schedule(static)
    for (int n = 0; n < N; ++n)
        for (int m = 0; m < M; ++m)
            for (int g = 0; g < G; ++g) {
                int32_t acc = 0;
                for (int k = g * group; k < (g + 1) * group; ++k)
                    acc += (int32_t)a_q[(size_t)m * K + k] * (int32_t)q[(size_t)n * K + k];
                P[((size_t)m * N + n) * G + g] = acc;
            }
}

// W4A8: y[m, n] = a_scale[m] * sum_g s[n, g] * (P[m, n, g] - z[n, g] * A_g[m, g]), fp64.
void orc_linear_w4a8(const float* x, const uint8_t* q, const uint16_t* scale_bits,
                     const uint16_t* zero_bits, int M, int N, int K, int group, double* y) {
    const int G = K / group;
    int8_t* a_q = new int8_t[(size_t)M * K];
    float* a_scale = new float[M];
    int32_t* A_g = new int32_t[(size_t)M * G];
    orc_act_quant(x, M, K, group, a_q, a_scale, A_g);
#pragma omp parallel for schedule(static)
    for (int n = 0; n < N; ++n)
        for (int m = 0; m < M; ++m) {
            double acc = 0.0;
            for (int g = 0; g < G; ++g) {
                int32_t P = 0;
                for (int k = g * group; k < (g + 1) * group; ++k)
                    P += (int32_t)a_q[(size_t)m * K + k] * (int32_t)q[(size_t)n * K + k];
                const double s = (double)orc_f16_to_f32(scale_bits[(size_t)n * G + g]);
                const double z = (double)orc_f16_to_f32(zero_bits[(size_t)n * G + g]);
                acc += s * ((double)P - z * (double)A_g[(size_t)m * G + g]);
            }
            y[(size_t)m * N + n] = (double)a_scale[m] * acc;
        }
    delete[] a_q;
    delete[] a_scale;
    delete[] A_g;
}

// W8A8 (Section 4.2), per-channel int8 weights (one scale and zero point per weight row, codes
// 0..255) and per-token int8 activations:
//   y[m, n] = a_scale[m] * s[n] * (sum_k a_q[m, k] q[n, k]  -  z[n] * sum_k a_q[m, k]), fp64.
void orc_linear_w8a8(const float* x, const uint8_t* q, const uint16_t* scale_bits,
                     const uint16_t* zero_bits, int M, int N, int K, double* y) {
    int8_t* a_q = new int8_t[(size_t)M * K];
    float* a_scale = new float[M];
    int32_t* A = new int32_t[M];
    orc_act_quant(x, M, K, K, a_q, a_scale, A);   // one group = the whole row: A[m] = sum_k a_q[m, k]
#pragma omp parallel for schedule(static)
    for (int n = 0; n < N; ++n) {
        const double s = (double)orc_f16_to_f32(scale_bits[n]);
        const double z = (double)orc_f16_to_f32(zero_bits[n]);
        for (int m = 0; m < M; ++m) {
            int64_t P = 0;
            for (int k = 0; k < K; ++k)
                P += (int64_t)a_q[(size_t)m * K + k] * (int64_t)q[(size_t)n * K + k];
            y[(size_t)m * N + n] = (double)a_scale[m] * (s * ((double)P - z * (double)A[m]));
        }
    }
    delete[] a_q;
    delete[] a_scale;
    delete[] A;
}

// LoRA bypass (Section 5.5, Table 3): y[m, n] += sum_j A[n, j] * t[m, j],  t[m, j] = sum_k B[j, k] x[m, k],
// i.e. LoRA_A (LoRA_B x) in the order the paper chooses (the small product first).  A is [N, r],
// B is [r, K], both given as the fp32 values of their fp16 entries; everything in fp64.
void orc_lora_bypass(const float* x, const float* A, const float* B, int M, int N, int K, int r,
                     double* y) {
    double* t = new double[(size_t)M * r];
    for (int m = 0; m < M; ++m)
        for (int j = 0; j < r; ++j) {
            double acc = 0.0;
            for (int k = 0; k < K; ++k) acc += (double)B[(size_t)j * K + k] * (double)x[(size_t)m * K + k];
            t[(size_t)m * r + j] = acc;
        }
#pragma omp parallel for schedule(static)
    for (int n = 0; n < N; ++n)
        for (int m = 0; m < M; ++m) {
            double acc = 0.0;
            for (int j = 0; j < r; ++j) acc += (double)A[(size_t)n * r + j] * t[(size_t)m * r + j];
            y[(size_t)m * N + n] += acc;
        }
    delete[] t;
}

// ---- fp8 E4M3 (1 sign, 4 exponent bits with bias 7, 3 fraction bits; no infinities, S.1111.111 is
// NaN, largest finite value 448; subnormals 2^-9 .. 7 * 2^-9) -------------------------------------
float orc_e4m3_to_f32(uint8_t b) {
    const int sign = b >> 7, e = (b >> 3) & 15, f = b & 7;
    double v;
    if (e == 15 && f == 7) return std::nanf("");
    if (e == 0) v = std::ldexp((double)f, -9);
    else v = std::ldexp(1.0 + (double)f / 8.0, e - 7);
    return (float)(sign ? -v : v);
}

// Round to nearest, ties to the even code; magnitudes above 448 (and infinities) saturate at 448.
uint8_t orc_f32_to_e4m3(float x) {
    if (std::isnan(x)) return 0x7F;
    const uint8_t sign = std::signbit(x) ? 0x80 : 0;
    const double a = std::fabs((double)x);
    if (a >= 448.0) return sign | 0x7E;
    // the codes 0 .. 0x7E are increasing in value: find the two neighbours and take the nearer one
    int lo = 0;
    for (int c = 0; c <= 0x7E; ++c)
        if ((double)orc_e4m3_to_f32((uint8_t)c) <= a) lo = c;
    if (lo == 0x7E) return sign | 0x7E;
    const double vlo = (double)orc_e4m3_to_f32((uint8_t)lo), vhi = (double)orc_e4m3_to_f32((uint8_t)(lo + 1));
    int pick;
    if (a - vlo < vhi - a) pick = lo;
    else if (a - vlo > vhi - a) pick = lo + 1;
    else pick = (lo & 1) ? lo + 1 : lo;   // tie: the code with an even fraction
    return sign | (uint8_t)pick;
}

// Values to E4M3, entry by entry (nothing in the cache depends on any other entry).
void orc_quantize_values(const float* v, long long n, uint8_t* out) {
#pragma omp parallel for schedule(static)
    for (long long i = 0; i < n; ++i) out[i] = orc_f32_to_e4m3(v[i]);
}

// Attention for one decoded token over a quantised KV cache (Section 4.2: keys int8, quantised per
// key vector along head_dim with Eq. 1; values fp8; Section 5.4: softmax in full precision, the
// query divided by sqrt(head_dim) before the product with the keys).
//   q        [H, D]       query values (fp16 widened to fp32)
//   k_codes  [Hk, S, D]   uint8 codes, k_scale / k_zero [Hk, S] fp16 bits: k_hat = s * (c - z)
//   v        [Hk, S, D]   E4M3 bytes
//   out      [H, D]       fp64;   query head h reads kv head h / (H / Hk)
//   score[h, t] = sum_d (q[h, d] / sqrt(D)) * k_hat[t, d];  p = softmax_t(score);  out[h, :] = sum_t p[t] * v[t, :]
void orc_attention_decode(const float* q, const uint8_t* k_codes, const uint16_t* k_scale,
                          const uint16_t* k_zero, const uint8_t* v, int H, int Hk, int S, int D,
                          double* out) {
    const int rep = H / Hk;
    const double inv = 1.0 / std::sqrt((double)D);
#pragma omp parallel for schedule(static)
    for (int h = 0; h < H; ++h) {
        const int hk = h / rep;
        double* score = new double[S];
        double mx = -INFINITY;
        for (int t = 0; t < S; ++t) {
            const size_t row = (size_t)hk * S + t;
            const double s = (double)orc_f16_to_f32(k_scale[row]), z = (double)orc_f16_to_f32(k_zero[row]);
            double acc = 0.0;
            for (int d = 0; d < D; ++d)
                acc += ((double)q[(size_t)h * D + d] * inv) * (s * ((double)k_codes[row * D + d] - z));
            score[t] = acc;
            if (acc > mx) mx = acc;
        }
        double denom = 0.0;
        for (int t = 0; t < S; ++t) {
            score[t] = std::exp(score[t] - mx);
            denom += score[t];
        }
        for (int d = 0; d < D; ++d) {
            double acc = 0.0;
            for (int t = 0; t < S; ++t)
                acc += (score[t] / denom) * (double)orc_e4m3_to_f32(v[((size_t)hk * S + t) * D + d]);
            out[(size_t)h * D + d] = acc;
        }
        delete[] score;
    }
}

int orc_num_threads(void) {
#ifdef _OPENMP
    int n = 1;
#pragma omp parallel
    {
#pragma omp single
        n = omp_get_num_threads();
    }
    return n;
#else
    return 1;
#endif
}

}  // extern "C"
