/*
 * CPU oracle for the W4A8-dINT quantized linear layer.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition that the
 * CUDA library is compared against.  It shares no code, header, table or
 * constant with the CUDA path, and nothing in the product may call it.
 *
 * What it defines (paper: "Enhancing Computation Efficiency in Large Language
 * Models through Weight and Activation Quantization", arXiv 2311.05161):
 *
 *   - the dINT number format: quantize (Eq. 5) and dequantize (Eq. 6), for any
 *     bit width b (p = 2^b - 3 uniform steps, Section 4.2);
 *   - output-channel-wise (or group-wise) Min-Max asymmetric weight
 *     quantization of W * diag(s) (Eq. 1, Appendix A.1 "Quantization
 *     Settings");
 *   - token-wise 8-bit activation quantization of diag(s)^-1 * X (Eq. 1,
 *     Appendix A.1) in the symmetric absmax variant;
 *   - the quantized matmul Q(W diag(s)) Q(diag(s)^-1 X) (Eq. 1) as an exact
 *     integer contraction followed by a floating-point rescale.
 *
 * Arithmetic: every rounding decision (a code, a zero-point, an INT8 value) is
 * taken in IEEE-754 binary32, one rounded operation per written operation,
 * round-to-nearest-even, no fused multiply-add unless fmaf() is written, no
 * flush-to-zero.  Build with -ffp-contract=off and without -ffast-math.  The
 * output rescale also exists in binary64 (oracle_linear_f64) as the tolerance
 * reference for the BF16 result.
 *
 * Readings of the paper where it is silent (each is a documented choice):
 *   - "n" in the conditions of Eq. 5 is the real value being quantized;
 *   - the inequalities of Eq. 5 are taken literally (x = s/4 is not special,
 *     x = 3s/4 is);
 *   - the rounding bracket of Eq. 5 is round-half-to-even;
 *   - the special codes are c1 = p + 1 (value +s/2) and c2 = p + 2 (-s/2);
 *   - the quantization range is [min(0, min w), max(0, max w)], optionally
 *     shrunk by a clip ratio, and z = clamp(rint(-lo / s), 0, p);
 *   - an all-zero row or group takes s = 1, z = 0.
 *
 * Parity pins: see tests/test_oracle_*.py.  The conventions listed above are
 * "parity unpinned" by the paper itself; everything Eq. 5 / Eq. 6 fix is
 * pinned by exhaustive and closed-form tests.
 */
#include <math.h>
#include <stdint.h>
#include <stddef.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* ------------------------------------------------------------------------- */
/* storage formats                                                           */
/* ------------------------------------------------------------------------- */

/* IEEE binary16 -> binary32, exact. */
static float half_bits_to_float(uint16_t h)
{
    uint32_t sign = (uint32_t)(h >> 15) & 1u;
    uint32_t expo = (uint32_t)(h >> 10) & 0x1Fu;
    uint32_t mant = (uint32_t)h & 0x3FFu;
    float v;
    if (expo == 0) {
        v = ldexpf((float)mant, -24);               /* zero and subnormals */
    } else if (expo == 31) {
        v = mant ? NAN : INFINITY;
    } else {
        v = ldexpf((float)(mant | 0x400u), (int)expo - 25);
    }
    return sign ? -v : v;
}

/* binary32 -> bfloat16 bits, round-to-nearest-even on the dropped 16 bits. */
static uint16_t float_to_bf16_bits(float f)
{
    uint32_t u;
    memcpy(&u, &f, 4);
    if ((u & 0x7F800000u) == 0x7F800000u && (u & 0x007FFFFFu)) {
        return (uint16_t)((u >> 16) | 0x0040u);     /* quiet NaN */
    }
    uint32_t keep = u >> 16;
    uint32_t drop = u & 0xFFFFu;
    if (drop > 0x8000u || (drop == 0x8000u && (keep & 1u))) keep += 1u;
    return (uint16_t)keep;
}

float oracle_half_to_float(uint16_t h) { return half_bits_to_float(h); }
uint16_t oracle_float_to_bf16(float f) { return float_to_bf16_bits(f); }

/* ------------------------------------------------------------------------- */
/* dINT format, Section 4.2                                                   */
/* ------------------------------------------------------------------------- */

/* Number of uniform steps p = 2^b - 3 (text below Eq. 6). */
int oracle_dint_p(int b) { return (1 << b) - 3; }

static int clampi(int v, int lo, int hi) { return v < lo ? lo : (v > hi ? hi : v); }

/* round-half-even of a float to an int; the float is first limited to a range
 * far outside any code so that the conversion itself is always defined. */
static int rint_to_int(float r)
{
    r = rintf(r);
    if (r > 1048576.0f) r = 1048576.0f;
    if (r < -1048576.0f) r = -1048576.0f;
    return (int)r;
}

/* Eq. 5: real value x -> b-bit dINT code, step size s, zero-point z.
 * Codes 0..p are the integer levels, p+1 is c1 (+s/2), p+2 is c2 (-s/2). */
int oracle_dint_quantize(float x, float s, int z, int b)
{
    const int p = oracle_dint_p(b);
    const float quarter = 0.25f * s;
    const float threeq = 0.75f * s;
    if (x > quarter && x <= threeq) return p + 1;
    if (x < -quarter && x >= -threeq) return p + 2;
    return clampi(rint_to_int(x / s) + z, 0, p);
}

/* Eq. 6: code -> real value. */
float oracle_dint_dequantize(int code, float s, int z, int b)
{
    const int p = oracle_dint_p(b);
    if (code == p + 1) return 0.5f * s;
    if (code == p + 2) return -0.5f * s;
    return (float)(code - z) * s;
}

/* Eq. 6 in units of s/2, so that every level is an integer:
 * t[code] = 2 (code - z) for the integer levels, +1 for c1, -1 for c2. */
void oracle_dint_table2(int z, int b, int8_t *t)
{
    const int p = oracle_dint_p(b);
    for (int c = 0; c <= p; ++c) t[c] = (int8_t)(2 * (c - z));
    t[p + 1] = 1;
    t[p + 2] = -1;
}

/* ------------------------------------------------------------------------- */
/* weight side of Eq. 1: Q(W diag(s)), b = 4                                 */
/* ------------------------------------------------------------------------- */

/* W      [N][K] binary16 bits, row-major (N output features, K input features)
 * s_in   [K] binary32 per-input-channel scale of Eq. 1, or NULL for all-ones
 * group  0: one (step, zero-point) per output row; else per `group` consecutive
 *        k of a row (K % group == 0)
 * clip   ratio applied to both range ends (1.0f = plain Min-Max)
 * codes  [N][K/2]: byte k/2 holds code[k] (low nibble) and code[k+1] (high)
 * scales [G][N] step sizes, zeros [G][N] zero-points, G = group ? K/group : 1 */
void oracle_pack_weights(const uint16_t *W, const float *s_in, int N, int K,
                         int group, float clip, uint8_t *codes, float *scales,
                         uint8_t *zeros)
{
    const int glen = group ? group : K;
    const int G = K / glen;
#pragma omp parallel for schedule(static)
    for (int n = 0; n < N; ++n) {
        for (int g = 0; g < G; ++g) {
            float lo = 0.0f, hi = 0.0f;
            for (int k = g * glen; k < (g + 1) * glen; ++k) {
                float w = half_bits_to_float(W[(size_t)n * K + k]);
                if (s_in) w = w * s_in[k];
                if (w < lo) lo = w;
                if (w > hi) hi = w;
            }
            lo = lo * clip;
            hi = hi * clip;
            float s = (hi - lo) / 13.0f;
            if (s == 0.0f) s = 1.0f;
            const int z = clampi(rint_to_int((-lo) / s), 0, 13);
            scales[(size_t)g * N + n] = s;
            zeros[(size_t)g * N + n] = (uint8_t)z;
            for (int k = g * glen; k < (g + 1) * glen; k += 2) {
                float w0 = half_bits_to_float(W[(size_t)n * K + k]);
                float w1 = half_bits_to_float(W[(size_t)n * K + k + 1]);
                if (s_in) { w0 = w0 * s_in[k]; w1 = w1 * s_in[k + 1]; }
                const int c0 = oracle_dint_quantize(w0, s, z, 4);
                const int c1 = oracle_dint_quantize(w1, s, z, 4);
                codes[(size_t)n * (K / 2) + k / 2] = (uint8_t)(c0 | (c1 << 4));
            }
        }
    }
}

/* ------------------------------------------------------------------------- */
/* activation side of Eq. 1: Q(diag(s)^-1 X), token-wise INT8                 */
/* ------------------------------------------------------------------------- */

/* X [M][K] binary16 bits (M tokens), inv_s_in [K] = 1/s or NULL,
 * Xq [M][K] INT8, tok_scale [M] step size of each token. */
void oracle_quantize_act(const uint16_t *X, const float *inv_s_in, int M, int K,
                         int8_t *Xq, float *tok_scale)
{
#pragma omp parallel for schedule(static)
    for (int m = 0; m < M; ++m) {
        float amax = 0.0f;
        for (int k = 0; k < K; ++k) {
            float x = half_bits_to_float(X[(size_t)m * K + k]);
            if (inv_s_in) x = x * inv_s_in[k];
            const float a = fabsf(x);
            if (a > amax) amax = a;
        }
        if (amax == 0.0f) {
            tok_scale[m] = 0.0f;
            for (int k = 0; k < K; ++k) Xq[(size_t)m * K + k] = 0;
            continue;
        }
        const float r = 127.0f / amax;
        tok_scale[m] = amax / 127.0f;
        for (int k = 0; k < K; ++k) {
            float x = half_bits_to_float(X[(size_t)m * K + k]);
            if (inv_s_in) x = x * inv_s_in[k];
            Xq[(size_t)m * K + k] = (int8_t)clampi(rint_to_int(x * r), -127, 127);
        }
    }
}

/* ------------------------------------------------------------------------- */
/* the contraction                                                           */
/* ------------------------------------------------------------------------- */

/* acc[g][m][n] = sum over k in group g of Xq[m][k] * t2_{z[g][n]}[code[n][k]],
 * in 64-bit so that a test can prove the 32-bit result cannot overflow. */
void oracle_linear_acc_i64(const int8_t *Xq, const uint8_t *codes,
                           const uint8_t *zeros, int M, int N, int K, int group,
                           int64_t *acc)
{
    const int glen = group ? group : K;
    const int G = K / glen;
#pragma omp parallel for schedule(static)
    for (int n = 0; n < N; ++n) {
        for (int g = 0; g < G; ++g) {
            int8_t t2[16];
            oracle_dint_table2(zeros[(size_t)g * N + n], 4, t2);
            for (int m = 0; m < M; ++m) {
                int64_t sum = 0;
                for (int k = g * glen; k < (g + 1) * glen; ++k) {
                    const uint8_t byte = codes[(size_t)n * (K / 2) + k / 2];
                    const int code = (k & 1) ? (byte >> 4) : (byte & 15);
                    sum += (int64_t)Xq[(size_t)m * K + k] * (int64_t)t2[code];
                }
                acc[((size_t)g * M + m) * N + n] = sum;
            }
        }
    }
}

/* The same sums in 32-bit, the width the method accumulates in. */
void oracle_linear_acc_i32(const int8_t *Xq, const uint8_t *codes,
                           const uint8_t *zeros, int M, int N, int K, int group,
                           int32_t *acc)
{
    const int glen = group ? group : K;
    const int G = K / glen;
#pragma omp parallel for schedule(static)
    for (int n = 0; n < N; ++n) {
        for (int g = 0; g < G; ++g) {
            int8_t t2[16];
            oracle_dint_table2(zeros[(size_t)g * N + n], 4, t2);
            for (int m = 0; m < M; ++m) {
                int32_t sum = 0;
                for (int k = g * glen; k < (g + 1) * glen; ++k) {
                    const uint8_t byte = codes[(size_t)n * (K / 2) + k / 2];
                    const int code = (k & 1) ? (byte >> 4) : (byte & 15);
                    sum += (int32_t)Xq[(size_t)m * K + k] * (int32_t)t2[code];
                }
                acc[((size_t)g * M + m) * N + n] = sum;
            }
        }
    }
}

/* ------------------------------------------------------------------------- */
/* rescale to real values                                                    */
/* ------------------------------------------------------------------------- */

/* True weight = t2 * (s/2) and true activation = q * tok_scale, so
 *   y[m][n] = tok_scale[m] * sum_g (s[g][n]/2) * acc[g][m][n]  (+ bias[n]).
 * binary32 evaluation order:
 *   one group : t = (float(acc) * tok_scale[m]) * (0.5f * s[n])
 *   G groups  : u = 0; for g ascending u = fmaf(float(acc_g), 0.5f * s[g][n], u);
 *               t = u * tok_scale[m]
 *   then t = t + bias[n] when bias is given, and Y = bf16(t), nearest-even. */
/* The layer's FP32 value t before the BF16 rounding (Y, may be NULL) and, optionally, that
 * value itself (T32, may be NULL). */
void oracle_linear_f32(const int8_t *Xq, const float *tok_scale, const uint8_t *codes,
                       const float *scales, const uint8_t *zeros, const float *bias,
                       int M, int N, int K, int group, uint16_t *Y, float *T32)
{
    const int glen = group ? group : K;
    const int G = K / glen;
#pragma omp parallel for schedule(static)
    for (int n = 0; n < N; ++n) {
        for (int m = 0; m < M; ++m) {
            float u = 0.0f;
            float t = 0.0f;
            for (int g = 0; g < G; ++g) {
                int8_t t2[16];
                oracle_dint_table2(zeros[(size_t)g * N + n], 4, t2);
                int32_t sum = 0;
                for (int k = g * glen; k < (g + 1) * glen; ++k) {
                    const uint8_t byte = codes[(size_t)n * (K / 2) + k / 2];
                    const int code = (k & 1) ? (byte >> 4) : (byte & 15);
                    sum += (int32_t)Xq[(size_t)m * K + k] * (int32_t)t2[code];
                }
                const float h = 0.5f * scales[(size_t)g * N + n];
                if (G == 1) {
                    t = ((float)sum * tok_scale[m]) * h;
                } else {
                    u = fmaf((float)sum, h, u);
                }
            }
            if (G != 1) t = u * tok_scale[m];
            if (bias) t = t + bias[n];
            if (Y) Y[(size_t)m * N + n] = float_to_bf16_bits(t);
            if (T32) T32[(size_t)m * N + n] = t;
        }
    }
}

void oracle_linear(const int8_t *Xq, const float *tok_scale, const uint8_t *codes,
                   const float *scales, const uint8_t *zeros, const float *bias,
                   int M, int N, int K, int group, uint16_t *Y)
{
    oracle_linear_f32(Xq, tok_scale, codes, scales, zeros, bias, M, N, K, group, Y, NULL);
}

/* Gate and up projections with the gated unit h = silu(g) * u between them and the next
 * quantized matmul ("all matrix multiplications in the Decoder layer", Appendix A.1; the unit
 * itself is the LLaMA block's, not the paper's).  Row 2 i of the weight matrix is row i of the
 * gate projection, row 2 i + 1 row i of the up projection; g and u are the layer's FP32 values
 * (bias included) before any BF16 rounding; h = (g / (1 + exp(-g))) * u is evaluated in binary64
 * on those FP32 values (H64, [M][F]) and rounded once to binary16 (H16 bits, may be NULL). */
void oracle_linear_swiglu(const int8_t *Xq, const float *tok_scale, const uint8_t *codes,
                          const float *scales, const uint8_t *zeros, const float *bias, int M,
                          int F, int K, int group, double *H64, float *T32)
{
    oracle_linear_f32(Xq, tok_scale, codes, scales, zeros, bias, M, 2 * F, K, group, NULL, T32);
    for (int m = 0; m < M; ++m)
        for (int f = 0; f < F; ++f) {
            const double g = (double)T32[(size_t)m * 2 * F + 2 * f];
            const double u = (double)T32[(size_t)m * 2 * F + 2 * f + 1];
            H64[(size_t)m * F + f] = g / (1.0 + exp(-g)) * u;
        }
}

/* The same value in binary64, not rounded to BF16: the tolerance reference. */
void oracle_linear_f64(const int8_t *Xq, const float *tok_scale,
                       const uint8_t *codes, const float *scales,
                       const uint8_t *zeros, const float *bias, int M, int N,
                       int K, int group, double *Y)
{
    const int glen = group ? group : K;
    const int G = K / glen;
#pragma omp parallel for schedule(static)
    for (int n = 0; n < N; ++n) {
        for (int m = 0; m < M; ++m) {
            double u = 0.0;
            for (int g = 0; g < G; ++g) {
                int8_t t2[16];
                oracle_dint_table2(zeros[(size_t)g * N + n], 4, t2);
                int64_t sum = 0;
                for (int k = g * glen; k < (g + 1) * glen; ++k) {
                    const uint8_t byte = codes[(size_t)n * (K / 2) + k / 2];
                    const int code = (k & 1) ? (byte >> 4) : (byte & 15);
                    sum += (int64_t)Xq[(size_t)m * K + k] * (int64_t)t2[code];
                }
                u += (double)sum * (0.5 * (double)scales[(size_t)g * N + n]);
            }
            double t = u * (double)tok_scale[m];
            if (bias) t += (double)bias[n];
            Y[(size_t)m * N + n] = t;
        }
    }
}

/* ------------------------------------------------------------------------- */
/* asymmetric token-wise activations (the paper's own activation quantizer)   */
/* ------------------------------------------------------------------------- */

/* App. A.1 quantizes activations token-wise with an asymmetric Min-Max quantizer.  The paper
 * gives no formula; the reading here mirrors the weight side (range widened to contain
 * zero, 2^8 - 1 steps) in binary32:
 *   x'[k] = float(X[m][k]) * inv_s_in[k]
 *   lo = min(0, min_k x'), hi = max(0, max_k x'), d = hi - lo
 *   d == 0: all codes 0, zero-point 0, step 0
 *   step = d / 255, r = 255 / d, zx = clamp(rint((-lo) * r), 0, 255)
 *   Q[m][k] = clamp(rint(x'[k] * r) + zx, 0, 255)        so that x' ~ step * (Q - zx). */
void oracle_quantize_act_asym(const uint16_t *X, const float *inv_s_in, int M, int K,
                              uint8_t *Q, float *tok_scale, int32_t *tok_zero)
{
#pragma omp parallel for schedule(static)
    for (int m = 0; m < M; ++m) {
        float lo = 0.0f, hi = 0.0f;
        for (int k = 0; k < K; ++k) {
            float x = half_bits_to_float(X[(size_t)m * K + k]);
            if (inv_s_in) x = x * inv_s_in[k];
            if (x < lo) lo = x;
            if (x > hi) hi = x;
        }
        const float d = hi - lo;
        if (d == 0.0f) {
            tok_scale[m] = 0.0f;
            tok_zero[m] = 0;
            for (int k = 0; k < K; ++k) Q[(size_t)m * K + k] = 0;
            continue;
        }
        const float r = 255.0f / d;
        tok_scale[m] = d / 255.0f;
        const int zx = clampi(rint_to_int((-lo) * r), 0, 255);
        tok_zero[m] = zx;
        for (int k = 0; k < K; ++k) {
            float x = half_bits_to_float(X[(size_t)m * K + k]);
            if (inv_s_in) x = x * inv_s_in[k];
            Q[(size_t)m * K + k] = (uint8_t)clampi(rint_to_int(x * r) + zx, 0, 255);
        }
    }
}

/* acc[m][n] = sum_k (Q[m][k] - zx[m]) * t2_{z[n]}[code[n][k]]: the contraction of the
 * dequantized integers, per-output-channel weights (the paper's W4A8 setting), in 64-bit. */
void oracle_linear_asym_acc_i64(const uint8_t *Q, const int32_t *tok_zero,
                                const uint8_t *codes, const uint8_t *zeros, int M, int N,
                                int K, int64_t *acc)
{
#pragma omp parallel for schedule(static)
    for (int n = 0; n < N; ++n) {
        int8_t t2[16];
        oracle_dint_table2(zeros[n], 4, t2);
        for (int m = 0; m < M; ++m) {
            int64_t sum = 0;
            for (int k = 0; k < K; ++k) {
                const uint8_t byte = codes[(size_t)n * (K / 2) + k / 2];
                const int code = (k & 1) ? (byte >> 4) : (byte & 15);
                sum += (int64_t)((int)Q[(size_t)m * K + k] - tok_zero[m]) * (int64_t)t2[code];
            }
            acc[(size_t)m * N + n] = sum;
        }
    }
}

/* y = (float(acc) * tok_scale[m]) * (0.5f * s[n]) (+ bias[n]) -> BF16, as in oracle_linear;
 * `wide` (may be NULL) receives the same value in binary64, unrounded. */
void oracle_linear_asym(const uint8_t *Q, const float *tok_scale, const int32_t *tok_zero,
                        const uint8_t *codes, const float *scales, const uint8_t *zeros,
                        const float *bias, int M, int N, int K, uint16_t *Y, double *wide)
{
#pragma omp parallel for schedule(static)
    for (int n = 0; n < N; ++n) {
        int8_t t2[16];
        oracle_dint_table2(zeros[n], 4, t2);
        const float h = 0.5f * scales[n];
        for (int m = 0; m < M; ++m) {
            int32_t sum = 0;
            for (int k = 0; k < K; ++k) {
                const uint8_t byte = codes[(size_t)n * (K / 2) + k / 2];
                const int code = (k & 1) ? (byte >> 4) : (byte & 15);
                sum += ((int32_t)Q[(size_t)m * K + k] - tok_zero[m]) * (int32_t)t2[code];
            }
            float t = ((float)sum * tok_scale[m]) * h;
            if (bias) t = t + bias[n];
            if (Y) Y[(size_t)m * N + n] = float_to_bf16_bits(t);
            if (wide) {
                double w = (double)sum * (double)tok_scale[m] * (0.5 * (double)scales[n]);
                if (bias) w += (double)bias[n];
                wide[(size_t)m * N + n] = w;
            }
        }
    }
}

/* The same layer with group-wise weight steps (128 consecutive k share a step and a
 * zero-point): the token's zero-point leaves every group's integer sum before that sum is
 * scaled, acc_g = sum_{k in g} (Q - zx) * t2, then the FP32 accumulation over the groups of
 * oracle_linear: u = fmaf(float(acc_g), 0.5 s_g, u), y = u * tok_scale (+ bias).  acc
 * ([G][M][N], may be NULL), Y (BF16 bits, may be NULL), wide (binary64, may be NULL). */
void oracle_linear_asym_group(const uint8_t *Q, const float *tok_scale, const int32_t *tok_zero,
                              const uint8_t *codes, const float *scales, const uint8_t *zeros,
                              const float *bias, int M, int N, int K, int group, int64_t *acc,
                              uint16_t *Y, double *wide)
{
    const int G = K / group;
#pragma omp parallel for schedule(static)
    for (int n = 0; n < N; ++n) {
        for (int m = 0; m < M; ++m) {
            float u = 0.0f;
            double w = 0.0;
            for (int g = 0; g < G; ++g) {
                int8_t t2[16];
                oracle_dint_table2(zeros[(size_t)g * N + n], 4, t2);
                int32_t sum = 0;
                for (int k = g * group; k < (g + 1) * group; ++k) {
                    const uint8_t byte = codes[(size_t)n * (K / 2) + k / 2];
                    const int code = (k & 1) ? (byte >> 4) : (byte & 15);
                    sum += ((int32_t)Q[(size_t)m * K + k] - tok_zero[m]) * (int32_t)t2[code];
                }
                if (acc) acc[((size_t)g * M + m) * N + n] = sum;
                const float h = 0.5f * scales[(size_t)g * N + n];
                u = fmaf((float)sum, h, u);
                w += (double)sum * (double)h;
            }
            float t = u * tok_scale[m];
            w *= (double)tok_scale[m];
            if (bias) { t = t + bias[n]; w += (double)bias[n]; }
            if (Y) Y[(size_t)m * N + n] = float_to_bf16_bits(t);
            if (wide) wide[(size_t)m * N + n] = w;
        }
    }
}

/* ------------------------------------------------------------------------- */
/* other special values: c = s / 2^j (App. A.5 sweeps c/s = 0.5, 0.25, 0.125)  */
/* ------------------------------------------------------------------------- */

/* Section 4.2 asks for a special value that is the step size over a power of two; Eq. 5 and
 * Eq. 6 are written for c = s/2 and the appendix gives no formulas for the others.  The
 * reading here keeps Eq. 5's structure: a value goes to +-c when it lies between the midpoints
 * of (0, c) and (c, s), i.e. c/2 < |x| <= (c + s)/2, with the same strictness as Eq. 5, and is
 * rounded to the integer grid otherwise.  j = 1 reproduces Eq. 5 / Eq. 6 exactly. */
int oracle_dint_quantize_fmt(float x, float s, int z, int b, int j)
{
    const int p = oracle_dint_p(b);
    const float lower = ldexpf(s, -(j + 1));          /* c / 2 */
    const float upper = 0.5f * s + lower;              /* (c + s) / 2 */
    if (x > lower && x <= upper) return p + 1;
    if (x < -lower && x >= -upper) return p + 2;
    return clampi(rint_to_int(x / s) + z, 0, p);
}

float oracle_dint_dequantize_fmt(int code, float s, int z, int b, int j)
{
    const int p = oracle_dint_p(b);
    if (code == p + 1) return ldexpf(s, -j);
    if (code == p + 2) return -ldexpf(s, -j);
    return (float)(code - z) * s;
}

/* Levels in units of c = s / 2^j: 2^j (code - z) for the integer levels, +1 and -1. */
void oracle_dint_table_fmt(int z, int b, int j, int8_t *t)
{
    const int p = oracle_dint_p(b);
    for (int c = 0; c <= p; ++c) t[c] = (int8_t)((c - z) * (1 << j));
    t[p + 1] = 1;
    t[p + 2] = -1;
}

/* oracle_pack_weights for the b-bit format (p = 2^b - 3 uniform steps, Section 4.2; b = 4 in
 * the paper's main results, b = 3 in Tables 10-11) with the special value s / 2^j.  Codes are
 * stored two per byte whatever b is (a 3-bit code occupies the low bits of its nibble). */
void oracle_pack_weights_bits(const uint16_t *W, const float *s_in, int N, int K, int group,
                              float clip, int b, int j, uint8_t *codes, float *scales,
                              uint8_t *zeros)
{
    const int p = oracle_dint_p(b);
    const int glen = group ? group : K;
    const int G = K / glen;
#pragma omp parallel for schedule(static)
    for (int n = 0; n < N; ++n) {
        for (int g = 0; g < G; ++g) {
            float lo = 0.0f, hi = 0.0f;
            for (int k = g * glen; k < (g + 1) * glen; ++k) {
                float w = half_bits_to_float(W[(size_t)n * K + k]);
                if (s_in) w = w * s_in[k];
                if (w < lo) lo = w;
                if (w > hi) hi = w;
            }
            lo = lo * clip;
            hi = hi * clip;
            float s = (hi - lo) / (float)p;
            if (s == 0.0f) s = 1.0f;
            const int z = clampi(rint_to_int((-lo) / s), 0, p);
            scales[(size_t)g * N + n] = s;
            zeros[(size_t)g * N + n] = (uint8_t)z;
            for (int k = g * glen; k < (g + 1) * glen; k += 2) {
                float w0 = half_bits_to_float(W[(size_t)n * K + k]);
                float w1 = half_bits_to_float(W[(size_t)n * K + k + 1]);
                if (s_in) { w0 = w0 * s_in[k]; w1 = w1 * s_in[k + 1]; }
                const int c0 = oracle_dint_quantize_fmt(w0, s, z, b, j);
                const int c1 = oracle_dint_quantize_fmt(w1, s, z, b, j);
                codes[(size_t)n * (K / 2) + k / 2] = (uint8_t)(c0 | (c1 << 4));
            }
        }
    }
}

/* oracle_pack_weights with the special value s / 2^j (4-bit format). */
void oracle_pack_weights_fmt(const uint16_t *W, const float *s_in, int N, int K, int group,
                             float clip, int j, uint8_t *codes, float *scales, uint8_t *zeros)
{
    oracle_pack_weights_bits(W, s_in, N, K, group, clip, 4, j, codes, scales, zeros);
}

/* The layer with levels in units of s / 2^j: integer sums acc [G][M][N] (may be NULL), BF16
 * output Y (may be NULL) in the evaluation order of oracle_linear with the level unit
 * 2^-j * s in place of 0.5 * s, and the same value in binary64 (may be NULL). */
void oracle_linear_bits(const int8_t *Xq, const float *tok_scale, const uint8_t *codes,
                        const float *scales, const uint8_t *zeros, const float *bias, int M,
                        int N, int K, int group, int b, int j, int64_t *acc, uint16_t *Y,
                        double *wide)
{
    const int glen = group ? group : K;
    const int G = K / glen;
#pragma omp parallel for schedule(static)
    for (int n = 0; n < N; ++n) {
        for (int m = 0; m < M; ++m) {
            float u = 0.0f, t = 0.0f;
            double w = 0.0;
            for (int g = 0; g < G; ++g) {
                int8_t lv[16];
                oracle_dint_table_fmt(zeros[(size_t)g * N + n], b, j, lv);
                int64_t sum = 0;
                for (int k = g * glen; k < (g + 1) * glen; ++k) {
                    const uint8_t byte = codes[(size_t)n * (K / 2) + k / 2];
                    const int code = (k & 1) ? (byte >> 4) : (byte & 15);
                    sum += (int64_t)Xq[(size_t)m * K + k] * (int64_t)lv[code];
                }
                if (acc) acc[((size_t)g * M + m) * N + n] = sum;
                const float h = ldexpf(scales[(size_t)g * N + n], -j);
                if (G == 1) t = ((float)(int32_t)sum * (tok_scale ? tok_scale[m] : 0.0f)) * h;
                else u = fmaf((float)(int32_t)sum, h, u);
                w += (double)sum * (double)h;
            }
            if (G != 1) t = u * (tok_scale ? tok_scale[m] : 0.0f);
            w *= tok_scale ? (double)tok_scale[m] : 0.0;
            if (bias) { t = t + bias[n]; w += (double)bias[n]; }
            if (Y) Y[(size_t)m * N + n] = float_to_bf16_bits(t);
            if (wide) wide[(size_t)m * N + n] = w;
        }
    }
}

void oracle_linear_fmt(const int8_t *Xq, const float *tok_scale, const uint8_t *codes,
                       const float *scales, const uint8_t *zeros, const float *bias, int M,
                       int N, int K, int group, int j, int64_t *acc, uint16_t *Y, double *wide)
{
    oracle_linear_bits(Xq, tok_scale, codes, scales, zeros, bias, M, N, K, group, 4, j, acc, Y, wide);
}

/* ---------------------------------------------------------------------------
 * Activation side of Eq. 1 with the scale diag(s)^-1 merged into the
 * normalisation in front of the matmul (Fig. 1(a), Section 3.1): the layer's
 * input is norm(X), the normalisation's weight (and bias) already carry 1/s,
 * and the token-wise INT8 quantizer (Appendix A.1) follows at once.
 *
 * kind 0, RMSNorm:    d_k = x_k,        ms = (sum_k d_k^2) / K
 * kind 1, LayerNorm:  d_k = x_k - mu,   mu = (sum_k x_k) / K,  ms = (sum_k d_k^2) / K
 * both:               r = 1 / sqrt(ms + eps),  x'_k = (d_k * r) * w_k (+ b_k)
 *
 * Precision (the paper gives none; this is the reading): a sum over the K
 * features is taken in binary32 inside each run of 8 consecutive features
 * (ascending k; the squares enter by fmaf, and a binary16 value squared is
 * exact in binary32), and the K / 8 partial sums are added in binary64
 * (ascending); mu, ms and r are binary64, mu and r are rounded once to
 * binary32, and everything per element (x - mu, the products, the bias) is
 * binary32, one rounded operation per written operation.  Then the symmetric
 * absmax quantizer exactly as in oracle_quantize_act.  K % 8 == 0.
 * ------------------------------------------------------------------------- */
void oracle_norm_quantize_act(const uint16_t *X, const float *w, const float *b, int kind,
                              float eps, int M, int K, int8_t *Xq, float *tok_scale)
{
#pragma omp parallel for schedule(static)
    for (int m = 0; m < M; ++m) {
        const uint16_t *row = X + (size_t)m * K;
        float mu32 = 0.0f;
        if (kind == 1) {
            double sum = 0.0;
            for (int g = 0; g < K; g += 8) {
                float part = 0.0f;
                for (int k = g; k < g + 8; ++k) part = part + half_bits_to_float(row[k]);
                sum += (double)part;
            }
            mu32 = (float)(sum / (double)K);
        }
        double ss = 0.0;
        for (int g = 0; g < K; g += 8) {
            float part = 0.0f;
            for (int k = g; k < g + 8; ++k) {
                const float d = kind == 1 ? half_bits_to_float(row[k]) - mu32
                                          : half_bits_to_float(row[k]);
                part = fmaf(d, d, part);
            }
            ss += (double)part;
        }
        const float r = (float)(1.0 / sqrt(ss / (double)K + (double)eps));
        float amax = 0.0f;
        for (int pass = 0; pass < 2; ++pass) {
            float q_r = 0.0f;
            if (pass == 1) {
                if (amax == 0.0f) {
                    tok_scale[m] = 0.0f;
                    for (int k = 0; k < K; ++k) Xq[(size_t)m * K + k] = 0;
                    break;
                }
                q_r = 127.0f / amax;
                tok_scale[m] = amax / 127.0f;
            }
            for (int k = 0; k < K; ++k) {
                float x = half_bits_to_float(row[k]);
                if (kind == 1) x = x - mu32;
                x = x * r;
                x = x * w[k];
                if (b) x = x + b[k];
                if (pass == 0) {
                    const float a = fabsf(x);
                    if (a > amax) amax = a;
                } else {
                    Xq[(size_t)m * K + k] = (int8_t)clampi(rint_to_int(x * q_r), -127, 127);
                }
            }
        }
    }
}

/* ------------------------------------------------------------------------- */
/* threading of the outermost loops (sums are integer, so order-free)         */
/* ------------------------------------------------------------------------- */
void oracle_set_threads(int n)
{
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
#else
    (void)n;
#endif
}

int oracle_get_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
