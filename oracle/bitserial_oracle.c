/*
 * Oracle for bit-serial ultra-low-bit convolution.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is a plain, slow, obviously-correct CPU
 * statement of what the GPU library computes.  It shares no code, header, table
 * or helper with the CUDA path and must never be linked into, imported by or
 * called from it; only the test-suite, the smoke check and the reported CPU
 * baseline of the benchmark may use it.
 *
 * What is the definition and what is an encoding
 * ----------------------------------------------
 * Section V of the paper computes the dot product of low-bit weights and
 * activations as POPCOUNT(W & A) for 1-bit unipolar operands and, for w-bit
 * weights and a-bit activations, as the sum over all bitplane pairs (i, j) of
 * POPCOUNT(W[i] & A[j]) << (i + j).  That sum reaches *exactly* the ordinary
 * integer dot product of the unpacked values, so the oracle for the
 * convolution and the matrix product is that ordinary definition, written out
 * on unpacked int8 codes (oracle_conv2d_i32, oracle_gemm_i32).
 *
 * The bitplane formula itself is restated separately, with explicit bit loops
 * and no popcount primitive (oracle_bitserial_dot), so that the tests can pin
 * "plane-pair sum == integer dot" on small inputs.
 *
 * The quantiser follows the Section IV equation t_bar = round(clip(t / s,
 * -Q_N, Q_P)) with Q_P = 2^(b-1) - 1 and Q_N = 2^(b-1).  The bracket in the
 * printed equation is read as round-to-nearest, ties to even (the result is
 * declared an integer).  Unsigned activations use the limits [0, 2^b - 1].
 * Arithmetic is IEEE binary32 because a floating-point value decides an
 * integer code here and the GPU takes the same decision in binary32.
 *
 * The requantisation epilogue (per-channel scale and bias, optional residual,
 * optional ReLU, clip, round-half-even) is not spelled out in the paper (it
 * only mentions a calibrated scale and bias for activations, Section IV); the
 * operation order used here is the reading fixed for this library:
 *     v = fma((float)acc, scale[o], bias[o])
 *     v = fma(res_scale, (float)res_code, v)      if a residual is given
 *     v = max(v, 0)                               if relu
 *     v = min(max(v, qmin), qmax)
 *     code = (int) rint(v)                        ties to even
 *
 * Value conventions: sign 0 = unsigned codes in [0, 2^b - 1]; sign 1 = two's
 * complement codes in [-2^(b-1), 2^(b-1) - 1]; sign 2 = bipolar, 1 bit, codes
 * in {-1, +1}.
 *
 * The packing functions restate the documented storage encodings (bit c%32 of
 * word c/32 holds channel c; plane index innermost) so packed buffers can be
 * compared word for word.
 *
 * Pins (tests/test_oracle_pins.py): worked examples under tests/golden/,
 * exhaustive small cases, closed-form border counts, float64 library
 * convolution, int64 matrix product, bipolar XOR identity.
 */
#include <math.h>
#include <stdint.h>
#include <stddef.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { ORA_UNSIGNED = 0, ORA_SIGNED = 1, ORA_BIPOLAR = 2 };

int oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void oracle_set_threads(int n)
{
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
#else
    (void)n;
#endif
}

/* Clipping limits of the quantiser (Section IV): signed [-2^(b-1), 2^(b-1)-1];
 * unsigned reading [0, 2^b - 1]; bipolar {-1, +1}. */
static void code_limits(int bits, int sign, int *qmin, int *qmax)
{
    if (sign == ORA_SIGNED)       { *qmin = -(1 << (bits - 1)); *qmax = (1 << (bits - 1)) - 1; }
    else if (sign == ORA_BIPOLAR) { *qmin = -1;                  *qmax = 1; }
    else                          { *qmin = 0;                   *qmax = (1 << bits) - 1; }
}

/* Section IV quantiser: code = round_half_even(clip(x / s, qmin, qmax)).
 * Bipolar: code = +1 when x >= 0, else -1 (the paper gives no 1-bit bipolar
 * quantiser; sign() is the reading used). */
void oracle_quantize(const float *x, long n, float s, int bits, int sign, int8_t *codes)
{
    int qmin, qmax;
    code_limits(bits, sign, &qmin, &qmax);
    for (long k = 0; k < n; ++k) {
        if (sign == ORA_BIPOLAR) { codes[k] = (x[k] >= 0.0f) ? 1 : -1; continue; }
        volatile float t = x[k] / s;               /* IEEE binary32 division */
        float c = fminf(fmaxf(t, (float)qmin), (float)qmax);
        codes[k] = (int8_t)(int)rintf(c);           /* FE_TONEAREST: ties to even */
    }
}

/* Section IV: t_hat = t_bar * s. */
void oracle_dequantize(const int8_t *codes, long n, float s, float *x_hat)
{
    for (long k = 0; k < n; ++k) x_hat[k] = (float)codes[k] * s;
}

/* Direct integer convolution, the quantity the Section V plane-pair sum equals.
 *   acc[n][o][p][q] = sum_{c,r,s} a[n][c][p*stride - pad + r][q*stride - pad + s] * w[o][c][r][s]
 * with a = 0 outside the image.  a: NCHW int8 codes, w: OIHW int8 codes,
 * out: [N][O][P][Q] int32, P = (H + 2 pad - R)/stride + 1 (same for Q). */
int oracle_conv2d_i32(const int8_t *a, const int8_t *w, int N, int C, int H, int W, int O, int R,
                      int S, int stride, int pad, int32_t *out)
{
    if (stride < 1 || pad < 0 || H + 2 * pad < R || W + 2 * pad < S) return 1;
    const int P = (H + 2 * pad - R) / stride + 1;
    const int Q = (W + 2 * pad - S) / stride + 1;
#pragma omp parallel for collapse(2) schedule(static)
    for (int n = 0; n < N; ++n)
        for (int o = 0; o < O; ++o) {
            int32_t *dst = out + ((size_t)n * O + o) * P * Q;
            memset(dst, 0, sizeof(int32_t) * (size_t)P * Q);
            for (int c = 0; c < C; ++c)
                for (int r = 0; r < R; ++r)
                    for (int s = 0; s < S; ++s) {
                        const int32_t wv = w[(((size_t)o * C + c) * R + r) * S + s];
                        for (int p = 0; p < P; ++p) {
                            const int y = p * stride - pad + r;
                            if (y < 0 || y >= H) continue;          /* zero padding */
                            const int8_t *row = a + (((size_t)n * C + c) * H + y) * W;
                            for (int q = 0; q < Q; ++q) {
                                const int x = q * stride - pad + s;
                                if (x < 0 || x >= W) continue;      /* zero padding */
                                dst[(size_t)p * Q + q] += (int32_t)row[x] * wv;
                            }
                        }
                    }
        }
    return 0;
}

/* out[m][n] = sum_k a[m][k] * w[n][k]; both operands K-contiguous int8 codes. */
int oracle_gemm_i32(const int8_t *a, const int8_t *w, int M, int N, int K, int32_t *out)
{
#pragma omp parallel for schedule(static)
    for (int m = 0; m < M; ++m)
        for (int n = 0; n < N; ++n) {
            int32_t acc = 0;
            for (int k = 0; k < K; ++k) acc += (int32_t)a[(size_t)m * K + k] * (int32_t)w[(size_t)n * K + k];
            out[(size_t)m * N + n] = acc;
        }
    return 0;
}

/* Requantisation epilogue over a tensor viewed as [outer][O][inner]
 * (NCHW accumulators: outer = N, inner = P*Q; row-major GEMM output
 * [M][N]: outer = M, O = N, inner = 1).  res may be NULL. */
void oracle_requantize(const int32_t *acc, long outer, int O, long inner, const float *scale,
                       const float *bias, const int8_t *res, float res_scale, int relu,
                       int out_bits, int out_sign, int8_t *codes)
{
    int qmin, qmax;
    code_limits(out_bits, out_sign, &qmin, &qmax);
#pragma omp parallel for schedule(static)
    for (long u = 0; u < outer; ++u)
        for (int o = 0; o < O; ++o)
            for (long t = 0; t < inner; ++t) {
                const size_t idx = ((size_t)u * O + o) * inner + t;
                float v = fmaf((float)acc[idx], scale[o], bias[o]);
                if (res) v = fmaf(res_scale, (float)res[idx], v);
                if (relu) v = fmaxf(v, 0.0f);
                if (out_sign == ORA_BIPOLAR) { codes[idx] = (v >= 0.0f) ? 1 : -1; continue; }
                v = fminf(fmaxf(v, (float)qmin), (float)qmax);
                codes[idx] = (int8_t)(int)rintf(v);
            }
}

/* Bit b of the stored pattern of a code.  Unsigned and two's-complement codes
 * store their low `bits` bits; a bipolar code stores 1 for +1 and 0 for -1. */
static int stored_bit(int code, int sign, int b)
{
    if (sign == ORA_BIPOLAR) return (b == 0 && code > 0) ? 1 : 0;
    return (int)(((unsigned)code >> b) & 1u);
}

/* The Section V plane-pair formula restated with explicit bit loops:
 *   sum_i sum_j popcount(W[i] & A[j]) << (i + j)
 * where popcount over the K positions is a plain count of positions whose two
 * plane bits are both 1.  Readings added to the printed (unsigned) formula:
 * the top plane of a two's-complement operand carries weight -2^(b-1); a
 * bipolar operand is v = 2*bit - 1, which is expanded algebraically:
 *   (2x-1) * y = 2xy - y,  x * (2y-1) = 2xy - x,  (2x-1)(2y-1) = 4xy - 2x - 2y + 1.
 */
int32_t oracle_bitserial_dot(const int8_t *a, const int8_t *w, int K, int a_bits, int a_sign,
                             int w_bits, int w_sign)
{
    long and_sum = 0;   /* signed, shifted sum over plane pairs of AND counts */
    long a_sum = 0;     /* signed, shifted sum over activation planes of bit counts */
    long w_sum = 0;     /* same for weight planes */
    for (int i = 0; i < w_bits; ++i) {
        const long ci = (w_sign == ORA_SIGNED && i == w_bits - 1) ? -1 : 1;
        long cnt = 0;
        for (int k = 0; k < K; ++k) cnt += stored_bit(w[k], w_sign, i);
        w_sum += ci * (cnt << i);
    }
    for (int j = 0; j < a_bits; ++j) {
        const long dj = (a_sign == ORA_SIGNED && j == a_bits - 1) ? -1 : 1;
        long cnt = 0;
        for (int k = 0; k < K; ++k) cnt += stored_bit(a[k], a_sign, j);
        a_sum += dj * (cnt << j);
    }
    for (int i = 0; i < w_bits; ++i)
        for (int j = 0; j < a_bits; ++j) {
            const long ci = (w_sign == ORA_SIGNED && i == w_bits - 1) ? -1 : 1;
            const long dj = (a_sign == ORA_SIGNED && j == a_bits - 1) ? -1 : 1;
            long popc = 0;
            for (int k = 0; k < K; ++k)
                popc += stored_bit(w[k], w_sign, i) & stored_bit(a[k], a_sign, j);
            and_sum += ci * dj * (popc << (i + j));
        }
    const int ab = (a_sign == ORA_BIPOLAR), wb = (w_sign == ORA_BIPOLAR);
    if (ab && wb) return (int32_t)(4 * and_sum - 2 * a_sum - 2 * w_sum + K);
    if (wb) return (int32_t)(2 * and_sum - a_sum);
    if (ab) return (int32_t)(2 * and_sum - w_sum);
    return (int32_t)and_sum;
}

/* Bipolar identity: dot = K - 2 * popcount(a XOR w), popcount by bit loop. */
int32_t oracle_bipolar_xor_dot(const int8_t *a, const int8_t *w, int K)
{
    int diff = 0;
    for (int k = 0; k < K; ++k) diff += stored_bit(a[k], ORA_BIPOLAR, 0) ^ stored_bit(w[k], ORA_BIPOLAR, 0);
    return K - 2 * diff;
}

/* Storage encoding of packed activations: uint32 [N][H][W][Cw][bits],
 * Cw = ceil(C/32); bit (c % 32) of word (c / 32) of plane j is bit j of the
 * stored pattern of channel c; channels beyond C are 0.  Input codes NCHW. */
void oracle_pack_activations(const int8_t *codes, int N, int C, int H, int W, int bits, int sign,
                             uint32_t *packed)
{
    const int Cw = (C + 31) / 32;
    memset(packed, 0, sizeof(uint32_t) * (size_t)N * H * W * Cw * bits);
    for (int n = 0; n < N; ++n)
        for (int c = 0; c < C; ++c)
            for (int y = 0; y < H; ++y)
                for (int x = 0; x < W; ++x) {
                    const int code = codes[(((size_t)n * C + c) * H + y) * W + x];
                    for (int j = 0; j < bits; ++j)
                        if (stored_bit(code, sign, j))
                            packed[((((size_t)n * H + y) * W + x) * Cw + c / 32) * bits + j] |= 1u << (c % 32);
                }
}

/* Inverse of oracle_pack_activations. */
void oracle_unpack_activations(const uint32_t *packed, int N, int C, int H, int W, int bits, int sign,
                               int8_t *codes)
{
    const int Cw = (C + 31) / 32;
    for (int n = 0; n < N; ++n)
        for (int c = 0; c < C; ++c)
            for (int y = 0; y < H; ++y)
                for (int x = 0; x < W; ++x) {
                    unsigned pat = 0;
                    for (int j = 0; j < bits; ++j)
                        pat |= ((packed[((((size_t)n * H + y) * W + x) * Cw + c / 32) * bits + j] >> (c % 32)) & 1u) << j;
                    int v = (int)pat;
                    if (sign == ORA_SIGNED && (pat >> (bits - 1))) v -= 1 << bits;
                    if (sign == ORA_BIPOLAR) v = pat ? 1 : -1;
                    codes[(((size_t)n * C + c) * H + y) * W + x] = (int8_t)v;
                }
}

/* Storage encoding of packed weights: uint32 [O][R][S][Cw][bits]; input OIHW. */
void oracle_pack_weights(const int8_t *codes, int O, int C, int R, int S, int bits, int sign,
                         uint32_t *packed)
{
    const int Cw = (C + 31) / 32;
    memset(packed, 0, sizeof(uint32_t) * (size_t)O * R * S * Cw * bits);
    for (int o = 0; o < O; ++o)
        for (int c = 0; c < C; ++c)
            for (int r = 0; r < R; ++r)
                for (int s = 0; s < S; ++s) {
                    const int code = codes[(((size_t)o * C + c) * R + r) * S + s];
                    for (int i = 0; i < bits; ++i)
                        if (stored_bit(code, sign, i))
                            packed[((((size_t)o * R + r) * S + s) * Cw + c / 32) * bits + i] |= 1u << (c % 32);
                }
}

/* Storage encoding of packed matrix rows: uint32 [rows][Kw][bits], Kw = ceil(K/32). */
void oracle_pack_rows(const int8_t *codes, int rows, int K, int bits, int sign, uint32_t *packed)
{
    const int Kw = (K + 31) / 32;
    memset(packed, 0, sizeof(uint32_t) * (size_t)rows * Kw * bits);
    for (int m = 0; m < rows; ++m)
        for (int k = 0; k < K; ++k)
            for (int j = 0; j < bits; ++j)
                if (stored_bit(codes[(size_t)m * K + k], sign, j))
                    packed[((size_t)m * Kw + k / 32) * bits + j] |= 1u << (k % 32);
}
