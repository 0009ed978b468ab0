/*
 * Oracle for the layers that stay in floating point (TEST INFRASTRUCTURE ONLY, same rules as bitserial_oracle.c: no code
 * shared with the CUDA path, called by the tests, the smoke check and the benchmark's CPU baseline only).
 *
 * The paper keeps a few quantisation-sensitive layers in FP32 and quantises the rest (Section VII-D, mixed precision;
 * Section VI pipeline): in a residual classifier these are the first convolution with its pooling and the final
 * pooling + fully-connected layer.  The paper gives no arithmetic for them beyond "FP32"; the reading fixed here, which the
 * CUDA side must follow operation by operation because a quantiser turns the stem's output into integer codes:
 *
 *   conv      acc = bias[o];  for c, r, s ascending (c outermost, s innermost):  acc = fma(x, w, acc)  over the taps that
 *             fall inside the image (zero padding adds nothing);  ReLU if asked.  IEEE binary32, one rounding per fma.
 *   max pool  the maximum over the window positions inside the image (padding never wins).
 *   avg pool  over integer activation codes: the exact integer sum of the window (here the whole image), converted to
 *             binary32 (exact: far below 2^24) and multiplied once by `inv` = code step / number of pixels.
 *   fc        acc = bias[j];  for k ascending:  acc = fma(x[k], w[j][k], acc).
 *
 * Pins (tests/test_oracle_pins.py): hand-worked small cases with exactly representable values, float64 library routines
 * within the rounding bound of a chain of that length, a single-tap filter (pins the correlation direction and the
 * stride/pad arithmetic), the pooling routines against their library counterparts (exact).
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>

void oracle_conv2d_f32(const float *x, const float *w, const float *bias, int N, int C, int H, int W, int O, int R, int S,
                       int stride, int pad, int relu, float *out)
{
    const int P = (H + 2 * pad - R) / stride + 1, Q = (W + 2 * pad - S) / stride + 1;
#pragma omp parallel for collapse(2) schedule(static)
    for (int n = 0; n < N; ++n)
        for (int o = 0; o < O; ++o)
            for (int p = 0; p < P; ++p)
                for (int q = 0; q < Q; ++q) {
                    float acc = bias ? bias[o] : 0.0f;
                    for (int c = 0; c < C; ++c)
                        for (int r = 0; r < R; ++r)
                            for (int s = 0; s < S; ++s) {
                                const int y = p * stride - pad + r, xx = q * stride - pad + s;
                                if (y < 0 || y >= H || xx < 0 || xx >= W) continue;
                                acc = fmaf(x[(((size_t)n * C + c) * H + y) * W + xx], w[(((size_t)o * C + c) * R + r) * S + s], acc);
                            }
                    if (relu) acc = fmaxf(acc, 0.0f);
                    out[(((size_t)n * O + o) * P + p) * Q + q] = acc;
                }
}

void oracle_maxpool2d_f32(const float *x, int N, int C, int H, int W, int k, int stride, int pad, float *out)
{
    const int P = (H + 2 * pad - k) / stride + 1, Q = (W + 2 * pad - k) / stride + 1;
#pragma omp parallel for schedule(static)
    for (long nc = 0; nc < (long)N * C; ++nc)
        for (int p = 0; p < P; ++p)
            for (int q = 0; q < Q; ++q) {
                float m = -INFINITY;
                for (int r = 0; r < k; ++r)
                    for (int s = 0; s < k; ++s) {
                        const int y = p * stride - pad + r, xx = q * stride - pad + s;
                        if (y < 0 || y >= H || xx < 0 || xx >= W) continue;
                        m = fmaxf(m, x[((size_t)nc * H + y) * W + xx]);
                    }
                out[((size_t)nc * P + p) * Q + q] = m;
            }
}

/* Global average pooling of integer codes [N][C][H][W] -> [N][C]: exact integer sum, one multiplication by inv. */
void oracle_avgpool_codes(const int8_t *codes, int N, int C, int H, int W, float inv, float *out)
{
    for (long nc = 0; nc < (long)N * C; ++nc) {
        int sum = 0;
        for (int i = 0; i < H * W; ++i) sum += codes[(size_t)nc * H * W + i];
        out[nc] = (float)sum * inv;
    }
}

/* out[n][j] = bias[j] + sum_k x[n][k] * w[j][k], accumulated as a chain of fma over ascending k. */
void oracle_fc_f32(const float *x, const float *w, const float *bias, int N, int K, int J, float *out)
{
#pragma omp parallel for collapse(2) schedule(static)
    for (int n = 0; n < N; ++n)
        for (int j = 0; j < J; ++j) {
            float acc = bias ? bias[j] : 0.0f;
            for (int k = 0; k < K; ++k) acc = fmaf(x[(size_t)n * K + k], w[(size_t)j * K + k], acc);
            out[(size_t)n * J + j] = acc;
        }
}
