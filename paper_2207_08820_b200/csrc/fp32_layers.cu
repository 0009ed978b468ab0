// The layers a mixed-precision network keeps in floating point (paper, Section VII-D: a few quantisation-sensitive layers
// stay FP32, the rest is quantised): the first convolution with its max pooling, and the final average pooling + fully
// connected layer.  The paper gives no arithmetic for them beyond "FP32".  Fixed here, because a quantiser turns the stem's
// output into integer codes and every rounding matters: IEEE binary32; a convolution output is a chain of fused multiply-adds
// that starts at the bias and walks the taps channel-outermost, then row, then column, all ascending; the fully connected
// layer walks its inputs ascending; the average pool sums integer codes exactly and multiplies once.
#include "common.cuh"

namespace bs {

// ----------------------------------------------------------------------------- convolution, register-tiled
//
// CTA tile: TH x TW output pixels of one image x 64 filters; thread = 8 filters x 8 consecutive output columns.
// Weights of the 64 filters ([c][r][s][64], 16-byte vectors of four filters) and the input halo sit in shared memory.  For a
// fixed (c, r) a thread keeps the input row segment of its eight outputs in registers and walks the S columns: per column two
// 128-bit weight loads feed 64 fused multiply-adds (with four filters per thread the shared-memory pipe, not the FMA pipe, set
// the pace: 22 TFLOP/s).  A warp is 8 filter octets x 4 strips: its weight loads are 8 distinct vectors, its input loads four
// broadcasts.
constexpr int F32_TH = 16, F32_TW = 16, F32_STRIP = 8, F32_OT = 64, F32_THREADS = 256, F32_FPT = 8;

struct ConvF32Args {
    const float* x;
    const float* w;
    const float* bias;
    float* out;
    int N, C, H, W, O, R, stride, pad, relu, P, Q;
    int in_h, in_w, pitch;        // staged input tile: rows, columns, row pitch (floats, multiple of 4)
    int tiles_p, tiles_q, tiles_o;
};

template <int S, int STRIDE>
__global__ void __launch_bounds__(F32_THREADS, 2) conv2d_f32_tiled_kernel(const ConvF32Args g)
{
    extern __shared__ __align__(16) float f32_smem[];
    constexpr int WIN = (F32_STRIP - 1) * STRIDE + S;            // input columns one strip needs
    constexpr int WIN4 = (WIN + 3) / 4;
    float* s_w = f32_smem;                                       // [C][R][S][2][8][4]
    float* s_x0 = f32_smem + g.C * g.R * S * F32_OT;             // [2][C][in_h][pitch]: the halo of the next tile lands while this one is computed
    const int halo_floats = g.C * g.in_h * g.pitch;
    const int tid = threadIdx.x;
    const int to = blockIdx.y, o0 = to * F32_OT;

    // weights once per CTA: global [O][C][R][S] -> shared [c][r][s][o - o0] (zero beyond O).  Consecutive threads take
    // consecutive filters of one tap: the shared-memory writes are conflict-free, the strided global reads stay in L1/L2
    // (the filter bank is a few tens of KB) and are amortised over all the tiles the CTA walks.
    const int taps = g.C * g.R * S;
    for (int i = tid; i < taps * F32_OT; i += F32_THREADS) {
        // filter o = 8 * octet + k sits at [tap][k / 4][octet][k % 4]: the eight threads of a quarter warp, one octet each, read
        // 128 contiguous bytes with each of their two vector loads
        const int t = i >> 6, o = i & 63;
        s_w[t * F32_OT + ((o & 7) >> 2) * 32 + (o >> 3) * 4 + (o & 3)] = (o0 + o < g.O) ? g.w[static_cast<size_t>(o0 + o) * taps + t] : 0.0f;
    }
    const int tiles = g.N * g.tiles_p * g.tiles_q;
    // Input halo of a tile, zero outside the image (a zero tap leaves the chain unchanged: fma(0, w, acc) == acc), fetched with
    // 4-byte asynchronous copies (zero-filled where the source is outside): a thread owns column tid % 64 of every fourth
    // halo row, so no division is needed per element, and the copies of tile k + 1 fly while tile k is computed.
    auto stage = [&](int tile, float* dst) {
        int b = tile;
        const int tq = b % g.tiles_q; b /= g.tiles_q;
        const int tp = b % g.tiles_p; b /= g.tiles_p;
        const int n = b;
        const int y0 = tp * F32_TH * STRIDE - g.pad, x0 = tq * F32_TW * STRIDE - g.pad;
        const int rows = g.C * g.in_h;
        int yy = tid >> 6, c = 0;
        while (yy >= g.in_h) { yy -= g.in_h; ++c; }
        for (int xx = tid & 63; xx < g.pitch; xx += 64) {
            int y2 = yy, c2 = c;
            const int x = x0 + xx;
            const bool xok = xx < g.in_w && x >= 0 && x < g.W;
            for (int row = tid >> 6; row < rows; row += F32_THREADS / 64) {
                const int y = y0 + y2;
                const bool ok = xok && y >= 0 && y < g.H;
                const float* src = ok ? g.x + ((static_cast<size_t>(n) * g.C + c2) * g.H + y) * g.W + x : g.x;
                const unsigned d = static_cast<unsigned>(__cvta_generic_to_shared(dst + row * g.pitch + xx));
                asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"(d), "l"(src), "r"(ok ? 4 : 0) : "memory");
                y2 += F32_THREADS / 64;
                while (y2 >= g.in_h) { y2 -= g.in_h; ++c2; }
            }
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };
    if (static_cast<int>(blockIdx.x) < tiles) stage(blockIdx.x, s_x0);
    int buf = 0;
    for (int tile = blockIdx.x; tile < tiles; tile += gridDim.x, buf ^= 1) {
    int b = tile;
    const int tq = b % g.tiles_q; b /= g.tiles_q;
    const int tp = b % g.tiles_p; b /= g.tiles_p;
    const int n = b;
    const int p0 = tp * F32_TH, q0 = tq * F32_TW;
    const float* s_x = s_x0 + buf * halo_floats;
    // the other buffer was read by the tile before this one: every thread is past that (barrier at the end of the loop body)
    if (tile + static_cast<int>(gridDim.x) < tiles) {
        stage(tile + gridDim.x, s_x0 + (buf ^ 1) * halo_floats);
        asm volatile("cp.async.wait_group 1;" ::: "memory");     // this tile's copies have landed; the next tile's may still fly
    } else {
        asm volatile("cp.async.wait_group 0;" ::: "memory");
    }
    __syncthreads();

    const int cq = tid & 7, strip = tid >> 3;                    // filter octet, strip (row-major over TH x TW / 8)
    const int sp = strip / (F32_TW / F32_STRIP), sq = strip % (F32_TW / F32_STRIP);
    float acc[F32_STRIP][F32_FPT];
    {
        float bq[F32_FPT];
#pragma unroll
        for (int k = 0; k < F32_FPT; ++k) bq[k] = (g.bias && o0 + cq * F32_FPT + k < g.O) ? g.bias[o0 + cq * F32_FPT + k] : 0.0f;
#pragma unroll
        for (int j = 0; j < F32_STRIP; ++j)
#pragma unroll
            for (int k = 0; k < F32_FPT; ++k) acc[j][k] = bq[k];  // the chain starts at the bias
    }
    for (int c = 0; c < g.C; ++c) {
        for (int r = 0; r < g.R; ++r) {
            const float* row = s_x + (c * g.in_h + sp * STRIDE + r) * g.pitch + sq * F32_STRIP * STRIDE;
            float xr[WIN4 * 4];
#pragma unroll
            for (int v = 0; v < WIN4; ++v) {
                const float4 t = *reinterpret_cast<const float4*>(row + 4 * v);
                xr[4 * v] = t.x; xr[4 * v + 1] = t.y; xr[4 * v + 2] = t.z; xr[4 * v + 3] = t.w;
            }
            const float* wrow = s_w + ((c * g.R + r) * S) * F32_OT + cq * 4;
#pragma unroll
            for (int s = 0; s < S; ++s) {
                const float4 wa = *reinterpret_cast<const float4*>(wrow + s * F32_OT);
                const float4 wb = *reinterpret_cast<const float4*>(wrow + s * F32_OT + 32);
#pragma unroll
                for (int j = 0; j < F32_STRIP; ++j) {
                    const float xv = xr[j * STRIDE + s];
                    acc[j][0] = fmaf(xv, wa.x, acc[j][0]);
                    acc[j][1] = fmaf(xv, wa.y, acc[j][1]);
                    acc[j][2] = fmaf(xv, wa.z, acc[j][2]);
                    acc[j][3] = fmaf(xv, wa.w, acc[j][3]);
                    acc[j][4] = fmaf(xv, wb.x, acc[j][4]);
                    acc[j][5] = fmaf(xv, wb.y, acc[j][5]);
                    acc[j][6] = fmaf(xv, wb.z, acc[j][6]);
                    acc[j][7] = fmaf(xv, wb.w, acc[j][7]);
                }
            }
        }
    }
    const int p = p0 + sp, qb = q0 + sq * F32_STRIP;
#pragma unroll
    for (int k = 0; k < F32_FPT; ++k) {
        const int o = o0 + cq * F32_FPT + k;
        if (o >= g.O || p >= g.P) continue;
        float* dst = g.out + ((static_cast<size_t>(n) * g.O + o) * g.P + p) * g.Q + qb;
        float v[F32_STRIP];
#pragma unroll
        for (int j = 0; j < F32_STRIP; ++j) v[j] = g.relu ? fmaxf(acc[j][k], 0.0f) : acc[j][k];
        if (qb + F32_STRIP <= g.Q && (g.Q & 3) == 0) {
            reinterpret_cast<float4*>(dst)[0] = make_float4(v[0], v[1], v[2], v[3]);
            reinterpret_cast<float4*>(dst)[1] = make_float4(v[4], v[5], v[6], v[7]);
        } else {
#pragma unroll
            for (int j = 0; j < F32_STRIP; ++j)
                if (qb + j < g.Q) dst[j] = v[j];
        }
    }
    __syncthreads();                                             // every thread is done reading this tile's halo buffer
    }   // tiles
}

// Any other shape: one thread per output, the same chain in the same order (slow; the stem shapes take the tiled kernel).
__global__ void conv2d_f32_direct_kernel(const float* __restrict__ x, const float* __restrict__ w, const float* __restrict__ bias,
                                         float* __restrict__ out, int N, int C, int H, int W, int O, int R, int S, int stride, int pad,
                                         int relu, int P, int Q)
{
    const long long total = static_cast<long long>(N) * O * P * Q;
    for (long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; i < total; i += static_cast<long long>(gridDim.x) * blockDim.x) {
        long long t = i;
        const int q = static_cast<int>(t % Q); t /= Q;
        const int p = static_cast<int>(t % P); t /= P;
        const int o = static_cast<int>(t % O);
        const int n = static_cast<int>(t / O);
        float acc = bias ? bias[o] : 0.0f;
        for (int c = 0; c < C; ++c)
            for (int r = 0; r < R; ++r)
                for (int s = 0; s < S; ++s) {
                    const int y = p * stride - pad + r, xx = q * stride - pad + s;
                    if (y < 0 || y >= H || xx < 0 || xx >= W) continue;
                    acc = fmaf(x[((static_cast<size_t>(n) * C + c) * H + y) * W + xx], w[((static_cast<size_t>(o) * C + c) * R + r) * S + s], acc);
                }
        out[i] = relu ? fmaxf(acc, 0.0f) : acc;
    }
}

// ----------------------------------------------------------------------------- pooling and the classifier

__global__ void maxpool2d_f32_kernel(const float* __restrict__ x, float* __restrict__ out, long long planes, int H, int W, int k, int stride,
                                     int pad, int P, int Q)
{
    const long long total = planes * P * Q;
    for (long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; i < total; i += static_cast<long long>(gridDim.x) * blockDim.x) {
        const int q = static_cast<int>(i % Q);
        const int p = static_cast<int>((i / Q) % P);
        const long long pl = i / (static_cast<long long>(P) * Q);
        const float* src = x + pl * H * W;
        float m = -INFINITY;
        for (int r = 0; r < k; ++r) {
            const int y = p * stride - pad + r;
            if (y < 0 || y >= H) continue;
            for (int s = 0; s < k; ++s) {
                const int xx = q * stride - pad + s;
                if (xx < 0 || xx >= W) continue;
                m = fmaxf(m, src[static_cast<size_t>(y) * W + xx]);
            }
        }
        out[i] = m;
    }
}

// 3x3 window, stride 2, pad 1 on rows whose width is a multiple of 8 (the stem's pooling): a thread produces four consecutive
// outputs from three rows of eight inputs read as 128-bit vectors plus the column to their left.  The maximum does not depend
// on the order of its operands, so this is the same result as the generic kernel.
__global__ void maxpool3x3s2p1_f32_kernel(const float* __restrict__ x, float* __restrict__ out, long long planes, int H, int W, int P, int Q)
{
    const int q4n = Q >> 2;
    const long long total = planes * P * q4n;
    for (long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; i < total; i += static_cast<long long>(gridDim.x) * blockDim.x) {
        const int q4 = static_cast<int>(i % q4n);
        const int p = static_cast<int>((i / q4n) % P);
        const long long pl = i / (static_cast<long long>(P) * q4n);
        const float* src = x + pl * H * W;
        float m[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
        for (int r = 0; r < 3; ++r) {
            const int y = 2 * p - 1 + r;
            if (y < 0 || y >= H) continue;
            const float* row = src + static_cast<size_t>(y) * W + 8 * q4;
            const float4 a = *reinterpret_cast<const float4*>(row), b = *reinterpret_cast<const float4*>(row + 4);
            const float left = q4 > 0 ? row[-1] : -INFINITY;
            m[0] = fmaxf(m[0], fmaxf(left, fmaxf(a.x, a.y)));
            m[1] = fmaxf(m[1], fmaxf(a.y, fmaxf(a.z, a.w)));
            m[2] = fmaxf(m[2], fmaxf(a.w, fmaxf(b.x, b.y)));
            m[3] = fmaxf(m[3], fmaxf(b.y, fmaxf(b.z, b.w)));
        }
        *reinterpret_cast<float4*>(out + (pl * P + p) * Q + 4 * q4) = make_float4(m[0], m[1], m[2], m[3]);
    }
}

// Global average pool of packed activation codes [N][H][W][Cw][bits] -> float [N][C]: exact integer sum, one multiplication.
__global__ void avgpool_codes_kernel(const uint32_t* __restrict__ packed, float* __restrict__ out, int N, int C, int HW, int Cw, int bits,
                                     int sign, float inv)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= N * C) return;
    const int n = i / C, c = i - n * C;
    const uint32_t* src = packed + (static_cast<size_t>(n) * HW * Cw + (c >> 5)) * bits;
    int sum = 0;
    for (int px = 0; px < HW; ++px) {
        unsigned pat = 0;
        for (int j = 0; j < bits; ++j) pat |= ((src[static_cast<size_t>(px) * Cw * bits + j] >> (c & 31)) & 1u) << j;
        sum += pattern_value(pat, bits, sign);
    }
    out[i] = static_cast<float>(sum) * inv;
}

// out[n][j] = bias[j] + sum_k x[n][k] w[j][k], a chain of fused multiply-adds over ascending k.
// Block: 32 outputs j x 8 rows n; weights and inputs are staged in chunks of 64 k (the chain crosses the chunks in order).
constexpr int FC_KC = 64;
__global__ void __launch_bounds__(256) fc_f32_kernel(const float* __restrict__ x, const float* __restrict__ w, const float* __restrict__ bias,
                                                      float* __restrict__ out, int N, int K, int J)
{
    __shared__ float s_w[32][FC_KC + 1];
    __shared__ float s_x[8][FC_KC];
    const int jl = threadIdx.x & 31, nl = threadIdx.x >> 5;
    const int j = blockIdx.x * 32 + jl, n = blockIdx.y * 8 + nl;
    float acc = (bias && j < J) ? bias[j] : 0.0f;
    for (int k0 = 0; k0 < K; k0 += FC_KC) {
        for (int i = threadIdx.x; i < 32 * FC_KC; i += 256) {
            const int r = i / FC_KC, kk = i - r * FC_KC;
            const int jj = blockIdx.x * 32 + r;
            s_w[r][kk] = (jj < J && k0 + kk < K) ? w[static_cast<size_t>(jj) * K + k0 + kk] : 0.0f;
        }
        for (int i = threadIdx.x; i < 8 * FC_KC; i += 256) {
            const int r = i / FC_KC, kk = i - r * FC_KC;
            const int nn = blockIdx.y * 8 + r;
            s_x[r][kk] = (nn < N && k0 + kk < K) ? x[static_cast<size_t>(nn) * K + k0 + kk] : 0.0f;
        }
        __syncthreads();
        const int kn = K - k0 < FC_KC ? K - k0 : FC_KC;
        for (int kk = 0; kk < kn; ++kk) acc = fmaf(s_x[nl][kk], s_w[jl][kk], acc);
        __syncthreads();
    }
    if (j < J && n < N) out[static_cast<size_t>(n) * J + j] = acc;
}

template <int S, int STRIDE>
static int launch_conv_tiled(const ConvF32Args& g, size_t smem, cudaStream_t st)
{
    auto kern = conv2d_f32_tiled_kernel<S, STRIDE>;
    if (smem > 48 * 1024 && cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)) != cudaSuccess) {
        cudaGetLastError();
        return BS_ERR_CUDA;
    }
    const long long tiles = static_cast<long long>(g.N) * g.tiles_p * g.tiles_q;
    if (tiles > 0x7fffffffLL || g.tiles_o > 65535) return BS_ERR_UNSUPPORTED;
    int sms = device_sm_count();
    if (sms <= 0) return BS_ERR_CUDA;
    long long per_o = static_cast<long long>(sms) * 2 / g.tiles_o;         // two CTAs per SM (registers), persistent over the tiles
    if (per_o < 1) per_o = 1;
    if (per_o > tiles) per_o = tiles;
    kern<<<dim3(static_cast<unsigned>(per_o), static_cast<unsigned>(g.tiles_o)), F32_THREADS, smem, st>>>(g);
    return cudaGetLastError() == cudaSuccess ? BS_OK : BS_ERR_CUDA;
}

}  // namespace bs

extern "C" int bs_conv2d_f32(const float* x, const float* w, const float* bias, int N, int C, int H, int W, int O, int R, int S, int stride,
                             int pad, int relu, float* out, void* stream)
{
    if (!x || !w || !out || N <= 0 || C <= 0 || H <= 0 || W <= 0 || O <= 0 || R <= 0 || S <= 0 || stride < 1 || pad < 0) return BS_ERR_INVALID_ARG;
    if (H + 2 * pad < R || W + 2 * pad < S) return BS_ERR_INVALID_ARG;
    if (!bs::aligned16(x) || !bs::aligned16(w) || !bs::aligned16(out) || (bias && (reinterpret_cast<uintptr_t>(bias) & 3u))) return BS_ERR_ALIGNMENT;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    bs::ConvF32Args g{};
    g.x = x; g.w = w; g.bias = bias; g.out = out;
    g.N = N; g.C = C; g.H = H; g.W = W; g.O = O; g.R = R; g.stride = stride; g.pad = pad; g.relu = relu;
    g.P = (H + 2 * pad - R) / stride + 1;
    g.Q = (W + 2 * pad - S) / stride + 1;
    const bool tiled = (S == 7 && stride == 2) || (S == 3 && stride == 1) || (S == 3 && stride == 2) || (S == 1 && stride == 1);
    if (tiled) {
        g.in_h = (bs::F32_TH - 1) * stride + R;
        g.in_w = (bs::F32_TW - 1) * stride + S;
        // every strip reads whole 16-byte vectors: the last one may run a few floats past the halo
        const int win4 = ((bs::F32_STRIP - 1) * stride + S + 3) / 4 * 4;
        const int need = (bs::F32_TW / bs::F32_STRIP - 1) * bs::F32_STRIP * stride + win4;
        g.pitch = ((need > g.in_w ? need : g.in_w) + 3) / 4 * 4;
        g.tiles_p = bs::ceil_div(g.P, bs::F32_TH); g.tiles_q = bs::ceil_div(g.Q, bs::F32_TW); g.tiles_o = bs::ceil_div(O, bs::F32_OT);
        const size_t smem = (static_cast<size_t>(C) * R * S * bs::F32_OT + 2 * static_cast<size_t>(C) * g.in_h * g.pitch) * 4;
        if (smem <= 200 * 1024) {
            if (S == 7) return bs::launch_conv_tiled<7, 2>(g, smem, st);
            if (S == 3 && stride == 1) return bs::launch_conv_tiled<3, 1>(g, smem, st);
            if (S == 3) return bs::launch_conv_tiled<3, 2>(g, smem, st);
            return bs::launch_conv_tiled<1, 1>(g, smem, st);
        }
    }
    const long long total = static_cast<long long>(N) * O * g.P * g.Q;
    long long blocks = (total + 255) / 256;
    if (blocks > 148 * 32) blocks = 148 * 32;
    bs::conv2d_f32_direct_kernel<<<static_cast<unsigned>(blocks), 256, 0, st>>>(x, w, bias, out, N, C, H, W, O, R, S, stride, pad, relu, g.P, g.Q);
    return cudaGetLastError() == cudaSuccess ? BS_OK : BS_ERR_CUDA;
}

extern "C" int bs_maxpool2d_f32(const float* x, int N, int C, int H, int W, int k, int stride, int pad, float* out, void* stream)
{
    if (!x || !out || N <= 0 || C <= 0 || H <= 0 || W <= 0 || k <= 0 || stride < 1 || pad < 0 || 2 * pad > k) return BS_ERR_INVALID_ARG;
    if (H + 2 * pad < k || W + 2 * pad < k) return BS_ERR_INVALID_ARG;
    const int P = (H + 2 * pad - k) / stride + 1, Q = (W + 2 * pad - k) / stride + 1;
    const long long planes = static_cast<long long>(N) * C, total = planes * P * Q;
    if (k == 3 && stride == 2 && pad == 1 && W % 8 == 0 && Q * 2 == W && bs::aligned16(x) && bs::aligned16(out)) {
        long long blocks4 = (total / 4 + 255) / 256;
        if (blocks4 > 148 * 64) blocks4 = 148 * 64;
        bs::maxpool3x3s2p1_f32_kernel<<<static_cast<unsigned>(blocks4), 256, 0, static_cast<cudaStream_t>(stream)>>>(x, out, planes, H, W, P, Q);
        return cudaGetLastError() == cudaSuccess ? BS_OK : BS_ERR_CUDA;
    }
    long long blocks = (total + 255) / 256;
    if (blocks > 148 * 64) blocks = 148 * 64;
    bs::maxpool2d_f32_kernel<<<static_cast<unsigned>(blocks), 256, 0, static_cast<cudaStream_t>(stream)>>>(x, out, planes, H, W, k, stride, pad, P, Q);
    return cudaGetLastError() == cudaSuccess ? BS_OK : BS_ERR_CUDA;
}

extern "C" int bs_avgpool_codes_f32(const uint32_t* packed, int N, int C, int H, int W, int a_bits, bs_sign_t a_sign, float inv, float* out,
                                    void* stream)
{
    if (!packed || !out || N <= 0 || C <= 0 || H <= 0 || W <= 0 || !bs::bits_ok(a_bits, a_sign)) return BS_ERR_INVALID_ARG;
    if (static_cast<long long>(N) * C > 0x7fffffffLL || static_cast<long long>(H) * W * ((1 << a_bits)) >= (1LL << 24)) return BS_ERR_UNSUPPORTED;
    const int total = N * C;
    bs::avgpool_codes_kernel<<<(total + 127) / 128, 128, 0, static_cast<cudaStream_t>(stream)>>>(packed, out, N, C, H * W, (C + 31) / 32, a_bits,
                                                                                                 a_sign, inv);
    return cudaGetLastError() == cudaSuccess ? BS_OK : BS_ERR_CUDA;
}

extern "C" int bs_fc_f32(const float* x, const float* w, const float* bias, int N, int K, int J, float* out, void* stream)
{
    if (!x || !w || !out || N <= 0 || K <= 0 || J <= 0) return BS_ERR_INVALID_ARG;
    const dim3 grid(static_cast<unsigned>((J + 31) / 32), static_cast<unsigned>((N + 7) / 8));
    if (grid.y > 65535) return BS_ERR_UNSUPPORTED;
    bs::fc_f32_kernel<<<grid, 256, 0, static_cast<cudaStream_t>(stream)>>>(x, w, bias, out, N, K, J);
    return cudaGetLastError() == cudaSuccess ? BS_OK : BS_ERR_CUDA;
}
