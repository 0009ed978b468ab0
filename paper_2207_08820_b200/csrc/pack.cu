// Quantise + bitplane split of activations (Section IV quantiser, Section V plane split), the inverse
// unpack, and the offline plane split of weights / matrix rows.
#include "common.cuh"

namespace bs {

constexpr int PACK_THREADS = 256;
constexpr int CODE_PITCH_PAD = 4;   // bytes added to each code row so that byte reads by 32 lanes hit 32 banks

template <typename T> struct In4;
template <> struct In4<float> { using type = float4; };
template <> struct In4<int8_t> { using type = char4; };

template <typename T>
__device__ __forceinline__ int to_code(T v, float s, int qmin, int qmax, int sign);
template <>
__device__ __forceinline__ int to_code<float>(float v, float s, int qmin, int qmax, int sign)
{
    return quantize_code(v, s, qmin, qmax, sign);
}
template <>
__device__ __forceinline__ int to_code<int8_t>(int8_t v, float, int, int, int) { return v; }

// One block packs TP consecutive pixels (flattened y*W + x) of one image, all channels.
//   NCHW: per 32-channel word, lanes read 4 consecutive pixels of one channel (coalesced, vectorised
//         when H*W % 4 == 0), quantise, park the patterns as bytes in shared memory; then one warp per
//         pixel reads lane = channel and __ballot_sync gives one word per plane.
//   NHWC: lane = channel directly; ballot straight from the quantised value.
// The packed pixel records of the tile are contiguous in global memory and leave through 128-bit stores.
template <typename T, bool NHWC>
__global__ void __launch_bounds__(PACK_THREADS)
bitpack_kernel(const T* __restrict__ x, uint32_t* __restrict__ out, int C, int HW, int Cw, int bits, int sign,
               float s, int TP)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    uint32_t* out_s = reinterpret_cast<uint32_t*>(smem_raw);                     // [TP][Cw][bits]
    const int rec = Cw * bits;
    unsigned char* codes_s = smem_raw + static_cast<size_t>(TP) * rec * 4;       // [32][TP + pad] (NCHW only)
    const int pitch = TP + CODE_PITCH_PAD;

    const int n = blockIdx.y;
    const int hw0 = blockIdx.x * TP;
    const int npix = min(TP, HW - hw0);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    constexpr int NWARP = PACK_THREADS / 32;
    int qmin, qmax;
    code_limits(bits, sign, qmin, qmax);

    if (NHWC) {
        const T* xin = x + (static_cast<size_t>(n) * HW + hw0) * C;
        for (int cw = 0; cw < Cw; ++cw) {
            const int c = cw * 32 + lane;
            const bool cvalid = c < C;
            for (int px0 = warp; px0 < TP; px0 += NWARP * 4) {
                T v[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int px = px0 + u * NWARP;
                    v[u] = (cvalid && px < npix) ? xin[static_cast<size_t>(px) * C + c] : T(0);
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int px = px0 + u * NWARP;
                    unsigned pat = 0;
                    if (cvalid && px < npix) pat = stored_pattern(to_code<T>(v[u], s, qmin, qmax, sign), bits, sign);
                    for (int j = 0; j < bits; ++j) {
                        const unsigned word = __ballot_sync(0xffffffffu, (pat >> j) & 1u);
                        if (lane == j && px < TP) out_s[(px * Cw + cw) * bits + j] = word;
                    }
                }
            }
        }
    } else {
        const bool vec = (HW % 4 == 0);
        // Each thread owns up to 4 items (channel cl, 4 consecutive pixels) per 32-channel word.  The loads of
        // word cw + 1 are issued before the ballot phase of word cw so that global reads stay in flight.
        constexpr int MAXI = 4;                       // TP <= 128  =>  32 * (TP / 4) / PACK_THREADS <= 4
        const int q4n = TP / 4;
        T v[MAXI][4];
        auto load_items = [&](int cw) {
#pragma unroll
            for (int it = 0; it < MAXI; ++it) {
                const int item = threadIdx.x + it * PACK_THREADS;
                const int cl = item / q4n, px = (item % q4n) * 4;
                const int c = cw * 32 + cl;
#pragma unroll
                for (int u = 0; u < 4; ++u) v[it][u] = T(0);
                if (item < 32 * q4n && c < C && px < npix) {
                    const T* src = x + (static_cast<size_t>(n) * C + c) * HW + hw0 + px;
                    if (vec) {   // npix is a multiple of 4 here, so all four are inside the image
                        typename In4<T>::type q = *reinterpret_cast<const typename In4<T>::type*>(src);
                        v[it][0] = q.x; v[it][1] = q.y; v[it][2] = q.z; v[it][3] = q.w;
                    } else {
#pragma unroll
                        for (int u = 0; u < 4; ++u)
                            if (px + u < npix) v[it][u] = src[u];
                    }
                }
            }
        };
        load_items(0);
        for (int cw = 0; cw < Cw; ++cw) {
            // phase 1: 32 channels x TP pixels -> byte patterns
#pragma unroll
            for (int it = 0; it < MAXI; ++it) {
                const int item = threadIdx.x + it * PACK_THREADS;
                if (item >= 32 * q4n) continue;
                const int cl = item / q4n, px = (item % q4n) * 4;
                const int c = cw * 32 + cl;
                unsigned packed4 = 0;
                if (c < C) {
#pragma unroll
                    for (int u = 0; u < 4; ++u)
                        if (px + u < npix)
                            packed4 |= stored_pattern(to_code<T>(v[it][u], s, qmin, qmax, sign), bits, sign) << (8 * u);
                }
                *reinterpret_cast<unsigned*>(codes_s + cl * pitch + px) = packed4;
            }
            if (cw + 1 < Cw) load_items(cw + 1);
            __syncthreads();
            // phase 2: one warp per pixel, lane = channel, one ballot per plane
            for (int px = warp; px < TP; px += NWARP) {
                const unsigned pat = codes_s[lane * pitch + px];
                for (int j = 0; j < bits; ++j) {
                    const unsigned word = __ballot_sync(0xffffffffu, (pat >> j) & 1u);
                    if (lane == j) out_s[(px * Cw + cw) * bits + j] = word;
                }
            }
            __syncthreads();
        }
    }
    __syncthreads();
    // write-out: npix * rec contiguous words; the tile start is 16-byte aligned when TP*rec % 4 == 0
    uint32_t* dst = out + (static_cast<size_t>(n) * HW + hw0) * rec;
    const int nwords = npix * rec;
    if ((static_cast<size_t>(HW) * rec) % 4 == 0 && (static_cast<size_t>(TP) * rec) % 4 == 0) {
        const int nvec = nwords / 4;
        for (int k = threadIdx.x; k < nvec; k += PACK_THREADS)
            reinterpret_cast<uint4*>(dst)[k] = reinterpret_cast<const uint4*>(out_s)[k];
        for (int k = nvec * 4 + threadIdx.x; k < nwords; k += PACK_THREADS) dst[k] = out_s[k];
    } else {
        for (int k = threadIdx.x; k < nwords; k += PACK_THREADS) dst[k] = out_s[k];
    }
}

__global__ void bitunpack_kernel(const uint32_t* __restrict__ packed, int8_t* __restrict__ codes, long long total,
                                 int C, int HW, int Cw, int bits, int sign, int nhwc)
{
    const long long idx = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (idx >= total) return;
    // idx enumerates the OUTPUT layout
    long long n, c, hw;
    if (nhwc) { c = idx % C; hw = (idx / C) % HW; n = idx / (static_cast<long long>(C) * HW); }
    else      { hw = idx % HW; c = (idx / HW) % C; n = idx / (static_cast<long long>(C) * HW); }
    const uint32_t* rec = packed + ((n * HW + hw) * Cw + c / 32) * bits;
    unsigned pat = 0;
    for (int j = 0; j < bits; ++j) pat |= ((rec[j] >> (c % 32)) & 1u) << j;
    codes[idx] = static_cast<int8_t>(pattern_value(pat, bits, sign));
}

// One thread per packed word group (o, tap, cw): reads 32 channel codes, emits `bits` plane words.
__global__ void pack_weights_kernel(const int8_t* __restrict__ w, uint32_t* __restrict__ out, long long ngroups,
                                    int C, int RS, int Cw, int bits, int sign, int ohwi)
{
    const long long g = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (g >= ngroups) return;
    const int cw = static_cast<int>(g % Cw);
    const int tap = static_cast<int>((g / Cw) % RS);
    const long long o = g / (static_cast<long long>(Cw) * RS);
    unsigned words[4] = {0, 0, 0, 0};
    for (int b = 0; b < 32; ++b) {
        const int c = cw * 32 + b;
        if (c >= C) break;
        const long long src = ohwi ? ((o * RS + tap) * C + c) : ((o * C + c) * RS + tap);
        const unsigned pat = stored_pattern(w[src], bits, sign);
#pragma unroll
        for (int i = 0; i < 4; ++i) words[i] |= ((pat >> i) & 1u) << b;
    }
#pragma unroll
    for (int i = 0; i < 4; ++i)
        if (i < bits) out[g * bits + i] = words[i];
}

}  // namespace bs

using namespace bs;

extern "C" size_t bs_packed_act_bytes(int N, int C, int H, int W, int a_bits)
{
    if (N <= 0 || C <= 0 || H <= 0 || W <= 0 || a_bits < 1 || a_bits > 4) return 0;
    return static_cast<size_t>(N) * H * W * ceil_div(C, 32) * a_bits * sizeof(uint32_t);
}

extern "C" size_t bs_packed_wgt_bytes(int O, int C, int R, int S, int w_bits)
{
    if (O <= 0 || C <= 0 || R <= 0 || S <= 0 || w_bits < 1 || w_bits > 4) return 0;
    return static_cast<size_t>(O) * R * S * ceil_div(C, 32) * w_bits * sizeof(uint32_t);
}

extern "C" size_t bs_packed_rows_bytes(int rows, int K, int bits)
{
    if (rows <= 0 || K <= 0 || bits < 1 || bits > 4) return 0;
    return static_cast<size_t>(rows) * ceil_div(K, 32) * bits * sizeof(uint32_t);
}

template <typename T, bool NHWC>
static int launch_bitpack(const void* x, uint32_t* out, int N, int C, int HW, int bits, int sign, float s,
                          cudaStream_t st)
{
    const int Cw = ceil_div(C, 32);
    const int rec = Cw * bits;
    int TP = 128;
    auto smem_for = [&](int tp) { return static_cast<size_t>(tp) * rec * 4 + (NHWC ? 0 : 32 * (tp + CODE_PITCH_PAD)); };
    if (smem_for(TP) > 64 * 1024) TP = 32;
    const size_t smem = smem_for(TP);
    if (smem > 200 * 1024) return BS_ERR_UNSUPPORTED;
    auto kern = bitpack_kernel<T, NHWC>;
    if (smem > 48 * 1024 &&
        cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)) != cudaSuccess)
        return BS_ERR_CUDA;
    dim3 grid(ceil_div(HW, TP), N);
    kern<<<grid, PACK_THREADS, smem, st>>>(static_cast<const T*>(x), out, C, HW, Cw, bits, sign, s, TP);
    return cudaGetLastError() == cudaSuccess ? BS_OK : BS_ERR_CUDA;
}

extern "C" int bitpack_activations(const void* x, int x_is_fp32, bs_layout_t layout, int N, int C, int H, int W,
                                   float act_scale, int a_bits, bs_sign_t a_sign, uint32_t* packed_out, void* stream)
{
    if (!x || !packed_out || N <= 0 || C <= 0 || H <= 0 || W <= 0) return BS_ERR_INVALID_ARG;
    if (!bits_ok(a_bits, a_sign) || (layout != BS_NCHW && layout != BS_NHWC)) return BS_ERR_INVALID_ARG;
    if (x_is_fp32 && !(act_scale > 0.0f && act_scale < 3.0e38f)) return BS_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(packed_out)) return BS_ERR_ALIGNMENT;
    if (static_cast<long long>(H) * W > 0x7fffffffLL || N > 65535) return BS_ERR_UNSUPPORTED;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int HW = H * W;
    if (x_is_fp32)
        return layout == BS_NHWC ? launch_bitpack<float, true>(x, packed_out, N, C, HW, a_bits, a_sign, act_scale, st)
                                 : launch_bitpack<float, false>(x, packed_out, N, C, HW, a_bits, a_sign, act_scale, st);
    return layout == BS_NHWC ? launch_bitpack<int8_t, true>(x, packed_out, N, C, HW, a_bits, a_sign, 1.0f, st)
                             : launch_bitpack<int8_t, false>(x, packed_out, N, C, HW, a_bits, a_sign, 1.0f, st);
}

extern "C" int bitunpack_activations(const uint32_t* packed, int N, int C, int H, int W, int a_bits, bs_sign_t a_sign,
                                     bs_layout_t layout, int8_t* codes_out, void* stream)
{
    if (!packed || !codes_out || N <= 0 || C <= 0 || H <= 0 || W <= 0) return BS_ERR_INVALID_ARG;
    if (!bits_ok(a_bits, a_sign) || (layout != BS_NCHW && layout != BS_NHWC)) return BS_ERR_INVALID_ARG;
    if (!aligned16(packed) || !aligned16(codes_out)) return BS_ERR_ALIGNMENT;
    const long long total = static_cast<long long>(N) * C * H * W;
    const long long blocks = ceil_div_ll(total, 256);
    if (blocks > 0x7fffffffLL) return BS_ERR_UNSUPPORTED;
    bitunpack_kernel<<<static_cast<unsigned>(blocks), 256, 0, static_cast<cudaStream_t>(stream)>>>(
        packed, codes_out, total, C, H * W, ceil_div(C, 32), a_bits, a_sign, layout == BS_NHWC);
    return cudaGetLastError() == cudaSuccess ? BS_OK : BS_ERR_CUDA;
}

static int launch_pack_weights(const int8_t* w, int ohwi, long long O, int C, int RS, int bits, int sign,
                               uint32_t* out, cudaStream_t st)
{
    const int Cw = ceil_div(C, 32);
    const long long ngroups = O * RS * Cw;
    const long long blocks = ceil_div_ll(ngroups, 128);
    if (blocks > 0x7fffffffLL) return BS_ERR_UNSUPPORTED;
    pack_weights_kernel<<<static_cast<unsigned>(blocks), 128, 0, st>>>(w, out, ngroups, C, RS, Cw, bits, sign, ohwi);
    return cudaGetLastError() == cudaSuccess ? BS_OK : BS_ERR_CUDA;
}

extern "C" int pack_weights(const int8_t* w_codes, bs_layout_t layout, int O, int C, int R, int S, int w_bits,
                            bs_sign_t w_sign, uint32_t* packed_out, void* stream)
{
    if (!w_codes || !packed_out || O <= 0 || C <= 0 || R <= 0 || S <= 0) return BS_ERR_INVALID_ARG;
    if (!bits_ok(w_bits, w_sign) || (layout != BS_NCHW && layout != BS_NHWC)) return BS_ERR_INVALID_ARG;
    if (!aligned16(w_codes) || !aligned16(packed_out)) return BS_ERR_ALIGNMENT;
    return launch_pack_weights(w_codes, layout == BS_NHWC, O, C, R * S, w_bits, w_sign, packed_out,
                               static_cast<cudaStream_t>(stream));
}

extern "C" int bs_pack_rows(const int8_t* codes, int rows, int K, int bits, bs_sign_t sign, uint32_t* packed_out,
                            void* stream)
{
    if (!codes || !packed_out || rows <= 0 || K <= 0) return BS_ERR_INVALID_ARG;
    if (!bits_ok(bits, sign)) return BS_ERR_INVALID_ARG;
    if (!aligned16(codes) || !aligned16(packed_out)) return BS_ERR_ALIGNMENT;
    return launch_pack_weights(codes, 1, rows, K, 1, bits, sign, packed_out, static_cast<cudaStream_t>(stream));
}
