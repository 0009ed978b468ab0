// Quantise + bitplane split of activations (Section IV quantiser, Section V plane split), the inverse
// unpack, and the offline plane split of weights / matrix rows.
#include <cmath>
#include <cstring>

#include "common.cuh"

namespace bs {

constexpr int PACK_THREADS = 256;
constexpr int PACK_WARPS = PACK_THREADS / 32;
constexpr int PACK_UNROLL = 8;      // NHWC: pixels in flight per warp

// Quantiser of Section IV prepared for the device.  The decision
//     code = round_half_even(clip(x / s, qmin, qmax))
// is monotone in x, so it equals qmin + #{k : x >= bound[k]} where bound[k] is the smallest binary32 value whose
// code is >= qmin + k + 1.  The host finds those bounds by bisection over the ordered float bit patterns using the very
// same IEEE division, clip and rint, so the comparison form takes exactly the decision of the formula while costing
// a few subtractions instead of a division (a binary search over the bounds for 3 and 4 bits).
struct QuantParams {
    float below[15];    // largest binary32 value below bound[k] (never -0): x >= bound[k]  <=>  sign bit of (below[k] - x) is set
    int bits, sign;
};

// Stored pattern of an int8 code as plane bits (the two's-complement low bits; bipolar: bit 0 = code > 0).
template <int BITS>
__device__ __forceinline__ unsigned code_pattern(int8_t x, int sign)
{
    if (sign == BS_BIPOLAR) return x > 0 ? 1u : 0u;
    return static_cast<unsigned>(static_cast<int>(x)) & ((1u << BITS) - 1u);
}

// A warp copies the contiguous packed records of its tile from shared to global memory, as 128-bit stores when the
// tile starts on a 16-byte boundary.
__device__ __forceinline__ void store_tile_records(const uint32_t* stage, uint32_t* dst, int nwords, bool vec, int lane)
{
    if (vec) {
        const int nvec = nwords / 4;
        for (int k = lane; k < nvec; k += 32) reinterpret_cast<uint4*>(dst)[k] = reinterpret_cast<const uint4*>(stage)[k];
        for (int k = nvec * 4 + lane; k < nwords; k += 32) dst[k] = stage[k];
    } else {
        for (int k = lane; k < nwords; k += 32) dst[k] = stage[k];
    }
}

// Fallback for int8 codes in shapes the vector kernels below refuse (H*W not a multiple of 4 in NCHW, C not a multiple
// of 32 in NHWC, bipolar codes).  One warp packs 32 consecutive pixels (flattened y*W + x) of one image, all channels,
// with no block-wide barrier.
//   NCHW: lane = pixel.  Every channel row is read with one coalesced request per warp, a whole 32-channel word in
//         flight; each lane sets bit c of its own plane words from the pattern of channel c.
//   NHWC: lane = channel.  One coalesced request per (pixel, 32-channel word); __ballot_sync over the 32 channels
//         yields one plane word per vote.
// The packed records of the 32 pixels are contiguous in global memory; they are parked in the warp's slice of
// shared memory and leave through coalesced 128-bit stores.
template <bool NHWC, int BITS>
__global__ void __launch_bounds__(PACK_THREADS)
bitpack_codes_kernel(const int8_t* __restrict__ x, uint32_t* __restrict__ out, int C, int HW, int Cw, long long ntiles,
                     int tiles_per_img, int sign)
{
    extern __shared__ __align__(16) uint32_t pack_smem[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const long long tile = static_cast<long long>(blockIdx.x) * PACK_WARPS + warp;
    if (tile >= ntiles) return;                       // whole warps leave; only __syncwarp is used below
    const int rec = Cw * BITS;
    uint32_t* stage = pack_smem + static_cast<size_t>(warp) * 32 * rec;      // [32 pixels][rec]
    const long long n = tile / tiles_per_img;
    const int hw0 = static_cast<int>(tile % tiles_per_img) * 32;
    const int npix = min(32, HW - hw0);

    if (NHWC) {
        const int8_t* xin = x + (static_cast<size_t>(n) * HW + hw0) * C;
        for (int cw = 0; cw < Cw; ++cw) {
            const int c = cw * 32 + lane;
            const bool cvalid = c < C;
            for (int p0 = 0; p0 < 32; p0 += PACK_UNROLL) {
                unsigned pat[PACK_UNROLL];
#pragma unroll
                for (int u = 0; u < PACK_UNROLL; ++u)
                    pat[u] = (cvalid && p0 + u < npix) ? code_pattern<BITS>(xin[static_cast<size_t>(p0 + u) * C + c], sign) : 0u;
#pragma unroll
                for (int u = 0; u < PACK_UNROLL; ++u) {
#pragma unroll
                    for (int j = 0; j < BITS; ++j) {
                        const unsigned word = __ballot_sync(0xffffffffu, (pat[u] >> j) & 1u);
                        if (lane == j) stage[(p0 + u) * rec + cw * BITS + j] = word;
                    }
                }
            }
        }
    } else {
        const bool pvalid = lane < npix;
        const int8_t* xin = x + static_cast<size_t>(n) * C * HW + hw0 + lane;
        for (int cw = 0; cw < Cw; ++cw) {
            uint32_t words[BITS];
#pragma unroll
            for (int j = 0; j < BITS; ++j) words[j] = 0u;
            unsigned pat[32];
#pragma unroll
            for (int u = 0; u < 32; ++u) {
                const int c = cw * 32 + u;
                pat[u] = (pvalid && c < C) ? code_pattern<BITS>(xin[static_cast<size_t>(c) * HW], sign) : 0u;
            }
#pragma unroll
            for (int u = 0; u < 32; ++u)
#pragma unroll
                for (int j = 0; j < BITS; ++j) words[j] |= ((pat[u] >> j) & 1u) << u;
#pragma unroll
            for (int j = 0; j < BITS; ++j) stage[lane * rec + cw * BITS + j] = words[j];
        }
    }
    __syncwarp();
    store_tile_records(stage, out + (static_cast<size_t>(n) * HW + hw0) * rec, npix * rec,
                       (static_cast<size_t>(HW) * rec) % 4 == 0 && (32 * rec) % 4 == 0, lane);
}

// Stores the BITS plane words of one (pixel, channel word) with the widest aligned store.
template <int BITS>
__device__ __forceinline__ void store_planes(uint32_t* dst, const uint32_t (&w)[BITS])
{
    if constexpr (BITS == 4) *reinterpret_cast<uint4*>(dst) = make_uint4(w[0], w[1], w[2], w[3]);
    else if constexpr (BITS == 2) *reinterpret_cast<uint2*>(dst) = make_uint2(w[0], w[1]);
    else {
#pragma unroll
        for (int j = 0; j < BITS; ++j) dst[j] = w[j];
    }
}

// Sign-bit form of the comparison quantiser for fp32 input.
//   With p the largest binary32 value below the bound b:  x >= b  <=>  x > p  <=>  the sign bit of p - x is set.
//   An IEEE subtraction never rounds across zero and x == p gives +0; p is stored as +0 when it is a zero, so neither
//   signed zero of x yields -0.  A NaN input gives the canonical NaN (sign clear): no level reached, the lowest
//   code, which is what clip() makes of a NaN in the formula.  +-inf behave like the comparison.
//   2-bit codes: plane 1 = (x >= b1); plane 0 = parity of the three comparisons = sign((p0-x) ^ (p1-x) ^ (p2-x)).
//   3- and 4-bit codes search the 7 or 15 bounds binarily: one subtraction, one sign test and one funnel shift per bit
//   plus the selects that pick the next bound.
// One funnel shift moves a sign bit into a plane word (w = 2 w + bit); the inputs of a word are walked from position 31
// down to 0 so that input i ends at bit i.  Per element of a 2-bit tensor: one load, three subtractions, one three-input
// xor and two funnel shifts, which leaves the kernels waiting on HBM rather than on the issue slots.
// Shifts the BITS plane bits of one input into the plane words w (w = 2 w + bit), in the sign-bit comparison form.
template <int BITS>
__device__ __forceinline__ void quant_push(const QuantParams& q, float v, uint32_t (&w)[BITS])
{
    if constexpr (BITS == 1) {
        w[0] = __funnelshift_l(__float_as_uint(q.below[0] - v), w[0], 1);
    } else if constexpr (BITS == 2) {
        const uint32_t d0 = __float_as_uint(q.below[0] - v), d1 = __float_as_uint(q.below[1] - v),
                       d2 = __float_as_uint(q.below[2] - v);
        w[1] = __funnelshift_l(d1, w[1], 1);
        w[0] = __funnelshift_l(d0 ^ d1 ^ d2, w[0], 1);
    } else {
        // binary search for the count of bounds reached, top bit first: with the higher bits m decided, bit L is
        // "bound number m * 2^(L+1) + 2^L reached"; the candidates are folded with selects on the decided bits
        bool c[BITS];
#pragma unroll
        for (int L = BITS - 1; L >= 0; --L) {
            constexpr int MAXC = 1 << (BITS - 1);
            float sel[MAXC];
            const int nd = BITS - 1 - L;
#pragma unroll
            for (int m = 0; m < MAXC; ++m)
                if (m < (1 << nd)) sel[m] = q.below[m * (2 << L) + (1 << L) - 1];
#pragma unroll
            for (int d = 0; d < BITS - 1; ++d)
                if (d < nd) {
#pragma unroll
                    for (int m = 0; m < MAXC / 2; ++m)
                        if (m < (1 << (nd - d - 1))) sel[m] = c[L + 1 + d] ? sel[2 * m + 1] : sel[2 * m];
                }
            const uint32_t e = __float_as_uint(sel[0] - v);
            c[L] = static_cast<int>(e) < 0;
            w[L] = __funnelshift_l(e, w[L], 1);
        }
    }
}

// Transpose of the 32 x 32 bit matrix whose row r is the word held by lane r: afterwards lane r holds column r.  Five
// butterfly stages; stage k swaps the off-diagonal k x k blocks between lanes r and r ^ k.
__device__ __forceinline__ uint32_t warp_transpose32(uint32_t x, int lane)
{
#pragma unroll
    for (int k = 16; k >= 1; k >>= 1) {
        const uint32_t mask = k == 16 ? 0x0000FFFFu : k == 8 ? 0x00FF00FFu : k == 4 ? 0x0F0F0F0Fu : k == 2 ? 0x33333333u : 0x55555555u;
        const uint32_t y = __shfl_xor_sync(0xffffffffu, x, k);
        x = (lane & k) ? ((x & ~mask) | ((y & ~mask) >> k)) : ((x & mask) | ((y & mask) << k));
    }
    return x;
}

// fp32 NCHW.  Work unit of a warp = 32 consecutive pixels of one image x one 32-channel word (lane = pixel): all 32
// channel rows are in flight at once (32 coalesced 128-byte requests per warp), walked from channel 31 down, and each lane
// stores the BITS plane words of its pixel straight to the packed record (8-byte stores for 2-bit codes; the words of
// the other channel groups of the record come from the neighbouring warps of the block, so the sectors fill up in L2).
// Units are small and numerous, which keeps the tail of the grid short; no shared memory, no barrier.
constexpr int FAST_THREADS = 128;
constexpr int FAST_WARPS = FAST_THREADS / 32;

template <int BITS>
__global__ void __launch_bounds__(FAST_THREADS, 8)
bitpack_nchw_f32_kernel(const float* __restrict__ x, uint32_t* __restrict__ out, int C, int HW, int Cw, long long nunits,
                        int units_per_img, const QuantParams q)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const long long unit = static_cast<long long>(blockIdx.x) * FAST_WARPS + warp;
    if (unit >= nunits) return;
    const long long n = unit / units_per_img;
    const int rem = static_cast<int>(unit % units_per_img);
    const int cw = rem % Cw;
    const int hw0 = (rem / Cw) * 32;
    const bool pvalid = lane < HW - hw0;
    // lanes beyond the image re-read the first pixel of the tile (always in bounds) and store nothing
    const float* xin = x + (static_cast<size_t>(n) * C + cw * 32) * HW + hw0 + (pvalid ? lane : 0);
    uint32_t w[BITS];
#pragma unroll
    for (int j = 0; j < BITS; ++j) w[j] = 0u;
    auto push = [&](float v) { quant_push<BITS>(q, v, w); };
    const int nvalid = min(32, C - cw * 32);
    if (nvalid == 32) {
        // a full channel word: unconditional loads, walking the channel rows downward from channel 31
        const ptrdiff_t row = HW;
        const float* pc = xin + 31 * row;
        float v[32];
#pragma unroll
        for (int u = 0; u < 32; ++u) {
            v[u] = __ldcs(pc);
            pc -= row;
        }
#pragma unroll
        for (int u = 0; u < 32; ++u) push(v[u]);
    } else {
        // the ragged last word: channels past C count as "no level reached"
        for (int u = 31; u >= 0; --u) push(u < nvalid ? __ldcs(xin + static_cast<size_t>(u) * HW) : -INFINITY);
    }
    if (!pvalid) return;
    const unsigned fl = nvalid == 32 ? 0xffffffffu : ((1u << nvalid) - 1u);
    // pattern = (qmin + count) mod 2^BITS: two's-complement codes (qmin = -2^(BITS-1)) flip the top plane only
    if (q.sign == BS_SIGNED) w[BITS - 1] ^= fl;
    store_planes<BITS>(out + ((static_cast<size_t>(n) * HW + hw0 + lane) * Cw + cw) * BITS, w);
}

// fp32 NHWC input, comparison form at any width.  Work unit of a warp = 32 consecutive pixels x one 32-channel word, lane
// = channel: the 32 channels of a pixel are one coalesced 128-byte request and all 32 pixels of the unit are in flight
// at once.  A lane shifts the plane bits of its channel into words indexed by PIXEL (pixels walked from 31 down), a
// 32 x 32 bit transpose across the warp (five shuffles per plane) turns them into words indexed by channel held by lane
// = pixel, and the records leave as one store per lane like in the NCHW kernel.  No votes, no shared memory.
template <int BITS>
__global__ void __launch_bounds__(FAST_THREADS, 8)
bitpack_nhwc_f32_kernel(const float* __restrict__ x, uint32_t* __restrict__ out, int C, int HW, int Cw, long long nunits,
                        int units_per_img, const QuantParams q)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const long long unit = static_cast<long long>(blockIdx.x) * FAST_WARPS + warp;
    if (unit >= nunits) return;
    const long long n = unit / units_per_img;
    const int rem = static_cast<int>(unit % units_per_img);
    const int cw = rem % Cw;
    const int hw0 = (rem / Cw) * 32;
    const int npix = min(32, HW - hw0);
    const bool cvalid = cw * 32 + lane < C;
    const unsigned valid_word = __ballot_sync(0xffffffffu, cvalid);
    // lanes past the last channel re-read the first channel of the word (always in bounds); their words are cleared
    const float* xin = x + (static_cast<size_t>(n) * HW + hw0) * C + cw * 32 + (cvalid ? lane : 0);
    uint32_t w[BITS];
#pragma unroll
    for (int j = 0; j < BITS; ++j) w[j] = 0u;
    if (npix == 32) {
        const ptrdiff_t row = C;
        const float* pc = xin + 31 * row;
        float v[32];
#pragma unroll
        for (int u = 0; u < 32; ++u) {
            v[u] = __ldcs(pc);
            pc -= row;
        }
#pragma unroll
        for (int u = 0; u < 32; ++u) quant_push<BITS>(q, v[u], w);
    } else {
        // the ragged last tile of an image: pixels past the end count as "no level reached" and are not stored
        for (int u = 31; u >= 0; --u) quant_push<BITS>(q, u < npix ? __ldcs(xin + static_cast<size_t>(u) * C) : -INFINITY, w);
    }
#pragma unroll
    for (int j = 0; j < BITS; ++j) w[j] = warp_transpose32(cvalid ? w[j] : 0u, lane);
    if (lane >= npix) return;
    if (q.sign == BS_SIGNED) w[BITS - 1] ^= valid_word;
    store_planes<BITS>(out + ((static_cast<size_t>(n) * HW + hw0 + lane) * Cw + cw) * BITS, w);
}

// int8 codes, NCHW (unsigned or two's-complement codes: plane j is bit j of the byte).  At one byte per element the
// HBM roofline leaves about five thread instructions per element, so the plane split works on four pixels at a time:
// a lane owns four consecutive pixels and reads them as one 32-bit word per channel row (a warp = 128 pixels, 128-byte
// requests); (r >> j) & 0x01010101 is bit j of the four codes, and a = 2 a + that, over eight channel rows from the
// highest down, leaves in byte k of a the eight channel bits of pixel k.  A byte permute drops each finished byte into
// the plane word of its pixel.  About 1.8 instructions per element for 2-bit codes.  Needs H*W to be a multiple of 4
// (aligned 32-bit loads); work unit of a warp = 128 pixels x one 32-channel word.
// Stores: with CW = 0 every lane writes the plane words of its pixels straight to the records (8-byte pieces of 32-byte
// sectors, four partial writes per sector).  When the channel words of a record number CW = 1, 2 or 4, the four warps of
// a block hold complete records of 4 / CW tiles: they park their words in shared memory as [warp][plane][pixel] (128-bit
// stores, no bank conflicts), and after one barrier the block writes the records as whole 128-bit pieces.
template <int BITS, int CW>
__global__ void __launch_bounds__(FAST_THREADS, 8)
bitpack_nchw_i8_kernel(const int8_t* __restrict__ x, uint32_t* __restrict__ out, int C, int HW, int Cw, long long nunits,
                       int units_per_img)
{
    constexpr bool STAGED = CW != 0;
    __shared__ __align__(16) uint32_t stage[STAGED ? FAST_WARPS * BITS * 128 : 4];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const long long unit = static_cast<long long>(blockIdx.x) * FAST_WARPS + warp;
    const bool active = unit < nunits;
    if (!STAGED && !active) return;
    if (active) {
        const long long n = unit / units_per_img;
        const int rem = static_cast<int>(unit % units_per_img);
        const int cw = rem % Cw;
        const int hw0 = (rem / Cw) * 128;
        const int pix = hw0 + 4 * lane;
        const bool pvalid = pix < HW;      // H*W is a multiple of 4: the four pixels of a lane are inside or outside together
        const uint32_t* xin = reinterpret_cast<const uint32_t*>(x + (static_cast<size_t>(n) * C + cw * 32) * HW + (pvalid ? pix : hw0));
        const int nvalid = min(32, C - cw * 32);
        const size_t row = static_cast<size_t>(HW / 4);
        uint32_t v[32];
        if (nvalid == 32) {
#pragma unroll
            for (int u = 0; u < 32; ++u) v[u] = __ldcs(xin + u * row);
        } else {
#pragma unroll
            for (int u = 0; u < 32; ++u) v[u] = u < nvalid ? __ldcs(xin + u * row) : 0u;
        }
        uint32_t w[4][BITS];
#pragma unroll
        for (int k = 0; k < 4; ++k)
#pragma unroll
            for (int j = 0; j < BITS; ++j) w[k][j] = 0u;
#pragma unroll
        for (int g = 0; g < 4; ++g) {
            uint32_t a[BITS];
#pragma unroll
            for (int j = 0; j < BITS; ++j) a[j] = 0u;
#pragma unroll
            for (int i = 7; i >= 0; --i) {
                const uint32_t r = v[8 * g + i];
#pragma unroll
                for (int j = 0; j < BITS; ++j) a[j] = a[j] * 2u + ((r >> j) & 0x01010101u);
            }
#pragma unroll
            for (int k = 0; k < 4; ++k)
#pragma unroll
                for (int j = 0; j < BITS; ++j)      // byte k of a[j] becomes byte g of the plane word of pixel k
                    w[k][j] = __byte_perm(w[k][j], a[j], (0x3210u & ~(0xfu << (4 * g))) | ((4u + k) << (4 * g)));
        }
        if constexpr (STAGED) {
#pragma unroll
            for (int j = 0; j < BITS; ++j)
                *reinterpret_cast<uint4*>(stage + (warp * BITS + j) * 128 + 4 * lane) = make_uint4(w[0][j], w[1][j], w[2][j], w[3][j]);
        } else {
            if (!pvalid) return;
#pragma unroll
            for (int k = 0; k < 4; ++k)
                store_planes<BITS>(out + ((static_cast<size_t>(n) * HW + pix + k) * Cw + cw) * BITS, w[k]);
        }
    }
    if constexpr (STAGED) {
        __syncthreads();
        // the block's first unit is a multiple of 4, hence of CW: warp t * CW + c holds channel word c of the block's tile t
        constexpr int REC = CW * BITS;                 // words of a pixel record
        constexpr int PIECE = REC % 4 == 0 ? 4 : (REC % 2 == 0 ? 2 : 1);     // words per store
#pragma unroll
        for (int t = 0; t < FAST_WARPS / CW; ++t) {
            const long long unit_t = static_cast<long long>(blockIdx.x) * FAST_WARPS + t * CW;
            if (unit_t >= nunits) break;
            const long long n = unit_t / units_per_img;
            const int hw0 = (static_cast<int>(unit_t % units_per_img) / CW) * 128;
            const int nwords = min(128, HW - hw0) * REC;            // a multiple of 4: H*W and the tile start are
            uint32_t* dst = out + (static_cast<size_t>(n) * HW + hw0) * REC;
            for (int i = threadIdx.x * PIECE; i < nwords; i += FAST_THREADS * PIECE) {
                uint32_t piece[PIECE];
#pragma unroll
                for (int e = 0; e < PIECE; ++e) {
                    const int idx = i + e, p = idx / REC, r = idx % REC;          // (pixel, word of its record)
                    piece[e] = stage[((t * CW + r / BITS) * BITS + r % BITS) * 128 + p];
                }
                if constexpr (PIECE == 4) *reinterpret_cast<uint4*>(dst + i) = make_uint4(piece[0], piece[1], piece[2], piece[3]);
                else if constexpr (PIECE == 2) *reinterpret_cast<uint2*>(dst + i) = make_uint2(piece[0], piece[1]);
                else dst[i] = piece[0];
            }
        }
    }
}

// int8 codes, NHWC, C a multiple of 32: the 32 channels of a (pixel, channel word) are 32 contiguous, aligned bytes.
// Lane = pixel; a warp takes 128 pixels x one channel word (four pixels per lane, eight 128-bit loads in flight).  For
// each word of four codes, ((q >> j) & 0x01010101) * 0x01020408 gathers bit j of the four bytes in bits 24..27 (all
// partial products fall on distinct bits, so nothing carries).  About 2.5 instructions per element for 2-bit codes.
template <int BITS>
__global__ void __launch_bounds__(FAST_THREADS, 8)
bitpack_nhwc_i8_kernel(const int8_t* __restrict__ x, uint32_t* __restrict__ out, int C, int HW, int Cw, long long nunits,
                       int units_per_img)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const long long unit = static_cast<long long>(blockIdx.x) * FAST_WARPS + warp;
    if (unit >= nunits) return;
    const long long n = unit / units_per_img;
    const int rem = static_cast<int>(unit % units_per_img);
    const int cw = rem % Cw;
    const int hw0 = (rem / Cw) * 128;
    uint4 q[4][2];
#pragma unroll
    for (int t = 0; t < 4; ++t) {
        const int pix = min(hw0 + 32 * t + lane, HW - 1);       // clamped: always in bounds, stored only when inside
        const uint4* src = reinterpret_cast<const uint4*>(x + (static_cast<size_t>(n) * HW + pix) * C + cw * 32);
        q[t][0] = __ldcs(src);
        q[t][1] = __ldcs(src + 1);
    }
#pragma unroll
    for (int t = 0; t < 4; ++t) {
        const uint32_t words[8] = {q[t][0].x, q[t][0].y, q[t][0].z, q[t][0].w, q[t][1].x, q[t][1].y, q[t][1].z, q[t][1].w};
        uint32_t w[BITS];
#pragma unroll
        for (int j = 0; j < BITS; ++j) w[j] = 0u;
#pragma unroll
        for (int i = 0; i < 8; ++i)
#pragma unroll
            for (int j = 0; j < BITS; ++j)
                w[j] |= ((((words[i] >> j) & 0x01010101u) * 0x01020408u) >> 24) << (4 * i);
        const int pix = hw0 + 32 * t + lane;
        if (pix < HW) store_planes<BITS>(out + ((static_cast<size_t>(n) * HW + pix) * Cw + cw) * BITS, w);
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

// Host copy of the Section IV quantiser (IEEE binary32 division, clip, round-half-even) used to derive the bounds.
static int host_quantize(float x, float s, int qmin, int qmax)
{
    volatile float t = x / s;
    float c = fminf(fmaxf(t, static_cast<float>(qmin)), static_cast<float>(qmax));
    return static_cast<int>(nearbyintf(c));
}

// Ordered integer key of a float (monotone in the float order) and back.
static uint32_t float_key(float f)
{
    uint32_t u;
    memcpy(&u, &f, 4);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
static float key_float(uint32_t k)
{
    uint32_t u = (k & 0x80000000u) ? (k & 0x7fffffffu) : ~k;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

// Comparison-form quantiser for scale s: below[k] = the binary32 value just under bound[k], the smallest input whose code
// is >= qmin + k + 1 (bounds are never -inf: -inf always quantises to the lowest code; unreachable levels get +inf).
// bound[k], k = 0 .. 14: smallest binary32 input whose code is >= qmin + k + 1; +inf for levels that do not exist.
static void quantiser_bounds(float s, int bits, int sign, float (&bound)[15])
{
    int qmin, qmax;
    code_limits(bits, sign, qmin, qmax);
    for (int k = 0; k < 15; ++k) bound[k] = INFINITY;
    if (sign == BS_BIPOLAR) {                 // +1 iff x >= 0
        bound[0] = 0.0f;
        return;
    }
    const uint32_t lo_key = float_key(-INFINITY), hi_key = float_key(INFINITY);
    for (int k = 1; k <= qmax - qmin; ++k) {
        // smallest x (in float order) with code >= qmin + k; the code is monotone in x and reaches qmax at +inf
        uint32_t lo = lo_key, hi = hi_key;
        while (lo < hi) {
            const uint32_t mid = lo + (hi - lo) / 2;
            if (host_quantize(key_float(mid), s, qmin, qmax) >= qmin + k) hi = mid;
            else lo = mid + 1;
        }
        bound[k - 1] = key_float(lo);
    }
}

static QuantParams make_quant_params(float s, int bits, int sign)
{
    QuantParams q{};
    q.bits = bits; q.sign = sign;
    float bound[15];
    quantiser_bounds(s, bits, sign, bound);
    for (int k = 0; k < 15; ++k) {
        float p = bound[k] == 0.0f ? -1.401298464e-45f : key_float(float_key(bound[k]) - 1u);
        if (p == 0.0f) p = fabsf(p);          // drops the sign of a zero
        q.below[k] = p;
    }
    return q;
}

extern "C" int bs_quantiser_bounds(float act_scale, int a_bits, bs_sign_t a_sign, float* bounds_out)
{
    if (!bounds_out || !bits_ok(a_bits, a_sign) || !(act_scale > 0.0f && act_scale < 3.0e38f)) return BS_ERR_INVALID_ARG;
    float bound[15];
    quantiser_bounds(act_scale, a_bits, a_sign, bound);
    const int n = a_sign == BS_BIPOLAR ? 1 : (1 << a_bits) - 1;
    for (int k = 0; k < n; ++k) bounds_out[k] = bound[k];
    return BS_OK;
}

template <bool NHWC, int BITS>
static int launch_bitpack_codes(const void* x, uint32_t* out, int N, int C, int HW, int sign, cudaStream_t st)
{
    const int Cw = ceil_div(C, 32);
    const size_t smem = static_cast<size_t>(PACK_WARPS) * 32 * Cw * BITS * 4;
    if (smem > 200 * 1024) return BS_ERR_UNSUPPORTED;
    auto kern = bitpack_codes_kernel<NHWC, BITS>;
    if (smem > 48 * 1024 &&
        cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)) != cudaSuccess)
        return BS_ERR_CUDA;
    const int tiles_per_img = ceil_div(HW, 32);
    const long long ntiles = static_cast<long long>(N) * tiles_per_img;
    const long long blocks = ceil_div_ll(ntiles, PACK_WARPS);
    if (blocks > 0x7fffffffLL) return BS_ERR_UNSUPPORTED;
    kern<<<static_cast<unsigned>(blocks), PACK_THREADS, smem, st>>>(static_cast<const int8_t*>(x), out, C, HW, Cw, ntiles,
                                                                  tiles_per_img, sign);
    return cudaGetLastError() == cudaSuccess ? BS_OK : BS_ERR_CUDA;
}

template <typename P, typename... R> static P first_param(void (*)(P, R...));

// Launch of a kernel whose warps each take `pix_per_unit` pixels x one channel word.
template <typename K, typename... Extra>
static int launch_units(K kern, const void* x, uint32_t* out, int N, int C, int HW, int pix_per_unit, cudaStream_t st, Extra... extra)
{
    const int Cw = ceil_div(C, 32);
    const long long units_per_img = static_cast<long long>(ceil_div(HW, pix_per_unit)) * Cw;
    const long long nunits = N * units_per_img;
    const long long blocks = ceil_div_ll(nunits, FAST_WARPS);
    if (units_per_img > 0x7fffffffLL || blocks > 0x7fffffffLL) return BS_ERR_UNSUPPORTED;
    kern<<<static_cast<unsigned>(blocks), FAST_THREADS, 0, st>>>(
        static_cast<decltype(first_param(kern))>(x), out, C, HW, Cw, nunits, static_cast<int>(units_per_img), extra...);
    return cudaGetLastError() == cudaSuccess ? BS_OK : BS_ERR_CUDA;
}

template <int BITS>
static int launch_bitpack_nchw_i8(const void* x, uint32_t* out, int N, int C, int HW, cudaStream_t st)
{
    switch (ceil_div(C, 32)) {      // records of 1, 2 or 4 channel words leave through the block-staged stores
        case 1: return launch_units(bitpack_nchw_i8_kernel<BITS, 1>, x, out, N, C, HW, 128, st);
        case 2: return launch_units(bitpack_nchw_i8_kernel<BITS, 2>, x, out, N, C, HW, 128, st);
        case 4: return launch_units(bitpack_nchw_i8_kernel<BITS, 4>, x, out, N, C, HW, 128, st);
        default: return launch_units(bitpack_nchw_i8_kernel<BITS, 0>, x, out, N, C, HW, 128, st);
    }
}

template <bool NHWC>
static int launch_bitpack_i8(const void* x, uint32_t* out, int N, int C, int HW, int bits, cudaStream_t st)
{
    switch (bits) {
        case 1: return NHWC ? launch_units(bitpack_nhwc_i8_kernel<1>, x, out, N, C, HW, 128, st) : launch_bitpack_nchw_i8<1>(x, out, N, C, HW, st);
        case 2: return NHWC ? launch_units(bitpack_nhwc_i8_kernel<2>, x, out, N, C, HW, 128, st) : launch_bitpack_nchw_i8<2>(x, out, N, C, HW, st);
        case 3: return NHWC ? launch_units(bitpack_nhwc_i8_kernel<3>, x, out, N, C, HW, 128, st) : launch_bitpack_nchw_i8<3>(x, out, N, C, HW, st);
        default: return NHWC ? launch_units(bitpack_nhwc_i8_kernel<4>, x, out, N, C, HW, 128, st) : launch_bitpack_nchw_i8<4>(x, out, N, C, HW, st);
    }
}

// fp32 tensors: comparison-form kernels with one (32 pixels, channel word) unit per warp.
template <bool NHWC>
static int launch_bitpack_f32(const void* x, uint32_t* out, int N, int C, int HW, const QuantParams& q, cudaStream_t st)
{
    switch (q.bits) {
        case 1: return NHWC ? launch_units(bitpack_nhwc_f32_kernel<1>, x, out, N, C, HW, 32, st, q)
                            : launch_units(bitpack_nchw_f32_kernel<1>, x, out, N, C, HW, 32, st, q);
        case 2: return NHWC ? launch_units(bitpack_nhwc_f32_kernel<2>, x, out, N, C, HW, 32, st, q)
                            : launch_units(bitpack_nchw_f32_kernel<2>, x, out, N, C, HW, 32, st, q);
        case 3: return NHWC ? launch_units(bitpack_nhwc_f32_kernel<3>, x, out, N, C, HW, 32, st, q)
                            : launch_units(bitpack_nchw_f32_kernel<3>, x, out, N, C, HW, 32, st, q);
        default: return NHWC ? launch_units(bitpack_nhwc_f32_kernel<4>, x, out, N, C, HW, 32, st, q)
                             : launch_units(bitpack_nchw_f32_kernel<4>, x, out, N, C, HW, 32, st, q);
    }
}

// int8 codes: the vector kernels where the shape allows aligned vector loads and the planes are the low bits of the byte,
// else the fallback.
template <bool NHWC>
static int launch_bitpack_codes_any(const void* x, uint32_t* out, int N, int C, int HW, int bits, int sign, cudaStream_t st)
{
    if (sign != BS_BIPOLAR && (NHWC ? C % 32 == 0 : HW % 4 == 0)) return launch_bitpack_i8<NHWC>(x, out, N, C, HW, bits, st);
    switch (bits) {
        case 1: return launch_bitpack_codes<NHWC, 1>(x, out, N, C, HW, sign, st);
        case 2: return launch_bitpack_codes<NHWC, 2>(x, out, N, C, HW, sign, st);
        case 3: return launch_bitpack_codes<NHWC, 3>(x, out, N, C, HW, sign, st);
        default: return launch_bitpack_codes<NHWC, 4>(x, out, N, C, HW, sign, st);
    }
}

extern "C" int bitpack_activations(const void* x, int x_is_fp32, bs_layout_t layout, int N, int C, int H, int W,
                                   float act_scale, int a_bits, bs_sign_t a_sign, uint32_t* packed_out, void* stream)
{
    if (!x || !packed_out || N <= 0 || C <= 0 || H <= 0 || W <= 0) return BS_ERR_INVALID_ARG;
    if (!bits_ok(a_bits, a_sign) || (layout != BS_NCHW && layout != BS_NHWC)) return BS_ERR_INVALID_ARG;
    if (x_is_fp32 && !(act_scale > 0.0f && act_scale < 3.0e38f)) return BS_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(packed_out)) return BS_ERR_ALIGNMENT;
    if (static_cast<long long>(H) * W > 0x7fffffffLL) return BS_ERR_UNSUPPORTED;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int HW = H * W;
    if (x_is_fp32) {
        const QuantParams q = make_quant_params(act_scale, a_bits, a_sign);
        return layout == BS_NHWC ? launch_bitpack_f32<true>(x, packed_out, N, C, HW, q, st)
                                 : launch_bitpack_f32<false>(x, packed_out, N, C, HW, q, st);
    }
    return layout == BS_NHWC ? launch_bitpack_codes_any<true>(x, packed_out, N, C, HW, a_bits, a_sign, st)
                             : launch_bitpack_codes_any<false>(x, packed_out, N, C, HW, a_bits, a_sign, st);
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
