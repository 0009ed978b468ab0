// Implicit-GEMM bit-serial convolution on the SM integer pipes (Section V plane-pair popcount sum).
//
// One CTA computes a tile of (TNI images x TH rows x TW columns) output pixels by TN filters.  The
// reduction runs over channel-word chunks; each chunk stages, for all R*S taps at once,
//   - the packed activation halo  [TNI][hh][hw][CWC][A]   (TMA tiled load, out-of-image = 0 = padding)
//   - the packed filter slice     [TN][R*S][CWC][WB]      (TMA tiled load)
// in a ring of shared-memory stages guarded by mbarriers with bounded waits.  Tensors whose packed
// records are not 16-byte multiples cannot be described to TMA and are gathered with cp.async instead.
// Each thread owns PB pixels x FB filters of int32 accumulators and runs, per reduction word,
//   acc += coef[i][j] * popc(A_j & W_i)   over all plane pairs,
// with coef carrying 2^(i+j), the -2^(b-1) top-plane sign and the bipolar factors.
#pragma once
#include <cuda.h>

#include "common.cuh"

namespace bs {

constexpr int MAX_STAGES = 4;
constexpr unsigned WAIT_LIMIT = 1u << 22;   // bounded mbarrier polling (each poll may suspend briefly)

struct ConvArgs {
    CUtensorMap tmA;   // activations: dims (Cw*A, W, H, N) words
    CUtensorMap tmW;   // weights:     dims (Cw*WB, R*S, O) words
    const uint32_t* act;
    const uint32_t* wgt;
    int32_t* out_i32;
    uint32_t* out_packed;
    const float* scale;
    const float* bias;
    const uint32_t* residual;
    int* status;
    float res_scale;
    // problem
    int N, C, H, W, O, R, S, stride, pad, P, Q, Cw;
    int a_sign, w_sign;
    int relu, out_bits, out_sign, out_cw_off, out_cw_total;
    int res_bits, res_sign, res_c_off, res_cw_total;
    int i32_nhwc;
    // tiling
    int NFG, NPG, TNI, TH, TWB, used_pg;
    int hh, hw, CWC, nchunks, nstage;
    int stageA_words, stageW_words;          // padded to multiples of 32 words (128 B)
    int aux_off_words;                       // barriers and window sums live behind the ring / epilogue area
    int tiles_o, tiles_q, tiles_p, tiles_n;
    int tma_a, tma_w;                        // 1 = TMA tiled load, 0 = cp.async gather
    int boxA_w, nboxA;                       // a row tile (hh == 1, TNI == 1) may be split into nboxA boxes of boxA_w pixels
    int unitA, unitW;                        // cp.async unit in words (1, 2 or 4)
    // arithmetic
    int coef[4][4];                          // [i][j]
    int rs_coef[4];                          // per activation plane, used when the weights are bipolar
    int cs_coef[4];                          // per weight plane, used when the activations are bipolar
    int kconst;                              // + K when both operands are bipolar
    int need_rs, need_cs;
    // split of the reduction over several CTAs of one tile (needs a zeroed workspace; left zeroed on exit)
    int ksplit, chunks_per_split;
    int* ws_acc;                             // [tiles][PB*FB][threads] partial accumulators
    unsigned* ws_cnt;                        // [tiles] arrival counters
    int acc_small;                           // |acc| < 2^22 guaranteed by the shape: the exact mantissa trick applies
};

// ----------------------------------------------------------------------------- PTX wrappers

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, unsigned count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, unsigned bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, unsigned parity)
{
    unsigned ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait: returns false (and never blocks forever) if the phase does not complete.
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, unsigned parity, unsigned limit = WAIT_LIMIT)
{
    for (unsigned it = 0; it < limit; ++it)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}
__device__ __forceinline__ void fence_barrier_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ void tma_load_4d(void* dst, const CUtensorMap* tm, uint64_t* bar, int c0, int c1, int c2, int c3)
{
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cta.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(tm)), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
        : "memory");
}
__device__ __forceinline__ void tma_load_3d(void* dst, const CUtensorMap* tm, uint64_t* bar, int c0, int c1, int c2)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cta.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(tm)), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2)
        : "memory");
}

__device__ __forceinline__ void cp_unit(uint32_t* dst, const uint32_t* src, bool valid, int unit_words)
{
    const unsigned d = smem_u32(dst);
    if (unit_words == 4) {
        const unsigned n = valid ? 16u : 0u;
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(d), "l"(src), "r"(n) : "memory");
    } else if (unit_words == 2) {
        const unsigned n = valid ? 8u : 0u;
        asm volatile("cp.async.ca.shared.global [%0], [%1], 8, %2;" ::"r"(d), "l"(src), "r"(n) : "memory");
    } else {
        const unsigned n = valid ? 4u : 0u;
        asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"(d), "l"(src), "r"(n) : "memory");
    }
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_pending(int pending)
{
    switch (pending) {
        case 0: asm volatile("cp.async.wait_group 0;" ::: "memory"); break;
        case 1: asm volatile("cp.async.wait_group 1;" ::: "memory"); break;
        case 2: asm volatile("cp.async.wait_group 2;" ::: "memory"); break;
        default: asm volatile("cp.async.wait_group 3;" ::: "memory"); break;
    }
}

// ----------------------------------------------------------------------------- exact conversions off the XU pipe

// (float)i for |i| < 2^22, exact: the integer is planted in the mantissa of 1.5 * 2^23 and the offset subtracted.
// Keeps int->float conversions (which share the population-count pipe) out of the epilogue.
__device__ __forceinline__ float int_to_float_exact(int i)
{
    return __int_as_float(0x4B400000 + i) - 12582912.0f;
}
// Round-to-nearest-even of a float already clamped to a small range (|v| <= 2^21): adding 1.5 * 2^23 rounds to an
// integer in the mantissa with the IEEE default rounding, which is ties-to-even.
__device__ __forceinline__ int small_float_to_int_rn(float v)
{
    return __float_as_int(v + 12582912.0f) - 0x4B400000;
}

// ----------------------------------------------------------------------------- operand loads

template <int NB>
__device__ __forceinline__ void load_planes(const uint32_t* p, uint32_t (&v)[NB])
{
    if (NB == 2) { const uint2 t = *reinterpret_cast<const uint2*>(p); v[0] = t.x; v[1] = t.y; }
    else if (NB == 4) { const uint4 t = *reinterpret_cast<const uint4*>(p); v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w; }
    else {
#pragma unroll
        for (int k = 0; k < NB; ++k) v[k] = p[k];
    }
}

// ----------------------------------------------------------------------------- staging

struct TileOrigin { int n0, p0, q0, o0; };

// Issue the loads of reduction chunk `chunk` into the stage buffers sA / sW.
// TMA parts: one elected thread arms the mbarrier with the byte count and issues the tiled copies.
// cp.async parts: every thread copies its share of 4/8/16-byte units, zero-filling what lies outside
// the image, the batch, the filter bank or the channel words.  Every thread commits one group.
template <int A, int WB>
__device__ __forceinline__ void stage_issue(const ConvArgs& g, int chunk, uint32_t* sA, uint32_t* sW, uint64_t* bar,
                                            const TileOrigin& t, int TN)
{
    const int tid = threadIdx.x, nthreads = blockDim.x;
    const int c0 = chunk * g.CWC;
    const int recA = g.CWC * A, recW = g.CWC * WB, RS = g.R * g.S;
    const int y0 = t.p0 * g.stride - g.pad, x0 = t.q0 * g.stride - g.pad;
    if ((g.tma_a || g.tma_w) && tid == 0) {
        unsigned bytes = 0;
        if (g.tma_a) bytes += static_cast<unsigned>(g.TNI * g.hh * g.nboxA * g.boxA_w * recA) * 4u;
        if (g.tma_w) bytes += static_cast<unsigned>(TN * RS * recW) * 4u;
        mbar_expect_tx(bar, bytes);
        if (g.tma_a)
            for (int b = 0; b < g.nboxA; ++b)
                tma_load_4d(sA + b * g.boxA_w * recA, &g.tmA, bar, c0 * A, x0 + b * g.boxA_w, y0, t.n0);
        if (g.tma_w) tma_load_3d(sW, &g.tmW, bar, c0 * WB, 0, t.o0);
    }
    if (!g.tma_a) {
        const int upr = recA / g.unitA;                       // units per pixel record
        const int total = g.TNI * g.hh * g.hw * upr;
        const int fullA = g.Cw * A;
        for (int k = tid; k < total; k += nthreads) {
            const int u = k % upr, pix = k / upr;
            const int x = pix % g.hw, yy = (pix / g.hw) % g.hh, ni = pix / (g.hw * g.hh);
            const int n = t.n0 + ni, y = y0 + yy, xx = x0 + x;
            const int wofs = c0 * A + u * g.unitA;
            const bool valid = n < g.N && y >= 0 && y < g.H && xx >= 0 && xx < g.W && wofs < fullA;
            const uint32_t* src = valid ? g.act + ((static_cast<size_t>(n) * g.H + y) * g.W + xx) * fullA + wofs : g.act;
            cp_unit(sA + pix * recA + u * g.unitA, src, valid, g.unitA);
        }
    }
    if (!g.tma_w) {
        const int upr = recW / g.unitW;
        const int total = TN * RS * upr;
        const int fullW = g.Cw * WB;
        for (int k = tid; k < total; k += nthreads) {
            const int u = k % upr, ft = k / upr;               // ft = f * RS + tap
            const int o = t.o0 + ft / RS, tap = ft % RS;
            const int wofs = c0 * WB + u * g.unitW;
            const bool valid = o < g.O && wofs < fullW;
            const uint32_t* src = valid ? g.wgt + (static_cast<size_t>(o) * RS + tap) * fullW + wofs : g.wgt;
            cp_unit(sW + ft * recW + u * g.unitW, src, valid, g.unitW);
        }
    }
    cp_async_commit();
}

// ----------------------------------------------------------------------------- the kernel

template <int A, int WB, int PB, int FB>
__global__ void __launch_bounds__(256, (PB * FB <= 32) ? 3 : 1) bitserial_conv_kernel(const __grid_constant__ ConvArgs g)
{
    extern __shared__ __align__(128) uint32_t smem[];
    const int tid = threadIdx.x, nthreads = blockDim.x;
    const int TN = g.NFG * FB;
    const int TW = g.TWB * PB;
    const int used_pix = g.used_pg * PB;

    // shared-memory carve-up
    uint32_t* stageA = smem;
    uint32_t* stageW = stageA + static_cast<size_t>(g.nstage) * g.stageA_words;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + g.aux_off_words);
    int* rs_s = reinterpret_cast<int*>(bars + MAX_STAGES);     // [used_pix]
    int* cs_s = rs_s + used_pix;                               // [TN]

    // reduction split fastest, then filter tile, columns, rows, images
    const int ks = static_cast<int>(blockIdx.x % static_cast<unsigned>(g.ksplit));
    const int tile_id = static_cast<int>(blockIdx.x / static_cast<unsigned>(g.ksplit));
    const int c_begin = ks * g.chunks_per_split;
    const int c_end = min(g.nchunks, c_begin + g.chunks_per_split);
    const int my_chunks = c_end - c_begin;
    TileOrigin t;
    {
        int b = tile_id;
        t.o0 = (b % g.tiles_o) * TN;       b /= g.tiles_o;
        t.q0 = (b % g.tiles_q) * TW;       b /= g.tiles_q;
        t.p0 = (b % g.tiles_p) * g.TH;     b /= g.tiles_p;
        t.n0 = b * g.TNI;
    }

    // thread -> (filter group, pixel group).  Filters of a thread: fg + NFG*u; pixels: column tb + TWB*v.
    const int fg = tid % g.NFG;
    const int pg_raw = tid / g.NFG;
    const bool pg_used = pg_raw < g.used_pg;
    const int pg = pg_used ? pg_raw : 0;
    const int tb = pg % g.TWB;
    const int ty = (pg / g.TWB) % g.TH;
    const int ni = pg / (g.TWB * g.TH);

    const int recA = g.CWC * A, recW = g.CWC * WB, RS = g.R * g.S;
    const int a_off0 = ((ni * g.hh + ty * g.stride) * g.hw + tb * g.stride) * recA;
    const int a_pstep = g.TWB * g.stride * recA;
    const int w_off0 = fg * RS * recW;
    const int w_fstep = g.NFG * RS * recW;

    const bool any_tma = g.tma_a || g.tma_w;
    const bool any_cp = !g.tma_a || !g.tma_w;
    if (any_tma && tid == 0) {
        for (int s = 0; s < g.nstage; ++s) mbar_init(&bars[s], 1);
        fence_barrier_init();
        fence_proxy_async();
    }
    __syncthreads();

    // prologue: fill the ring (every thread commits exactly nstage groups, possibly empty)
    for (int s = 0; s < g.nstage; ++s) {
        if (s < my_chunks) stage_issue<A, WB>(g, c_begin + s, stageA + static_cast<size_t>(s) * g.stageA_words,
                                              stageW + static_cast<size_t>(s) * g.stageW_words, &bars[s], t, TN);
        else cp_async_commit();
    }

    int acc[PB][FB];
#pragma unroll
    for (int v = 0; v < PB; ++v)
#pragma unroll
        for (int u = 0; u < FB; ++u) acc[v][u] = 0;
    int coef[WB][A];
#pragma unroll
    for (int i = 0; i < WB; ++i)
#pragma unroll
        for (int j = 0; j < A; ++j) coef[i][j] = g.coef[i][j];
    int coef2[WB][A];
#pragma unroll
    for (int i = 0; i < WB; ++i)
#pragma unroll
        for (int j = 0; j < A; ++j) coef2[i][j] = 2 * g.coef[i][j];

    // window sums for the bipolar corrections: thread tid covers tile pixels tid, tid + nthreads, ...
    int rs_acc[4] = {0, 0, 0, 0};
    int cs_acc = 0;
    bool dead = false;   // set once a bounded wait ran out; later waits are skipped so the CTA still ends

    for (int c = 0; c < my_chunks; ++c) {
        const int s = c % g.nstage;
        const uint32_t* sA = stageA + static_cast<size_t>(s) * g.stageA_words;
        const uint32_t* sW = stageW + static_cast<size_t>(s) * g.stageW_words;
        if (any_cp) cp_async_wait_pending(g.nstage - 1);
        if (any_tma && !dead) {
            if (!mbar_wait_bounded(&bars[s], (c / g.nstage) & 1)) {
                dead = true;
                atomicOr(g.status, STATUS_TIMEOUT);
            }
        }
        if (any_cp) __syncthreads();

        // ---- plane-pair popcount MACs over all taps and words of this chunk (idle pixel groups skip them).
        // Within a filter row the reduction words (tap column, channel word) are contiguous for both operands.  They
        // are taken three at a time through a carry-save adder: with x_q = a_q & w_q,
        //     popc(x0) + popc(x1) + popc(x2) = popc(x0 ^ x1 ^ x2) + 2 * popc(maj(x0, x1, x2)),
        // i.e. two population counts (the scarce pipe: 16 lanes per clock per SM) and two 3-input logic operations
        // instead of three counts.  A remainder of one or two words takes the plain form.
        // A 1x1 layer (a matrix product) whose channel words do not fill the last chunk: the staged words past the
        // end are zero and add nothing, so the loops stop at the last live word (576 channels = 18 words in chunks of 8
        // would otherwise pay for 24).  With several taps the zero words sit between the taps and are kept.
        const int cw_live = RS == 1 ? min(g.CWC, g.Cw - (c_begin + c) * g.CWC) : g.CWC;
        if (pg_used)
        for (int r = 0; r < g.R; ++r) {
            const uint32_t* par = sA + a_off0 + r * g.hw * recA;
            const uint32_t* pwr = sW + w_off0 + r * g.S * recW;
            const int M = g.S * cw_live;
            int m = 0;
            for (; m + 3 <= M; m += 3) {
                uint32_t w[3][FB][WB];
#pragma unroll
                for (int q = 0; q < 3; ++q)
#pragma unroll
                    for (int u = 0; u < FB; ++u) load_planes<WB>(pwr + u * w_fstep + (m + q) * WB, w[q][u]);
#pragma unroll
                for (int v = 0; v < PB; ++v) {
                    uint32_t a[3][A];
#pragma unroll
                    for (int q = 0; q < 3; ++q) load_planes<A>(par + v * a_pstep + (m + q) * A, a[q]);
#pragma unroll
                    for (int u = 0; u < FB; ++u)
#pragma unroll
                        for (int i = 0; i < WB; ++i)
#pragma unroll
                            for (int j = 0; j < A; ++j) {
                                const uint32_t x0 = a[0][j] & w[0][u][i], x1 = a[1][j] & w[1][u][i], x2 = a[2][j] & w[2][u][i];
                                const uint32_t sum = x0 ^ x1 ^ x2, carry = (x0 & x1) | (x2 & (x0 ^ x1));
                                acc[v][u] += coef[i][j] * __popc(sum) + coef2[i][j] * __popc(carry);
                            }
                }
            }
            for (; m < M; ++m) {
                uint32_t a[PB][A], w[FB][WB];
#pragma unroll
                for (int v = 0; v < PB; ++v) load_planes<A>(par + v * a_pstep + m * A, a[v]);
#pragma unroll
                for (int u = 0; u < FB; ++u) load_planes<WB>(pwr + u * w_fstep + m * WB, w[u]);
#pragma unroll
                for (int v = 0; v < PB; ++v)
#pragma unroll
                    for (int u = 0; u < FB; ++u)
#pragma unroll
                        for (int i = 0; i < WB; ++i)
#pragma unroll
                            for (int j = 0; j < A; ++j)
                                acc[v][u] += coef[i][j] * __popc(a[v][j] & w[u][i]);
            }
        }
        // ---- window sums (only when an operand is bipolar)
        if (g.need_rs) {
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const int tp = tid + k * nthreads;
                if (tp < used_pix) {
                    const int row = tp / TW, x = tp - row * TW;          // row = ni * TH + ty
                    const int rni = row / g.TH, rty = row - rni * g.TH;
                    const uint32_t* base = sA + ((rni * g.hh + rty * g.stride) * g.hw + x * g.stride) * recA;
                    int sum = 0;
                    for (int tap = 0; tap < RS; ++tap) {
                        const int r = tap / g.S, sx = tap - r * g.S;
                        const uint32_t* p = base + (r * g.hw + sx) * recA;
                        for (int cw = 0; cw < cw_live; ++cw)
#pragma unroll
                            for (int j = 0; j < A; ++j) sum += g.rs_coef[j] * __popc(p[cw * A + j]);
                    }
                    rs_acc[k] += sum;
                }
            }
        }
        if (g.need_cs && tid < TN) {
            const uint32_t* base = sW + tid * RS * recW;
            int sum = 0;
            for (int k = 0; k < (RS == 1 ? cw_live : RS * g.CWC); ++k)
#pragma unroll
                for (int i = 0; i < WB; ++i) sum += g.cs_coef[i] * __popc(base[k * WB + i]);
            cs_acc += sum;
        }
        __syncthreads();   // everyone is done with stage s
        if (c + g.nstage < my_chunks)
            stage_issue<A, WB>(g, c_begin + c + g.nstage, stageA + static_cast<size_t>(s) * g.stageA_words,
                               stageW + static_cast<size_t>(s) * g.stageW_words, &bars[s], t, TN);
        else
            cp_async_commit();
    }

    // ---- corrections through shared memory
    if (g.need_rs) {
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const int tp = tid + k * nthreads;
            if (tp < used_pix) rs_s[tp] = rs_acc[k];
        }
    }
    if (g.need_cs && tid < TN) cs_s[tid] = cs_acc;
    if (g.need_rs || g.need_cs) __syncthreads();

    const int n = t.n0 + ni, p = t.p0 + ty;
    const bool row_ok = pg_used && n < g.N && p < g.P;
#pragma unroll
    for (int v = 0; v < PB; ++v) {
        const int x = tb + g.TWB * v;
        int add = ks == 0 ? g.kconst : 0;
        if (g.need_rs) add += rs_s[(ni * g.TH + ty) * TW + x];
#pragma unroll
        for (int u = 0; u < FB; ++u) {
            acc[v][u] += add;
            if (g.need_cs) acc[v][u] += cs_s[fg + g.NFG * u];
        }
    }

    // ---- reduction split: add partial sums into the workspace; the last CTA of the tile picks up the totals,
    //      clears what it read (the workspace stays zero for the next launch) and runs the epilogue
    if (g.ksplit > 1) {
        int* ws = g.ws_acc + static_cast<size_t>(tile_id) * (PB * FB) * nthreads + tid;
#pragma unroll
        for (int v = 0; v < PB; ++v)
#pragma unroll
            for (int u = 0; u < FB; ++u) atomicAdd(ws + (v * FB + u) * nthreads, acc[v][u]);
        __threadfence();
        __syncthreads();
        __shared__ unsigned s_arrival;
        if (tid == 0) s_arrival = atomicAdd(g.ws_cnt + tile_id, 1u);
        __syncthreads();
        if (s_arrival != static_cast<unsigned>(g.ksplit - 1)) return;
        __threadfence();
#pragma unroll
        for (int v = 0; v < PB; ++v)
#pragma unroll
            for (int u = 0; u < FB; ++u) {
                acc[v][u] = __ldcg(ws + (v * FB + u) * nthreads);
                __stcg(ws + (v * FB + u) * nthreads, 0);
            }
        if (tid == 0) g.ws_cnt[tile_id] = 0u;
    }

    // ---- raw accumulators
    if (g.out_i32 && row_ok) {
#pragma unroll
        for (int v = 0; v < PB; ++v) {
            const int q = t.q0 + tb + g.TWB * v;
            if (q >= g.Q) continue;
#pragma unroll
            for (int u = 0; u < FB; ++u) {
                const int o = t.o0 + fg + g.NFG * u;
                if (o >= g.O) continue;
                const size_t idx = g.i32_nhwc ? ((static_cast<size_t>(n) * g.P + p) * g.Q + q) * g.O + o
                                              : ((static_cast<size_t>(n) * g.O + o) * g.P + p) * g.Q + q;
                g.out_i32[idx] = acc[v][u];
            }
        }
    }

    // ---- fused requantisation epilogue and plane re-packing
    if (g.out_packed) {
        // the stage buffers are free now (the loop ended with a barrier); park patterns as bytes [tile_pix][TN + 4]
        unsigned char* codes_s = reinterpret_cast<unsigned char*>(smem);
        const int pitch = TN + 4;
        int qmin, qmax;
        code_limits(g.out_bits, g.out_sign, qmin, qmax);
        const float fqmin = static_cast<float>(qmin), fqmax = static_cast<float>(qmax);
        float sc[FB], bi[FB];
#pragma unroll
        for (int u = 0; u < FB; ++u) {
            const int o = t.o0 + fg + g.NFG * u;
            sc[u] = o < g.O ? g.scale[o] : 0.f;
            bi[u] = o < g.O ? g.bias[o] : 0.f;
        }
#pragma unroll
        for (int v = 0; v < PB; ++v) {
            const int x = tb + g.TWB * v;
            const int q = t.q0 + x;
            const bool pix_ok = row_ok && q < g.Q;
            const size_t pix = (static_cast<size_t>(n) * g.P + p) * g.Q + q;
            // residual planes are fetched once per 32-channel word, not once per output
            uint32_t rw[4] = {0, 0, 0, 0};
            int rw_word = -1;
#pragma unroll
            for (int u = 0; u < FB; ++u) {
                const int of = fg + g.NFG * u;
                const int o = t.o0 + of;
                unsigned pat = 0;
                if (pix_ok && o < g.O) {
                    float val = fmaf(g.acc_small ? int_to_float_exact(acc[v][u]) : static_cast<float>(acc[v][u]), sc[u], bi[u]);
                    if (g.residual) {
                        const int rc = g.res_c_off + o;
                        if ((rc >> 5) != rw_word) {
                            rw_word = rc >> 5;
                            const uint32_t* rp = g.residual + (pix * g.res_cw_total + rw_word) * g.res_bits;
#pragma unroll
                            for (int j = 0; j < 4; ++j)
                                if (j < g.res_bits) rw[j] = rp[j];
                        }
                        unsigned rpat = 0;
#pragma unroll
                        for (int j = 0; j < 4; ++j)
                            if (j < g.res_bits) rpat |= ((rw[j] >> (rc & 31)) & 1u) << j;
                        val = fmaf(g.res_scale, static_cast<float>(pattern_value(rpat, g.res_bits, g.res_sign)), val);
                    }
                    if (g.relu) val = fmaxf(val, 0.0f);
                    int code;
                    if (g.out_sign == BS_BIPOLAR) code = val >= 0.0f ? 1 : -1;
                    else code = small_float_to_int_rn(fminf(fmaxf(val, fqmin), fqmax));
                    pat = stored_pattern(code, g.out_bits, g.out_sign);
                }
                if (pg_used) codes_s[((ni * g.TH + ty) * TW + x) * pitch + of] = static_cast<unsigned char>(pat);
            }
        }
        __syncthreads();
        // one task per (tile pixel, 32-filter word): gather bit j of 32 byte patterns into plane word j
        const int words_per_pix = TN / 32;
        const int ntask = used_pix * words_per_pix;
        for (int task = tid; task < ntask; task += nthreads) {
            const int wi = task % words_per_pix, tp = task / words_per_pix;
            const int row = tp / TW, x = tp - row * TW;
            const int rni = row / g.TH, rty = row - rni * g.TH;
            const int nn = t.n0 + rni, pp = t.p0 + rty, qq = t.q0 + x;
            const int ow = (t.o0 >> 5) + wi;                              // word index inside this layer's O range
            if (nn >= g.N || pp >= g.P || qq >= g.Q || ow * 32 >= g.O) continue;
            const uint32_t* src = reinterpret_cast<const uint32_t*>(codes_s + tp * pitch + wi * 32);
            uint32_t b[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) b[k] = src[k];
            uint32_t* dst = g.out_packed +
                (((static_cast<size_t>(nn) * g.P + pp) * g.Q + qq) * g.out_cw_total + g.out_cw_off + ow) * g.out_bits;
            for (int j = 0; j < g.out_bits; ++j) {
                uint32_t word = 0;
#pragma unroll
                for (int k = 0; k < 8; ++k)
                    word |= ((((b[k] >> j) & 0x01010101u) * 0x01020408u) >> 24 & 0xFu) << (4 * k);
                dst[j] = word;
            }
        }
    }
}

}  // namespace bs
