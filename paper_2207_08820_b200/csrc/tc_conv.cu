// Exact integer tensor-core formulation of the bit-serial convolution (tcgen05.mma kind::i8, accumulators in TMEM).
//
// The Section V plane-pair popcount sum equals the integer dot product of the unpacked codes, so the same int32
// accumulators come out of an int8 x int8 -> int32 matrix product on the 5th-generation tensor cores.  Activations
// stay bit-packed in HBM (the library's format); a CTA
//   - TMA-loads the packed halo of a channel chunk and a pre-expanded int8 filter slice (cp.async.bulk),
//   - expands the bitplanes to int8 in shared memory, directly in the K-major core-matrix layout UMMA reads
//     ([16-channel group][halo pixel][16 bytes]); a tap (r, s) of the implicit GEMM is then only a different
//     descriptor start address, no im2col copy,
//   - one elected thread issues tcgen05.mma (M = 128 pixels, N = filters of the tile, K = 32 channels each),
//   - four warps read the accumulator rows back with tcgen05.ld (one pixel per thread), apply the same fused
//     requantisation epilogue as the popcount kernel and build the output plane words thread-locally.
// Every wait on an mbarrier is bounded; a wait that runs out sets the device status word and the CTA drains.
#include <cstdio>
#include <cstdlib>
#include <array>
#include <map>
#include <mutex>

#include "conv_kernel.cuh"
#include "requant_bounds.h"

namespace bs {

constexpr int TC_THREADS = 320;       // warps 0-3 and 6-9: expand + epilogue, warp 4: TMA producer, warp 5: MMA issuer
constexpr int TC_WORKERS = 256;       // threads of the eight expand + epilogue warps
constexpr int TC_M = 128;             // pixels per tile = 16 row groups x 8 columns (or 128 flat pixels)
constexpr int TC_MAX_STAGES = 4;

struct TcArgs {
    CUtensorMap tmA;                  // packed activations: (W*Cw*A, H, N) words when a halo row fits one box row, else (Cw*A, W, H, N)
    const uint32_t* act;              // packed activations (flat mode copies whole pixel records with cp.async.bulk)
    const int8_t* wgt;                // prepared int8 filters [chunk][O/8][tap][CK/16][8][16]
    int32_t* out_i32;
    uint32_t* out_packed;
    const float* scale;
    const float* bias;
    const uint32_t* residual;
    int* status;
    float res_scale;
    int N, H, W, O, R, S, stride, pad, P, Q;
    int A;                            // activation bits
    int relu, out_bits, out_sign, out_cw_off, out_cw_total;
    int res_bits, res_sign, res_c_off, res_cw_total;
    int i32_nhwc, acc_small;
    int acc_bound;                    // |accumulator| <= acc_bound
    int thr_packed;                   // thresholds stored for two filters per entry (16-bit lanes), see tc_compare_pairs
    // tiling
    int flat;                         // 1: 128 consecutive pixels of the flattened image (1x1, stride 1)
    int NM;                           // filters of one MMA (TN when TN <= 128, else 256: a wider tile issues TN / NM MMAs per step)
    int TN, CK, MB, CWC, nchunks, nsp, nse;   // CK: channels per filter-layout block, MB: blocks per pipeline chunk, CWC: words per chunk
    int fullA;                        // words of one packed pixel record (Cw * A)
    int pitchA;                       // words between the staged records of consecutive pixels (fullA, or seg_words)
    int ld_stride;                    // 2: a 1x1 stride-2 layer fetched through a tensor map that skips every other row and column
                                      // (the kernels then see a stride-1 layer on the subsampled image: `stride` is 1)
    int seg_words, seg_chunks, nseg;  // flat tiles with long records: the 128 rows are staged seg_words at a time (0: whole records)
    int pmode;                        // how a tile's packed halo is fetched: 0 flat bulk copy, 1 rows merged with W, 2 4-D box
    int TNI, GI, hh, hw;              // packed halo: TNI images x hh rows x hw columns; GI row groups per image
    int hwb, xsh;                     // row pitch of the staged halo in pixels, and pixels skipped at the start of a row
                                      // (8-byte records: the box starts one pixel early to stay 16-byte aligned)
    int HWP, HWH, HPE;                // expanded layout: row pitch, half-row offset (stride 2), pixels per 16-channel plane
    int tiles_o, tiles_q, tiles_p, tiles_n;
    int opad8;                        // padded filter count / 8 in the prepared weights
    int pa_bytes, pa_tx_bytes, b_bytes, e_bytes;   // per stage (pa_tx_bytes: bytes the activation box delivers)
    int off_p, off_e, off_sb, off_bar, off_lut;
    int off_thr, thr_pats;            // integer thresholds of the epilogue: offset (0 = not used) and residual patterns (1 or 4)   // shared-memory offsets (bytes)
    int persistent;
    int PT;                           // streaming kernel: pixel tiles per CTA (they share every streamed filter chunk)
    int tmem_cols;
    unsigned idesc;
    unsigned mul[4];                  // byte value of plane j (2^j, or 256 - 2^(A-1) for a two's-complement top plane)
    unsigned xormask;                 // 0xFFFFFFFF for bipolar activations
    RequantBounds rb;                 // comparison form of the epilogue (1- and 2-bit outputs)
};

// ----------------------------------------------------------------------------- timeline trace (tuning builds only)
//
// Built with -DBS_TUNING, the first 148 CTAs of a launch record the SM cycle counter at the hand-offs between their roles
// (per tile, for the first 24 tiles); bs_tc_trace_read copies the table to the host.  Compiled out of the normal library.
enum { TR_START = 0, TR_SETUP, TR_PDL, TR_WGT, TR_LOAD, TR_XBEG, TR_XEND, TR_MBEG, TR_MEND, TR_EBEG, TR_EEND, TR_END, TR_E_LD, TR_E_CMP,
       TR_E_ST, TR_E_LOOP, TR_M_ISSUED, TR_X_DONE0, TR_X_BEG0 };
#ifdef BS_TUNING
constexpr int TC_TRACE_EVENTS = 24, TC_TRACE_TILES = 24, TC_TRACE_CTAS = 148;
__device__ long long g_tc_trace[TC_TRACE_CTAS * TC_TRACE_EVENTS * TC_TRACE_TILES];
__device__ __forceinline__ void tc_trace(int ev, int tile)
{
    if (blockIdx.x < TC_TRACE_CTAS && tile >= 0 && tile < TC_TRACE_TILES)
        g_tc_trace[(blockIdx.x * TC_TRACE_EVENTS + ev) * TC_TRACE_TILES + tile] = clock64();
}
#define TC_TRACE(ev, tile) tc_trace(ev, tile)
#else
#define TC_TRACE(ev, tile) do { } while (0)
#endif

// Position in a ring of `n` stages guarded by mbarriers: stage index and phase bit, advanced without any division (a
// division by a run-time ring size costs a lone issuing thread hundreds of cycles per hand-off).  A consumer waits for
// full[idx] with `phase`; a producer waits for empty[idx] with `phase ^ 1`, which a freshly initialised barrier already
// satisfies, so the first round needs no special case.
struct TcRing {
    int idx;
    unsigned phase;
    __device__ __forceinline__ TcRing() : idx(0), phase(0) {}
    __device__ __forceinline__ void advance(int n) { if (++idx == n) { idx = 0; phase ^= 1u; } }
};

// ----------------------------------------------------------------------------- tcgen05 wrappers

__device__ __forceinline__ void mbar_arrive(uint64_t* bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// Barrier among the threads of one warp group (expanders or epilogue); ids 1 and 2, id 0 is __syncthreads.
__device__ __forceinline__ void group_sync(int id, int nthreads = 128) { asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory"); }
// Bounded wait for the tensor-core pipeline: try_wait parks the thread for at most ~2 us per attempt (measured: a
// shorter hint, no hint or a test_wait spin make no difference to the layer times); 2^20 attempts bound a wait that
// nothing satisfies to about two seconds, after which the caller sets the status word and the CTA drains.
__device__ __forceinline__ bool mbar_spin_bounded(uint64_t* bar, unsigned parity)
{
    const uint32_t addr = smem_u32(bar);
    for (unsigned it = 0; it < (1u << 20); ++it) {
        unsigned ok;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(ok) : "r"(addr), "r"(parity), "r"(2000u) : "memory");     // park for at most ~2 us per attempt
        if (ok) return true;
    }
    return false;
}
// Group-wide AND of a per-thread flag (also a barrier): every thread of the group gets the same answer, so a wait
// that ran out makes the whole group leave its loop together and nobody is left behind at a later group_sync.
__device__ __forceinline__ bool group_all(int id, bool ok, int nthreads = 128)
{
    unsigned r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.u32 q, %1, 0;\n\t"
        "bar.red.and.pred p, %2, %3, q;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(r) : "r"(ok ? 1u : 0u), "r"(id), "r"(nthreads) : "memory");
    return r != 0;
}
// One lane polls the mbarrier for its warp (128 threads hammering one shared-memory word is slow); result is broadcast.
__device__ __forceinline__ bool mbar_wait_warp(uint64_t* bar, unsigned parity, int lane)
{
    unsigned ok = 1;
    if (lane == 0) ok = mbar_spin_bounded(bar, parity) ? 1u : 0u;
    return __shfl_sync(0xffffffffu, ok, 0) != 0;
}
// Programmatic dependent launch: `pdl_release` lets the next kernel of the stream start its prologue once every CTA of
// this grid has passed it; `pdl_acquire` returns when the preceding grid has completed and its writes are visible.
// Both are no-ops when the launches involved do not carry the programmatic-serialisation attribute.
__device__ __forceinline__ void pdl_release() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_acquire() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

__device__ __forceinline__ void tmem_alloc(uint32_t* slot, unsigned ncols)
{
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(slot)), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() { asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, unsigned ncols)
{
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void umma_i8(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t* bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&v)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
          "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
          "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ void bulk_load(void* dst, const void* src, unsigned bytes, uint64_t* bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* tm, uint64_t* bar, int c0, int c1)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cta.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(tm)), "r"(smem_u32(bar)), "r"(c0), "r"(c1) : "memory");
}

// K-major, no-swizzle shared-memory matrix descriptor: 8-row x 16-byte core matrices of 128 contiguous bytes;
// lbo = byte distance between the two core matrices of one K = 32 step, sbo = byte distance between 8-row groups.
__device__ __forceinline__ uint64_t umma_desc(uint32_t smem_addr, uint32_t lbo, uint32_t sbo)
{
    return static_cast<uint64_t>((smem_addr >> 4) & 0x3FFFu) | (static_cast<uint64_t>((lbo >> 4) & 0x3FFFu) << 16) |
           (static_cast<uint64_t>((sbo >> 4) & 0x3FFFu) << 32) | (1ull << 46);
}

// ----------------------------------------------------------------------------- building blocks

struct TcTile { int n0, p0, q0; };

__device__ __forceinline__ TcTile tc_decode_tile(const TcArgs& g, int mt)
{
    TcTile t;
    if (g.flat) { t.q0 = mt * TC_M; t.p0 = 0; t.n0 = 0; return t; }      // tiles_p = tiles_n = 1
    t.q0 = (mt % g.tiles_q) * 8;   mt /= g.tiles_q;
    t.p0 = (mt % g.tiles_p) * 16;                    mt /= g.tiles_p;
    t.n0 = mt * g.TNI;
    return t;
}

// Walks the pixel tiles first, first + step, ... of a CTA: the decomposition of the step is found once, each further
// tile costs a few additions and carries instead of two divisions.
struct TcTileWalker {
    int iq, ip, in;            // tile coordinates
    int dq, dp, dn;            // decomposition of the step
    int mt;                    // linear tile index
    int step;
};

__device__ __forceinline__ TcTileWalker tc_walk_init(const TcArgs& g, int first, int step)
{
    TcTileWalker w;
    w.mt = first; w.step = step;
    int t = first;
    w.iq = t % g.tiles_q; t /= g.tiles_q; w.ip = t % g.tiles_p; w.in = t / g.tiles_p;
    t = step;
    w.dq = t % g.tiles_q; t /= g.tiles_q; w.dp = t % g.tiles_p; w.dn = t / g.tiles_p;
    return w;
}
__device__ __forceinline__ TcTile tc_walk_tile(const TcArgs& g, const TcTileWalker& w)
{
    TcTile t;
    if (g.flat) { t.q0 = w.mt * TC_M; t.p0 = 0; t.n0 = 0; return t; }
    t.q0 = w.iq * 8; t.p0 = w.ip * 16; t.n0 = w.in * g.TNI;
    return t;
}
__device__ __forceinline__ void tc_walk_next(const TcArgs& g, TcTileWalker& w)
{
    w.mt += w.step;
    w.iq += w.dq; w.ip += w.dp; w.in += w.dn;
    if (w.iq >= g.tiles_q) { w.iq -= g.tiles_q; ++w.ip; }
    if (w.ip >= g.tiles_p) { w.ip -= g.tiles_p; ++w.in; }
}

// Fetch the packed halo of one tile (whole pixel records, all channel chunks) and arm `bar` with its byte count.
// Rows of a TMA box cost a fixed overhead each, so the copy is shaped to have few, long rows: a flat tile is one
// contiguous cp.async.bulk; otherwise a halo row (hw pixels x record) is one box row whenever it fits 256 elements.
__device__ __forceinline__ void tc_load_tile(const TcArgs& g, void* dst, uint64_t* bar, const TcTile& tile)
{
    if (g.pmode == 0) {
        const long long npix = static_cast<long long>(g.N) * g.P * g.Q;
        long long rows = npix - tile.q0;
        if (rows > TC_M) rows = TC_M;
        const unsigned bytes = static_cast<unsigned>(rows) * static_cast<unsigned>(g.fullA) * 4u;
        mbar_expect_tx(bar, bytes);
        bulk_load(dst, g.act + static_cast<size_t>(tile.q0) * g.fullA, bytes, bar);
    } else {
        mbar_expect_tx(bar, static_cast<unsigned>(g.pa_tx_bytes));
        const int x0 = tile.q0 * g.stride * g.ld_stride - g.pad, y0 = tile.p0 * g.stride * g.ld_stride - g.pad;
        if (g.pmode == 1) tma_load_3d(dst, &g.tmA, bar, (x0 - g.xsh) * g.fullA, y0, tile.n0);
        else tma_load_4d(dst, &g.tmA, bar, 0, x0, y0, tile.n0);
    }
}

// Look-up tables of the expansion, built once per CTA.
// A == 2 (the 2-bit activations of the headline networks): one table of 256 words indexed by a nibble of plane 0
// (low four index bits) and the same nibble of plane 1 (high four): the entry is the four finished int8 codes.
// Other widths: entry [j][b] holds, for the eight bits of byte b of plane j, eight int8 lanes with value mul[j] where
// the bit is set (two 32-bit words); adding the entries of all planes gives eight codes at once.
constexpr int TC_LUT_BYTES_PER_PLANE = 256 * 8;

__device__ __forceinline__ void tc_build_lut(const TcArgs& g, uint2* lut, int tid, int nthreads)
{
    if (g.A == 2) {
        uint32_t* lut4 = reinterpret_cast<uint32_t*>(lut);
        for (int e = tid; e < 256; e += nthreads) {
            const unsigned n0 = e & 15u, n1 = static_cast<unsigned>(e) >> 4;
            const unsigned s0 = (n0 * 0x00204081u) & 0x01010101u, s1 = (n1 * 0x00204081u) & 0x01010101u;
            lut4[e] = s0 * g.mul[0] + s1 * g.mul[1];      // per byte: at most 1 + 254, no carry between lanes
        }
        return;
    }
    for (int e = tid; e < g.A * 256; e += nthreads) {
        const unsigned b = e & 255u, m = g.mul[e >> 8];
        const unsigned lo = (((b & 0xFu) * 0x00204081u) & 0x01010101u) * m;
        const unsigned hi = (((b >> 4) * 0x00204081u) & 0x01010101u) * m;
        lut[e] = make_uint2(lo, hi);
    }
}

// Where an expander thread starts in the item grid of a chunk, and how 128 items further move it: found once per
// kernel so that the per-item loop has no division.  Items are (pixel, channel word) pairs, channel word fastest;
// a chunk has one or two channel words.
struct TcExpand {
    int cw;            // channel word of this thread's items (the item stride is a multiple of the words per chunk)
    int x2, y2;        // first item's position in the (possibly subsampled) halo grid
    int dx, dy;        // movement of `step` items
    int nx, items;
    int step;          // threads of the expander group
};

__device__ __forceinline__ TcExpand tc_expand_init(const TcArgs& g, int et, int nthreads)
{
    TcExpand x;
    x.step = nthreads;
    const int sub = (!g.flat && g.stride == 2 && g.R == 1) ? 2 : 1;
    x.nx = g.flat ? TC_M : (g.hw + sub - 1) / sub;
    const int ny = g.flat ? 1 : (g.TNI * g.hh + sub - 1) / sub;   // hh is even for stride 2: rows of all images keep their parity
    x.items = x.nx * ny * g.CWC;
    const int sh = __ffs(g.CWC) - 1;                               // CWC is a power of two (1 .. 8)
    x.cw = et & (g.CWC - 1);
    const int pp = et >> sh, pstep = nthreads >> sh;
    x.y2 = pp / x.nx; x.x2 = pp - x.y2 * x.nx;
    x.dy = pstep / x.nx; x.dx = pstep - x.dy * x.nx;
    return x;
}

// Expansion of channel chunk c of the staged tile: bitplanes of (pixel, 32-channel word) -> 32 int8 values, written as
// two 16-byte rows of the K-major core-matrix layout [16-channel group][halo pixel][16 bytes].  `et` = 0..127 within
// the expander group.  A 1x1 stride-2 layer only ever reads even halo rows and columns, so only those are expanded.
// MODE: 0 flat tile, 1 2-D tile stride 1, 2 2-D tile stride 2, 3 2-D tile 1x1 stride 2 (even rows and columns only).
// The mode is a template parameter so that the per-item body is straight-line code.
template <int A, int MODE>
__device__ __forceinline__ void tc_expand_items(const TcArgs& g, const TcExpand& x, const uint32_t* pa, unsigned char* eb,
                                                const uint2* lut, int et, int c)
{
    constexpr int step = MODE == 3 ? 2 : 1;
    const uint32_t xormask = g.xormask;
    const int plane_bytes = g.HPE * 16;
    const int cw = x.cw;
    int x2 = x.x2, y2 = x.y2;
    const uint32_t* src_c = pa + (c * g.CWC + cw) * A;
    unsigned char* dst_c = eb + static_cast<size_t>(2 * cw) * plane_bytes;
    for (int it = et; it < x.items; it += x.step) {
        int hp, ep;
        if (MODE == 0) {
            hp = ep = x2;
        } else {
            const int hy = y2 * step, hx = x2 * step;
            hp = hy * g.hwb + hx + g.xsh;
            ep = hy * g.HWP + (MODE == 1 ? hx : (hx & 1) * g.HWH + (hx >> 1));
        }
        uint32_t w[A];
        load_planes<A>(src_c + static_cast<size_t>(hp) * g.pitchA, w);
        uint32_t out[8];
        if (A == 2) {
            // byte j of t / u: table index of nibble 2j / 2j+1 (plane 0 in the low four bits, plane 1 in the high four)
            const char* lut4 = reinterpret_cast<const char*>(lut);
            const uint32_t t = (w[0] & 0x0F0F0F0Fu) | ((w[A - 1] << 4) & 0xF0F0F0F0u);
            const uint32_t u = ((w[0] >> 4) & 0x0F0F0F0Fu) | (w[A - 1] & 0xF0F0F0F0u);
            out[0] = *reinterpret_cast<const uint32_t*>(lut4 + ((t << 2) & 0x3FCu));
            out[1] = *reinterpret_cast<const uint32_t*>(lut4 + ((u << 2) & 0x3FCu));
            out[2] = *reinterpret_cast<const uint32_t*>(lut4 + ((t >> 6) & 0x3FCu));
            out[3] = *reinterpret_cast<const uint32_t*>(lut4 + ((u >> 6) & 0x3FCu));
            out[4] = *reinterpret_cast<const uint32_t*>(lut4 + ((t >> 14) & 0x3FCu));
            out[5] = *reinterpret_cast<const uint32_t*>(lut4 + ((u >> 14) & 0x3FCu));
            out[6] = *reinterpret_cast<const uint32_t*>(lut4 + ((t >> 22) & 0x3FCu));
            out[7] = *reinterpret_cast<const uint32_t*>(lut4 + ((u >> 22) & 0x3FCu));
        } else {
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                uint2 acc = lut[(w[0] >> (8 * q)) & 0xFFu];
#pragma unroll
                for (int j = 1; j < A; ++j) {
                    const uint2 tt = lut[j * 256 + ((w[j] >> (8 * q)) & 0xFFu)];
                    acc.x += tt.x; acc.y += tt.y;
                }
                out[2 * q] = acc.x ^ xormask;
                out[2 * q + 1] = acc.y ^ xormask;
            }
        }
        unsigned char* d = dst_c + static_cast<size_t>(ep) * 16;
        *reinterpret_cast<uint4*>(d) = make_uint4(out[0], out[1], out[2], out[3]);
        *reinterpret_cast<uint4*>(d + plane_bytes) = make_uint4(out[4], out[5], out[6], out[7]);
        x2 += x.dx; y2 += x.dy;
        if (x2 >= x.nx) { x2 -= x.nx; ++y2; }
    }
}

template <int A>
__device__ __forceinline__ void tc_expand_chunk(const TcArgs& g, const TcExpand& x, const uint32_t* pa, unsigned char* eb,
                                                const uint2* lut, int et, int c)
{
    if (g.flat) tc_expand_items<A, 0>(g, x, pa, eb, lut, et, c);
    else if (g.stride == 1) tc_expand_items<A, 1>(g, x, pa, eb, lut, et, c);
    else if (g.R == 1) tc_expand_items<A, 3>(g, x, pa, eb, lut, et, c);
    else tc_expand_items<A, 2>(g, x, pa, eb, lut, et, c);
}

// All MMAs of one chunk: R*S taps x CK/32 steps of K = 32; a tap only moves the descriptor start address.
// One thread issues them.  A lone thread cannot hide the latency of a load in front of every MMA (a tabulated
// offset per MMA measured 120-160 cycles per MMA against 64 for the MMA itself), so the start addresses are produced
// by register arithmetic alone: the filter operand advances by a constant per MMA, the activation operand by the
// tap's column, row and K-half offsets (16-byte units; shared-memory addresses fit the 14-bit field without a mask).
struct TcIssue {
    uint32_t a_lo, a_hi, b_lo, b_hi;   // descriptor words with a zero start-address field
    uint32_t idesc;
    uint32_t row16, half16, kstep16;   // halo row, odd-column plane (stride 2) and second K half, in 16-byte units
    int R, S;
    bool stride2;                      // even/odd column split
    int ksteps;                        // K = 32 steps per tap and layout block (block channels / 32)
    int blocks;                        // layout blocks per chunk
    uint32_t blk_b16;                  // filter tile of one layout block, in 16-byte units
};

__device__ __forceinline__ TcIssue tc_make_issue(const TcArgs& g)
{
    TcIssue is;
    const uint32_t lbo_a = static_cast<uint32_t>(g.HPE) * 16u;
    const uint32_t sbo_a = g.flat ? 128u : static_cast<uint32_t>(g.stride * g.HWP) * 16u;
    const uint32_t k16 = static_cast<uint32_t>(g.CK >> 4);
    const uint32_t sbo_b = static_cast<uint32_t>(g.R * g.S) * k16 * 128u;
    const uint64_t ad = umma_desc(0, lbo_a, sbo_a), bd = umma_desc(0, 128u, sbo_b);
    is.a_lo = static_cast<uint32_t>(ad); is.a_hi = static_cast<uint32_t>(ad >> 32);
    is.b_lo = static_cast<uint32_t>(bd); is.b_hi = static_cast<uint32_t>(bd >> 32);
    is.idesc = g.idesc;
    is.row16 = static_cast<uint32_t>(g.HWP);
    is.half16 = static_cast<uint32_t>(g.HWH);
    is.kstep16 = 2u * (lbo_a >> 4);
    is.R = g.R; is.S = g.S;
    is.stride2 = !g.flat && g.stride == 2;
    is.ksteps = g.CK >> 5;
    is.blocks = g.MB;
    is.blk_b16 = static_cast<uint32_t>(g.b_bytes / g.MB) >> 4;
    return is;
}

__device__ __forceinline__ void umma_i8_words(uint32_t d_tmem, uint32_t a_lo, uint32_t a_hi, uint32_t b_lo, uint32_t b_hi,
                                              uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
        "mov.b64 da, {%1, %2};\n\t"
        "mov.b64 db, {%3, %4};\n\t"
        "setp.ne.b32 p, %6, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], da, db, %5, p;\n\t}"
        ::"r"(d_tmem), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate) : "memory");
}

// Fully unrolled issue of one layout block for the commonest shape classes (stride 1, two K steps per tap): no loop
// counters or branches between the MMAs of the lone issuing thread.
template <int R, int S, bool STRIDE2, int KS>
__device__ __forceinline__ void tc_issue_block_unrolled(const TcIssue& is, uint32_t arow, uint32_t b, uint32_t tmem_acc, uint32_t acc)
{
#pragma unroll
    for (int r = 0; r < R; ++r) {
#pragma unroll
        for (int sx = 0; sx < S; ++sx) {
            const uint32_t a = arow + (STRIDE2 ? static_cast<uint32_t>(sx & 1) * is.half16 + static_cast<uint32_t>(sx >> 1) : static_cast<uint32_t>(sx));
            umma_i8_words(tmem_acc, a, is.a_hi, b, is.b_hi, is.idesc, (r == 0 && sx == 0) ? acc : 1u);
            if (KS == 2) umma_i8_words(tmem_acc, a + is.kstep16, is.a_hi, b + 16, is.b_hi, is.idesc, 1u);
            b += 16 * KS;
        }
        arow += is.row16;
    }
}

__device__ __forceinline__ void tc_issue_chunk(const TcIssue& is, uint32_t ea, uint32_t ba, uint32_t tmem_acc, bool first_chunk)
{
    if (is.ksteps <= 2 && is.R == is.S && (is.R == 3 || is.R == 1)) {
        uint32_t arow0 = is.a_lo + (ea >> 4), b0 = is.b_lo + (ba >> 4), acc0 = first_chunk ? 0u : 1u;
        for (int blk = 0; blk < is.blocks; ++blk) {
            if (is.ksteps == 2) {
                if (is.R == 1) tc_issue_block_unrolled<1, 1, false, 2>(is, arow0, b0, tmem_acc, acc0);     // a lone tap has no column offset
                else if (is.stride2) tc_issue_block_unrolled<3, 3, true, 2>(is, arow0, b0, tmem_acc, acc0);
                else tc_issue_block_unrolled<3, 3, false, 2>(is, arow0, b0, tmem_acc, acc0);
            } else {
                if (is.R == 1) tc_issue_block_unrolled<1, 1, false, 1>(is, arow0, b0, tmem_acc, acc0);
                else if (is.stride2) tc_issue_block_unrolled<3, 3, true, 1>(is, arow0, b0, tmem_acc, acc0);
                else tc_issue_block_unrolled<3, 3, false, 1>(is, arow0, b0, tmem_acc, acc0);
            }
            acc0 = 1u;
            arow0 += static_cast<uint32_t>(is.ksteps) * is.kstep16;
            b0 += is.blk_b16;
        }
        return;
    }
    uint32_t acc = first_chunk ? 0u : 1u;          // the first MMA of a tile overwrites the accumulator
    uint32_t ablk = is.a_lo + (ea >> 4);
    uint32_t bblk = is.b_lo + (ba >> 4);
    for (int blk = 0; blk < is.blocks; ++blk) {
        uint32_t arow = ablk;
        uint32_t b = bblk;                         // filters of a block: [tap][K half] tiles of 16 x 16 bytes, one after the other
        for (int r = 0; r < is.R; ++r) {
            for (int sx = 0; sx < is.S; ++sx) {
                const uint32_t a = arow + (is.stride2 ? static_cast<uint32_t>(sx & 1) * is.half16 + static_cast<uint32_t>(sx >> 1)
                                                      : static_cast<uint32_t>(sx));
                // straight-line per tap: a loop over the K steps costs the lone issuing thread tens of cycles per MMA
                umma_i8_words(tmem_acc, a, is.a_hi, b, is.b_hi, is.idesc, acc);
                acc = 1u;
                b += 16;
                if (is.ksteps == 2) {
                    umma_i8_words(tmem_acc, a + is.kstep16, is.a_hi, b, is.b_hi, is.idesc, 1u);
                    b += 16;
                }
            }
            arow += is.row16;
        }
        ablk += static_cast<uint32_t>(is.ksteps) * is.kstep16;     // the block's 16-channel groups follow each other
        bblk += is.blk_b16;
    }
}

// Comparison-form epilogue of 32 accumulators of one pixel: plane bits of the 1- or 2-bit code into ow[0], ow[1].
template <bool SMALL, int RES>      // RES: 0 no residual, 1 residual of 1-2 bits, 2 residual of 3-4 bits
__device__ __forceinline__ void tc_compare_block(const uint32_t (&v)[32], const float2* sb32, const float4* s_bounds, const float4 bnd0,
                                                 const uint32_t (&rw)[4], uint32_t (&ow)[4])
{
    uint32_t w0 = 0, w1 = 0;
#pragma unroll
    for (int f = 0; f < 32; ++f) {
        const int acc = static_cast<int>(v[f]);
        const float2 sb = sb32[f];
        const float t = fmaf(SMALL ? int_to_float_exact(acc) : static_cast<float>(acc), sb.x, sb.y);
        float b0 = bnd0.x, b1 = bnd0.y, b2 = bnd0.z;
        if (RES != 0) {
            unsigned rpat = ((rw[0] >> f) & 1u) | (((rw[1] >> f) & 1u) << 1);      // planes beyond res_bits are zero
            if (RES == 2) rpat |= (((rw[2] >> f) & 1u) << 2) | (((rw[3] >> f) & 1u) << 3);
            const float4 bb = s_bounds[rpat];
            b0 = bb.x; b1 = bb.y; b2 = bb.z;
        }
        const uint32_t m1 = t >= b0 ? 0xffffffffu : 0u, m2 = t >= b1 ? 0xffffffffu : 0u, m3 = t >= b2 ? 0xffffffffu : 0u;
        w0 |= (m1 ^ m2 ^ m3) & (1u << f);      // count = c1 + c2 + c3 with c1 >= c2 >= c3: bit 0 is the parity
        w1 |= m2 & (1u << f);                  // bit 1 is c2
    }
    ow[0] = w0;
    ow[1] = w1;
}

// Integer form of the comparison epilogue.  t = fmaf((float)acc, scale, bias) is monotone in the integer accumulator
// when scale > 0, so "t >= bound" is "acc >= T" for the smallest accumulator T that satisfies it.  The thresholds are
// found per (residual pattern, filter) once per CTA: an estimate (bound - bias) / scale, corrected by evaluating the
// very fmaf of the formula at T - 1 and T until  f(T - 1) < bound <= f(T)  holds, which pins T exactly.  Accumulators
// and thresholds stay within +-2^29, so differences cannot overflow.  Anything unusual (scale <= 0, non-finite
// numbers, no convergence) clears *ok and the CTA keeps the floating-point comparison.
constexpr int TC_THR_LIM = 1 << 29;

__device__ __forceinline__ int tc_threshold(float s, float b, float bound, int* ok)
{
    if (!(bound == bound)) { *ok = 0; return TC_THR_LIM; }
    float x = (bound - b) / s;
    x = fminf(fmaxf(x, -6.0e8f), 6.0e8f);             // NaN cannot occur: s > 0 and b finite are checked by the caller
    int T = static_cast<int>(ceilf(x));
    T = T < -TC_THR_LIM ? -TC_THR_LIM : (T > TC_THR_LIM ? TC_THR_LIM : T);
    int it = 0;
    while (T > -TC_THR_LIM && fmaf(static_cast<float>(T - 1), s, b) >= bound && it < 8) { --T; ++it; }
    if (it == 8) *ok = 0;
    it = 0;
    while (T < TC_THR_LIM && !(fmaf(static_cast<float>(T), s, b) >= bound) && it < 8) { ++T; ++it; }
    if (it == 8) *ok = 0;
    return T;
}

// thr[filter * patterns + pattern] = (T1, T2, T3, -) for the filters of this CTA (the patterns of one filter share a
// 64-byte line, so lanes with different residuals do not collide on banks); called by `nthreads` threads (index `t`).
__device__ __forceinline__ void tc_build_thresholds(const TcArgs& g, int4* thr, int* ok, const float2* s_sb, const float4* s_bounds,
                                                    int o0, int t, int nthreads)
{
    if (g.thr_packed) {
        // entry (group of 32 filters, j = 0..15) serves filters j and j + 16 of the group: per level the word
        // (2^15 - T[j + 16]) << 16 | (2^15 - T[j]).  Thresholds are clamped to +-(acc_bound + 1), which decides the same
        // for every possible accumulator and keeps each 16-bit lane of  acc + 2^15 - T  inside (0, 2^16).
        const int lim = g.acc_bound + 1;
        for (int e = t; e < g.TN / 2; e += nthreads) {
            const int grp = e >> 4, j = e & 15;
            unsigned d[3] = {0u, 0u, 0u};
            for (int half = 0; half < 2; ++half) {
                const int f = grp * 32 + half * 16 + j;
                int T[3] = {lim, lim, lim};                                      // filters past O: never reached, masked anyway
                if (o0 + f < g.O) {
                    const float2 sb = s_sb[f];
                    if (!(sb.x > 0.0f) || !(sb.x < 3.0e38f) || !(fabsf(sb.y) < 3.0e38f)) {
                        *ok = 0;
                    } else {
                        const float4 bb = s_bounds[0];
                        T[0] = tc_threshold(sb.x, sb.y, bb.x, ok);
                        T[1] = tc_threshold(sb.x, sb.y, bb.y, ok);
                        T[2] = tc_threshold(sb.x, sb.y, bb.z, ok);
                    }
                }
                for (int k = 0; k < 3; ++k) {
                    const int Tc = T[k] < -lim ? -lim : (T[k] > lim ? lim : T[k]);
                    d[k] |= static_cast<unsigned>(32768 - Tc) << (16 * half);
                }
            }
            thr[e] = make_int4(static_cast<int>(d[0]), static_cast<int>(d[1]), static_cast<int>(d[2]), 0);
        }
        return;
    }
    for (int e = t; e < g.thr_pats * g.TN; e += nthreads) {
        const int f = e % g.TN, pat = e / g.TN;
        int4 T = make_int4(TC_THR_LIM, TC_THR_LIM, TC_THR_LIM, 0);         // filters past O: never reached, masked anyway
        if (o0 + f < g.O) {
            const float2 sb = s_sb[f];
            if (!(sb.x > 0.0f) || !(sb.x < 3.0e38f) || !(fabsf(sb.y) < 3.0e38f)) {
                *ok = 0;
            } else {
                const float4 bb = s_bounds[pat];
                T.x = tc_threshold(sb.x, sb.y, bb.x, ok);
                T.y = tc_threshold(sb.x, sb.y, bb.y, ok);
                T.z = tc_threshold(sb.x, sb.y, bb.z, ok);
            }
        }
        thr[f * g.thr_pats + pat] = T;
    }
}

__device__ __forceinline__ int4 lds_int4(uint32_t addr)
{
    int4 r;
    asm volatile("ld.shared.v4.s32 {%0, %1, %2, %3}, [%4];" : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "r"(addr));
    return r;
}
// Bits of the low half of x moved to the even bit positions.
__device__ __forceinline__ uint32_t spread16(uint32_t x)
{
    x &= 0xFFFFu;
    x = (x | (x << 8)) & 0x00FF00FFu;
    x = (x | (x << 4)) & 0x0F0F0F0Fu;
    x = (x | (x << 2)) & 0x33333333u;
    x = (x | (x << 1)) & 0x55555555u;
    return x;
}

// 32 accumulators of one pixel, two per 32-bit word (filters j and j + 16 in the 16-bit lanes), against packed thresholds:
// lane value acc + 2^15 - T_k has bit 15 set exactly when level k is reached, and no carry crosses the lanes.  Three
// additions, one xor and four shift/merge operations per PAIR of outputs, and half the threshold loads.
__device__ __forceinline__ void tc_compare_pairs(const uint32_t (&v)[32], uint32_t thr_addr, uint32_t (&ow)[4])
{
    uint32_t w0 = 0, w1 = 0;
#pragma unroll
    for (int j = 0; j < 16; ++j) {
        const uint32_t q = v[j + 16] * 65536u + v[j];           // (acc_hi << 16) + acc_lo as one integer sum
        const int4 D = lds_int4(thr_addr + j * 16);
        const uint32_t x1 = q + static_cast<uint32_t>(D.x), x2 = q + static_cast<uint32_t>(D.y), x3 = q + static_cast<uint32_t>(D.z);
        w1 = (w1 >> 1) | (x2 & 0x80008000u);                    // after 16 steps: filter j at bit j, filter j + 16 at bit 16 + j
        w0 = (w0 >> 1) | ((x1 ^ x2 ^ x3) & 0x80008000u);
    }
    ow[0] = w0;         // parity of the levels reached
    ow[1] = w1;         // level 2 reached
}

// 32 accumulators of one pixel against their integer thresholds.  The sign bit of acc - T_k says "below level k";
// a funnel shift collects it, so an output costs three subtractions, one three-way xor and two shifts.
// thr_addr: shared-memory address of the thresholds of filter 0 of this group of 32.
template <int RES>      // 0: no residual, 1: residual of 1-2 bits selects one of four threshold sets
__device__ __forceinline__ void tc_compare_int(const uint32_t (&v)[32], uint32_t thr_addr, const uint32_t (&rw)[4], uint32_t (&ow)[4])
{
    uint32_t w0 = 0, w1 = 0;
    // residual pattern of filter f at bits 2f, 2f+1 of (z_hi : z_lo)
    const uint32_t z_lo = RES ? (spread16(rw[0]) | (spread16(rw[1]) << 1)) : 0u;
    const uint32_t z_hi = RES ? (spread16(rw[0] >> 16) | (spread16(rw[1] >> 16) << 1)) : 0u;
#pragma unroll
    for (int f = 31; f >= 0; --f) {
        const uint32_t acc = v[f];
        int4 T;
        if (RES == 0) {
            T = lds_int4(thr_addr + f * 16);
        } else {
            const uint32_t z = f < 16 ? z_lo : z_hi;
            const int sh = 2 * (f & 15) - 4;                                  // pattern * 16 bytes
            const uint32_t off = (sh >= 0 ? (z >> sh) : (z << -sh)) & 0x30u;
            T = lds_int4(thr_addr + f * 64 + off);
        }
        const uint32_t d1 = acc - static_cast<uint32_t>(T.x), d2 = acc - static_cast<uint32_t>(T.y), d3 = acc - static_cast<uint32_t>(T.z);
        w1 = __funnelshift_l(d2, w1, 1);                 // (w1 << 1) | sign(d2)
        w0 = __funnelshift_l(d1 ^ d2 ^ d3, w0, 1);
    }
    ow[0] = ~w0;        // levels reached = 3 - (number of set signs): bit 0 is the complemented parity,
    ow[1] = ~w1;        // bit 1 is "level 2 reached"
}

// (scale, bias) of the CTA's filters, the comparison bounds and the "thresholds are valid" flag, written by the
// `nthreads` threads that run the epilogue (index t); the caller synchronises them afterwards.
__device__ __forceinline__ void tc_epilogue_tables(const TcArgs& g, unsigned char* tc_smem, float2* s_sb, float4* s_bounds, int o0,
                                                   int t, int nthreads)
{
    for (int f = t; f < g.TN; f += nthreads) {
        const int o = o0 + f;
        s_sb[f] = (g.out_packed && o < g.O) ? make_float2(g.scale[o], g.bias[o]) : make_float2(0.f, 0.f);
    }
    if (t < 16) s_bounds[t] = make_float4(g.rb.bound[t][0], g.rb.bound[t][1], g.rb.bound[t][2], 0.f);
    if (t == 32 && g.off_thr) *reinterpret_cast<int*>(tc_smem + g.off_thr + g.thr_pats * g.TN * 16) = 1;
}

// Where accumulator row m (= tensor-memory lane = tile pixel) sits inside a 2-D tile: image of the stack, row, column.
// Depends on the thread only, so it is found once per kernel (stacked small images need a division).
struct TcEpiThread { int ni, ty, tx; };

__device__ __forceinline__ TcEpiThread tc_epi_thread(const TcArgs& g, int m)
{
    TcEpiThread t;
    const int grp = m >> 3;
    t.tx = m & 7; t.ni = 0; t.ty = grp;
    if (!g.flat && g.GI != 16) { t.ni = grp / g.GI; t.ty = grp - t.ni * g.GI; }
    return t;
}

// Epilogue of one tile: thread `tid` (0..127, warp = TMEM lane quadrant) owns accumulator row tid = one output pixel.
__device__ __forceinline__ void tc_epilogue_tile(const TcArgs& g, uint32_t tmem_acc, int tid, int warp, const TcTile& tile, const TcEpiThread& et,
                                                 int o0, const float2* s_sb, const float4* s_bounds, uint32_t thr_addr, int cc0 = 0,
                                                 int ccstep = 1, int trace_tile = -1, bool res_l2 = false, unsigned char* stage = nullptr)
{
    const int n0 = tile.n0, p0 = tile.p0, q0 = tile.q0;
    const int m = tid;                               // TMEM lane = tile pixel
    int n = 0, p = 0, q = 0;
    bool valid;
    size_t pix;
    if (g.flat) {
        // a flat tile is 128 consecutive pixels of the [N][P][Q] order: the pixel index is all the packed output and the
        // NHWC accumulators need; (n, p, q) cost two divisions and are found only for NCHW accumulators
        const unsigned upix = static_cast<unsigned>(q0) + static_cast<unsigned>(m);      // N*P*Q < 2^31 (checked on the host)
        valid = upix < static_cast<unsigned>(g.N) * static_cast<unsigned>(g.P * g.Q);
        pix = upix;
        if (g.out_i32 && !g.i32_nhwc) {
            const unsigned hwsz = static_cast<unsigned>(g.P * g.Q);
            n = static_cast<int>(upix / hwsz);
            const unsigned rem = upix - static_cast<unsigned>(n) * hwsz;
            p = static_cast<int>(rem / static_cast<unsigned>(g.Q));
            q = static_cast<int>(rem - static_cast<unsigned>(p) * static_cast<unsigned>(g.Q));
        }
    } else {
        const int ni = et.ni, ty = et.ty, tx = et.tx;                        // stacked small images: ni > 0
        n = n0 + ni; p = p0 + ty; q = q0 + tx;
        valid = n < g.N && p < g.P && q < g.Q && ni < g.TNI && (g.GI == 16 || ty < g.P);
        pix = (static_cast<size_t>(n) * g.P + p) * g.Q + q;
    }
    int qmin, qmax;
    code_limits(g.out_bits > 0 ? g.out_bits : 1, g.out_sign, qmin, qmax);
    const float fqmin = static_cast<float>(qmin), fqmax = static_cast<float>(qmax);
    const float4 bnd0 = s_bounds[0];
    for (int cc = cc0; cc < g.TN / 32; cc += ccstep) {       // groups of 32 filters; two warps may share a lane quadrant
        uint32_t v[32];
        tmem_ld32(tmem_acc + (static_cast<uint32_t>(warp * 32) << 16) + static_cast<uint32_t>(cc * 32), v);
        tmem_ld_wait();
        if (tid == 0 && cc == cc0) TC_TRACE(TR_E_LD, trace_tile);
        const int ob = o0 + cc * 32;
        // Flat tiles with channel-innermost int32 outputs (matrix products): the 32 x 32 block of this warp goes through 4 KB of
        // shared memory so that a store instruction writes four whole 128-byte lines (eight lanes per row) instead of 16 bytes of 32
        // different lines.  16-byte chunks are swizzled by the row, which keeps both passes free of bank conflicts.
        const bool staged = stage != nullptr && g.out_i32 && g.i32_nhwc && g.flat && (g.O & 3) == 0 && g.O - ob >= 32;      // warp-uniform
        if (staged) {
            uint4* sw = reinterpret_cast<uint4*>(stage);
            const int l = tid & 31;
#pragma unroll
            for (int c = 0; c < 8; ++c) sw[l * 8 + (c ^ (l & 7))] = make_uint4(v[4 * c], v[4 * c + 1], v[4 * c + 2], v[4 * c + 3]);
            __syncwarp();
            const unsigned row0 = static_cast<unsigned>(q0) + static_cast<unsigned>(tid & ~31);
            const unsigned npix = static_cast<unsigned>(g.N) * static_cast<unsigned>(g.P * g.Q);
#pragma unroll
            for (int it = 0; it < 8; ++it) {
                const int rr = it * 4 + (l >> 3), ch = l & 7;
                const uint4 val = sw[rr * 8 + (ch ^ (rr & 7))];
                const unsigned upix = row0 + static_cast<unsigned>(rr);
                if (upix < npix) *reinterpret_cast<uint4*>(g.out_i32 + static_cast<size_t>(upix) * g.O + ob + ch * 4) = val;
            }
            __syncwarp();                 // the next group of 32 filters reuses the block
        }
        if (valid && ob < g.O) {
        if (g.out_i32 && !staged) {
            if (g.i32_nhwc && (g.O & 3) == 0 && g.O - ob >= 32) {
                // channel-innermost accumulators: the 32 values of this thread are 128 contiguous, 16-byte aligned bytes
                uint4* dst4 = reinterpret_cast<uint4*>(g.out_i32 + pix * g.O + ob);
#pragma unroll
                for (int f = 0; f < 8; ++f) dst4[f] = make_uint4(v[4 * f], v[4 * f + 1], v[4 * f + 2], v[4 * f + 3]);
            } else {
#pragma unroll
                for (int f = 0; f < 32; ++f) {
                    const int o = ob + f;
                    if (o < g.O) {
                        const size_t idx = g.i32_nhwc ? pix * g.O + o : ((static_cast<size_t>(n) * g.O + o) * g.P + p) * g.Q + q;
                        g.out_i32[idx] = static_cast<int>(v[f]);
                    }
                }
            }
        }
        if (g.out_packed) {
            uint32_t rw[4] = {0, 0, 0, 0};
            if (g.residual) {
                const uint32_t* rp = g.residual + (pix * g.res_cw_total + ((g.res_c_off + ob) >> 5)) * g.res_bits;
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    if (j < g.res_bits) rw[j] = res_l2 ? __ldcg(rp + j) : rp[j];     // inside a chain another SM may just have written it: read at L2
            }
            uint32_t ow[4] = {0, 0, 0, 0};
            if (g.rb.enabled) {
                // comparison form: t = fmaf(acc, scale, bias) against the bounds of the residual pattern.  The
                // uniform switches are resolved once per 32 outputs, so the unrolled body is straight-line code.
                const unsigned valid_mask = (g.O - ob >= 32) ? 0xffffffffu : ((1u << (g.O - ob)) - 1u);
                const float2* sb32 = s_sb + cc * 32;
                if (thr_addr && g.thr_packed) {
                    tc_compare_pairs(v, thr_addr + cc * 256, ow);
                } else if (thr_addr) {
                    if (!g.residual) tc_compare_int<0>(v, thr_addr + cc * 512, rw, ow);
                    else tc_compare_int<1>(v, thr_addr + cc * 2048, rw, ow);
                } else if (!g.residual) {
                    if (g.acc_small) tc_compare_block<true, 0>(v, sb32, s_bounds, bnd0, rw, ow);
                    else tc_compare_block<false, 0>(v, sb32, s_bounds, bnd0, rw, ow);
                } else if (g.res_bits <= 2) {
                    if (g.acc_small) tc_compare_block<true, 1>(v, sb32, s_bounds, bnd0, rw, ow);
                    else tc_compare_block<false, 1>(v, sb32, s_bounds, bnd0, rw, ow);
                } else {
                    if (g.acc_small) tc_compare_block<true, 2>(v, sb32, s_bounds, bnd0, rw, ow);
                    else tc_compare_block<false, 2>(v, sb32, s_bounds, bnd0, rw, ow);
                }
                ow[0] = (ow[0] ^ ((g.rb.flip & 1u) ? 0xffffffffu : 0u)) & valid_mask;
                ow[1] = (ow[1] ^ ((g.rb.flip & 2u) ? 0xffffffffu : 0u)) & valid_mask;
            } else {
#pragma unroll
            for (int f = 0; f < 32; ++f) {
                if (ob + f < g.O) {
                    const int acc = static_cast<int>(v[f]);
                    const float2 sb = s_sb[cc * 32 + f];
                    float val = fmaf(g.acc_small ? int_to_float_exact(acc) : static_cast<float>(acc), sb.x, sb.y);
                    if (g.residual) {
                        unsigned rpat = 0;
#pragma unroll
                        for (int j = 0; j < 4; ++j)
                            if (j < g.res_bits) rpat |= ((rw[j] >> f) & 1u) << j;
                        val = fmaf(g.res_scale, static_cast<float>(pattern_value(rpat, g.res_bits, g.res_sign)), val);
                    }
                    if (g.relu) val = fmaxf(val, 0.0f);
                    int code;
                    if (g.out_sign == BS_BIPOLAR) code = val >= 0.0f ? 1 : -1;
                    else code = small_float_to_int_rn(fminf(fmaxf(val, fqmin), fqmax));
                    const unsigned pat = stored_pattern(code, g.out_bits, g.out_sign);
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        if (j < g.out_bits) ow[j] |= ((pat >> j) & 1u) << f;
                }
            }
            }
            uint32_t* dst = g.out_packed + (pix * g.out_cw_total + g.out_cw_off + (ob >> 5)) * g.out_bits;
#pragma unroll
            for (int j = 0; j < 4; ++j)
                if (j < g.out_bits) dst[j] = ow[j];
        }
        }
        __syncwarp();                 // the next tcgen05.ld is warp-collective
        if (tid == 0 && cc == cc0) TC_TRACE(TR_E_ST, trace_tile);
    }
}

// ----------------------------------------------------------------------------- one tile per CTA (filters streamed per chunk)

// SEG: the packed rows of a flat tile are staged in segments (matrix products with a long reduction, see the plan); a
// template parameter so that the common instantiation carries none of that code (with a run-time switch the residual stack
// measured 1.2 % slower).
template <int A, bool SEG>
__global__ void __launch_bounds__(TC_THREADS) bitserial_conv_tc_kernel(const __grid_constant__ TcArgs g)
{
    extern __shared__ __align__(128) unsigned char tc_smem[];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int RS = g.R * g.S;
    const int stage_p_bytes = g.b_bytes;                                    // filter ring; the packed tile sits at off_p
    float2* s_sb = reinterpret_cast<float2*>(tc_smem + g.off_sb);           // (scale, bias) per filter of the tile
    float4* s_bounds = reinterpret_cast<float4*>(tc_smem + g.off_sb + g.TN * 8);   // comparison bounds per residual pattern
    uint2* s_lut = reinterpret_cast<uint2*>(tc_smem + g.off_lut);
    uint64_t* bars = reinterpret_cast<uint64_t*>(tc_smem + g.off_bar);
    uint64_t* full_p = bars;                       // [TC_MAX_STAGES]
    uint64_t* empty_p = bars + TC_MAX_STAGES;
    uint64_t* full_e = bars + 2 * TC_MAX_STAGES;
    uint64_t* empty_e = bars + 3 * TC_MAX_STAGES;
    uint64_t* accum_full = bars + 4 * TC_MAX_STAGES;
    uint64_t* full_a = bars + 4 * TC_MAX_STAGES + 1;      // [2] packed tile (or segment of its rows) landed
    uint64_t* empty_a = bars + 4 * TC_MAX_STAGES + 3;     // [2] segment buffer expanded (segmented rows only)
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 4 * TC_MAX_STAGES + 5);

    const int o0 = static_cast<int>(blockIdx.x % static_cast<unsigned>(g.tiles_o)) * g.TN;   // filter tile fastest
    const int tiles_m = g.tiles_q * g.tiles_p * g.tiles_n;
    const int mt0 = static_cast<int>(blockIdx.x / static_cast<unsigned>(g.tiles_o)) * g.PT;      // first pixel tile of this CTA
    const int nt = tiles_m - mt0 < g.PT ? tiles_m - mt0 : g.PT;                                   // 1..PT pixel tiles
    const int e_stage = g.PT * g.e_bytes;

    if (tid == 0) TC_TRACE(TR_START, 0);
    pdl_release();
    if (tid == 0) {
        for (int s = 0; s < TC_MAX_STAGES; ++s) {
            mbar_init(&full_p[s], 1);
            mbar_init(&empty_p[s], 1);
            mbar_init(&full_e[s], 1);
            mbar_init(&empty_e[s], 1);
        }
        mbar_init(accum_full, 1);
        mbar_init(&full_a[0], static_cast<unsigned>(nt));
        if (SEG) {
            mbar_init(&full_a[1], 1);
            mbar_init(&empty_a[0], 1);
            mbar_init(&empty_a[1], 1);
        }
        fence_barrier_init();
        fence_proxy_async();
    }
    if (warp == 5) {
        tmem_alloc(tmem_slot, static_cast<unsigned>(g.tmem_cols));
        tmem_relinquish();
    }
    // Only the barriers and the tensor-memory address are needed by every role: the producer starts fetching right
    // after this barrier; the byte table and the scale/bias/bounds tables are set up by the warps that use them.
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (SEG && warp == 4) {
        // ------------------------------------------------------------------ producer, rows staged in segments
        // A matrix product with a long reduction: the packed rows of the tile are too large to stay resident (4608 channels at
        // 2 bits: 147 KB), so they are fetched seg_words per row at a time into two buffers.  The 128 row pieces of a segment
        // are separate bulk copies, four per lane, requested one segment ahead of the expanders.
        const int early = g.nchunks < g.nsp ? g.nchunks : g.nsp;
        const int blk_bytes = g.b_bytes / g.MB;
        const size_t blk_stride = static_cast<size_t>(g.opad8) * RS * (g.CK >> 4) * 128;
        const int8_t* src = g.wgt + static_cast<size_t>(o0 >> 3) * RS * (g.CK >> 4) * 128;
        const int seg_bytes = g.pa_bytes / 2;
        const TcTile tile = tc_decode_tile(g, mt0);
        const long long npix = static_cast<long long>(g.N) * g.P * g.Q;
        const int rows = static_cast<int>(npix - tile.q0 < TC_M ? npix - tile.q0 : TC_M);
        auto load_segment = [&](int sg) {
            const int w0 = sg * g.seg_words;
            const int words = g.fullA - w0 < g.seg_words ? g.fullA - w0 : g.seg_words;
            uint64_t* bar = &full_a[sg & 1];
            if (lane == 0) mbar_expect_tx(bar, static_cast<unsigned>(rows) * static_cast<unsigned>(words) * 4u);
            __syncwarp();
            unsigned char* dst = tc_smem + g.off_p + (sg & 1) * seg_bytes;
            for (int r = lane; r < rows; r += 32)
                bulk_load(dst + static_cast<size_t>(r) * g.seg_words * 4, g.act + (static_cast<size_t>(tile.q0) + r) * g.fullA + w0,
                          static_cast<unsigned>(words) * 4u, bar);
        };
        TcRing rp;
        unsigned ok = 1;
        for (int c = 0; c < g.nchunks; ++c) {
            if (c == early) {
                pdl_acquire();
                load_segment(0);
                if (g.nseg > 1) load_segment(1);
            }
            if (lane == 0) {
                ok = mbar_spin_bounded(&empty_p[rp.idx], rp.phase ^ 1u) ? 1u : 0u;
                if (ok) {
                    TC_TRACE(TR_LOAD, c);
                    mbar_expect_tx(&full_p[rp.idx], static_cast<unsigned>(g.b_bytes));
                    for (int j = 0; j < g.MB; ++j, src += blk_stride)
                        bulk_load(tc_smem + rp.idx * stage_p_bytes + j * blk_bytes, src, static_cast<unsigned>(blk_bytes), &full_p[rp.idx]);
                }
            }
            ok = __shfl_sync(0xffffffffu, ok, 0);
            if (!ok) break;
            rp.advance(g.nsp);
            if (c >= early && c % g.seg_chunks == 0 && c / g.seg_chunks >= 1 && c / g.seg_chunks + 1 < g.nseg) {
                // the filters of the first chunk of segment c / seg_chunks are on their way, so the expanders are about to leave
                // the segment before it: its buffer takes the segment after this one (needed a whole segment from now)
                const int sg = c / g.seg_chunks + 1;
                if (lane == 0) ok = mbar_spin_bounded(&empty_a[sg & 1], ((sg >> 1) - 1) & 1) ? 1u : 0u;
                ok = __shfl_sync(0xffffffffu, ok, 0);
                if (!ok) break;
                load_segment(sg);
            }
        }
        if (!ok && lane == 0) atomicOr(g.status, STATUS_TIMEOUT);
        __syncwarp();
    } else if (warp == 4) {
        // ------------------------------------------------------------------ producer
        if (lane == 0) {
            // the first ring of filter chunks does not depend on the preceding kernel: fetch it before waiting for it
            const int early = g.nchunks < g.nsp ? g.nchunks : g.nsp;
            const int blk_bytes = g.b_bytes / g.MB;
            const size_t blk_stride = static_cast<size_t>(g.opad8) * RS * (g.CK >> 4) * 128;      // one layout block, all filters
            const int8_t* src = g.wgt + static_cast<size_t>(o0 >> 3) * RS * (g.CK >> 4) * 128;
            TcRing rp;
            for (int c = 0; c < g.nchunks; ++c) {
                if (c == early) {
                    pdl_acquire();
                    for (int t = 0; t < nt; ++t) tc_load_tile(g, tc_smem + g.off_p + t * g.pa_bytes, full_a, tc_decode_tile(g, mt0 + t));
                }
                if (!mbar_spin_bounded(&empty_p[rp.idx], rp.phase ^ 1u)) { atomicOr(g.status, STATUS_TIMEOUT); break; }
                TC_TRACE(TR_LOAD, c);
                mbar_expect_tx(&full_p[rp.idx], static_cast<unsigned>(g.b_bytes));
                for (int j = 0; j < g.MB; ++j, src += blk_stride)
                    bulk_load(tc_smem + rp.idx * stage_p_bytes + j * blk_bytes, src, static_cast<unsigned>(blk_bytes), &full_p[rp.idx]);
                rp.advance(g.nsp);
            }
            if (early == g.nchunks) {
                pdl_acquire();
                for (int t = 0; t < nt; ++t) tc_load_tile(g, tc_smem + g.off_p + t * g.pa_bytes, full_a, tc_decode_tile(g, mt0 + t));
            }
        }
        __syncwarp();
    } else if (warp == 5) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            const uint32_t e_base = smem_u32(tc_smem + g.off_e), p_base = smem_u32(tc_smem);
            const TcIssue is = tc_make_issue(g);
            const int nmt = g.TN / g.NM;
            const uint32_t nm_b_bytes = static_cast<uint32_t>(g.NM >> 3) * static_cast<uint32_t>(RS * (g.CK >> 4)) * 128u;   // NM / 8 groups of 8 filters
            TcRing rp, re;
            for (int c = 0; c < g.nchunks; ++c) {
                if (!(mbar_spin_bounded(&full_p[rp.idx], rp.phase) && mbar_spin_bounded(&full_e[re.idx], re.phase))) {
                    atomicOr(g.status, STATUS_TIMEOUT);
                    break;
                }
                TC_TRACE(TR_MBEG, c);
                tc_fence_after();
                for (int t = 0; t < nt; ++t)
                    for (int nm = 0; nm < nmt; ++nm)      // a tile wider than one MMA: the same expanded chunk against each slice of NM filters
                        tc_issue_chunk(is, e_base + static_cast<uint32_t>(re.idx * e_stage + t * g.e_bytes),
                                       p_base + static_cast<uint32_t>(rp.idx * stage_p_bytes) + static_cast<uint32_t>(nm) * nm_b_bytes,
                                       tmem_base + static_cast<uint32_t>(t * g.TN + nm * g.NM), c == 0);
                umma_commit(&empty_e[re.idx]);
                umma_commit(&empty_p[rp.idx]);
                TC_TRACE(TR_MEND, c);
                rp.advance(g.nsp);
                re.advance(g.nse);
            }
            umma_commit(accum_full);      // arrives when every MMA issued above has completed
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------------ expanders (warps 0-3, 6-9), then epilogue
        pdl_acquire();                    // the epilogue reads the residual and overwrites buffers the preceding kernel may use
        const int ct = warp < 4 ? tid : tid - 64;          // 0..255 among the workers
        tc_build_lut(g, s_lut, ct, TC_WORKERS);
        tc_epilogue_tables(g, tc_smem, s_sb, s_bounds, o0, ct, TC_WORKERS);
        group_sync(1, TC_WORKERS);
        const TcExpand xp = tc_expand_init(g, ct, TC_WORKERS);
        const TcEpiThread eth = tc_epi_thread(g, (warp & 3) * 32 + lane);
        if (tid == 0) TC_TRACE(TR_SETUP, 0);
        bool ok = SEG ? true : mbar_wait_warp(&full_a[0], 0, lane);
        if (tid == 0) TC_TRACE(TR_PDL, 0);
        TcRing re;
        int sg = 0, cl = 0;               // segmented rows: segment and chunk within it
        for (int c = 0; c < g.nchunks; ++c) {
            if (SEG && cl == 0 && ok) ok = mbar_wait_warp(&full_a[sg & 1], (sg >> 1) & 1, lane);
            if (ok) ok = mbar_wait_warp(&empty_e[re.idx], re.phase ^ 1u, lane);
            if (!ok) atomicOr(g.status, STATUS_TIMEOUT);
            if (tid == 0) TC_TRACE(TR_XBEG, c);
            if (SEG) {
                tc_expand_chunk<A>(g, xp, reinterpret_cast<const uint32_t*>(tc_smem + g.off_p + (sg & 1) * (g.pa_bytes / 2)),
                                   tc_smem + g.off_e + re.idx * e_stage, s_lut, ct, cl);
            } else {
                for (int t = 0; t < nt; ++t)
                    tc_expand_chunk<A>(g, xp, reinterpret_cast<const uint32_t*>(tc_smem + g.off_p + t * g.pa_bytes),
                                       tc_smem + g.off_e + re.idx * e_stage + t * g.e_bytes, s_lut, ct, c);
            }
            fence_proxy_async();          // make the generic-proxy writes visible to the tensor core's reads
            group_sync(1, TC_WORKERS);
            if (tid == 0) TC_TRACE(TR_XEND, c);
            if (tid == 0) mbar_arrive(&full_e[re.idx]);
            re.advance(g.nse);
            if (SEG && ++cl == g.seg_chunks) {
                if (tid == 0) mbar_arrive(&empty_a[sg & 1]);      // after the group barrier: every thread has read the segment
                cl = 0;
                ++sg;
            }
        }
        // the last chunks are still in the tensor core: time to turn the comparison bounds into integer thresholds
        uint32_t thr = 0;                 // shared-memory address of the thresholds, 0: floating-point comparison
        if (g.off_thr) {
            int4* s_thr = reinterpret_cast<int4*>(tc_smem + g.off_thr);
            int* thr_ok = reinterpret_cast<int*>(s_thr + g.thr_pats * g.TN);
            tc_build_thresholds(g, s_thr, thr_ok, s_sb, s_bounds, o0, ct, TC_WORKERS);
            group_sync(1, TC_WORKERS);
            if (*thr_ok) thr = smem_u32(s_thr);
        }
        if (tid == 0) TC_TRACE(TR_E_CMP, 0);
        if (ok) ok = mbar_wait_warp(accum_full, 0, lane);
        if (!ok) atomicOr(g.status, STATUS_TIMEOUT);
        if (tid == 0) TC_TRACE(TR_EBEG, 0);
        tc_fence_after();
        // every MMA has completed, so the filter ring is free: each of the eight warps takes 4 KB of it to stage its int32 stores
        unsigned char* i32_stage = nullptr;
        if (g.flat && g.out_i32 && g.nsp * g.b_bytes >= 8 * 4096) {
            fence_proxy_async();          // the ring was last written by bulk copies
            i32_stage = tc_smem + (warp < 4 ? warp : warp - 2) * 4096;
        }
        for (int t = 0; t < nt; ++t)
            // a warp reads the tensor-memory lanes of quadrant (warp % 4): warps 0-3 take the even groups of 32 filters,
            // warps 6-9 (quadrants 2, 3, 0, 1) the odd ones
            tc_epilogue_tile(g, tmem_base + static_cast<uint32_t>(t * g.TN), (warp & 3) * 32 + lane, warp & 3, tc_decode_tile(g, mt0 + t), eth, o0,
                             s_sb, s_bounds, thr, warp < 4 ? 0 : 1, 2, -1, false, i32_stage);
        if (tid == 0) TC_TRACE(TR_EEND, 0);
        tc_fence_before();
    }
    __syncthreads();
    if (tid == 0) TC_TRACE(TR_END, 0);
    if (warp == 5) {
        tc_fence_after();
        tmem_dealloc(tmem_base, static_cast<unsigned>(g.tmem_cols));
    }
}

// ----------------------------------------------------------------------------- persistent CTAs, filters resident
//
// A CTA keeps the int8 filters of its filter tile (all channel chunks) in shared memory and walks over pixel tiles.
// A chain of layers run by one launch: the same geometry in every layer (stride 1, output as large as the input, same
// channels and filters), so that all layers share one shared-memory plan and one tiling, and a pixel tile of layer l + 1
// reads only its own and the adjacent pixel tiles of layer l.  The work items (layer, pixel tile) are numbered layer by
// layer and dealt to the CTAs round-robin; every role of a CTA walks its items in that order, the pipeline rings simply
// continue across a layer boundary and only the filters are swapped.  What keeps the order of the layers is a counter
// per (layer, pixel tile) in global memory, raised by the epilogue once the tile's outputs are stored; the producer
// of a CTA waits (bounded) for the up to nine counters its next halo depends on.  All CTAs of the grid are resident
// at once (the host sizes the grid by the occupancy of the kernel), and an item only ever waits for items that come
// earlier in the common order, so the CTA holding the earliest unfinished item can always proceed.
// MAXL = 1 is the plain one-layer kernel: no counters, no waits.
constexpr int TC_CHAIN_MAX = 4;

template <int MAXL>
struct TcChainArgs {
    TcArgs L[MAXL];
    int nlayers;
    unsigned* flags;       // [nlayers][pixel tiles] filter tiles finished, summed over all launches on this workspace
    unsigned* ctl;         // [0] launches completed on this workspace, [1] CTAs of the running launch that have finished
};

__device__ __forceinline__ unsigned ld_acquire_gpu(const unsigned* p)
{
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void fence_proxy_async_global() { asm volatile("fence.proxy.async.global;" ::: "memory"); }

// Bounded wait until the counter has reached `target` (wrap-safe).  About a second before it gives up.
__device__ __forceinline__ bool tc_flag_wait(const unsigned* flag, unsigned target)
{
    for (unsigned it = 0; it < (1u << 22); ++it) {
        if (static_cast<int>(ld_acquire_gpu(flag) - target) >= 0) return true;
        __nanosleep(200);
    }
    return false;
}

// Position of a role in the item sequence of its CTA: layer and pixel tile, advanced without divisions.
struct TcItemWalker {
    TcTileWalker w;            // tile within the layer (w.mt is the tile index inside the layer)
    int l, dl;                 // layer, and whole layers per step
};

__device__ __forceinline__ TcItemWalker tc_item_init(const TcArgs& g, int first, int step, int tiles_m)
{
    TcItemWalker x;
    x.l = first / tiles_m; x.dl = step / tiles_m;
    x.w = tc_walk_init(g, first - x.l * tiles_m, step - x.dl * tiles_m);
    return x;
}
__device__ __forceinline__ void tc_item_next(const TcArgs& g, TcItemWalker& x, int tiles_m)
{
    tc_walk_next(g, x.w);
    x.l += x.dl;
    if (x.w.mt >= tiles_m) { x.w.mt -= tiles_m; x.w.in -= g.tiles_n; ++x.l; }
}

// Warps 0-3: epilogue (TMEM lane quadrants), warps 4-7: bitplane expansion, warp 8: TMA producer, warp 9: MMA issuer.
// Packed and expanded activation chunks travel through two mbarrier rings; two TMEM accumulator buffers let the
// epilogue of tile i overlap the MMAs of tile i + 1.

constexpr int TCP_THREADS = 320;
constexpr int TCP_THREADS_WIDE = 448;   // with a second set of four epilogue warps (10-13)
constexpr int TCP_NSP = 3;            // packed-tile ring (at most)
constexpr int TCP_NSE = 3;            // expanded-chunk ring (at most)

// CPS: CTAs per SM the registers are budgeted for (3: 64 registers per thread; 1: no cap, for plans whose shared memory
// leaves room for one or two CTAs anyway).
// WIDE: eight epilogue warps (0-3 and 10-13, two per tensor-memory lane quadrant, sharing the groups of 32 filters).
template <int A, int CPS, bool WIDE, int MAXL>
__global__ void __launch_bounds__(WIDE ? TCP_THREADS_WIDE : TCP_THREADS, CPS)
bitserial_conv_tc_persistent_kernel(const __grid_constant__ TcChainArgs<MAXL> ch)
{
    extern __shared__ __align__(128) unsigned char tc_smem[];
    const TcArgs& g0 = ch.L[0];                     // geometry, tiling and shared-memory plan: the same in every layer
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int RS = g0.R * g0.S;
    unsigned char* s_w = tc_smem;                                               // [nchunks][b_bytes]
    unsigned char* s_p = tc_smem + g0.off_p;                                    // [nsp][pa_bytes] packed tiles
    unsigned char* s_e = tc_smem + g0.off_e;                                    // [nse][e_bytes]
    float2* s_sb = reinterpret_cast<float2*>(tc_smem + g0.off_sb);
    float4* s_bounds = reinterpret_cast<float4*>(tc_smem + g0.off_sb + g0.TN * 8);
    uint2* s_lut = reinterpret_cast<uint2*>(tc_smem + g0.off_lut);
    uint64_t* bars = reinterpret_cast<uint64_t*>(tc_smem + g0.off_bar);
    uint64_t* full_p = bars;                        // [TCP_NSP]
    uint64_t* empty_p = bars + TCP_NSP;             // [TCP_NSP]
    uint64_t* full_e = bars + 2 * TCP_NSP;          // [TCP_NSE]
    uint64_t* empty_e = full_e + TCP_NSE;           // [TCP_NSE]
    uint64_t* full_acc = empty_e + TCP_NSE;         // [2]
    uint64_t* empty_acc = full_acc + 2;             // [2]
    uint64_t* wgt_full = empty_acc + 2;             // [1] filters of the current layer have landed
    uint64_t* wgt_free = wgt_full + 1;              // [1] every MMA that reads the filters of the layer just finished has completed
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(wgt_free + 1);

    const int nlayers = MAXL > 1 ? ch.nlayers : 1;
    const int o0 = static_cast<int>(blockIdx.x % static_cast<unsigned>(g0.tiles_o)) * g0.TN;
    const int first_tile = static_cast<int>(blockIdx.x / static_cast<unsigned>(g0.tiles_o));
    const int tile_step = static_cast<int>(gridDim.x / static_cast<unsigned>(g0.tiles_o));
    const int tiles_m = g0.tiles_q * g0.tiles_p * g0.tiles_n;
    const int items = nlayers * tiles_m;

    if (tid == 0) TC_TRACE(TR_START, 0);
    pdl_release();
    if (tid == 0) {
        for (int s = 0; s < TCP_NSP; ++s) { mbar_init(&full_p[s], 1); mbar_init(&empty_p[s], 1); }
        for (int s = 0; s < TCP_NSE; ++s) { mbar_init(&full_e[s], 1); mbar_init(&empty_e[s], 1); }
        for (int s = 0; s < 2; ++s) { mbar_init(&full_acc[s], 1); mbar_init(&empty_acc[s], 1); }
        mbar_init(wgt_full, 1);
        mbar_init(wgt_free, 1);
        fence_barrier_init();
        fence_proxy_async();
    }
    if (warp == 9) {
        tmem_alloc(tmem_slot, static_cast<unsigned>(g0.tmem_cols));
        tmem_relinquish();
    }
    // Only the barriers and the tensor-memory address are needed by every role: the producer starts fetching right
    // after this barrier; the byte table and the scale/bias/bounds tables are set up by the warps that use them.
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (MAXL == 1 && warp == 8) {
        // ------------------------------------------------------------------ producer of the one-layer kernel: filters once, then packed tiles
        if (lane == 0) {
            mbar_expect_tx(wgt_full, static_cast<unsigned>(g0.nchunks * g0.b_bytes));
            const int blk_bytes = g0.b_bytes / g0.MB;
            const size_t blk_stride = static_cast<size_t>(g0.opad8) * RS * (g0.CK >> 4) * 128;     // one layout block, all filters
            const int8_t* src = g0.wgt + static_cast<size_t>(o0 >> 3) * RS * (g0.CK >> 4) * 128;
            unsigned char* dst = s_w;
            for (int c = 0; c < g0.nchunks * g0.MB; ++c, src += blk_stride, dst += blk_bytes)      // layout blocks, consecutive in shared memory
                bulk_load(dst, src, static_cast<unsigned>(blk_bytes), wgt_full);
            TC_TRACE(TR_SETUP, 0);
            pdl_acquire();                // activations come from the preceding kernel; the filters above do not
            TC_TRACE(TR_PDL, 0);
            TcTileWalker tw = tc_walk_init(g0, first_tile, tile_step);
            TcRing rp;
            bool ok = true;
            for (int i = 0; tw.mt < tiles_m; tc_walk_next(g0, tw), ++i) {
                if (!mbar_spin_bounded(&empty_p[rp.idx], rp.phase ^ 1u)) { ok = false; break; }
                TC_TRACE(TR_LOAD, i);
                tc_load_tile(g0, s_p + rp.idx * g0.pa_bytes, &full_p[rp.idx], tc_walk_tile(g0, tw));
                rp.advance(g0.nsp);
            }
            if (!ok) atomicOr(g0.status, STATUS_TIMEOUT);
        }
        __syncwarp();
    } else if (warp == 8) {
        // ------------------------------------------------------------------ producer of a chain: packed tiles, in item order
        if (lane == 0) TC_TRACE(TR_SETUP, 0);
        pdl_acquire();                    // activations come from the preceding kernel
        if (lane == 0) TC_TRACE(TR_PDL, 0);
        unsigned target = 0;
        if (MAXL > 1 && nlayers > 1) target = (ld_acquire_gpu(ch.ctl) + 1u) * static_cast<unsigned>(g0.tiles_o);
        TcItemWalker x = tc_item_init(g0, first_tile, tile_step, tiles_m);
        TcRing rp;
        bool ok = true;
        int i = 0;
        // One copy of the loop per layer: the layer's arguments are then read at fixed offsets of the parameter block
        // (operands of the instructions) instead of being fetched through a run-time index after every barrier.
#pragma unroll
        for (int l = 0; l < MAXL; ++l) {
            const TcArgs& g = ch.L[l];
            for (; ok && x.l == l && l < nlayers; tc_item_next(g0, x, tiles_m), ++i) {
                if (MAXL > 1 && l > 0) {
                    // the halo of this tile was written by the tile itself and its neighbours in the preceding layer
                    bool mine = true;
                    if (lane < 9) {
                        const int dy = g.flat ? 0 : lane / 3 - 1, dx = g.flat ? 0 : lane % 3 - 1;
                        const int ip = x.w.ip + dy, iq = x.w.iq + dx;
                        const bool exists = g.flat ? lane == 4 : (ip >= 0 && ip < g.tiles_p && iq >= 0 && iq < g.tiles_q);
                        if (exists) {
                            const int nb = g.flat ? x.w.mt : (x.w.in * g.tiles_p + ip) * g.tiles_q + iq;
                            mine = tc_flag_wait(ch.flags + static_cast<size_t>(l - 1) * tiles_m + nb, target);
                        }
                    }
                    ok = __all_sync(0xffffffffu, mine);
                    if (!ok) break;
                }
                unsigned mine_ok = 1;
                if (lane == 0) {
                    if (MAXL > 1 && l > 0) fence_proxy_async_global();       // stores of other SMs, read by the copy engine
                    mine_ok = mbar_spin_bounded(&empty_p[rp.idx], rp.phase ^ 1u) ? 1u : 0u;
                    if (mine_ok) {
                        TC_TRACE(TR_LOAD, i);
                        tc_load_tile(g, s_p + rp.idx * g.pa_bytes, &full_p[rp.idx], tc_walk_tile(g, x.w));
                    }
                }
                ok = __shfl_sync(0xffffffffu, mine_ok, 0) != 0;
                if (!ok) break;
                rp.advance(g0.nsp);
            }
        }
        if (!ok && lane == 0) atomicOr(g0.status, STATUS_TIMEOUT);
        __syncwarp();
    } else if (warp == 9) {
        // ------------------------------------------------------------------ MMA issuer (in a chain it also fetches the filters of each layer)
        if (MAXL == 1 && lane == 0) {
            const TcIssue is = tc_make_issue(g0);
            const uint32_t e_base = smem_u32(s_e), w_base = smem_u32(s_w);
            bool ok = mbar_spin_bounded(wgt_full, 0);       // also keeps the CTA alive until the filter copy has landed
            TC_TRACE(TR_WGT, 0);
            TcRing re, ra;                                  // expanded chunks; accumulator buffers
            int i = 0;
            for (int mt = first_tile; mt < tiles_m && ok; mt += tile_step, ++i) {
                ok = mbar_spin_bounded(&empty_acc[ra.idx], ra.phase ^ 1u);
                if (!ok) break;
                tc_fence_after();
                const uint32_t tmem_acc = tmem_base + static_cast<uint32_t>(ra.idx * g0.TN);
                uint32_t wa = w_base;
                for (int c = 0; c < g0.nchunks; ++c, wa += static_cast<uint32_t>(g0.b_bytes)) {
                    if (!mbar_spin_bounded(&full_e[re.idx], re.phase)) { ok = false; break; }
                    if (c == 0) TC_TRACE(TR_MBEG, i);
                    tc_fence_after();
                    tc_issue_chunk(is, e_base + static_cast<uint32_t>(re.idx * g0.e_bytes), wa, tmem_acc, c == 0);
                    if (c == 0) TC_TRACE(TR_M_ISSUED, i);
                    umma_commit(&empty_e[re.idx]);
                    re.advance(g0.nse);
                }
                if (ok) umma_commit(&full_acc[ra.idx]);
                TC_TRACE(TR_MEND, i);
                ra.advance(2);
            }
            if (!ok) atomicOr(g0.status, STATUS_TIMEOUT);
        } else if (lane == 0) {
            const TcIssue is = tc_make_issue(g0);
            const uint32_t e_base = smem_u32(s_e), w_base = smem_u32(s_w);
            const int blk_bytes = g0.b_bytes / g0.MB;
            const size_t blk_stride = static_cast<size_t>(g0.opad8) * RS * (g0.CK >> 4) * 128;    // one layout block, all filters
            TcRing re, ra;                                  // expanded chunks; accumulator buffers
            bool ok = true;
            int cur_l = -1;
            unsigned wphase = 0;
            int l = first_tile / tiles_m, rem = first_tile - l * tiles_m;
            const int dl = tile_step / tiles_m, drem = tile_step - dl * tiles_m;
            for (int i = 0; l < nlayers && ok; ++i) {
                if (l != cur_l) {
                    if (cur_l >= 0) {       // the filters in shared memory are still being read: wait for those MMAs
                        umma_commit(wgt_free);
                        ok = mbar_spin_bounded(wgt_free, wphase ^ 1u);
                        if (!ok) break;
                    }
                    const TcArgs& g = ch.L[MAXL > 1 ? l : 0];
                    mbar_expect_tx(wgt_full, static_cast<unsigned>(g0.nchunks * g0.b_bytes));
                    const int8_t* src = g.wgt + static_cast<size_t>(o0 >> 3) * RS * (g0.CK >> 4) * 128;
                    unsigned char* dst = s_w;
                    for (int c = 0; c < g0.nchunks * g0.MB; ++c, src += blk_stride, dst += blk_bytes)   // layout blocks, consecutive in shared memory
                        bulk_load(dst, src, static_cast<unsigned>(blk_bytes), wgt_full);
                    ok = mbar_spin_bounded(wgt_full, wphase);       // also keeps the CTA alive until the filter copy has landed
                    if (!ok) break;
                    if (cur_l < 0) TC_TRACE(TR_WGT, 0);
                    wphase ^= 1u;
                    cur_l = l;
                }
                ok = mbar_spin_bounded(&empty_acc[ra.idx], ra.phase ^ 1u);
                if (!ok) break;
                tc_fence_after();
                const uint32_t tmem_acc = tmem_base + static_cast<uint32_t>(ra.idx * g0.TN);
                uint32_t wa = w_base;
                for (int c = 0; c < g0.nchunks; ++c, wa += static_cast<uint32_t>(g0.b_bytes)) {
                    if (!mbar_spin_bounded(&full_e[re.idx], re.phase)) { ok = false; break; }
                    if (c == 0) TC_TRACE(TR_MBEG, i);
                    tc_fence_after();
                    tc_issue_chunk(is, e_base + static_cast<uint32_t>(re.idx * g0.e_bytes), wa, tmem_acc, c == 0);
                    if (c == 0) TC_TRACE(TR_M_ISSUED, i);
                    umma_commit(&empty_e[re.idx]);
                    re.advance(g0.nse);
                }
                if (ok) umma_commit(&full_acc[ra.idx]);
                TC_TRACE(TR_MEND, i);
                ra.advance(2);
                l += dl; rem += drem;
                if (rem >= tiles_m) { rem -= tiles_m; ++l; }
            }
            if (!ok) atomicOr(g0.status, STATUS_TIMEOUT);
        }
        __syncwarp();
    } else if (warp >= 4 && warp < 8) {
        // ------------------------------------------------------------------ expanders (warps 4-7)
        const int et = tid - 128;
        tc_build_lut(g0, s_lut, et, 128);
        group_sync(1);
        const TcExpand xp = tc_expand_init(g0, et, 128);
        TcRing rp, re;
        bool ok = true;
        for (int i = 0, it = first_tile; it < items && ok; it += tile_step, ++i) {
            ok = mbar_wait_warp(&full_p[rp.idx], rp.phase, lane);
            if (et == 0) TC_TRACE(TR_XBEG, i);
            const uint32_t* pa = reinterpret_cast<const uint32_t*>(s_p + rp.idx * g0.pa_bytes);
            for (int c = 0; c < g0.nchunks; ++c) {
                if (ok) ok = mbar_wait_warp(&empty_e[re.idx], re.phase ^ 1u, lane);
                ok = group_all(1, ok);
                if (!ok) break;
                if (et == 0 && c == 0) TC_TRACE(TR_X_BEG0, i);
                tc_expand_chunk<A>(g0, xp, pa, s_e + re.idx * g0.e_bytes, s_lut, et, c);
                fence_proxy_async();
                group_sync(1);                       // all 128 expander threads have written and fenced
                if (et == 0 && c == 0) TC_TRACE(TR_X_DONE0, i);
                if (et == 0) mbar_arrive(&full_e[re.idx]);
                re.advance(g0.nse);
            }
            if (et == 0) TC_TRACE(TR_XEND, i);
            if (ok && et == 0) mbar_arrive(&empty_p[rp.idx]);   // ordered after the last group_sync: every thread is done reading
            rp.advance(g0.nsp);
        }
        if (!ok) atomicOr(g0.status, STATUS_TIMEOUT);
    } else {
        // ------------------------------------------------------------------ epilogue (warps 0-3, and 10-13 when WIDE)
        constexpr int EPI_THREADS = WIDE ? 256 : 128;
        const int second = warp >= 10 ? 1 : 0;                 // second set: the odd groups of 32 filters
        const int ei = second ? tid - 192 : tid;               // 0 .. EPI_THREADS-1
        if constexpr (MAXL == 1) {
            // the one-layer kernel keeps its own, simpler loop: the chain form of it below measured 1.5 % slower on a whole network
            tc_epilogue_tables(g0, tc_smem, s_sb, s_bounds, o0, ei, EPI_THREADS);
            group_sync(2, EPI_THREADS);
            uint32_t thr = 0;                 // shared-memory address of the thresholds, 0: floating-point comparison
            if (g0.off_thr) {                  // while the pipeline fills: comparison bounds -> integer thresholds
                int4* s_thr = reinterpret_cast<int4*>(tc_smem + g0.off_thr);
                int* thr_ok = reinterpret_cast<int*>(s_thr + g0.thr_pats * g0.TN);
                tc_build_thresholds(g0, s_thr, thr_ok, s_sb, s_bounds, o0, ei, EPI_THREADS);
                group_sync(2, EPI_THREADS);
                if (*thr_ok) thr = smem_u32(s_thr);
            }
            const TcEpiThread eth = tc_epi_thread(g0, (warp & 3) * 32 + lane);
            TcTileWalker tw = tc_walk_init(g0, first_tile, tile_step);
            pdl_acquire();                    // the epilogue reads the residual and overwrites buffers the preceding kernel may use
            TcRing ra;
            bool ok = true;
            for (int i = 0; tw.mt < tiles_m; tc_walk_next(g0, tw), ++i) {
                ok = group_all(2, mbar_wait_warp(&full_acc[ra.idx], ra.phase, lane), EPI_THREADS);
                if (!ok) break;
                if (tid == 0) TC_TRACE(TR_EBEG, i);
                tc_fence_after();
                tc_epilogue_tile(g0, tmem_base + static_cast<uint32_t>(ra.idx * g0.TN), (warp & 3) * 32 + lane, warp & 3, tc_walk_tile(g0, tw), eth, o0,
                                 s_sb, s_bounds, thr, WIDE ? second : 0, WIDE ? 2 : 1, i);
                tc_fence_before();
                group_sync(2, EPI_THREADS);              // every epilogue warp has read its accumulator rows
                if (tid == 0) TC_TRACE(TR_EEND, i);
                if (tid == 0) mbar_arrive(&empty_acc[ra.idx]);
                ra.advance(2);
            }
            if (!ok) atomicOr(g0.status, STATUS_TIMEOUT);
        } else {
            const TcEpiThread eth = tc_epi_thread(g0, (warp & 3) * 32 + lane);
            TcItemWalker x = tc_item_init(g0, first_tile, tile_step, tiles_m);
            TcRing ra;
            bool ok = true;
            int i = 0;
#pragma unroll
            for (int l = 0; l < MAXL; ++l) {          // one copy of the loop per layer, see the producer
                const TcArgs& g = ch.L[l];
                if (!ok || x.l != l || l >= nlayers) continue;
                // tables of the layer (the preceding tile's group_sync has every thread past its last use of the old ones)
                tc_epilogue_tables(g, tc_smem, s_sb, s_bounds, o0, ei, EPI_THREADS);
                group_sync(2, EPI_THREADS);
                uint32_t thr = 0;                 // shared-memory address of the thresholds, 0: floating-point comparison
                if (g.off_thr) {                  // while the pipeline fills: comparison bounds -> integer thresholds
                    int4* s_thr = reinterpret_cast<int4*>(tc_smem + g.off_thr);
                    int* thr_ok = reinterpret_cast<int*>(s_thr + g.thr_pats * g.TN);
                    tc_build_thresholds(g, s_thr, thr_ok, s_sb, s_bounds, o0, ei, EPI_THREADS);
                    group_sync(2, EPI_THREADS);
                    if (*thr_ok) thr = smem_u32(s_thr);
                }
                if (i == 0) pdl_acquire();        // the epilogue reads the residual and overwrites buffers the preceding kernel may use
                for (; x.l == l; tc_item_next(g0, x, tiles_m), ++i) {
                    ok = group_all(2, mbar_wait_warp(&full_acc[ra.idx], ra.phase, lane), EPI_THREADS);
                    if (!ok) break;
                    if (tid == 0) TC_TRACE(TR_EBEG, i);
                    tc_fence_after();
                    tc_epilogue_tile(g, tmem_base + static_cast<uint32_t>(ra.idx * g0.TN), (warp & 3) * 32 + lane, warp & 3, tc_walk_tile(g, x.w), eth, o0,
                                     s_sb, s_bounds, thr, WIDE ? second : 0, WIDE ? 2 : 1, i, true);
                    if (l + 1 < nlayers) fence_proxy_async_global();     // the next layer reads these stores through the copy engine
                    tc_fence_before();
                    group_sync(2, EPI_THREADS);              // every epilogue warp has read its accumulator rows
                    if (tid == 0) TC_TRACE(TR_EEND, i);
                    if (tid == 0) {
                        mbar_arrive(&empty_acc[ra.idx]);
                        if (l + 1 < nlayers) {
                            __threadfence();                 // cumulative: orders the stores of the whole group (seen through the barrier) before the counter
                            atomicAdd(ch.flags + static_cast<size_t>(l) * tiles_m + x.w.mt, 1u);
                        }
                    }
                    ra.advance(2);
                }
            }
            if (!ok) atomicOr(g0.status, STATUS_TIMEOUT);
        }
    }
    tc_fence_before();
    __syncthreads();
    if (tid == 0) TC_TRACE(TR_END, 0);
    if (warp == 9) {
        tc_fence_after();
        tmem_dealloc(tmem_base, static_cast<unsigned>(g0.tmem_cols));
    }
    if (MAXL > 1 && nlayers > 1 && tid == 0) {
        // the last CTA out counts the launch: every CTA has read ctl[0] long before
        __threadfence();
        if (atomicAdd(ch.ctl + 1, 1u) == gridDim.x - 1) {
            atomicExch(ch.ctl + 1, 0u);
            __threadfence();
            atomicAdd(ch.ctl, 1u);
        }
    }
}


// One thread per 16-byte vector of the prepared filter layout [chunk][O/8][tap][CK/16][8 filters][16 channels].
__global__ void tc_prepare_weights_kernel(const uint32_t* __restrict__ packed, int8_t* __restrict__ out, long long nvec,
                                          int O, int RS, int Cw, int WB, int sign, int CK, int opad8)
{
    const long long idx = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (idx >= nvec) return;
    const int k16n = CK >> 4;
    long long t = idx;
    const int row = static_cast<int>(t % 8);        t /= 8;
    const int k16 = static_cast<int>(t % k16n);     t /= k16n;
    const int tap = static_cast<int>(t % RS);       t /= RS;
    const int og = static_cast<int>(t % opad8);     t /= opad8;
    const int kc = static_cast<int>(t);
    const int o = og * 8 + row;
    const int c0 = kc * CK + k16 * 16;
    uint32_t vals[4] = {0, 0, 0, 0};
    if (o < O) {
        const uint32_t* w = packed + ((static_cast<size_t>(o) * RS + tap) * Cw + (c0 >> 5)) * WB;
        for (int ch = 0; ch < 16; ++ch) {
            unsigned pat = 0;
            for (int i = 0; i < WB; ++i) pat |= ((w[i] >> ((c0 & 31) + ch)) & 1u) << i;
            const unsigned byte = static_cast<unsigned>(pattern_value(pat, WB, sign)) & 0xFFu;
            vals[ch >> 2] |= byte << (8 * (ch & 3));
        }
    }
    reinterpret_cast<uint4*>(out)[idx] = make_uint4(vals[0], vals[1], vals[2], vals[3]);
}

static int round_up_i(int v, int m) { return (v + m - 1) / m * m; }

// Channels per block of the prepared filter layout.  A pipeline chunk is one or several consecutive blocks, chosen per
// layer by the plan (which knows stride and batch; the prepared filters do not depend on them).
static int tc_chunk_channels(int C, int /*a_bits*/)
{
    return C % 32 == 0 ? 32 : 0;
}

static typename std::add_pointer<CUresult(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                          const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                          CUtensorMapL2promotion, CUtensorMapFloatOOBfill)>::type
tc_encode_fn()
{
    typedef CUresult (*Fn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                           const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                           CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
    static Fn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<Fn>(p);
    });
    return fn;
}

static int tc_max_abs(int bits, int sign)
{
    if (sign == BS_BIPOLAR) return 1;
    if (sign == BS_SIGNED) return 1 << (bits - 1);
    return (1 << bits) - 1;
}

// Validation shared by the support query and the launch.  Returns BS_OK when the tensor-core path can run `p`.
static int tc_validate(const bs_conv_params* p)
{
    if (!p) return BS_ERR_INVALID_ARG;
    if (p->N <= 0 || p->C <= 0 || p->H <= 0 || p->W <= 0 || p->O <= 0 || p->R <= 0 || p->S <= 0) return BS_ERR_INVALID_ARG;
    if (!bits_ok(p->a_bits, p->a_sign) || !bits_ok(p->w_bits, p->w_sign)) return BS_ERR_INVALID_ARG;
    if (p->stride < 1 || p->pad < 0) return BS_ERR_INVALID_ARG;
    if (p->i32_layout != BS_NCHW && p->i32_layout != BS_NHWC) return BS_ERR_INVALID_ARG;
    if (p->R != p->S || (p->R != 1 && p->R != 3 && p->R != 5 && p->R != 7)) return BS_ERR_UNSUPPORTED;
    if (p->stride > 2 || p->pad >= p->R) return BS_ERR_UNSUPPORTED;
    if (p->a_sign == BS_BIPOLAR && p->pad != 0) return BS_ERR_UNSUPPORTED;
    if (p->H + 2 * p->pad < p->R || p->W + 2 * p->pad < p->S) return BS_ERR_INVALID_ARG;
    if (p->C % 32 != 0 || tc_chunk_channels(p->C, p->a_bits) == 0) return BS_ERR_UNSUPPORTED;
    {
        // packed pixel records must be 16-byte multiples, or 8-byte multiples on rows that are 16-byte multiples
        const int fullA = ceil_div(p->C, 32) * p->a_bits;
        const bool flat = p->R == 1 && p->stride == 1 && p->pad == 0;
        if (fullA % 4 != 0) {
            if (fullA % 2 != 0 || (p->W * fullA) % 4 != 0) return BS_ERR_UNSUPPORTED;
            if (flat && (static_cast<long long>(p->N) * p->H * p->W) % 2 != 0) return BS_ERR_UNSUPPORTED;
        }
    }
    const long long kred = static_cast<long long>(p->C) * p->R * p->S;
    if (kred * tc_max_abs(p->a_bits, p->a_sign) * tc_max_abs(p->w_bits, p->w_sign) >= (1LL << 31)) return BS_ERR_UNSUPPORTED;
    return BS_OK;
}

// Validates and plans one layer: tiles, shared-memory layout, kernel arguments (and the tensor map unless plan_only, which
// touches no tensor: the support query).  `smem` receives the dynamic shared memory of the plan.
// chain_n > 1: the layer is one of chain_n same-shaped layers run by one launch, which needs the resident-filter plan and has
// chain_n times the pixel tiles to spread over the SMs.
static int tc_plan(const uint32_t* act, const int8_t* wgt, const bs_conv_params* p, int32_t* out_i32, uint32_t* out_packed,
                   bool plan_only, TcArgs& g, size_t& smem_out, int chain_n = 1)
{
    int rc = tc_validate(p);
    if (rc != BS_OK) return rc;
    if (!plan_only) {
        if (!act || !wgt || (!out_i32 && !out_packed)) return BS_ERR_INVALID_ARG;
        if (!aligned16(act) || !aligned16(wgt) || (out_i32 && !aligned16(out_i32)) || (out_packed && !aligned16(out_packed)))
            return BS_ERR_ALIGNMENT;
    }
    g = TcArgs{};
    g.P = (p->H + 2 * p->pad - p->R) / p->stride + 1;
    g.Q = (p->W + 2 * p->pad - p->S) / p->stride + 1;
    if (out_packed) {
        if (!p->scale || !p->bias) return BS_ERR_INVALID_ARG;
        if (!bits_ok(p->out_bits, p->out_sign)) return BS_ERR_INVALID_ARG;
        if (p->out_c_offset < 0 || p->out_c_total < p->out_c_offset + p->O) return BS_ERR_INVALID_ARG;
        if (p->out_c_offset % 32 != 0) return BS_ERR_UNSUPPORTED;
        if (p->O % 32 != 0 && p->out_c_offset + p->O != p->out_c_total) return BS_ERR_UNSUPPORTED;
        if (p->residual) {
            if (!bits_ok(p->res_bits, p->res_sign)) return BS_ERR_INVALID_ARG;
            if (p->res_c_offset < 0 || p->res_c_total < p->res_c_offset + p->O) return BS_ERR_INVALID_ARG;
            if (p->res_c_offset % 32 != 0) return BS_ERR_UNSUPPORTED;
            if (!aligned16(p->residual)) return BS_ERR_ALIGNMENT;
        }
    }
    const int A = p->a_bits, RS = p->R * p->S, Cw = p->C / 32;
    g.wgt = wgt; g.out_i32 = out_i32; g.out_packed = out_packed; g.scale = p->scale; g.bias = p->bias;
    g.residual = out_packed ? p->residual : nullptr; g.res_scale = p->res_scale;
    if (!plan_only) {
        g.status = status_device_ptr();
        if (!g.status) return BS_ERR_CUDA;
    }
    g.N = p->N; g.H = p->H; g.W = p->W; g.O = p->O; g.R = p->R; g.S = p->S; g.stride = p->stride; g.pad = p->pad; g.A = A;
    // A 1x1 stride-2 layer (projection shortcut) reads one pixel in four: its tensor map traverses rows and columns with element
    // stride 2, so the tile arrives dense and everything after the fetch is a stride-1 1x1 layer on the subsampled image.
    g.ld_stride = 1;
    if (RS == 1 && p->stride == 2 && p->pad == 0 && (Cw * A) % 4 == 0 && Cw * A <= 256) { g.ld_stride = 2; g.stride = 1; }
    const int st = g.stride;          // the stride the tiling sees
    g.relu = p->relu; g.out_bits = p->out_bits; g.out_sign = p->out_sign;
    g.out_cw_off = p->out_c_offset / 32; g.out_cw_total = ceil_div(p->out_c_total > 0 ? p->out_c_total : 1, 32);
    g.res_bits = p->res_bits; g.res_sign = p->res_sign; g.res_c_off = p->res_c_offset;
    g.res_cw_total = ceil_div(p->res_c_total > 0 ? p->res_c_total : 1, 32);
    g.i32_nhwc = p->i32_layout == BS_NHWC;
    const long long kred = static_cast<long long>(p->C) * RS;
    g.acc_small = kred * tc_max_abs(p->a_bits, p->a_sign) * tc_max_abs(p->w_bits, p->w_sign) < (1LL << 22);
    {
        const long long bound = kred * tc_max_abs(p->a_bits, p->a_sign) * tc_max_abs(p->w_bits, p->w_sign);
        g.acc_bound = bound > 0x7fffffffLL ? 0x7fffffff : static_cast<int>(bound);
    }
    g.thr_packed = 0;

    g.CK = tc_chunk_channels(p->C, A);
    // Blocks per pipeline chunk: 64 channels when C allows (two MMAs per tap and hand-off), 128 for 1x1 stride-1 layers
    // (one tap per block is too little work per hand-off), a single 32-channel block for stride-2 3x3 layers of 128 and more channels, whose
    // expanded halo is four times larger per output and would otherwise push the plan to a narrower filter tile.
    g.MB = p->C % 64 == 0 ? 2 : 1;
    {
        int wide = 4;
#ifdef BS_TUNING
        if (const char* e = getenv("BS_TC_MB")) wide = atoi(e);
#endif
        if (RS == 1 && p->pad == 0 && (p->stride == 1 || g.ld_stride == 2))
            for (int mb = wide; mb > 1; mb /= 2)
                if (p->C % (g.CK * mb) == 0) { g.MB = mb; break; }
        if (RS > 1 && p->stride == 2 && p->C >= 128) g.MB = 1;
#ifdef BS_TUNING
        if (const char* e = getenv("BS_TC_MBALL")) { const int mb = atoi(e); if (p->C % (g.CK * mb) == 0) g.MB = mb; }
#endif
    }
    int CKP = g.CK * g.MB;                        // channels per pipeline chunk
    g.CWC = CKP / 32;
    g.fullA = Cw * A;
    g.pitchA = g.fullA;
    g.seg_words = g.seg_chunks = g.nseg = 0;
    g.act = act;
    g.nchunks = p->C / CKP;
    g.nsp = g.nse = g.nchunks < 2 ? g.nchunks : 2;
    g.opad8 = round_up_i(p->O, 128) / 8;
    g.flat = (p->R == 1 && p->stride == 1 && p->pad == 0);
    long long tiles_m;
    if (g.flat) {
        const long long npix = static_cast<long long>(p->N) * p->H * p->W;
        if (npix > 0x7fffffffLL) return BS_ERR_UNSUPPORTED;
        g.tiles_q = static_cast<int>(ceil_div_ll(npix, TC_M)); g.tiles_p = 1; g.tiles_n = 1;
        g.TNI = 1; g.GI = 16; g.hh = 1; g.hw = TC_M; g.hwb = TC_M; g.xsh = 0; g.HWP = TC_M; g.HWH = 0; g.HPE = TC_M;
        g.pa_tx_bytes = TC_M * g.fullA * 4;
        g.pmode = 0;
        tiles_m = g.tiles_q;
    } else {
        g.hw = 7 * st + p->S;
        g.xsh = (g.fullA % 4 != 0 && (p->pad & 1)) ? 1 : 0;
        g.hwb = g.fullA % 4 != 0 ? round_up_i(g.hw + g.xsh, 2) : g.hw;
        g.HWH = (g.hw + 1) / 2;
        g.HWP = st == 2 ? 2 * g.HWH : g.hw;
        if (g.P <= 16) {        // whole image height in one tile; stack as many images as fit in the 16 row groups
            g.hh = round_up_i((g.P - 1) * st + p->R, st);
            g.GI = g.hh / st;
            g.TNI = (16 - g.P) / g.GI + 1;
            if (g.TNI > p->N) g.TNI = p->N;
            g.tiles_p = 1;
        } else {
            g.hh = round_up_i(15 * st + p->R, st);
            g.GI = 16; g.TNI = 1;
            g.tiles_p = ceil_div(g.P, 16);
        }
        g.tiles_q = ceil_div(g.Q, 8);
        g.tiles_n = ceil_div(p->N, g.TNI);
        const int rows_box = g.TNI * g.hh;
        const int rows_read = 15 * st + p->R;
        g.HPE = (rows_box > rows_read ? rows_box : rows_read) * g.HWP;
        g.pa_tx_bytes = g.TNI * g.hh * g.hwb * g.fullA * 4;
        g.pmode = (g.hwb * g.fullA <= 256 && g.ld_stride == 1) ? 1 : 2;      // columns can only be skipped as a dimension of their own
        if (g.pmode == 2 && (g.fullA > 256 || g.fullA % 4 != 0)) return BS_ERR_UNSUPPORTED;
        tiles_m = static_cast<long long>(g.tiles_q) * g.tiles_p * g.tiles_n;
    }
    g.pa_bytes = round_up_i(g.pa_tx_bytes, 128);
    g.e_bytes = round_up_i((CKP / 16) * g.HPE * 16, 128);
    int sms = device_sm_count();
    if (sms <= 0) {
        if (!plan_only) return BS_ERR_CUDA;
        sms = 148;                     // support query without a device: plan for a full B200
    }
    // Persistent plan: the filters of a tile (all channel chunks) stay resident in shared memory.  Largest filter tile
    // that fits and still leaves one (pixel tile, filter tile) pair per SM.
    size_t smem = 0;
    g.persistent = 0;
    const int bar_bytes = (2 * TCP_NSP + 2 * TCP_NSE + 5) * 8 + 16;
    int tn_max = 128;
    bool force_stream = false, keep_narrow = false;
    int stream_pt = 1, stream_tn = 0;
#ifdef BS_TUNING
    // plan overrides for tuning runs (not compiled into the library by default)
    if (const char* e = getenv("BS_TC_TNMAX")) tn_max = atoi(e);
    force_stream = getenv("BS_TC_STREAM") != nullptr;
    keep_narrow = getenv("BS_TC_KEEP_NARROW") != nullptr;
    if (const char* e = getenv("BS_TC_PT")) stream_pt = atoi(e);
    if (const char* e = getenv("BS_TC_STN")) stream_tn = atoi(e);
#endif
    for (int TN = 128; TN >= 32; TN /= 2) {
        if (TN > tn_max) continue;
        if (TN / 2 >= round_up_i(p->O, 32)) continue;                      // tile twice as wide as the filter bank
        const long long pairs = tiles_m * chain_n * ceil_div(p->O, TN);
        if (TN > 32 && pairs < sms) continue;
        const size_t wbytes = static_cast<size_t>(g.nchunks) * TN * RS * CKP;
        const int shapes[4][2] = {{2, 2}, {2, 2}, {2, 2}, {1, 2}};      // (packed-tile stages, expanded-chunk stages)
        for (const auto& sh : shapes) {
            const int nsp = sh[0], nse = sh[1];
            const size_t total = wbytes + static_cast<size_t>(nsp) * g.pa_bytes + static_cast<size_t>(nse) * g.e_bytes +
                                 static_cast<size_t>(TN) * 8 + 256 + bar_bytes + 128 + 16 + static_cast<size_t>(A) * TC_LUT_BYTES_PER_PLANE;
            if (total <= 220 * 1024) {
                g.persistent = 1; g.TN = TN; g.b_bytes = TN * RS * CKP; g.nse = nse; g.nsp = nsp;
                g.off_p = static_cast<int>(wbytes);
                g.off_e = g.off_p + nsp * g.pa_bytes;
                g.off_sb = g.off_e + nse * g.e_bytes;
                g.off_bar = round_up_i(g.off_sb + TN * 8 + 256, 16);
                g.off_lut = round_up_i(g.off_bar + bar_bytes, 16);
                smem = static_cast<size_t>(g.off_lut) + static_cast<size_t>(A) * TC_LUT_BYTES_PER_PLANE;
                break;
            }
        }
        if (g.persistent) break;
    }
    // A resident plan that had to shrink the filter tile wastes the tensor core (an N = 32 MMA costs as many cycles
    // as N = 64, and N = 64 only a fifth less than N = 128): stream the filters instead when a 128-wide tile leaves
    // enough (pixel tile, filter tile) pairs -- always for N = 32, for N = 64 when the reduction is deep (measured).
    if (!keep_narrow && g.persistent && (g.TN == 32 || (g.TN == 64 && g.nchunks >= 4)) && p->O >= 128 &&
        tiles_m * ceil_div(p->O, 128) >= sms / 2)
        g.persistent = 0;
    // A resident plan also loses when its CTAs see hardly more than one pixel tile each: nothing amortises the filter
    // fetch, and the streaming kernel has twice the expand/epilogue warps.  Measured on the bottleneck stack for
    // reductions of 512 and more (shallower ones are epilogue-bound and stay resident).
    if (!keep_narrow && chain_n == 1 && g.persistent && kred >= 512) {        // (a chain exists to save launches: it stays resident)
        int cps_est = static_cast<int>((225 * 1024) / (smem + 1024));
        if (cps_est > 3) cps_est = 3;
        if (cps_est * 2 * g.TN > 512) cps_est = 512 / (2 * g.TN);
        if (cps_est < 1) cps_est = 1;
        const int tiles_o = ceil_div(p->O, g.TN);
        long long per_o = static_cast<long long>(sms) * cps_est / tiles_o;
        if (per_o < 1) per_o = 1;
        if (per_o > tiles_m) per_o = tiles_m;
        if (2 * tiles_m <= 3 * per_o) g.persistent = 0;       // at most 1.5 pixel tiles per CTA
    }
    // Wide matrix products (see the streaming plan below): a resident 128-filter tile would expand every pixel tile once per
    // filter tile; with four or more filter tiles the streaming kernel with 256- or 512-filter tiles does less work.
    if (!keep_narrow && g.persistent && g.flat && p->O >= 512 && p->O % 256 == 0 && tiles_m * (p->O / 256) >= sms) g.persistent = 0;
    if (force_stream) g.persistent = 0;
    g.PT = 1;
    if (!g.persistent) {
        // Filters streamed chunk by chunk; a CTA takes PT pixel tiles (PT accumulators in tensor memory) so that every
        // filter chunk fetched from L2 serves PT tiles.  Widest filter tile that keeps about one CTA per SM.
        g.nsp = g.nse = g.nchunks < 2 ? g.nchunks : 2;
#ifdef BS_TUNING
        if (const char* e = getenv("BS_TC_NSP")) { const int n = atoi(e); g.nsp = g.nchunks < n ? g.nchunks : n; }
#endif
        int TN = 128;
        while (TN > 32 && (TN / 2 >= round_up_i(p->O, 32) || tiles_m * ceil_div(p->O, TN) < sms / 2)) TN /= 2;
        int PT = stream_pt;
        // Matrix products with a long reduction: 128 packed rows of all K no longer fit beside useful filter and expansion stages
        // (K = 4608 at 2 bits: 147 KB, which left room for 32-channel chunks only: one or two MMAs per hand-off).  Their rows are
        // staged in segments of at most 72 words (a multiple of every chunk width), two buffers of 36 KB: 512-filter tiles with
        // 64-channel chunks (four N = 256 MMAs per hand-off).  Segments of 32 words with 128-channel chunks in 214 KB measured
        // slower (0.190 against 0.175 ms at 4096 x 4096 x 4608): the expansion of a chunk then takes longer than its MMAs.  Only for records that
        // crowd the stages out (K = 2304, 74 KB resident, measured faster whole: 0.091 against 0.103 ms at 4096 x 4096) and only
        // when the tiles fill the machine (1024 x 1024 x 4608 on 16 CTAs is latency-bound: 0.048 against 0.063 ms).
        int seg_words = 0;
        if (g.flat && PT == 1 && g.fullA % 4 == 0 && g.pa_tx_bytes > 96 * 1024 && tiles_m * ceil_div(p->O, 256) >= sms) {
            seg_words = 72 / (4 * A) * (4 * A);
            g.pa_bytes = 2 * round_up_i(TC_M * seg_words * 4, 128);
        }
        auto stream_bytes = [&](int tn, int pt) {
            return static_cast<size_t>(g.nsp) * tn * RS * CKP + static_cast<size_t>(pt) * g.pa_bytes +
                   static_cast<size_t>(g.nse) * pt * g.e_bytes + 2 * tn * 4 + 256 + (4 * TC_MAX_STAGES + 6) * 8 + 128 +
                   16 + static_cast<size_t>(A) * TC_LUT_BYTES_PER_PLANE;
        };
        // Matrix products and 1x1 layers with many filters: every filter tile of a pixel tile expands the same packed rows
        // again, and one K = 32 step is a single MMA, so the expansion, not the tensor core, sets the pace.  A CTA then
        // takes 256 or 512 filters (N = 256 MMAs, 256 or 512 accumulator columns) as long as a full wave of CTAs remains.
        if (g.flat && PT == 1 && !stream_tn) {
            for (int wide = 512; wide > 128; wide /= 2) {
                if (p->O % wide != 0 || tiles_m * (p->O / wide) < sms) continue;
                // int32 outputs of a short reduction are bound by their own stores (four bytes per output against 2 K operations:
                // K below ~1000): two CTAs of 256 filters per SM then overlap one's stores with the other's MMAs
                // (4096 x 4096 x 576: 64 against 72 us; at K = 2304 the 512-filter tile wins, 106 against 126 us)
                if (wide == 512 && out_i32 && !out_packed && kred < 1024 && p->O % 256 == 0) continue;
                int mb = g.MB;
                auto bytes_mb = [&](int m) {
                    const int ckp = g.CK * m;
                    return static_cast<size_t>(2) * wide * RS * ckp + g.pa_bytes + static_cast<size_t>(2) * round_up_i((ckp / 16) * g.HPE * 16, 128) +
                           2 * wide * 4 + 256 + (4 * TC_MAX_STAGES + 6) * 8 + 128 + 16 + static_cast<size_t>(A) * TC_LUT_BYTES_PER_PLANE +
                           static_cast<size_t>(wide) * 16 + 16;
                };
                while (mb > 1 && bytes_mb(mb) > 200 * 1024) mb /= 2;
                if (bytes_mb(mb) > 200 * 1024) continue;
                if (mb != g.MB) {
                    g.MB = mb; CKP = g.CK * mb; g.CWC = CKP / 32; g.nchunks = p->C / CKP;
                    g.e_bytes = round_up_i((CKP / 16) * g.HPE * 16, 128);
                    g.nsp = g.nse = g.nchunks < 2 ? g.nchunks : 2;
                }
                TN = wide;
                break;
            }
        }
        if (stream_tn) TN = stream_tn;
        while (PT > 1 && (PT * TN > 512 || stream_bytes(TN, PT) > 220 * 1024)) PT /= 2;
        // Large kernels (5x5, 7x7) over many channels: a 128-wide filter chunk of 64 channels does not fit the ring;
        // halve the chunk to one layout block before narrowing the filter tile.
        const size_t stream_cap = 200 * 1024;
        if (g.MB > 1 && stream_bytes(TN, PT) > stream_cap) {
            g.MB = 1; CKP = g.CK; g.CWC = CKP / 32; g.nchunks = p->C / CKP;
            g.e_bytes = round_up_i((CKP / 16) * g.HPE * 16, 128);
            g.nsp = g.nse = g.nchunks < 2 ? g.nchunks : 2;
        }
        while (TN > 32 && stream_bytes(TN, PT) > stream_cap) TN /= 2;
        // More CTAs than SMs: halve the chunk if that lets two CTAs share an SM (one wave instead of two)
        if (g.MB == 2 && RS > 1 && ceil_div_ll(tiles_m, PT) * ceil_div(p->O, TN) > sms) {
            const int e_keep = g.e_bytes, n_keep = g.nchunks;
            g.MB = 1; CKP = g.CK; g.CWC = CKP / 32; g.nchunks = p->C / CKP;
            g.e_bytes = round_up_i((CKP / 16) * g.HPE * 16, 128);
            g.nsp = g.nse = g.nchunks < 2 ? g.nchunks : 2;
            if (stream_bytes(TN, PT) + 5 * 1024 > 112 * 1024) {
                g.MB = 2; CKP = 2 * g.CK; g.CWC = CKP / 32; g.nchunks = n_keep; g.e_bytes = e_keep;
                g.nsp = g.nse = g.nchunks < 2 ? g.nchunks : 2;
            }
        }
        if (seg_words) {
            g.seg_words = seg_words;
            g.pitchA = seg_words;
            g.seg_chunks = seg_words / (g.CWC * A);
            g.nseg = ceil_div(g.fullA, seg_words);
            if (g.nchunks <= g.nsp || PT != 1) return BS_ERR_UNSUPPORTED;      // cannot happen: records of 64 KB / 128 rows are many chunks
        }
        g.TN = TN;
        g.PT = PT;
        g.b_bytes = TN * RS * CKP;
        g.off_p = g.nsp * g.b_bytes;
        g.off_e = g.off_p + PT * g.pa_bytes;
        g.off_sb = g.off_e + g.nse * PT * g.e_bytes;
        g.off_bar = round_up_i(g.off_sb + 2 * g.TN * 4 + 256, 16);
        g.off_lut = round_up_i(g.off_bar + (4 * TC_MAX_STAGES + 6) * 8, 16);
        smem = static_cast<size_t>(g.off_lut) + static_cast<size_t>(A) * TC_LUT_BYTES_PER_PLANE;
        if (smem > 220 * 1024) return BS_ERR_UNSUPPORTED;
    }
    g.tiles_o = ceil_div(p->O, g.TN);
    g.tmem_cols = g.persistent ? 2 * g.TN : g.PT * g.TN;      // TN is 32, 64 or 128, PT 1, 2 or 4: powers of two, 32..512 columns
    g.NM = g.TN > 128 ? 256 : g.TN;
    g.idesc = (2u << 4) | (1u << 7) | (1u << 10) | (static_cast<unsigned>(g.NM >> 3) << 17) | (static_cast<unsigned>(TC_M >> 4) << 24);
    for (int j = 0; j < 4; ++j) g.mul[j] = 1u << j;
    g.xormask = 0;
    if (p->a_sign == BS_SIGNED) g.mul[A - 1] = 256u - (1u << (A - 1));
    if (p->a_sign == BS_BIPOLAR) { g.mul[0] = 0xFEu; g.xormask = 0xFFFFFFFFu; }

    g.rb = cached_requant_bounds(g.residual != nullptr, p->res_scale, p->res_bits, p->res_sign, p->relu,
                               out_packed ? p->out_bits : 0, p->out_sign);
    if (!out_packed) g.rb.enabled = 0;

    // Integer thresholds for the comparison epilogue, when they fit without costing a resident CTA.  With 2-bit
    // activations the nibble-pair table fills only the first 1 KB of the 4 KB table region; the rest is reused.
    auto ctas_per_sm = [](size_t bytes) { return static_cast<int>((225 * 1024) / (bytes + 1024)); };
    g.off_thr = 0;
    g.thr_pats = g.residual ? 4 : 1;
    if (g.rb.enabled && (!g.residual || p->res_bits <= 2) &&
        static_cast<long long>(p->C) * RS * tc_max_abs(p->a_bits, p->a_sign) * tc_max_abs(p->w_bits, p->w_sign) < TC_THR_LIM) {
        const size_t bytes = static_cast<size_t>(g.thr_pats) * g.TN * 16 + 16;
        const size_t off = A == 2 ? static_cast<size_t>(g.off_lut) + 1024 : smem;
        const size_t grown = off + bytes > smem ? off + bytes : smem;
        const bool same_occupancy = !g.persistent || ctas_per_sm(grown) >= (ctas_per_sm(smem) < 3 ? ctas_per_sm(smem) : 3);
        if (grown <= 220 * 1024 && same_occupancy) {
            g.off_thr = static_cast<int>(off);
            smem = grown;
            g.thr_packed = (!g.residual && g.acc_bound <= 16383) ? 1 : 0;
        }
    }

    smem_out = smem;
    if (plan_only) return BS_OK;
    auto enc = tc_encode_fn();
    if (!enc) return BS_ERR_CUDA;
    const cuuint64_t fullA = static_cast<cuuint64_t>(Cw) * A;
    cuuint32_t estr[4] = {1, 1, 1, 1};
    CUresult cr = CUDA_SUCCESS;
    if (g.pmode == 1) {
        cuuint64_t dims[3] = {fullA * p->W, static_cast<cuuint64_t>(p->H), static_cast<cuuint64_t>(p->N)};
        cuuint64_t strides[2] = {fullA * 4 * p->W, fullA * 4 * p->W * p->H};
        cuuint32_t box[3] = {static_cast<cuuint32_t>(g.hwb * g.fullA), static_cast<cuuint32_t>(g.hh), static_cast<cuuint32_t>(g.TNI)};
        cr = enc(&g.tmA, CU_TENSOR_MAP_DATA_TYPE_UINT32, 3, const_cast<uint32_t*>(act), dims, strides, box, estr,
                 CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                 CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    } else if (g.pmode == 2) {
        cuuint64_t dims[4] = {fullA, static_cast<cuuint64_t>(p->W), static_cast<cuuint64_t>(p->H), static_cast<cuuint64_t>(p->N)};
        cuuint64_t strides[3] = {fullA * 4, fullA * 4 * p->W, fullA * 4 * p->W * p->H};
        // with an element stride s a box dimension counts the elements TRAVERSED: s * n of them deliver n
        const cuuint32_t ls = static_cast<cuuint32_t>(g.ld_stride);
        cuuint32_t box[4] = {static_cast<cuuint32_t>(g.fullA), static_cast<cuuint32_t>(g.hw) * ls, static_cast<cuuint32_t>(g.hh) * ls,
                             static_cast<cuuint32_t>(g.TNI)};
        estr[1] = estr[2] = ls;
        cr = enc(&g.tmA, CU_TENSOR_MAP_DATA_TYPE_UINT32, 4, const_cast<uint32_t*>(act), dims, strides, box, estr,
                 CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                 CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    }
    if (cr != CUDA_SUCCESS) return BS_ERR_CUDA;
    return BS_OK;
}

// CTAs of the resident-filter kernel that fit on one SM: shared memory, registers (launch bounds) and tensor-memory columns.
static int tcp_ctas_per_sm(size_t smem, int TN)
{
    int cps = static_cast<int>((225 * 1024) / (smem + 1024));
    if (cps > 3) cps = 3;
    if (cps * 2 * TN > 512) cps = 512 / (2 * TN);
#ifdef BS_TUNING
    if (const char* e = getenv("BS_TC_CPSMAX")) { const int m = atoi(e); if (cps > m) cps = m; }
#endif
    return cps < 1 ? 1 : cps;
}

// The instantiation for a plan: CTAs per SM and whether registers allow eight epilogue warps (one or two CTAs per SM and
// at least two groups of 32 filters in the tile).
template <int MAXL>
static void (*tcp_pick(int A, int cps, bool wide))(TcChainArgs<MAXL>)
{
    switch (A) {
#define BS_TCP_PICK(ABITS) (cps >= 3 ? bitserial_conv_tc_persistent_kernel<ABITS, 3, false, MAXL> \
                          : cps == 2 ? (wide ? bitserial_conv_tc_persistent_kernel<ABITS, 2, true, MAXL> : bitserial_conv_tc_persistent_kernel<ABITS, 2, false, MAXL>) \
                                     : (wide ? bitserial_conv_tc_persistent_kernel<ABITS, 1, true, MAXL> : bitserial_conv_tc_persistent_kernel<ABITS, 1, false, MAXL>))
        case 1: return BS_TCP_PICK(1);
        case 2: return BS_TCP_PICK(2);
        case 3: return BS_TCP_PICK(3);
        default: return BS_TCP_PICK(4);
#undef BS_TCP_PICK
    }
}

// Launch with or without the programmatic-serialisation attribute.  With it, the grid may begin (barrier and TMEM
// set-up, byte table, filter fetch) while the preceding kernel of the stream drains; everything it reads before
// pdl_acquire() must therefore have been final before that preceding kernel was launched.
template <typename Args>
static cudaError_t tc_launch(void (*kern)(Args), unsigned grid, unsigned block, size_t smem, cudaStream_t st, bool chained, const Args& g)
{
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(block);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = chained ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kern, g);
}

static int tc_conv_impl(const uint32_t* act, const int8_t* wgt, const bs_conv_params* p, int32_t* out_i32, uint32_t* out_packed,
                        cudaStream_t st, bool chained = false, bool plan_only = false)
{
    TcArgs g;
    size_t smem = 0;
    const int rc = tc_plan(act, wgt, p, out_i32, out_packed, plan_only, g, smem);
    if (rc != BS_OK || plan_only) return rc;
    const int A = p->a_bits;
    if (g.persistent) {
        const int sms = device_sm_count();
        const long long tiles_m = static_cast<long long>(g.tiles_q) * g.tiles_p * g.tiles_n;
        const int cps = tcp_ctas_per_sm(smem, g.TN);
        long long per_o = (static_cast<long long>(sms) * cps) / g.tiles_o;
        if (per_o < 1) per_o = 1;
        if (per_o > tiles_m) per_o = tiles_m;
        const long long grid = per_o * g.tiles_o;
        bool wide = cps <= 2 && g.TN >= 64;
#ifdef BS_TUNING
        if (const char* e = getenv("BS_TC_WIDE")) wide = wide && atoi(e) != 0;
#endif
        void (*kern)(TcChainArgs<1>) = tcp_pick<1>(A, cps, wide);
        if (smem > 48 * 1024 &&
            cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)) != cudaSuccess) {
            cudaGetLastError();
            return BS_ERR_CUDA;
        }
        TcChainArgs<1> ch{};
        ch.L[0] = g; ch.nlayers = 1; ch.flags = nullptr; ch.ctl = nullptr;
        if (tc_launch(kern, static_cast<unsigned>(grid), wide ? TCP_THREADS_WIDE : TCP_THREADS, smem, st, chained, ch) != cudaSuccess) {
            cudaGetLastError();
            return BS_ERR_CUDA;
        }
        return BS_OK;
    }
    const long long tiles_m = static_cast<long long>(g.tiles_q) * g.tiles_p * g.tiles_n;
    const long long grid = ceil_div_ll(tiles_m, g.PT) * g.tiles_o;
    if (grid > 0x7fffffffLL) return BS_ERR_UNSUPPORTED;
    void (*kern)(TcArgs) = nullptr;
    switch (A) {
        case 1: kern = g.seg_words ? bitserial_conv_tc_kernel<1, true> : bitserial_conv_tc_kernel<1, false>; break;
        case 2: kern = g.seg_words ? bitserial_conv_tc_kernel<2, true> : bitserial_conv_tc_kernel<2, false>; break;
        case 3: kern = g.seg_words ? bitserial_conv_tc_kernel<3, true> : bitserial_conv_tc_kernel<3, false>; break;
        default: kern = g.seg_words ? bitserial_conv_tc_kernel<4, true> : bitserial_conv_tc_kernel<4, false>; break;
    }
    if (smem > 48 * 1024 &&
        cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)) != cudaSuccess) {
        cudaGetLastError();
        return BS_ERR_CUDA;
    }
    if (tc_launch(kern, static_cast<unsigned>(grid), TC_THREADS, smem, st, chained, g) != cudaSuccess) {
        cudaGetLastError();
        return BS_ERR_CUDA;
    }
    return BS_OK;
}

// ----------------------------------------------------------------------------- several layers in one launch

// Pixel tiles of one layer of a chain, or 0 when the layers cannot run as one chain: 2..TC_CHAIN_MAX layers that all take
// the resident-filter plan with the same geometry (batch, image, channels = filters, kernel, stride 1, output as large as the
// input), the same activation and weight formats, and packed outputs whose width is the next layer's activation width.
static long long tc_chain_plan(int n, const uint32_t* const* act, const int8_t* const* wgt, const bs_conv_params* params,
                               uint32_t* const* out, bool plan_only, TcArgs* L, size_t& smem)
{
    if (n < 2 || n > TC_CHAIN_MAX || !params) return 0;
    smem = 0;
    for (int l = 0; l < n; ++l) {
        const bs_conv_params* p = &params[l];
        bs_conv_params q = *p;
        if (plan_only) {                        // the epilogue's kind (thresholds, residual patterns) still shapes the plan
            static const float dummy = 0.f;
            q.scale = &dummy; q.bias = &dummy;
        }
        size_t s = 0;
        // a non-null placeholder stands for the output in a query: only "packed output wanted" matters to the plan
        uint32_t* o = plan_only ? reinterpret_cast<uint32_t*>(16) : out[l];
        if (tc_plan(plan_only ? nullptr : act[l], plan_only ? nullptr : wgt[l], &q, nullptr, o, plan_only, L[l], s, n) != BS_OK) return 0;
        if (!L[l].persistent || q.out_bits <= 0) return 0;
        if (p->stride != 1 || L[l].P != p->H || L[l].Q != p->W || p->O != p->C) return 0;
        if (s > smem) smem = s;
        if (l == 0) continue;
        const bs_conv_params* p0 = &params[0];
        if (p->N != p0->N || p->C != p0->C || p->H != p0->H || p->W != p0->W || p->O != p0->O || p->R != p0->R || p->S != p0->S ||
            p->pad != p0->pad || p->a_bits != p0->a_bits || p->a_sign != p0->a_sign || p->w_bits != p0->w_bits || p->w_sign != p0->w_sign)
            return 0;
        if (params[l - 1].out_bits != p->a_bits || params[l - 1].out_sign != p->a_sign) return 0;
        const TcArgs &a = L[0], &b = L[l];
        if (a.TN != b.TN || a.MB != b.MB || a.nchunks != b.nchunks || a.nsp != b.nsp || a.nse != b.nse || a.off_p != b.off_p ||
            a.off_e != b.off_e || a.off_sb != b.off_sb || a.off_bar != b.off_bar || a.off_lut != b.off_lut || a.tmem_cols != b.tmem_cols ||
            a.b_bytes != b.b_bytes || a.pa_bytes != b.pa_bytes || a.e_bytes != b.e_bytes || a.pmode != b.pmode || a.flat != b.flat)
            return 0;
    }
    for (int l = 0; l < n; ++l) {
        if (params[l].out_c_offset != 0 || params[l].out_c_total != params[l].O) return 0;       // a layer's output is a whole tensor
        if (params[l].residual && (params[l].res_c_offset != 0 || params[l].res_c_total != params[l].O)) return 0;
    }
    if (!plan_only) {
        // a layer may read (activations, residual) what an EARLIER layer of the chain wrote, or tensors final before the launch
        for (int l = 0; l < n; ++l)
            for (int k = l; k < n; ++k)
                if (act[l] == out[k] || (params[l].residual && params[l].residual == out[k])) return 0;
    }
    return static_cast<long long>(L[0].tiles_q) * L[0].tiles_p * L[0].tiles_n;
}

static size_t tc_chain_ws_bytes(int n, long long tiles_m) { return (static_cast<size_t>(n) * tiles_m + 4) * sizeof(unsigned); }

static int tc_chain_impl(int n, const uint32_t* const* act, const int8_t* const* wgt, const bs_conv_params* params,
                         uint32_t* const* out, void* workspace, size_t workspace_bytes, cudaStream_t st, bool chained)
{
    if (!act || !wgt || !params || !out || !workspace) return BS_ERR_INVALID_ARG;
    if (n < 2 || n > TC_CHAIN_MAX) return BS_ERR_UNSUPPORTED;
    for (int l = 0; l < n; ++l)
        if (!act[l] || !wgt[l] || !out[l]) return BS_ERR_INVALID_ARG;
    TcChainArgs<TC_CHAIN_MAX> ch{};
    size_t smem = 0;
    const long long tiles_m = tc_chain_plan(n, act, wgt, params, out, false, ch.L, smem);
    if (tiles_m <= 0) return BS_ERR_UNSUPPORTED;
    if (workspace_bytes < tc_chain_ws_bytes(n, tiles_m)) return BS_ERR_INVALID_ARG;
    if (!aligned16(workspace)) return BS_ERR_ALIGNMENT;
    ch.nlayers = n;
    ch.ctl = static_cast<unsigned*>(workspace);
    ch.flags = ch.ctl + 4;
    const TcArgs& g = ch.L[0];
    const int A = params[0].a_bits;
    const int sms = device_sm_count();
    if (sms <= 0) return BS_ERR_CUDA;
    const int cps = tcp_ctas_per_sm(smem, g.TN);
    const bool wide = cps <= 2 && g.TN >= 64;
    void (*kern)(TcChainArgs<TC_CHAIN_MAX>) = tcp_pick<TC_CHAIN_MAX>(A, cps, wide);
    if (smem > 48 * 1024 &&
        cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)) != cudaSuccess) {
        cudaGetLastError();
        return BS_ERR_CUDA;
    }
    // Every CTA of the grid must be resident at once (tiles wait for tiles of other CTAs).  The grid is sized by the same
    // count the one-layer kernel uses -- shared memory with the largest carve-out, which the kernel asks for here, registers
    // through the launch bounds, tensor-memory columns -- because the runtime's occupancy query answers one CTA per SM for
    // every kernel that allocates tensor memory, whatever its shared memory and block size.  Should fewer CTAs be resident
    // than counted, the bounded waits end the launch with BS_ERR_TIMEOUT instead of hanging.
    if (cudaFuncSetAttribute(kern, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared) != cudaSuccess) {
        cudaGetLastError();
        return BS_ERR_CUDA;
    }
    long long per_o = (static_cast<long long>(sms) * cps) / g.tiles_o;
    if (per_o < 1) return BS_ERR_UNSUPPORTED;                       // more filter tiles than resident CTAs
    if (per_o > n * tiles_m) per_o = n * tiles_m;
    const long long grid = per_o * g.tiles_o;
    if (tc_launch(kern, static_cast<unsigned>(grid), wide ? TCP_THREADS_WIDE : TCP_THREADS, smem, st, chained, ch) != cudaSuccess) {
        cudaGetLastError();
        return BS_ERR_CUDA;
    }
    return BS_OK;
}

}  // namespace bs

#ifdef BS_TUNING
// Tuning builds: copies the timeline table of the last tensor-core launches to `out` (HOST, 148 x 24 x 24 cycle counts).
extern "C" int bs_tc_trace_read(long long* out, int clear)
{
    if (cudaDeviceSynchronize() != cudaSuccess) return BS_ERR_CUDA;
    if (cudaMemcpyFromSymbol(out, bs::g_tc_trace, sizeof(bs::g_tc_trace)) != cudaSuccess) return BS_ERR_CUDA;
    if (clear) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, bs::g_tc_trace) != cudaSuccess || cudaMemset(p, 0, sizeof(bs::g_tc_trace)) != cudaSuccess) return BS_ERR_CUDA;
    }
    return BS_OK;
}
#endif

extern "C" size_t bs_tc_weights_bytes(int O, int C, int R, int S)
{
    if (O <= 0 || C <= 0 || R <= 0 || S <= 0 || C % 32 != 0) return 0;
    return static_cast<size_t>((O + 127) / 128 * 128) * R * S * C;
}

extern "C" int bs_tc_prepare_weights(const uint32_t* wgt_packed, int O, int C, int R, int S, int w_bits, bs_sign_t w_sign,
                                     int a_bits, int8_t* out, void* stream)
{
    if (!wgt_packed || !out || O <= 0 || C <= 0 || R <= 0 || S <= 0) return BS_ERR_INVALID_ARG;
    if (!bs::bits_ok(w_bits, w_sign) || a_bits < 1 || a_bits > 4) return BS_ERR_INVALID_ARG;
    if (!bs::aligned16(wgt_packed) || !bs::aligned16(out)) return BS_ERR_ALIGNMENT;
    const int CK = C % 32 == 0 ? bs::tc_chunk_channels(C, a_bits) : 0;
    if (CK == 0) return BS_ERR_UNSUPPORTED;
    const int opad8 = (O + 127) / 128 * 16;
    const long long nvec = static_cast<long long>(C / CK) * opad8 * R * S * (CK / 16) * 8;
    const long long blocks = (nvec + 255) / 256;
    if (blocks > 0x7fffffffLL) return BS_ERR_UNSUPPORTED;
    bs::tc_prepare_weights_kernel<<<static_cast<unsigned>(blocks), 256, 0, static_cast<cudaStream_t>(stream)>>>(
        wgt_packed, out, nvec, O, R * S, C / 32, w_bits, w_sign, CK, opad8);
    return cudaGetLastError() == cudaSuccess ? BS_OK : BS_ERR_CUDA;
}

extern "C" int bs_tc_supported(const bs_conv_params* p)
{
    if (bs::tc_validate(p) != BS_OK) return 0;
    // the answer of the planner itself (a shape may pass validation and still find no tiling that fits shared memory);
    // the epilogue fields do not change the tiling, so the query plans for raw accumulators
    bs_conv_params q = *p;
    q.scale = nullptr; q.bias = nullptr; q.residual = nullptr; q.out_bits = 0;
    return bs::tc_conv_impl(nullptr, nullptr, &q, nullptr, nullptr, nullptr, false, true) == BS_OK ? 1 : 0;
}

extern "C" int bitserial_conv2d_tc(const uint32_t* act_packed, const int8_t* wgt_tc, const bs_conv_params* p, int32_t* out_i32,
                                   uint32_t* out_packed, void* stream)
{
    return bs::tc_conv_impl(act_packed, wgt_tc, p, out_i32, out_packed, static_cast<cudaStream_t>(stream));
}

extern "C" size_t bs_tc_chain_workspace_bytes(const bs_conv_params* layers, int nlayers)
{
    if (!layers || nlayers < 2 || nlayers > bs::TC_CHAIN_MAX) return 0;
    bs::TcArgs L[bs::TC_CHAIN_MAX];
    size_t smem = 0;
    const long long tiles_m = bs::tc_chain_plan(nlayers, nullptr, nullptr, layers, nullptr, true, L, smem);
    return tiles_m > 0 ? bs::tc_chain_ws_bytes(nlayers, tiles_m) : 0;
}

extern "C" int bitserial_conv2d_tc_chain(int nlayers, const uint32_t* const* act_packed, const int8_t* const* wgt_tc,
                                         const bs_conv_params* layers, uint32_t* const* out_packed, void* workspace,
                                         size_t workspace_bytes, int chained, void* stream)
{
    return bs::tc_chain_impl(nlayers, act_packed, wgt_tc, layers, out_packed, workspace, workspace_bytes,
                             static_cast<cudaStream_t>(stream), chained != 0);
}

extern "C" int bitserial_conv2d_tc_chained(const uint32_t* act_packed, const int8_t* wgt_tc, const bs_conv_params* p,
                                           int32_t* out_i32, uint32_t* out_packed, void* stream)
{
    return bs::tc_conv_impl(act_packed, wgt_tc, p, out_i32, out_packed, static_cast<cudaStream_t>(stream), true);
}

extern "C" int bitserial_gemm_tc(const uint32_t* a_packed, const int8_t* w_tc, int M, int N, int K, int a_bits, bs_sign_t a_sign,
                                 int w_bits, bs_sign_t w_sign, const float* scale, const float* bias, int relu, int out_bits,
                                 bs_sign_t out_sign, int32_t* out_i32, uint32_t* out_packed, void* stream)
{
    if (M <= 0 || N <= 0 || K <= 0) return BS_ERR_INVALID_ARG;
    bs_conv_params p{};
    p.N = 1; p.C = K; p.H = 1; p.W = M; p.O = N; p.R = 1; p.S = 1; p.stride = 1; p.pad = 0;
    p.a_bits = a_bits; p.a_sign = a_sign; p.w_bits = w_bits; p.w_sign = w_sign;
    p.scale = scale; p.bias = bias; p.relu = relu; p.out_bits = out_bits; p.out_sign = out_sign;
    p.out_c_offset = 0; p.out_c_total = N; p.i32_layout = BS_NHWC;
    return bs::tc_conv_impl(a_packed, w_tc, &p, out_i32, out_packed, static_cast<cudaStream_t>(stream));
}
