// Host side of bitserial_conv2d / bitserial_gemm: validation, tile planning, TMA descriptors, launch.
#include <array>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <map>
#include <mutex>

#include "conv_launch.cuh"
#include "requant_bounds.h"

namespace bs {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    });
    return fn;
}

static int round_up(int v, int m) { return (v + m - 1) / m * m; }

struct Plan {
    int PB, FB, NFG, NT, TWB, TH, TNI, CWC, nchunks, nstage;
    int hh, hw, stageA_words, stageW_words, aux_off_words;
    int tma_a, tma_w, boxA_w, nboxA, unitA, unitW;
    int ksplit, chunks_per_split;
    size_t smem, ws_bytes;
    long long tiles;
    double cost;
};

static int largest_unit(int a, int b)
{
    if (a % 4 == 0 && b % 4 == 0) return 4;
    if (a % 2 == 0 && b % 2 == 0) return 2;
    return 1;
}

// Fill the staging part of a plan; returns false if the tile cannot be staged in shared memory.
static bool plan_staging(Plan& pl, int Cw, int RS, int R, int S, int stride, int A, int WB, bool many_tiles = false)
{
    const int TN = pl.NFG * pl.FB;
    const int TW = pl.TWB * pl.PB;
    pl.hh = (pl.TH - 1) * stride + R;
    pl.hw = (TW - 1) * stride + S;
    pl.CWC = Cw < (RS == 1 ? 8 : 4) ? Cw : (RS == 1 ? 8 : 4);
    if (RS == 1 && Cw > 8) {
        // 1x1 layers and matrix products: channel words per chunk among 8, 6 and 4.  The reduction loop takes the words of
        // a chunk three at a time through the carry-save adder (two counts per three words, one count per left-over
        // word) and a chunk costs about 0.85 counts of hand-off (fitted to 4096 x 4096 products with 72 words: 640 / 605 /
        // 709 us for 8 / 6 / 4); six words are two clean triples, and 18 words (576 channels) are three full chunks of six
        // instead of 8 + 8 + 2.  A width that would take the activations off the TMA path (record not a multiple of
        // 16 bytes) is not considered; the filters may fall back to the gather.  More chunks are only accepted when the
        // tiles fill the machine several times over (`many_tiles`): with one or two tiles per SM every extra hand-off is
        // exposed latency (1024 x 1024 x 2304: 0.058 ms with chunks of 8, 0.065 ms with chunks of 6).
        double best_cost = 0.0;
        const int chunks8 = ceil_div(Cw, 8);
        for (int cwc = 8; cwc >= 4; cwc -= 2) {
            if ((cwc * A) % 4 != 0 && (8 * A) % 4 == 0) continue;
            const int full = Cw / cwc, tail = Cw % cwc;
            if (!many_tiles && full + (tail ? 1 : 0) > chunks8) continue;
            const double cost = full * (2 * (cwc / 3) + cwc % 3) + (tail ? 2 * (tail / 3) + tail % 3 : 0) + 0.85 * (full + (tail ? 1 : 0));
            if (cwc == 8 || cost < 0.95 * best_cost) { best_cost = cost; pl.CWC = cwc; }      // a clear gain only
        }
    }
#ifdef BS_TUNING
    if (const char* e = getenv("BS_CWC")) { const int v = atoi(e); if (v >= 1 && v <= 8 && v <= Cw) pl.CWC = v; }
#endif
    pl.nchunks = ceil_div(Cw, pl.CWC);
    const int recA = pl.CWC * A, recW = pl.CWC * WB;
    pl.tma_a = (recA % 4 == 0) && ((Cw * A) % 4 == 0);
    pl.tma_w = (recW % 4 == 0) && ((Cw * WB) % 4 == 0) && RS <= 256 && TN <= 256;
    pl.boxA_w = pl.hw;
    pl.nboxA = 1;
    if (pl.tma_a) {
        if (pl.hh > 256 || pl.TNI > 256 || recA > 256) pl.tma_a = 0;
        else if (pl.hw > 256) {
            // only a single-row, single-image tile keeps split boxes contiguous in shared memory
            const int nb = ceil_div(pl.hw, 256);
            if (pl.hh == 1 && pl.TNI == 1 && pl.hw % nb == 0) { pl.nboxA = nb; pl.boxA_w = pl.hw / nb; }
            else pl.tma_a = 0;
        }
    }
    pl.unitA = largest_unit(recA, Cw * A);
    pl.unitW = largest_unit(recW, Cw * WB);
    pl.stageA_words = round_up(pl.TNI * pl.hh * pl.hw * recA, 32);
    pl.stageW_words = round_up(TN * RS * recW, 32);
    const size_t stage_bytes = static_cast<size_t>(pl.stageA_words + pl.stageW_words) * 4;
    pl.nstage = pl.nchunks < 3 ? pl.nchunks : 3;
    while (pl.nstage > 1 && stage_bytes * pl.nstage > 96 * 1024) --pl.nstage;
    const size_t ring = stage_bytes * pl.nstage;
    const int used_pix = pl.TWB * pl.TH * pl.TNI * pl.PB;
    const size_t codes = static_cast<size_t>(used_pix) * (TN + 4);
    const size_t main_bytes = round_up(static_cast<int>(ring > codes ? ring : codes), 128);
    pl.aux_off_words = static_cast<int>(main_bytes / 4);
    pl.smem = main_bytes + MAX_STAGES * 8 + static_cast<size_t>(used_pix) * 4 + static_cast<size_t>(TN) * 4;
    return pl.smem <= 200 * 1024;
}

// Per-thread (pixels, filters) register blocks that are instantiated (must match BS_TILE_LIST).
static const int kTiles[][2] = {{8, 8}, {7, 8}, {4, 8}, {8, 4}, {7, 4}, {4, 4}, {8, 2}, {7, 2}, {4, 2}};

// Exhaustive search over register blocks and CTA tilings with a small analytic time model:
//   - the popcount pipe retires one warp instruction per 8 cycles per SM sub-partition, so a warp costs
//     steps * PB * FB * pairs * 8 cycles, divided by an efficiency that is best for 48..160 popcounts per
//     reduction step (larger bodies spill out of the instruction cache, smaller ones are load-issue bound);
//   - the busiest SM runs ceil(tiles / SMs) CTAs one after the other on its four sub-partitions;
//   - fewer than 8 resident warps leave the pipe partly idle.
static bool search_plan(Plan& best, int N, int P, int Q, int O, int Cw, int R, int S, int stride, int A, int WB,
                        bool allow_split, int sms)
{
    const int RS = R * S;
    const int pairs = A * WB;
    bool found = false;
    for (const auto& tile : kTiles) {
        const int PB = tile[0], FB = tile[1];
        const int qb = ceil_div(Q, PB);
        const double work = static_cast<double>(PB) * FB * pairs;
        double eff_block = 0.86;
        if (work > 160.0) eff_block -= 0.06 * log2(work / 160.0);
        if (work < 48.0) eff_block -= 0.08 * log2(48.0 / work);
        for (int NFG = 4; NFG <= 32; NFG *= 2) {
            const int TN = NFG * FB;
            if (TN % 32 != 0 || TN > 256) continue;          // packed output words must not straddle CTAs
            if (PB > 4 * NFG) continue;                      // window sums: at most 4 tile pixels per thread
            const long long tiles_o = ceil_div(O, TN);
            for (int NPG = 1; NPG * NFG <= 256; NPG *= 2) {
                for (int TWB = 1; TWB <= NPG && TWB <= qb; ++TWB) {
                    const int max_th = NPG / TWB;
                    for (int TH = 1; TH <= max_th && TH <= P; ++TH) {
                        int TNI = NPG / (TWB * TH);
                        if (TNI > N) TNI = N;
                        if (TNI < 1) continue;
                        const int used = TWB * TH * TNI;
                        if (2 * used <= NPG && NPG > 1) continue;           // a smaller NPG covers this tiling
                        Plan pl{};
                        pl.PB = PB; pl.FB = FB; pl.NFG = NFG; pl.TWB = TWB; pl.TH = TH; pl.TNI = TNI;
                        pl.NT = round_up(used * NFG, 32);
                        pl.tiles = tiles_o * ceil_div(qb, TWB) * ceil_div(P, TH) * ceil_div(N, TNI);
                        if (!plan_staging(pl, Cw, RS, R, S, stride, A, WB, pl.tiles >= 8LL * sms)) continue;
                        const double cta_warps = pl.NT / 32.0;
                        // warps of a CTA spread over the four sub-partitions; the fullest one sets the pace
                        double per_subpartition = 0.5 * (ceil(cta_warps / 4.0) + cta_warps / 4.0);
                        if (per_subpartition < 1.0) per_subpartition = 1.0;
                        const double halo = 1.0 + 0.01 * (static_cast<double>(pl.hh) * pl.hw / (TWB * PB * TH)) / (stride * stride);
                        // reduction split: only when the tiles alone cannot fill the machine
                        const int max_split = allow_split ? pl.nchunks : 1;
                        for (int ksplit = 1; ksplit <= max_split; ksplit *= 2) {
                            if (ksplit > 1 && pl.tiles * (ksplit / 2) >= 2LL * sms) break;
                            const int cps = ceil_div(pl.nchunks, ksplit);
                            const int eff_split = ceil_div(pl.nchunks, cps);
                            const double split_steps = static_cast<double>(cps) * pl.CWC * RS;
                            const double wc = split_steps * work * 8.0 / eff_block + 0.5 * (PB * FB * 15.0 + 1500.0) +
                                              (eff_split > 1 ? PB * FB * 40.0 + 2000.0 : 0.0);
                            const long long ctas = pl.tiles * eff_split;
                            const long long per_sm = ceil_div_ll(ctas, sms);
                            long long resident = static_cast<long long>((200 * 1024) / pl.smem);
                            if (resident > per_sm) resident = per_sm;
                            if (resident * pl.NT > 1536) resident = 1536 / pl.NT;
                            if (resident < 1) resident = 1;
                            const double warps = static_cast<double>(resident) * cta_warps;
                            const double occ = warps >= 8.0 ? 1.0 : warps / 8.0;
                            const double cost = static_cast<double>(per_sm) * per_subpartition * wc / occ * halo;
                            if (!found || cost < best.cost * 0.999) {
                                best = pl;
                                best.cost = cost;
                                best.ksplit = eff_split;
                                best.chunks_per_split = cps;
                                best.ws_bytes = eff_split > 1 ? static_cast<size_t>(pl.tiles) * (static_cast<size_t>(PB) * FB * pl.NT + 1) * 4 : 0;
                                found = true;
                            }
                        }
                    }
                }
            }
        }
    }
    return found;
}

// Plans depend on the shape only, so they are searched once per shape and remembered.
static bool make_plan(Plan& out, int N, int P, int Q, int O, int Cw, int R, int S, int stride, int A, int WB,
                      bool allow_split)
{
#ifdef BS_TUNING   // tile-plan tuning hook, compiled only into tuning builds: BS_PLAN="PB,FB,NFG,NT,TWB,TH,TNI"
    if (const char* ov = getenv("BS_PLAN")) {
        Plan pl{};
        if (sscanf(ov, "%d,%d,%d,%d,%d,%d,%d", &pl.PB, &pl.FB, &pl.NFG, &pl.NT, &pl.TWB, &pl.TH, &pl.TNI) == 7) {
            if (pl.TNI > N) pl.TNI = N;
            pl.NT = round_up(pl.TWB * pl.TH * pl.TNI * pl.NFG, 32);
            if (!plan_staging(pl, Cw, R * S, R, S, stride, A, WB)) return false;
            pl.ksplit = 1; pl.chunks_per_split = pl.nchunks; pl.ws_bytes = 0;
            out = pl;
            return true;
        }
    }
#endif
    // the plan (tiling, reduction split, workspace size) also depends on the multiprocessor count of the current device
    const int sms = device_sm_count();
    if (sms <= 0) return false;
    static std::map<std::array<int, 12>, std::pair<bool, Plan>> cache;
    static std::mutex mu;
    const std::array<int, 12> key = {N, P, Q, O, Cw, R, S, stride, A, WB, allow_split ? 1 : 0, sms};
    std::lock_guard<std::mutex> lock(mu);
    auto it = cache.find(key);
    if (it == cache.end()) {
        Plan pl{};
        const bool ok = search_plan(pl, N, P, Q, O, Cw, R, S, stride, A, WB, allow_split, sms);
        it = cache.emplace(key, std::make_pair(ok, pl)).first;
    }
    out = it->second.second;
#ifdef BS_TUNING
    if (getenv("BS_PLAN_VERBOSE")) {
        const Plan& q = out;
        fprintf(stderr, "popc plan: N%d %dx%d O%d Cw%d k%d s%d A%d W%d -> PB %d FB %d NFG %d NT %d TWB %d TH %d TNI %d CWC %d chunks %d stages %d split %d tiles %lld smem %zu cost %.0f\n",
                N, P, Q, O, Cw, R, stride, A, WB, q.PB, q.FB, q.NFG, q.NT, q.TWB, q.TH, q.TNI, q.CWC, q.nchunks, q.nstage, q.ksplit, q.tiles, q.smem, q.cost);
    }
#endif
    return it->second.first;
}

static bool encode_map(CUtensorMap* tm, const void* base, int rank, const cuuint64_t* dims, const cuuint64_t* strides_bytes,
                       const cuuint32_t* box)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint32_t estr[5] = {1, 1, 1, 1, 1};
    return fn(tm, CU_TENSOR_MAP_DATA_TYPE_UINT32, static_cast<cuuint32_t>(rank), const_cast<void*>(base), dims,
              strides_bytes, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
              CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

static int max_abs_code(int bits, int sign)
{
    if (sign == BS_BIPOLAR) return 1;
    if (sign == BS_SIGNED) return 1 << (bits - 1);
    return (1 << bits) - 1;
}

// `query_ws` != NULL: validate, plan with the reduction split allowed, report the workspace it wants, launch nothing.
static int conv_impl(const uint32_t* act, const uint32_t* wgt, const bs_conv_params* p, int32_t* out_i32,
                     uint32_t* out_packed, void* workspace, size_t workspace_bytes, cudaStream_t st,
                     size_t* query_ws = nullptr)
{
    if (!p) return BS_ERR_INVALID_ARG;
    if (!query_ws && (!act || !wgt || (!out_i32 && !out_packed))) return BS_ERR_INVALID_ARG;
    if (p->N <= 0 || p->C <= 0 || p->H <= 0 || p->W <= 0 || p->O <= 0 || p->R <= 0 || p->S <= 0) return BS_ERR_INVALID_ARG;
    if (!bits_ok(p->a_bits, p->a_sign) || !bits_ok(p->w_bits, p->w_sign)) return BS_ERR_INVALID_ARG;
    if (p->stride < 1 || p->pad < 0) return BS_ERR_INVALID_ARG;
    if (p->i32_layout != BS_NCHW && p->i32_layout != BS_NHWC) return BS_ERR_INVALID_ARG;
    if (p->R != p->S || (p->R != 1 && p->R != 3 && p->R != 5 && p->R != 7)) return BS_ERR_UNSUPPORTED;
    if (p->stride > 2 || p->pad >= p->R) return BS_ERR_UNSUPPORTED;
    if (p->a_sign == BS_BIPOLAR && p->pad != 0) return BS_ERR_UNSUPPORTED;
    if (p->H + 2 * p->pad < p->R || p->W + 2 * p->pad < p->S) return BS_ERR_INVALID_ARG;
    if (!aligned16(act) || !aligned16(wgt) || (out_i32 && !aligned16(out_i32)) || (out_packed && !aligned16(out_packed)) ||
        (workspace && !aligned16(workspace)))
        return BS_ERR_ALIGNMENT;
    const long long kred = static_cast<long long>(p->C) * p->R * p->S;
    if (kred * max_abs_code(p->a_bits, p->a_sign) * max_abs_code(p->w_bits, p->w_sign) >= (1LL << 31))
        return BS_ERR_UNSUPPORTED;

    ConvArgs g{};
    g.P = (p->H + 2 * p->pad - p->R) / p->stride + 1;
    g.Q = (p->W + 2 * p->pad - p->S) / p->stride + 1;
    g.Cw = ceil_div(p->C, 32);
    if (out_packed) {
        if (!p->scale || !p->bias) return BS_ERR_INVALID_ARG;
        if (!bits_ok(p->out_bits, p->out_sign)) return BS_ERR_INVALID_ARG;
        if (p->out_c_offset < 0 || p->out_c_total < p->out_c_offset + p->O) return BS_ERR_INVALID_ARG;
        if (p->out_c_offset % 32 != 0) return BS_ERR_UNSUPPORTED;
        if (p->O % 32 != 0 && p->out_c_offset + p->O != p->out_c_total) return BS_ERR_UNSUPPORTED;
        if (p->residual) {
            if (!bits_ok(p->res_bits, p->res_sign)) return BS_ERR_INVALID_ARG;
            if (p->res_c_offset < 0 || p->res_c_total < p->res_c_offset + p->O) return BS_ERR_INVALID_ARG;
            if (!aligned16(p->residual)) return BS_ERR_ALIGNMENT;
        }
    }

    const int A = p->a_bits, WB = p->w_bits;
    Plan pl{};
    const bool want_split = query_ws != nullptr || (workspace != nullptr && workspace_bytes > 0);
    if (!make_plan(pl, p->N, g.P, g.Q, p->O, g.Cw, p->R, p->S, p->stride, A, WB, want_split)) return BS_ERR_UNSUPPORTED;
    if (query_ws) { *query_ws = pl.ws_bytes; return BS_OK; }
    if (pl.ws_bytes > workspace_bytes &&      // the workspace is too small for the split plan: run unsplit
        !make_plan(pl, p->N, g.P, g.Q, p->O, g.Cw, p->R, p->S, p->stride, A, WB, false))
        return BS_ERR_UNSUPPORTED;

    g.act = act; g.wgt = wgt; g.out_i32 = out_i32; g.out_packed = out_packed;
    g.scale = p->scale; g.bias = p->bias;
    g.residual = out_packed ? p->residual : nullptr;
    g.res_scale = p->res_scale;
    g.status = status_device_ptr();
    if (!g.status) return BS_ERR_CUDA;
    g.N = p->N; g.C = p->C; g.H = p->H; g.W = p->W; g.O = p->O; g.R = p->R; g.S = p->S;
    g.stride = p->stride; g.pad = p->pad;
    g.a_sign = p->a_sign; g.w_sign = p->w_sign;
    g.relu = p->relu; g.out_bits = p->out_bits; g.out_sign = p->out_sign;
    g.out_cw_off = p->out_c_offset / 32; g.out_cw_total = ceil_div(p->out_c_total > 0 ? p->out_c_total : 1, 32);
    g.res_bits = p->res_bits; g.res_sign = p->res_sign; g.res_c_off = p->res_c_offset;
    g.res_cw_total = ceil_div(p->res_c_total > 0 ? p->res_c_total : 1, 32);
    g.i32_nhwc = p->i32_layout == BS_NHWC;
    g.NFG = pl.NFG; g.NPG = pl.NT / pl.NFG; g.TNI = pl.TNI; g.TH = pl.TH; g.TWB = pl.TWB;
    g.used_pg = pl.TWB * pl.TH * pl.TNI;
    g.hh = pl.hh; g.hw = pl.hw; g.CWC = pl.CWC; g.nchunks = pl.nchunks; g.nstage = pl.nstage;
    g.stageA_words = pl.stageA_words; g.stageW_words = pl.stageW_words; g.aux_off_words = pl.aux_off_words;
    const int TN = pl.NFG * pl.FB, TW = pl.TWB * pl.PB;
    g.tiles_o = ceil_div(p->O, TN); g.tiles_q = ceil_div(g.Q, TW); g.tiles_p = ceil_div(g.P, pl.TH);
    g.tiles_n = ceil_div(p->N, pl.TNI);
    g.tma_a = pl.tma_a; g.tma_w = pl.tma_w; g.boxA_w = pl.boxA_w; g.nboxA = pl.nboxA;
    g.unitA = pl.unitA; g.unitW = pl.unitW;

    const int alpha_a = p->a_sign == BS_BIPOLAR ? 2 : 1, alpha_w = p->w_sign == BS_BIPOLAR ? 2 : 1;
    for (int i = 0; i < 4; ++i) {
        const int ci = (p->w_sign == BS_SIGNED && i == WB - 1) ? -1 : 1;
        g.cs_coef[i] = -alpha_w * ci * (1 << i);
        for (int j = 0; j < 4; ++j) {
            const int dj = (p->a_sign == BS_SIGNED && j == A - 1) ? -1 : 1;
            g.coef[i][j] = alpha_a * alpha_w * ci * dj * (1 << (i + j));
            g.rs_coef[j] = -alpha_a * dj * (1 << j);
        }
    }
    g.need_rs = p->w_sign == BS_BIPOLAR;
    g.need_cs = p->a_sign == BS_BIPOLAR;
    g.kconst = (g.need_rs && g.need_cs) ? static_cast<int>(kred) : 0;
    g.ksplit = pl.ksplit; g.chunks_per_split = pl.chunks_per_split;
    if (pl.ksplit > 1) {
        g.ws_acc = static_cast<int*>(workspace);
        g.ws_cnt = reinterpret_cast<unsigned*>(g.ws_acc + static_cast<size_t>(pl.tiles) * pl.PB * pl.FB * pl.NT);
    }
    g.acc_small = kred * max_abs_code(p->a_bits, p->a_sign) * max_abs_code(p->w_bits, p->w_sign) < (1LL << 22);

    const long long tiles = static_cast<long long>(g.tiles_o) * g.tiles_q * g.tiles_p * g.tiles_n * pl.ksplit;
    if (tiles > 0x7fffffffLL) return BS_ERR_UNSUPPORTED;

    if (g.tma_a) {
        const cuuint64_t fullA = static_cast<cuuint64_t>(g.Cw) * A;
        cuuint64_t dims[4] = {fullA, static_cast<cuuint64_t>(p->W), static_cast<cuuint64_t>(p->H), static_cast<cuuint64_t>(p->N)};
        cuuint64_t strides[3] = {fullA * 4, fullA * 4 * p->W, fullA * 4 * p->W * p->H};
        cuuint32_t box[4] = {static_cast<cuuint32_t>(g.CWC * A), static_cast<cuuint32_t>(g.boxA_w),
                             static_cast<cuuint32_t>(g.hh), static_cast<cuuint32_t>(g.TNI)};
        if (!encode_map(&g.tmA, act, 4, dims, strides, box)) {
            g.tma_a = 0; g.nboxA = 1; g.boxA_w = g.hw;   // descriptor refused: gather instead
        }
    }
    if (g.tma_w) {
        const cuuint64_t fullW = static_cast<cuuint64_t>(g.Cw) * WB;
        const cuuint64_t RS = static_cast<cuuint64_t>(p->R) * p->S;
        cuuint64_t dims[3] = {fullW, RS, static_cast<cuuint64_t>(p->O)};
        cuuint64_t strides[2] = {fullW * 4, fullW * 4 * RS};
        cuuint32_t box[3] = {static_cast<cuuint32_t>(g.CWC * WB), static_cast<cuuint32_t>(RS), static_cast<cuuint32_t>(TN)};
        if (!encode_map(&g.tmW, wgt, 3, dims, strides, box)) g.tma_w = 0;
    }

    const unsigned grid = static_cast<unsigned>(tiles), block = static_cast<unsigned>(pl.NT);
    typedef int (*LaunchFn)(int, int, const ConvArgs&, unsigned, unsigned, size_t, cudaStream_t);
    static const LaunchFn table[4][3] = {{launch_conv_a1_f2, launch_conv_a1_f4, launch_conv_a1_f8},
                                         {launch_conv_a2_f2, launch_conv_a2_f4, launch_conv_a2_f8},
                                         {launch_conv_a3_f2, launch_conv_a3_f4, launch_conv_a3_f8},
                                         {launch_conv_a4_f2, launch_conv_a4_f4, launch_conv_a4_f8}};
    return table[A - 1][pl.FB == 8 ? 2 : (pl.FB == 4 ? 1 : 0)](WB, pl.PB, g, grid, block, pl.smem, st);
}

}  // namespace bs

static bs_conv_params gemm_as_conv(int M, int N, int K, int a_bits, int a_sign, int w_bits, int w_sign, const float* scale,
                                   const float* bias, int relu, int out_bits, int out_sign)
{
    // a matrix product is a 1x1 convolution over a 1 x M image with K channels and N filters
    bs_conv_params p{};
    p.N = 1; p.C = K; p.H = 1; p.W = M; p.O = N; p.R = 1; p.S = 1; p.stride = 1; p.pad = 0;
    p.a_bits = a_bits; p.a_sign = a_sign; p.w_bits = w_bits; p.w_sign = w_sign;
    p.scale = scale; p.bias = bias; p.relu = relu; p.out_bits = out_bits; p.out_sign = out_sign;
    p.residual = nullptr; p.out_c_offset = 0; p.out_c_total = N; p.i32_layout = BS_NHWC;
    return p;
}

extern "C" int bitserial_conv2d(const uint32_t* act_packed, const uint32_t* wgt_packed, const bs_conv_params* p,
                                int32_t* out_i32, uint32_t* out_packed, void* stream)
{
    return bs::conv_impl(act_packed, wgt_packed, p, out_i32, out_packed, nullptr, 0, static_cast<cudaStream_t>(stream));
}

extern "C" int bitserial_conv2d_ws(const uint32_t* act_packed, const uint32_t* wgt_packed, const bs_conv_params* p,
                                   int32_t* out_i32, uint32_t* out_packed, void* workspace, size_t workspace_bytes,
                                   void* stream)
{
    return bs::conv_impl(act_packed, wgt_packed, p, out_i32, out_packed, workspace, workspace_bytes,
                         static_cast<cudaStream_t>(stream));
}

extern "C" size_t bs_conv_workspace_bytes(const bs_conv_params* p)
{
    size_t need = 0;
    if (bs::conv_impl(nullptr, nullptr, p, nullptr, nullptr, nullptr, 0, nullptr, &need) != BS_OK) return 0;
    return need;
}

extern "C" int bitserial_gemm(const uint32_t* a_packed, const uint32_t* w_packed, int M, int N, int K, int a_bits,
                              bs_sign_t a_sign, int w_bits, bs_sign_t w_sign, const float* scale, const float* bias,
                              int relu, int out_bits, bs_sign_t out_sign, int32_t* out_i32, uint32_t* out_packed,
                              void* stream)
{
    if (M <= 0 || N <= 0 || K <= 0) return BS_ERR_INVALID_ARG;
    const bs_conv_params p = gemm_as_conv(M, N, K, a_bits, a_sign, w_bits, w_sign, scale, bias, relu, out_bits, out_sign);
    return bs::conv_impl(a_packed, w_packed, &p, out_i32, out_packed, nullptr, 0, static_cast<cudaStream_t>(stream));
}

extern "C" int bitserial_gemm_ws(const uint32_t* a_packed, const uint32_t* w_packed, int M, int N, int K, int a_bits,
                                 bs_sign_t a_sign, int w_bits, bs_sign_t w_sign, const float* scale, const float* bias,
                                 int relu, int out_bits, bs_sign_t out_sign, int32_t* out_i32, uint32_t* out_packed,
                                 void* workspace, size_t workspace_bytes, void* stream)
{
    if (M <= 0 || N <= 0 || K <= 0) return BS_ERR_INVALID_ARG;
    const bs_conv_params p = gemm_as_conv(M, N, K, a_bits, a_sign, w_bits, w_sign, scale, bias, relu, out_bits, out_sign);
    return bs::conv_impl(a_packed, w_packed, &p, out_i32, out_packed, workspace, workspace_bytes,
                         static_cast<cudaStream_t>(stream));
}

extern "C" size_t bs_gemm_workspace_bytes(int M, int N, int K, int a_bits, bs_sign_t a_sign, int w_bits, bs_sign_t w_sign)
{
    if (M <= 0 || N <= 0 || K <= 0) return 0;
    const bs_conv_params p = gemm_as_conv(M, N, K, a_bits, a_sign, w_bits, w_sign, nullptr, nullptr, 0, 0, 0);
    size_t need = 0;
    if (bs::conv_impl(nullptr, nullptr, &p, nullptr, nullptr, nullptr, 0, nullptr, &need) != BS_OK) return 0;
    return need;
}

// ---------------------------------------------------------------------------------------------------------------
// Matrix product with the reduction split for callers that cannot allocate device memory.
//
// The split needs a scratch area for partial sums.  Here it lives in the library image itself: a file-scope device
// array that every GPU loading the library holds until the process exits.  In host code the array's name is only a
// host-side stand-in for the symbol, not a device address, so the address is looked up once per device with
// cudaGetSymbolAddress (with that device current) and that pointer is what the kernel receives.
// ---------------------------------------------------------------------------------------------------------------
#define BS_STATIC_SCRATCH_BYTES (2u * 1024u * 1024u)

static __device__ __align__(256) unsigned char bs_static_scratch[BS_STATIC_SCRATCH_BYTES];

namespace bs {

constexpr int kMaxDevices = 64;
static void* g_scratch_ptr[kMaxDevices];   // per device, filled on the first call made with that device current
static std::mutex g_scratch_mu;

// Device address of the static scratch array on the current device, or nullptr with *status set.
static void* static_scratch_ptr(int* status)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) { *status = BS_ERR_CUDA; return nullptr; }
    std::lock_guard<std::mutex> lock(g_scratch_mu);
    if (!g_scratch_ptr[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, bs_static_scratch) != cudaSuccess || !p) {
            cudaGetLastError();
            *status = BS_ERR_CUDA;
            return nullptr;
        }
        g_scratch_ptr[dev] = p;
    }
    return g_scratch_ptr[dev];
}

}  // namespace bs

extern "C" size_t bs_gemm_noalloc_max_scratch_bytes(void) { return BS_STATIC_SCRATCH_BYTES; }

extern "C" int bitserial_gemm_noalloc(const uint32_t* a_packed, const uint32_t* w_packed, int M, int N, int K, int a_bits,
                                      bs_sign_t a_sign, int w_bits, bs_sign_t w_sign, const float* scale,
                                      const float* bias, int relu, int out_bits, bs_sign_t out_sign, int32_t* out_i32,
                                      uint32_t* out_packed, void* stream)
{
    if (M <= 0 || N <= 0 || K <= 0) return BS_ERR_INVALID_ARG;
    const bs_conv_params p = gemm_as_conv(M, N, K, a_bits, a_sign, w_bits, w_sign, scale, bias, relu, out_bits, out_sign);
    // how much scratch the split plan of this shape wants (host-only planning; also validates the shape)
    size_t need = 0;
    int st = bs::conv_impl(nullptr, nullptr, &p, nullptr, nullptr, nullptr, 0, nullptr, &need);
    if (st != BS_OK) return st;
    if (need > BS_STATIC_SCRATCH_BYTES) return BS_ERR_UNSUPPORTED;   // beyond the built-in scratch: use bitserial_gemm_ws
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    void* scratch = nullptr;
    if (need > 0) {
        scratch = bs::static_scratch_ptr(&st);
        if (!scratch) return st;
        // Partial sums and arrival counters must start at zero.  A call that completed leaves them zero again, so this
        // clearing is defensive: it covers a predecessor that gave up on a bounded wait (BS_ERR_TIMEOUT) half-way.
        if (cudaMemsetAsync(scratch, 0, need, cs) != cudaSuccess) { cudaGetLastError(); return BS_ERR_CUDA; }
    }
    return bs::conv_impl(a_packed, w_packed, &p, out_i32, out_packed, scratch, need, cs);
}

// Test aid: fills the built-in scratch with a byte value, standing in for a predecessor that did not finish cleanly,
// so that a test can show the clearing in bitserial_gemm_noalloc is what makes the next call right.
extern "C" int bs_selftest_dirty_noalloc_scratch(int byte_value, void* stream)
{
    int st = BS_OK;
    void* scratch = bs::static_scratch_ptr(&st);
    if (!scratch) return st;
    if (cudaMemsetAsync(scratch, byte_value & 0xFF, BS_STATIC_SCRATCH_BYTES, static_cast<cudaStream_t>(stream)) != cudaSuccess) {
        cudaGetLastError();
        return BS_ERR_CUDA;
    }
    return BS_OK;
}

// ---- self-test of the failure path: a wait that runs out ------------------------------------------------------------
namespace bs {
// One warp; lane 0 waits, with the kernels' own bounded wait, on a barrier at which nothing ever arrives, gives up after
// `polls` polls and reports through the status word exactly as the convolution kernels do.  Nothing traps or spins
// without limit: the kernel always returns and the context stays usable.
__global__ void wait_timeout_selftest_kernel(unsigned polls, int* status)
{
    __shared__ __align__(8) uint64_t bar;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        fence_barrier_init();
        if (!mbar_wait_bounded(&bar, 0, polls)) atomicOr(status, STATUS_TIMEOUT);
    }
}
}  // namespace bs

extern "C" int bs_selftest_wait_timeout(int polls, void* stream)
{
    if (polls < 1 || polls > 65536) return BS_ERR_INVALID_ARG;
    int* status = bs::status_device_ptr();
    if (!status) return BS_ERR_CUDA;
    bs::wait_timeout_selftest_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(static_cast<unsigned>(polls), status);
    return cudaGetLastError() == cudaSuccess ? BS_OK : BS_ERR_CUDA;
}

// ---- host-side view of the epilogue's comparison form (no device work) ------------------------------------------
extern "C" int bs_requant_bounds(int has_residual, float res_scale, int res_bits, bs_sign_t res_sign, int relu, int out_bits,
                                 bs_sign_t out_sign, float* bounds_out)
{
    if (!bounds_out || !bs::bits_ok(out_bits, out_sign)) return BS_ERR_INVALID_ARG;
    if (has_residual && !bs::bits_ok(res_bits, res_sign)) return BS_ERR_INVALID_ARG;
    const bs::RequantBounds rb = bs::make_requant_bounds(has_residual != 0, res_scale, res_bits, res_sign, relu, out_bits, out_sign);
    if (!rb.enabled) return BS_ERR_UNSUPPORTED;
    const int npat = has_residual ? (1 << res_bits) : 1;
    for (int r = 0; r < npat; ++r)
        for (int k = 0; k < 3; ++k) bounds_out[r * 3 + k] = rb.bound[r][k];
    return BS_OK;
}
