// Comparison form of the requantisation epilogue (host side).
//
// After  t = fmaf((float)acc, scale[o], bias[o])  the rest of the epilogue,
//     v = fmaf(res_scale, res, t);  ReLU;  clip;  round-half-even   (or sign for bipolar outputs),
// depends only on t and on the residual code, and is monotone non-decreasing in t.  For 1- and 2-bit outputs the code
// is therefore  qmin + #{k : t >= bound[r][k]}  where bound[r][k] is the smallest binary32 t whose code reaches
// qmin + k when the residual pattern is r.  The bounds are found here by bisection over the ordered float bit patterns
// with the very same operations (fmaf, fmaxf, fminf, nearbyintf in binary32), so comparing against them takes exactly
// the decision of the formula; the kernels then need three compares per output instead of the arithmetic chain.
#pragma once
#include <cmath>
#include <cstdint>
#include <cstring>
#include <map>
#include <mutex>
#include <tuple>

#include "bitserial.h"

namespace bs {

struct RequantBounds {
    float bound[16][3];   // [residual pattern][k]; +inf where a level does not exist
    int enabled;          // 0: the kernel evaluates the formula (outputs wider than 2 bits)
    unsigned flip;        // pattern = count ^ flip (two's-complement outputs)
};

inline uint32_t rb_float_key(float f)
{
    uint32_t u;
    memcpy(&u, &f, 4);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
inline float rb_key_float(uint32_t k)
{
    const uint32_t u = (k & 0x80000000u) ? (k & 0x7fffffffu) : ~k;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

inline int rb_pattern_value(unsigned pat, int bits, int sign)
{
    if (sign == BS_BIPOLAR) return pat ? 1 : -1;
    int v = static_cast<int>(pat);
    if (sign == BS_SIGNED && (pat >> (bits - 1))) v -= (1 << bits);
    return v;
}

// Level index (0 .. nlevels-1) that the epilogue assigns to t.
inline int rb_level(float t, bool has_res, float res_scale, float res_val, int relu, int out_bits, int out_sign)
{
    volatile float v = t;
    if (has_res) v = fmaf(res_scale, res_val, v);
    if (relu) v = fmaxf(v, 0.0f);
    if (out_sign == BS_BIPOLAR) return v >= 0.0f ? 1 : 0;
    const int qmin = out_sign == BS_SIGNED ? -(1 << (out_bits - 1)) : 0;
    const int qmax = out_sign == BS_SIGNED ? (1 << (out_bits - 1)) - 1 : (1 << out_bits) - 1;
    const float c = fminf(fmaxf(v, static_cast<float>(qmin)), static_cast<float>(qmax));
    return static_cast<int>(nearbyintf(c)) - qmin;
}

inline RequantBounds make_requant_bounds(bool has_res, float res_scale, int res_bits, int res_sign, int relu, int out_bits,
                                         int out_sign)
{
    RequantBounds rb{};
    for (auto& row : rb.bound)
        for (float& b : row) b = INFINITY;
    rb.enabled = (out_bits <= 2 && out_bits >= 1 && (!has_res || (res_bits >= 1 && res_bits <= 4))) ? 1 : 0;
    rb.flip = 0;
    if (!rb.enabled) return rb;
    const int nlev = out_sign == BS_BIPOLAR ? 2 : (1 << out_bits);
    const int qmin = out_sign == BS_SIGNED ? -(1 << (out_bits - 1)) : 0;
    if (out_sign == BS_SIGNED) rb.flip = static_cast<unsigned>(qmin) & ((1u << out_bits) - 1u);
    const int npat = has_res ? (1 << res_bits) : 1;
    const uint32_t lo_key = rb_float_key(-INFINITY), hi_key = rb_float_key(INFINITY);
    for (int r = 0; r < npat; ++r) {
        const float res_val = has_res ? static_cast<float>(rb_pattern_value(static_cast<unsigned>(r), res_bits, res_sign)) : 0.0f;
        for (int k = 1; k < nlev; ++k) {
            uint32_t lo = lo_key, hi = hi_key;      // smallest key whose level is >= k; +inf always reaches the top level
            if (rb_level(INFINITY, has_res, res_scale, res_val, relu, out_bits, out_sign) < k) { rb.bound[r][k - 1] = INFINITY; continue; }
            while (lo < hi) {
                const uint32_t mid = lo + (hi - lo) / 2;
                if (rb_level(rb_key_float(mid), has_res, res_scale, res_val, relu, out_bits, out_sign) >= k) hi = mid;
                else lo = mid + 1;
            }
            rb.bound[r][k - 1] = rb_key_float(lo);
        }
    }
    return rb;
}

// Memoised variant: layers of a network share a handful of epilogue configurations.
inline RequantBounds cached_requant_bounds(bool has_res, float res_scale, int res_bits, int res_sign, int relu, int out_bits,
                                           int out_sign)
{
    typedef std::tuple<int, uint32_t, int, int, int, int, int> Key;
    static std::map<Key, RequantBounds> cache;
    static std::mutex mu;
    uint32_t rs_bits;
    memcpy(&rs_bits, &res_scale, 4);
    const Key key(has_res ? 1 : 0, has_res ? rs_bits : 0u, has_res ? res_bits : 0, has_res ? res_sign : 0, relu ? 1 : 0, out_bits, out_sign);
    std::lock_guard<std::mutex> lock(mu);
    auto it = cache.find(key);
    if (it == cache.end()) it = cache.emplace(key, make_requant_bounds(has_res, res_scale, res_bits, res_sign, relu, out_bits, out_sign)).first;
    return it->second;
}

}  // namespace bs
