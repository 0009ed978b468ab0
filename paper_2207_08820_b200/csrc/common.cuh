// Shared host/device helpers of the bit-serial library (CUDA side only).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "bitserial.h"

namespace bs {

// Device status word: kernels OR error bits into it when a bounded wait runs out.
enum : int { STATUS_TIMEOUT = 1 };
int* status_device_ptr();   // device address of the status word of the current device (host call)
int device_sm_count();      // multiprocessors of the CURRENT device (looked up once per device ordinal; 0 on error)

inline int ceil_div(int a, int b) { return (a + b - 1) / b; }
inline long long ceil_div_ll(long long a, long long b) { return (a + b - 1) / b; }

inline bool bits_ok(int bits, int sign)
{
    if (bits < 1 || bits > 4) return false;
    if (sign != BS_UNSIGNED && sign != BS_SIGNED && sign != BS_BIPOLAR) return false;
    if (sign == BS_BIPOLAR && bits != 1) return false;
    return true;
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Stored pattern of a code: low `bits` bits, or (code > 0) for bipolar.
__device__ __forceinline__ unsigned stored_pattern(int code, int bits, int sign)
{
    return sign == BS_BIPOLAR ? (code > 0 ? 1u : 0u) : (static_cast<unsigned>(code) & ((1u << bits) - 1u));
}

// Value of a stored pattern.
__device__ __forceinline__ int pattern_value(unsigned pat, int bits, int sign)
{
    if (sign == BS_BIPOLAR) return pat ? 1 : -1;
    int v = static_cast<int>(pat);
    if (sign == BS_SIGNED && (pat >> (bits - 1))) v -= (1 << bits);
    return v;
}

__host__ __device__ __forceinline__ void code_limits(int bits, int sign, int& qmin, int& qmax)
{
    if (sign == BS_SIGNED) { qmin = -(1 << (bits - 1)); qmax = (1 << (bits - 1)) - 1; }
    else if (sign == BS_BIPOLAR) { qmin = -1; qmax = 1; }
    else { qmin = 0; qmax = (1 << bits) - 1; }
}

}  // namespace bs
