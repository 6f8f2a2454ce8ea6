// Order-preserving key of a score, shared by the ranking kernels.
#pragma once
#include <cstdint>

namespace pc {

// Monotone map float -> uint32 with "larger key = better".  NaN ranks worst, -0 == +0.
__device__ __forceinline__ uint32_t rank_key(float f, bool lower_is_better) {
  if (f != f) return 0u;
  if (lower_is_better) f = -f;
  uint32_t u = __float_as_uint(f);
  if (u == 0x80000000u) u = 0u;                       // -0 -> +0
  u = (u & 0x80000000u) ? ~u : (u | 0x80000000u);
  return u == 0u ? 1u : u;                            // keep 0 for NaN only (-NaN patterns never reach here)
}

}  // namespace pc
