// Pieces shared by the refinement / selection kernels (select.cu, finish.cu): the mean filter of Eq. 13 and
// the order-preserving integer image of a score.  Both files must produce bit-identical refined scores, so the
// order of the additions below is part of the contract.
#pragma once

#include "ahakv_internal.cuh"

namespace ahakv {

// gamma_j of Eq. 13: mean of nu over [j - half, j + half] cut to [0, n).  Away from the ends the sum is
// multiplied by inv_w = 1 / width; at the ends it is divided by the number of tokens in range, or multiplied
// by inv_w too when `zero_pad` is set.  `nu` is indexed by token.
__device__ __forceinline__ float pooled(const float* __restrict__ nu, int j, int n, int half, float inv_w,
                                        bool zero_pad) {
  const int lo = max(j - half, 0), hi = min(j + half, n - 1);
  float s;
  if (hi - lo == 6) {
    // the usual width (7) away from the ends: seven independent loads, added in the order of the loop below
    const float a0 = nu[lo], a1 = nu[lo + 1], a2 = nu[lo + 2], a3 = nu[lo + 3], a4 = nu[lo + 4], a5 = nu[lo + 5],
                a6 = nu[lo + 6];
    s = (((((a0 + a1) + a2) + a3) + a4) + a5) + a6;
  } else {
    s = 0.f;
    for (int t = lo; t <= hi; ++t) s += nu[t];
  }
  return (zero_pad || hi - lo == 2 * half) ? s * inv_w : s / (float)(hi - lo + 1);
}

// The accumulated score of a token from the `slots` partial scores the scoring kernels leave per head: row
// blocks add up; the per-head scores of a query group pooled by maximum (group_max) take the largest.
__device__ __forceinline__ float combine_slots(const float* __restrict__ s_raw, size_t at, int n, int slots,
                                               int group_max) {
  float s = s_raw[at];
  if (group_max) {
    for (int t = 1; t < slots; ++t) s = fmaxf(s, s_raw[at + (size_t)t * n]);
  } else {
    for (int t = 1; t < slots; ++t) s += s_raw[at + (size_t)t * n];
  }
  return s;
}

// Monotone map float -> uint32: a > b  <=>  key(a) > key(b) (for non-NaN values), and its inverse.
__device__ __forceinline__ uint32_t order_key(float x) {
  const uint32_t u = __float_as_uint(x);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float key_to_float(uint32_t key) {
  return __uint_as_float((key & 0x80000000u) ? (key & 0x7fffffffu) : ~key);
}

}  // namespace ahakv
