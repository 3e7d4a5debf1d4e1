// Which mask of the library keeps most of a kernel's energy, and that energy (pattern selection, Section 4.1 / 5.1).
#pragma once
#include "common.cuh"

namespace pat {

// wk: the nine fp32 weights of one kernel.  Returns the id of the best mask (lowest id on ties) and its energy in
// best_e: squares of fp32 values are exact in fp64 and are added in ascending bit order, so the value is the same bits
// on any IEEE machine.
//
// The argmax is first taken in fp32.  Nine squares and a sum of at most nine non-negative terms carry a relative
// error below 2^-20 (nine roundings of 2^-24 each) as long as nothing overflows and the result is far above the
// subnormal range, so an fp32 winner that leads the runner-up by a factor of more than 1 + 2^-18 is the exact winner
// too.  Every other case - a lead inside the error bound (exact ties among them), a tiny, huge or non-finite energy -
// takes the exact path over all masks.  The winner's energy itself is always computed exactly.
__device__ inline int best_mask(const float* __restrict__ wk, const MaskTable& lib, double& best_e) {
  float sqf[9];
#pragma unroll
  for (int b = 0; b < 9; ++b) {
    const float v = wk[b];
    sqf[b] = __fmul_rn(v, v);
  }
  float best32 = -1.0f, second32 = -1.0f;
  int best = 0;
  bool plain = true;                       // every fp32 energy is an ordinary finite number
  for (int j = 0; j < lib.K; ++j) {
    const unsigned m = lib.m[j];
    float e = 0.0f;
#pragma unroll
    for (int b = 0; b < 9; ++b)
      if (m & (1u << b)) e = __fadd_rn(e, sqf[b]);
    plain = plain && (e <= 3.0e38f);       // false for NaN and infinity
    if (e > best32) { second32 = best32; best32 = e; best = j; }
    else if (e > second32) second32 = e;   // e == best32 lands here: a tie is never a clear lead
  }
  constexpr float kLead = 1.0f + 3.814697265625e-6f;     // 1 + 2^-18
  constexpr float kFloor = 7.8886090522101181e-31f;      // 2^-100
  const bool clear = plain && best32 >= kFloor && best32 > second32 * kLead;
  if (clear) {
    best_e = 0.0;
    unsigned m = lib.m[best];
    while (m) {                            // ascending bit order
      const double v = (double)wk[__ffs(m) - 1];
      best_e += v * v;                     // the square of an fp32 value is exact in fp64
      m &= m - 1u;
    }
  } else {
    double sq[9];
#pragma unroll
    for (int b = 0; b < 9; ++b) {
      const double v = (double)wk[b];
      sq[b] = v * v;
    }
    best_e = -1.0;
    best = 0;
    for (int j = 0; j < lib.K; ++j) {
      const unsigned m = lib.m[j];
      double e = 0.0;
#pragma unroll
      for (int b = 0; b < 9; ++b)
        if (m & (1u << b)) e += sq[b];
      if (e > best_e) { best_e = e; best = j; }
    }
  }
  return best;
}

}  // namespace pat
