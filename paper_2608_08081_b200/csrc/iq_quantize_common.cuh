// Threshold decisions shared by the quantize-append kernels (Section 3.2, Step 3).
#pragma once
#include "iq_common.cuh"

namespace iq {

// Distance (in unit-variance units) from a decision threshold below which the fp32 decision is not
// trusted and the row is re-decided in fp64. The fp32 butterfly + block product carry at most a few
// 1e-6 of absolute error in these units for head_dim <= 256.
constexpr float GUARD_BAND = 3.0517578125e-05f;  // 2^-15

template <typename T>
__device__ __forceinline__ int decide_code(T u, const float (&th)[7], bool& near_boundary, T guard) {
  // Binary search over the 7 ascending thresholds; code = #{ j : u > t_j }. The three pivots visited
  // include both bounds of the final cell, so checking them covers every decision that could flip.
  const bool b2 = u > (T)th[3];
  const T p1 = b2 ? (T)th[5] : (T)th[1];
  const bool b1 = u > p1;
  const T p0 = b2 ? (b1 ? (T)th[6] : (T)th[4]) : (b1 ? (T)th[2] : (T)th[0]);
  const bool b0 = u > p0;
  T dmin = fabs(u - (T)th[3]);
  dmin = fmin(dmin, fabs(u - p1));
  dmin = fmin(dmin, fabs(u - p0));
  near_boundary = dmin <= guard;
  return (b2 ? 4 : 0) + (b1 ? 2 : 0) + (b0 ? 1 : 0);
}

// The same decision for a codebook that is symmetric about zero (t_3 = 0, t_{6-k} = -t_k; the Lloyd-Max codebooks of a
// symmetric density are): two compares on |u| and the sign. Exact ties fall inside the guard band and are re-decided.
// dmin carries the smallest distance to a threshold seen so far, so that one test serves all coordinates of a lane.
__device__ __forceinline__ int decide_code_sym(float u, float a1, float a2, float a3, float& dmin) {
  const float a = fabsf(u);
  const bool b1 = a > a2;
  const float p0 = b1 ? a3 : a1;
  const bool b0 = a > p0;
  dmin = fminf(fminf(dmin, a), fminf(fabsf(a - a2), fabsf(a - p0)));
  const int mag = (b1 ? 2 : 0) + (b0 ? 1 : 0);
  return u > 0.f ? 4 + mag : 3 - mag;
}

}  // namespace iq
