// One cache row appended by one warp (Algorithm 1 for a single row): shared by the few-rows append kernel and by the
// one-launch decode step, whose auxiliary warp appends the step's new K and V rows itself.
#pragma once
#include "iq_format.cuh"
#include "iq_quantize_common.cuh"

namespace iq {

// code = #{ j : u > t_j } over NT = 3, 7 or 15 ascending thresholds, and whether u is within `guard` of one of them: a
// binary search whose pivots are picked with selects (the thresholds stay in registers). The pivots visited include
// both bounds of the final cell, so checking them covers every decision that could flip.
template <typename T, int NT>
__device__ __forceinline__ int decide_code_n(T u, const float (&th)[NT], bool& near_boundary, T guard) {
  if constexpr (NT == 7) {
    return decide_code<T>(u, th, near_boundary, guard);
  } else if constexpr (NT == 3) {
    const bool b1 = u > (T)th[1];
    const T p0 = b1 ? (T)th[2] : (T)th[0];
    const bool b0 = u > p0;
    near_boundary = fmin(fabs(u - (T)th[1]), fabs(u - p0)) <= guard;
    return (b1 ? 2 : 0) + (b0 ? 1 : 0);
  } else {
    static_assert(NT == 15, "2, 3 or 4 bits");
    const bool b3 = u > (T)th[7];
    const T p2 = b3 ? (T)th[11] : (T)th[3];
    const bool b2 = u > p2;
    const T p1 = b3 ? (b2 ? (T)th[13] : (T)th[9]) : (b2 ? (T)th[5] : (T)th[1]);
    const bool b1 = u > p1;
    const T p0 = b3 ? (b2 ? (b1 ? (T)th[14] : (T)th[12]) : (b1 ? (T)th[10] : (T)th[8]))
                    : (b2 ? (b1 ? (T)th[6] : (T)th[4]) : (b1 ? (T)th[2] : (T)th[0]));
    const bool b0 = u > p0;
    near_boundary = fmin(fmin(fabs(u - (T)th[7]), fabs(u - p2)), fmin(fabs(u - p1), fabs(u - p0))) <= guard;
    return (b3 ? 8 : 0) + (b2 ? 4 : 0) + (b1 ? 2 : 0) + (b0 ? 1 : 0);
  }
}

template <int D, int BITS = 3>
struct WarpRowQuantizer {
  static constexpr int E = D / 32;  // coordinates per lane
  static constexpr int NB = E / 4;  // SO(4) blocks per lane
  static constexpr int NT = (1 << BITS) - 1;
  const float* qbase;
  float M[NB][4][4];
  float th[NT];

  __device__ __forceinline__ void init(const float* rot_head, const float* thresholds, int lane) {
    qbase = rot_head + (size_t)lane * NB * 8;
#pragma unroll
    for (int j = 0; j < NB; j++) so4_matrix<float>(qbase + 8 * j, M[j]);
#pragma unroll
    for (int i = 0; i < NT; i++) th[i] = thresholds[i];
  }

  __device__ __forceinline__ void set_thresholds(const float* thresholds) {
#pragma unroll
    for (int i = 0; i < NT; i++) th[i] = thresholds[i];
  }

  // Algorithm 1, steps 1-3 for one row: returns the fp32 scale, fills code[E]. `src` points at this lane's E values.
  __device__ __forceinline__ float run(const __half2 (&raw)[E / 2], int lane, int (&code)[E], uint32_t* status) const {
    float x[E];
#pragma unroll
    for (int k = 0; k < E / 2; k++) {
      x[2 * k] = __low2float(raw[k]);
      x[2 * k + 1] = __high2float(raw[k]);
    }
    double ss = 0.0;  // squares of fp16 values are exact in fp32; the sum in fp64 makes the stored scale the rounded norm
#pragma unroll
    for (int e = 0; e < E; e++) ss += (double)(x[e] * x[e]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(FULL, ss, o);
    float s = sqrtf((float)ss);
    {  // correct the fp32 estimate with exact fp64 midpoint tests
      const float up = __uint_as_float(__float_as_uint(s) + 1u);
      const float dn = (s > 0.f) ? __uint_as_float(__float_as_uint(s) - 1u) : 0.f;
      const double mu = 0.5 * ((double)s + (double)up), md = 0.5 * ((double)s + (double)dn);
      if (ss > mu * mu) s = up;
      else if (s > 0.f && ss < md * md) s = dn;
    }
    const float inv_s = (s > 0.f) ? __frcp_rn(s) : 0.f;
    float v[E];
#pragma unroll
    for (int e = 0; e < E; e++) v[e] = x[e];
    wht_warp<float, E>(v, lane);
    so4_apply<float, E, false>(M, v);
    bool any_near = false;
#pragma unroll
    for (int e = 0; e < E; e++) {
      bool nb;
      code[e] = decide_code_n<float, NT>(v[e] * inv_s, th, nb, GUARD_BAND);
      any_near |= nb;
    }
    if (__any_sync(FULL, any_near)) {  // re-decide the row in fp64: the +-1 sums of fp16 values are exact there
      double vd[E];
#pragma unroll
      for (int e = 0; e < E; e++) vd[e] = (double)x[e];
      wht_warp<double, E>(vd, lane);
      const double inv_sd = (ss > 0.0) ? 1.0 / sqrt(ss) : 0.0;
#pragma unroll
      for (int j = 0; j < NB; j++) {
        double Md[1][4][4];
        so4_matrix<double>(qbase + 8 * j, Md[0]);
        double blk[4] = {vd[4 * j], vd[4 * j + 1], vd[4 * j + 2], vd[4 * j + 3]};
        so4_apply<double, 4, false>(Md, blk);
#pragma unroll
        for (int r = 0; r < 4; r++) {
          bool nb;
          code[4 * j + r] = decide_code_n<double, NT>(blk[r] * inv_sd, th, nb, 0.0);
        }
      }
      if (lane == 0 && status) atomicAdd(&status[1], 1u);
    }
    return s;
  }
};

// What a row writer needs to know about the cache.
struct RowSink {
  uint8_t* k_codes;
  float* k_scales;
  uint8_t* v_codes;
  float* v_scales;
  uint32_t* status;
  int scale_f16;
};

// K row `row` (index into the cache arrays): lane l holds the codes of coordinates l E .. l E + E - 1.
template <int D, int BITS = 3>
__device__ __forceinline__ void warp_store_k_row(const RowSink& c, size_t row, const int (&code)[D / 32], float s, int lane) {
  constexpr int E = D / 32;
  if constexpr (BITS != 3) {
    // the lane's E coordinates lie in one word (8 or 16 entries per word): the lanes that share a word OR their parts
    constexpr int EPW = BITS == 4 ? 8 : 16, LPW = EPW / E;
    uint32_t w = 0u;
#pragma unroll
    for (int e = 0; e < E; e++) {
      int word, sh;
      packed_place<BITS>(lane * E + e, word, sh);
      w |= (uint32_t)code[e] << sh;
    }
#pragma unroll
    for (int o = 1; o < LPW; o <<= 1) w |= __shfl_xor_sync(FULL, w, o);
    uint32_t* row_words = reinterpret_cast<uint32_t*>(c.k_codes + row * (size_t)(BITS * D / 8));
    if (lane % LPW == 0) row_words[lane * E / EPW] = w;
    if (lane == 0) store_scale(c.k_scales, row, s, c.scale_f16, c.status);
    return;
  }
  constexpr int LPU = 32 / E;  // lanes per 32-coordinate packing unit
  // packed row: a packing unit is 32 coordinates = LPU lanes = 3 words
  uint32_t w[3] = {0u, 0u, 0u};
  const int c0 = (lane % LPU) * E;
#pragma unroll
  for (int e = 0; e < E; e++) {
    const int cc = c0 + e;
    const uint32_t cd = (uint32_t)code[e];
    if (cc < 24) {
      w[cc >> 3] |= cd << (4 * (cc & 7));
    } else {
      const int sh = 4 * (cc - 24) + 3;
      w[0] |= (cd & 1u) << sh;
      w[1] |= ((cd >> 1) & 1u) << sh;
      w[2] |= ((cd >> 2) & 1u) << sh;
    }
  }
#pragma unroll
  for (int o = 1; o < LPU; o <<= 1) {
    w[0] |= __shfl_xor_sync(FULL, w[0], o);
    w[1] |= __shfl_xor_sync(FULL, w[1], o);
    w[2] |= __shfl_xor_sync(FULL, w[2], o);
  }
  const int k = lane % LPU;
  uint32_t* row_words = reinterpret_cast<uint32_t*>(c.k_codes + row * (size_t)(3 * D / 8));
  if (k < 3) row_words[3 * (lane / LPU) + k] = (k == 0) ? w[0] : (k == 1 ? w[1] : w[2]);
  if (lane == 0) store_scale(c.k_scales, row, s, c.scale_f16, c.status);
}

// V row t of its sequence (at `row` in the cache arrays) into the token-transposed records: row t is entry r = t % 32
// of unit u = (t % 128) / 32 of block t / 128, for every coordinate; one read-modify-write per touched word.
template <int D, int BITS = 3>
__device__ __forceinline__ void warp_store_v_row(const RowSink& c, size_t row, long long t, const int (&code)[D / 32], float s, int lane) {
  constexpr int E = D / 32;
  const size_t blk = row / 128;  // (a page holds whole 128-row blocks: row / 128 is the block's index in the V array)
  if constexpr (BITS != 3) {
    int word, sh;
    packed_place<BITS>((int)(t % 128), word, sh);
#pragma unroll
    for (int e = 0; e < E; e++) {
      uint32_t* dst = reinterpret_cast<uint32_t*>(c.v_codes + (blk * D + lane * E + e) * (size_t)(16 * BITS)) + word;
      *dst = (*dst & ~(((1u << BITS) - 1u) << sh)) | ((uint32_t)code[e] << sh);
    }
    if (lane == 0) store_scale(c.v_scales, row, s, c.scale_f16, c.status);
    return;
  }
  const int u = (int)(t % 128) / 32, r = (int)(t % 32);
#pragma unroll
  for (int e = 0; e < E; e++) {
    const int cc = lane * E + e;
    const uint32_t cd = (uint32_t)code[e];
    uint32_t* dst = reinterpret_cast<uint32_t*>(c.v_codes + (blk * D + cc) * 48) + 3 * u;
    if (r < 24) {
      const int sh = 4 * (r & 7);
      dst[r >> 3] = (dst[r >> 3] & ~(7u << sh)) | (cd << sh);
    } else {
      const int sh = 4 * (r - 24) + 3;
#pragma unroll
      for (int k = 0; k < 3; k++) dst[k] = (dst[k] & ~(1u << sh)) | (((cd >> k) & 1u) << sh);
    }
  }
  if (lane == 0) store_scale(c.v_scales, row, s, c.scale_f16, c.status);
}

}  // namespace iq
