// Quantize-append kernels: Algorithm 1 (normalise, WHT, SO(4) blocks, 3-bit Lloyd-Max, bit-pack) for new
// K and V rows, one warp per row. K rows are packed row-major, V rows token-transposed.
#include "iq_common.cuh"
#include "iq_kernels.h"

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

// Per-warp state that does not change from row to row: the lane's SO(4) blocks and the thresholds.
template <int D>
struct RowQuantizer {
  static constexpr int E = D / 32;  // coordinates per lane: lane l owns coordinates l*E .. l*E+E-1
  static constexpr int NB = E / 4;  // SO(4) blocks per lane
  float q8[NB][8];
  float M[NB][4][4];
  float th[7];

  __device__ __forceinline__ void init(const float* rot_head, const float* thresholds, int lane) {
    const float* qbase = rot_head + (size_t)lane * NB * 8;
#pragma unroll
    for (int j = 0; j < NB; j++) {
#pragma unroll
      for (int i = 0; i < 8; i++) q8[j][i] = qbase[j * 8 + i];
      so4_matrix<float>(q8[j], M[j]);
    }
#pragma unroll
    for (int i = 0; i < 7; i++) th[i] = thresholds[i];
  }

  // Algorithm 1, steps 1-3 for one row: returns the fp32 scale, fills code[E]. `src` points at this lane's E values.
  __device__ __forceinline__ float run(const __half* src, int lane, int (&code)[E], uint32_t* status) const {
    float x[E];
    if (E == 4) {
      const uint2 raw = *reinterpret_cast<const uint2*>(src);
      const __half2 h0 = *reinterpret_cast<const __half2*>(&raw.x), h1 = *reinterpret_cast<const __half2*>(&raw.y);
      x[0] = __low2float(h0); x[1] = __high2float(h0); x[2] = __low2float(h1); x[3] = __high2float(h1);
    } else {
      const uint4 raw = *reinterpret_cast<const uint4*>(src);
      const uint32_t r[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
      for (int k = 0; k < 4; k++) {
        const __half2 hh = *reinterpret_cast<const __half2*>(&r[k]);
        x[2 * k] = __low2float(hh);
        x[2 * k + 1] = __high2float(hh);
      }
    }
    // Step 1: s = ||x||_2. Squares of fp16 values are exact in fp64; the sum is accumulated in fp64 so that
    // the stored fp32 scale is the correctly rounded norm.
    double ss = 0.0;
#pragma unroll
    for (int e = 0; e < E; e++) ss += (double)x[e] * (double)x[e];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(FULL, ss, o);
    // Stored scale = sqrt(ss) rounded to fp32. An fp32 estimate is corrected with exact fp64 midpoint tests
    // (x and its neighbours are fp32, so (x +- ulp/2)^2 is exact in fp64 up to one rounding): this avoids the
    // software double-precision square root on every row.
    float s = sqrtf((float)ss);
    {
      const float up = __uint_as_float(__float_as_uint(s) + 1u);
      const float dn = (s > 0.f) ? __uint_as_float(__float_as_uint(s) - 1u) : 0.f;
      const double mu = 0.5 * ((double)s + (double)up), md = 0.5 * ((double)s + (double)dn);
      if (ss > mu * mu) s = up;
      else if (s > 0.f && ss < md * md) s = dn;
    }
    const float inv_s = (s > 0.f) ? __frcp_rn(s) : 0.f;

    // Step 2: u = sqrt(d) * R x^ = M_b (H_unnormalised x) / s  (the two sqrt(d) factors cancel)
    float v[E];
#pragma unroll
    for (int e = 0; e < E; e++) v[e] = x[e];
    wht_warp<float, E>(v, lane);
    so4_apply<float, E, false>(M, v);

    // Step 3: codes, with a guard band around the thresholds
    bool any_near = false;
#pragma unroll
    for (int e = 0; e < E; e++) {
      bool nb;
      code[e] = decide_code<float>(v[e] * inv_s, th, nb, GUARD_BAND);
      any_near |= nb;
    }
    if (__any_sync(FULL, any_near)) {
      // Re-decide the whole row in fp64: the +-1 sums of fp16 values are exact in fp64.
      double vd[E];
      double Md[NB][4][4];
#pragma unroll
      for (int e = 0; e < E; e++) vd[e] = (double)x[e];
#pragma unroll
      for (int j = 0; j < NB; j++) so4_matrix<double>(q8[j], Md[j]);
      wht_warp<double, E>(vd, lane);
      so4_apply<double, E, false>(Md, vd);
#pragma unroll
      for (int e = 0; e < E; e++) {
        bool nb;
        const double u = (ss > 0.0) ? vd[e] / sqrt(ss) : 0.0;
        code[e] = decide_code<double>(u, th, nb, 0.0);
      }
      if (lane == 0 && status) atomicAdd(&status[1], 1u);
    }
    return s;
  }
};

// ---------------------------------------------------------------------------------------------------------
// K rows: one warp per row, packed row-major (3d/8 bytes per row).
// ---------------------------------------------------------------------------------------------------------
template <int D>
__global__ void __launch_bounds__(QA_WARPS * 32) quantize_append_k_kernel(const QuantizeParams p) {
  constexpr int E = D / 32;
  constexpr int LPU = 32 / E;      // lanes per 32-coordinate packing unit
  constexpr int WPR = 3 * D / 32;  // 32-bit words per packed row

  const int lane = threadIdx.x & 31;
  const int warp = threadIdx.x >> 5;
  const int b = blockIdx.z;
  const int h = blockIdx.y;

  int n_new = p.n_new ? p.n_new[b] : p.n_new_max;
  n_new = min(n_new, p.n_new_max);
  const int row_begin = (blockIdx.x * QA_WARPS + warp) * QA_ROWS_PER_WARP;
  if (row_begin >= n_new) return;
  const int row_end = min(n_new, row_begin + QA_ROWS_PER_WARP);
  const int pos0 = p.append_pos[b];

  RowQuantizer<D> rq;
  rq.init(p.rot + (size_t)h * (D / 4) * 8, p.thresholds, lane);
  const __half* src_base = p.k_new + (size_t)b * p.stride_b + (size_t)h * p.stride_h + lane * E;
  const size_t slab = ((size_t)b * p.n_kv_heads + h) * (size_t)p.t_cap;

  for (int i = row_begin; i < row_end; i++) {
    const long long t = (long long)pos0 + i;
    if (t < 0 || t >= p.t_cap) {
      if (lane == 0 && p.status) {
        atomicOr(&p.status[0], IQ_STATUS_ROW_OUT_OF_RANGE);
        atomicAdd(&p.status[2], 1u);
      }
      continue;
    }
    int code[E];
    const float s = rq.run(src_base + (size_t)i * p.stride_t, lane, code, p.status);

    // Step 4: bit-pack. A packing unit is 32 coordinates = LPU lanes = 3 words.
    uint32_t w[3] = {0u, 0u, 0u};
    const int c0 = (lane % LPU) * E;  // unit-local coordinate of this lane's first element
#pragma unroll
    for (int e = 0; e < E; e++) {
      const int c = c0 + e;
      const uint32_t cd = (uint32_t)code[e];
      if (c < 24) {
        const uint32_t val = cd << (4 * (c & 7));
        if ((c >> 3) == 0) w[0] |= val;
        else if ((c >> 3) == 1) w[1] |= val;
        else w[2] |= val;
      } else {
        const int sh = 4 * (c - 24) + 3;
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
    uint32_t* row_words = reinterpret_cast<uint32_t*>(p.k_codes + (slab + (size_t)t) * (size_t)(WPR * 4));
    if (k < 3) row_words[3 * (lane / LPU) + k] = (k == 0) ? w[0] : (k == 1 ? w[1] : w[2]);
    if (lane == 0) p.k_scales[slab + (size_t)t] = s;
  }
}

// ---------------------------------------------------------------------------------------------------------
// V rows: stored token-transposed. For every block of 128 cache rows and every coordinate c there is one
// 48-byte row holding the 128 codes of coordinate c, arranged like a packing unit sequence with the
// row-in-block in the role of the coordinate. One CTA handles one 32-row unit of one (sequence, KV head):
// its warps quantise the unit's new rows, the codes go through shared memory, and thread c assembles the
// three words of (unit, coordinate c). Words that are only partly covered by new rows are read, merged and
// written back; no other CTA touches them.
// ---------------------------------------------------------------------------------------------------------
template <int D>
__global__ void __launch_bounds__(128) quantize_append_v_kernel(const QuantizeParams p) {
  constexpr int E = D / 32;
  __shared__ uint8_t codes_s[32][D];

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int b = blockIdx.z;
  const int h = blockIdx.y;
  int n_new = p.n_new ? p.n_new[b] : p.n_new_max;
  n_new = min(n_new, p.n_new_max);
  if (n_new <= 0) return;
  const long long pos0 = p.append_pos[b];
  const long long unit = (pos0 >= 0 ? pos0 / 32 : -((-pos0 + 31) / 32)) + blockIdx.x;  // floor(pos0 / 32) + x
  const long long t_lo = max(unit * 32, pos0);                 // first cache row of this unit that is appended
  const long long t_hi = min(unit * 32 + 32, pos0 + n_new);    // one past the last
  if (t_lo >= t_hi) return;
  const size_t slab = ((size_t)b * p.n_kv_heads + h) * (size_t)p.t_cap;
  const bool in_cache = unit >= 0 && unit * 32 + 32 <= p.t_cap;  // t_cap is a multiple of 128

  RowQuantizer<D> rq;
  rq.init(p.rot + (size_t)h * (D / 4) * 8, p.thresholds, lane);
  const __half* src_base = p.v_new + (size_t)b * p.stride_b + (size_t)h * p.stride_h + lane * E;
  for (long long t = t_lo + warp; t < t_hi; t += 4) {
    if (!in_cache) {
      if (lane == 0 && p.status) {
        atomicOr(&p.status[0], IQ_STATUS_ROW_OUT_OF_RANGE);
        atomicAdd(&p.status[2], 1u);
      }
      continue;
    }
    int code[E];
    const float s = rq.run(src_base + (size_t)(t - pos0) * p.stride_t, lane, code, p.status);
    uint32_t packed = 0;
#pragma unroll
    for (int e = 0; e < E; e++) packed |= (uint32_t)code[e] << (8 * (e & 3));
    if (E == 4) {
      *reinterpret_cast<uint32_t*>(&codes_s[t & 31][lane * 4]) = packed;
    } else {
      uint32_t p0 = 0, p1 = 0;
#pragma unroll
      for (int e = 0; e < 4; e++) { p0 |= (uint32_t)code[e] << (8 * e); p1 |= (uint32_t)code[4 + e] << (8 * e); }
      *reinterpret_cast<uint2*>(&codes_s[t & 31][lane * 8]) = make_uint2(p0, p1);
    }
    if (lane == 0) p.v_scales[slab + (size_t)t] = s;
  }
  __syncthreads();
  if (!in_cache) return;

  const int c_lo = (int)(t_lo & 31), c_hi = (int)(t_hi - unit * 32);  // rows [c_lo, c_hi) of the unit are new
  const size_t blk = (size_t)(unit * 32) / 128;
  const int u = (int)((unit * 32) % 128) / 32;
#pragma unroll
  for (int j = 0; j < D / 128; j++) {
    const int c = tid + 128 * j;  // coordinate
    uint32_t w[3] = {0u, 0u, 0u}, m[3] = {0u, 0u, 0u};
    for (int r = c_lo; r < c_hi; r++) {
      const uint32_t cd = codes_s[r][c];
      if (r < 24) {
        const int sh = 4 * (r & 7);
        w[r >> 3] |= cd << sh;
        m[r >> 3] |= 7u << sh;
      } else {
        const int sh = 4 * (r - 24) + 3;
#pragma unroll
        for (int k = 0; k < 3; k++) {
          w[k] |= ((cd >> k) & 1u) << sh;
          m[k] |= 1u << sh;
        }
      }
    }
    uint32_t* dst = reinterpret_cast<uint32_t*>(p.v_codes + ((slab / 128 + blk) * D + c) * 48) + 3 * u;
    const bool full = (c_lo == 0 && c_hi == 32);
#pragma unroll
    for (int k = 0; k < 3; k++) {
      if (m[k] == 0u) continue;
      dst[k] = full ? w[k] : ((dst[k] & ~m[k]) | w[k]);
    }
  }
}

cudaError_t launch_quantize_append(const QuantizeParams& p, int head_dim, int batch, cudaStream_t stream) {
  if (p.n_new_max <= 0 || batch <= 0) return cudaSuccess;
  const int rows_per_cta = QA_WARPS * QA_ROWS_PER_WARP;
  dim3 kgrid((p.n_new_max + rows_per_cta - 1) / rows_per_cta, p.n_kv_heads, batch);
  dim3 vgrid((p.n_new_max + 31) / 32 + 1, p.n_kv_heads, batch);  // +1: the first row may sit in the middle of a unit
  if (head_dim == 128) {
    quantize_append_k_kernel<128><<<kgrid, QA_WARPS * 32, 0, stream>>>(p);
    quantize_append_v_kernel<128><<<vgrid, 128, 0, stream>>>(p);
  } else {
    quantize_append_k_kernel<256><<<kgrid, QA_WARPS * 32, 0, stream>>>(p);
    quantize_append_v_kernel<256><<<vgrid, 128, 0, stream>>>(p);
  }
  return cudaGetLastError();
}

}  // namespace iq
