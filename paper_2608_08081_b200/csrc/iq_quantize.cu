// Quantize-append kernels: Algorithm 1 (normalise, WHT, SO(4) blocks, 3-bit Lloyd-Max, bit-pack) for new
// K and V rows: bulk kernels (a row shared by d/16 lanes), the few-rows kernel of the decode step (a warp per row) and the
// calibration histogram. K rows are packed row-major, V rows token-transposed.
#include "iq_common.cuh"
#include "iq_kernels.h"
#include "iq_append_row.cuh"

namespace iq {

// Work mapping of the row kernels: a row is shared by LPR = d/16 lanes, 16 consecutive coordinates (4 whole SO(4)
// blocks) per lane, so a warp holds 32/LPR rows at a time (4 at d = 128, 2 at d = 256). The Walsh-Hadamard
// butterfly runs 4 stages inside the lane and log2(LPR) xor-shuffle stages across the row's lanes; a 32-coordinate
// packing unit is a pair of lanes.
template <int D>
struct RowQuantizer {
  static constexpr int E = 16;
  static constexpr int LPR = D / E;        // lanes per row: 8 or 16
  static constexpr int RPW = 32 / LPR;     // rows per warp: 4 or 2
  static constexpr int NB = E / 4;         // SO(4) blocks per lane
  // The head's d/4 block matrices live in shared memory, 4 blocks (64 floats) + 4 floats of padding per lane-in-row:
  // with the padding the 8 or 16 different 16-byte rows a warp reads at a time fall into different banks. Keeping
  // them in registers (64 per thread) halves the number of resident warps.
  static constexpr int M_STRIDE = NB * 16 + 4;
  static constexpr int M_FLOATS = LPR * M_STRIDE;
  const float* qbase;      // this lane's NB quaternion pairs
  const float* th_global;  // the 7 thresholds in memory (for the out-of-line fp64 path)
  const float4* Ms;        // this lane's NB matrices in shared memory, row-major
  float th[7];

  // Called by every thread of the CTA (then __syncthreads()): the matrices of the head's blocks into m_smem.
  __device__ __forceinline__ static void fill_matrices(const float* rot_head, float* m_smem, int tid, int n_threads) {
    for (int blk = tid; blk < D / 4; blk += n_threads) {
      float Mt[4][4];
      so4_matrix<float>(rot_head + (size_t)blk * 8, Mt);
      float* dst = m_smem + (blk / NB) * M_STRIDE + (blk % NB) * 16;
#pragma unroll
      for (int r = 0; r < 4; r++) *reinterpret_cast<float4*>(dst + 4 * r) = make_float4(Mt[r][0], Mt[r][1], Mt[r][2], Mt[r][3]);
    }
  }

  __device__ __forceinline__ void init(const float* rot_head, const float* thresholds, int lane, const float* m_smem) {
    qbase = rot_head + (size_t)(lane % LPR) * NB * 8;
    Ms = reinterpret_cast<const float4*>(m_smem + (lane % LPR) * M_STRIDE);
#pragma unroll
    for (int i = 0; i < 7; i++) th[i] = thresholds[i];
    th_global = thresholds;
  }

  // butterflies across the lanes of one row (strides 16, 32, ...): lane bit b of (lane % LPR) <-> stride 16 << b
  template <typename T>
  __device__ __forceinline__ static void wht(T (&v)[E], int lane) {
#pragma unroll
    for (int s = 1; s < E; s <<= 1)
#pragma unroll
      for (int i = 0; i < E; i++)
        if ((i & s) == 0) {
          const T a = v[i], c = v[i + s];
          v[i] = a + c;
          v[i + s] = a - c;
        }
#pragma unroll
    for (int o = 1; o < LPR; o <<= 1) {
      const T sgn = (lane & o) ? T(-1) : T(1);  // the upper lane of a pair keeps (other - own)
#pragma unroll
      for (int i = 0; i < E; i++) {
        const T other = shfl_xor_t<T>(v[i], o);
        v[i] = sgn * v[i] + other;  // one fused multiply-add, exact: sgn is +-1
      }
    }
  }

  __device__ __forceinline__ static void unpack16(const uint4& r0, const uint4& r1, float (&x)[E]) {
    const uint32_t r[8] = {r0.x, r0.y, r0.z, r0.w, r1.x, r1.y, r1.z, r1.w};
#pragma unroll
    for (int k = 0; k < 8; k++) {
      const __half2 hh = *reinterpret_cast<const __half2*>(&r[k]);
      x[2 * k] = __low2float(hh);
      x[2 * k + 1] = __high2float(hh);
    }
  }

  // The rare path: re-decide the warp's rows in fp64, where the +-1 sums of fp16 values are exact. Kept out of line
  // so that its registers do not count against the common path.
  __device__ __forceinline__ static uint2 redo_fp64(uint4 r0, uint4 r1, double ss, int lane, const float* qbase,
                                                 const float* th_global) {
    float th[7];
#pragma unroll
    for (int i = 0; i < 7; i++) th[i] = th_global[i];
    int code[E];
    float x[E];
    unpack16(r0, r1, x);
    double vd[E];
#pragma unroll
    for (int e = 0; e < E; e++) vd[e] = (double)x[e];
    wht<double>(vd, lane);
    const double inv_sd = (ss > 0.0) ? 1.0 / sqrt(ss) : 0.0;
#pragma unroll
    for (int j = 0; j < NB; j++) {
      float q8[8];
#pragma unroll
      for (int i = 0; i < 8; i++) q8[i] = qbase[j * 8 + i];
      double Md[1][4][4];
      so4_matrix<double>(q8, Md[0]);
      double blk[4] = {vd[4 * j], vd[4 * j + 1], vd[4 * j + 2], vd[4 * j + 3]};
      so4_apply<double, 4, false>(Md, blk);
#pragma unroll
      for (int r = 0; r < 4; r++) {
        bool nb;
        code[4 * j + r] = decide_code<double>(blk[r] * inv_sd, th, nb, 0.0);
      }
    }
    uint2 packed = make_uint2(0u, 0u);  // 16 codes as nibbles
#pragma unroll
    for (int n = 0; n < 8; n++) {
      packed.x |= (uint32_t)code[n] << (4 * n);
      packed.y |= (uint32_t)code[8 + n] << (4 * n);
    }
    return packed;
  }

  // Algorithm 1, steps 1-2 for the row this lane belongs to (r0, r1 = this lane's 16 fp16 values, zeros for the lanes
  // of a row that is not used; those lanes still take part in the shuffles): returns the fp32 scale s (and its fp64
  // square sum) and leaves M_b (H x) -- u * s, the rotated coordinates before the division by the norm -- in x.
  __device__ __forceinline__ float rotate(const uint4& r0, const uint4& r1, int lane, float (&x)[E], double& ss_out) const {
    unpack16(r0, r1, x);
    // Step 1: s = ||x||_2. Squares of fp16 values are exact in fp32 (22 bits); they are summed in fp64 so that the
    // stored fp32 scale is the correctly rounded norm.
    double ss = 0.0;
#pragma unroll
    for (int e = 0; e < E; e += 2) ss += (double)(x[e] * x[e]) + (double)(x[e + 1] * x[e + 1]);
#pragma unroll
    for (int o = 1; o < LPR; o <<= 1) ss += __shfl_xor_sync(FULL, ss, o);
    float s = sqrtf((float)ss);
    {  // correct the fp32 estimate with exact fp64 midpoint tests instead of a double-precision square root
      const float up = __uint_as_float(__float_as_uint(s) + 1u);
      const float dn = (s > 0.f) ? __uint_as_float(__float_as_uint(s) - 1u) : 0.f;
      const double mu = 0.5 * ((double)s + (double)up), md = 0.5 * ((double)s + (double)dn);
      if (ss > mu * mu) s = up;
      else if (s > 0.f && ss < md * md) s = dn;
    }
    ss_out = ss;
    // Step 2: u = sqrt(d) * R x^ = M_b (H_unnormalised x) / s  (the two sqrt(d) factors cancel)
    wht<float>(x, lane);
#pragma unroll
    for (int j = 0; j < NB; j++) {
      const float x0 = x[4 * j], x1 = x[4 * j + 1], x2 = x[4 * j + 2], x3 = x[4 * j + 3];
#pragma unroll
      for (int r = 0; r < 4; r++) {
        const float4 m = Ms[4 * j + r];
        x[4 * j + r] = m.x * x0 + m.y * x1 + m.z * x2 + m.w * x3;
      }
    }

    return s;
  }

  // Algorithm 1, steps 1-3: the codes of this lane's 16 coordinates; returns the fp32 scale.
  template <bool SYM>
  __device__ __forceinline__ float run(const uint4& r0, const uint4& r1, bool active, int lane, int (&code)[E],
                                       uint32_t* status) const {
    float x[E];
    double ss;
    const float s = rotate(r0, r1, lane, x, ss);
    const float inv_s = (s > 0.f) ? __frcp_rn(s) : 0.f;

    // Step 3: codes, with a guard band around the thresholds
    bool any_near = false;
    if (SYM) {
      float dmin = 1.f;
#pragma unroll
      for (int e = 0; e < E; e++) code[e] = decide_code_sym(x[e] * inv_s, th[4], th[5], th[6], dmin);
      any_near = dmin <= GUARD_BAND;
    } else {
#pragma unroll
      for (int e = 0; e < E; e++) {
        bool nb;
        code[e] = decide_code<float>(x[e] * inv_s, th, nb, GUARD_BAND);
        any_near |= nb;
      }
    }
    const unsigned rows_near = __ballot_sync(FULL, any_near && active);
    if (rows_near) {
      const uint2 packed = redo_fp64(r0, r1, ss, lane, qbase, th_global);
#pragma unroll
      for (int n = 0; n < 8; n++) {
        code[n] = (packed.x >> (4 * n)) & 7;
        code[8 + n] = (packed.y >> (4 * n)) & 7;
      }
      int n_rows = 0;
#pragma unroll
      for (int r = 0; r < RPW; r++) n_rows += ((rows_near >> (r * LPR)) & ((1u << (LPR - 1)) * 2u - 1u)) != 0u;
      if (lane == 0 && status) atomicAdd(&status[1], (unsigned)n_rows);
    }
    return s;
  }
};

// Packed words of one row from per-lane codes: a packing unit is the lane pair (2p, 2p+1). Returns, for even lanes,
// words 0 and 1 of the unit in (w0, w1); for odd lanes word 2 in w0.
__device__ __forceinline__ void pack_pair(const int (&code)[16], int lane, uint32_t& w0, uint32_t& w1) {
  uint32_t lo = 0, hi = 0;
#pragma unroll
  for (int n = 0; n < 8; n++) {
    lo |= (uint32_t)code[n] << (4 * n);
    hi |= (uint32_t)code[8 + n] << (4 * n);
  }
  // odd lane: lo = entries 16..23 (word 2), hi = entries 24..31 (the bit-sliced ones)
  const uint32_t xs = __shfl_xor_sync(FULL, hi, 1);  // even lanes receive the odd lane's sliced nibble word
  if (lane & 1) {
    w0 = lo | (((hi >> 2) & 0x11111111u) << 3);
    w1 = 0u;
  } else {
    w0 = lo | ((xs & 0x11111111u) << 3);
    w1 = hi | (((xs >> 1) & 0x11111111u) << 3);
  }
}

// ---------------------------------------------------------------------------------------------------------
// K rows: packed row-major (3d/8 bytes per row).
// ---------------------------------------------------------------------------------------------------------
template <int D, bool SYM>
__global__ void __launch_bounds__(QA_WARPS * 32, 5) quantize_append_k_kernel(const __grid_constant__ QuantizeParams p) {
  using RQ = RowQuantizer<D>;
  constexpr int LPR = RQ::LPR, RPW = RQ::RPW;
  grid_dependency_wait();
  allow_dependent_launch();
  const int lane = threadIdx.x & 31;
  const int warp = threadIdx.x >> 5;
  const int b = blockIdx.z;
  const int h = blockIdx.y;

  int n_new = p.n_new ? p.n_new[b] : p.n_new_max;
  n_new = min(n_new, p.n_new_max);
  if (blockIdx.x * QA_WARPS * QA_ROWS_PER_WARP >= n_new) return;  // the whole CTA
  __shared__ __align__(16) float m_s[RQ::M_FLOATS];
  RQ::fill_matrices(p.rot + (size_t)h * (D / 4) * 8, m_s, threadIdx.x, QA_WARPS * 32);
  __syncthreads();
  const int row_begin = (blockIdx.x * QA_WARPS + warp) * QA_ROWS_PER_WARP;
  if (row_begin >= n_new) return;
  const int row_end = min(n_new, row_begin + QA_ROWS_PER_WARP);
  const int pos0 = p.append_pos[b];

  RQ rq;
  rq.init(p.rot + (size_t)h * (D / 4) * 8, p.thresholds_k, lane, m_s);
  const int li = lane % LPR, sub = lane / LPR;  // lane within the row, row within the warp
  const __half* src_base = p.k_new + (size_t)b * p.stride_b + (size_t)h * p.stride_h + li * 16;

  auto fetch = [&](int i0, uint4& r0, uint4& r1, bool& exists, bool& active) {
    const int i = i0 + sub;
    const long long t = (long long)pos0 + i;
    exists = i < row_end;
    active = exists && t >= 0 && t < p.t_cap;
    r0 = r1 = make_uint4(0u, 0u, 0u, 0u);
    if (active) {
      const uint4* src = reinterpret_cast<const uint4*>(src_base + (size_t)i * p.stride_t);
      r0 = __ldg(src);
      r1 = __ldg(src + 1);
    }
  };
  uint4 n0, n1;
  bool n_exists, n_active;
  fetch(row_begin, n0, n1, n_exists, n_active);
  for (int i0 = row_begin; i0 < row_end; i0 += RPW) {
    const uint4 r0 = n0, r1 = n1;
    const bool exists = n_exists, active = n_active;
    if (i0 + RPW < row_end) fetch(i0 + RPW, n0, n1, n_exists, n_active);  // next rows in flight during this group's math
    const long long t = (long long)pos0 + i0 + sub;
    if (exists && !active && li == 0 && p.status) {
      atomicOr(&p.status[0], IQ_STATUS_ROW_OUT_OF_RANGE);
      atomicAdd(&p.status[2], 1u);
    }
    int code[16];
    const float s = rq.template run<SYM>(r0, r1, active, lane, code, p.status);
    uint32_t w0, w1;
    pack_pair(code, lane, w0, w1);
    if (active) {
      size_t row;
      if (cache_row_for_write(p.pm, b, h, t, p.status, row)) {
        uint32_t* unit_words = reinterpret_cast<uint32_t*>(p.k_codes + row * (size_t)(3 * D / 8)) + 3 * (li >> 1);
        if (li & 1) unit_words[2] = w0;
        else { unit_words[0] = w0; unit_words[1] = w1; }
        if (li == 0) store_scale(p.k_scales, row, s, p.scale_f16, p.status);
      } else if (li == 0 && p.status) {
        atomicAdd(&p.status[2], 1u);  // a row whose page does not exist is skipped and counted
      }
    }
  }
}

// ---------------------------------------------------------------------------------------------------------
// V rows: stored token-transposed. For every block of 128 cache rows and every coordinate c there is one
// 48-byte record holding the 128 codes of coordinate c, arranged like a packing unit sequence with the
// row-in-block in the role of the entry. One CTA handles one 128-row block of one (sequence, KV head): its warps
// quantise the block's new rows, the codes go through shared memory, and thread c assembles the record of
// coordinate c -- written whole (48 contiguous bytes per thread, 1536 per warp) when the block is entirely new,
// otherwise unit by unit with the words that keep old entries read, merged and written back; no other CTA touches
// them.
// ---------------------------------------------------------------------------------------------------------
template <int D, bool SYM>
__global__ void __launch_bounds__(128, 5) quantize_append_v_kernel(const __grid_constant__ QuantizeParams p) {
  using RQ = RowQuantizer<D>;
  constexpr int LPR = RQ::LPR, RPW = RQ::RPW;
  __shared__ __align__(16) uint8_t codes_s[128][D + 16];  // +16: the 16-byte stores of different rows hit different banks
  __shared__ __align__(16) float m_s[RQ::M_FLOATS];

  grid_dependency_wait();
  allow_dependent_launch();
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int b = blockIdx.z;
  const int h = blockIdx.y;
  int n_new = p.n_new ? p.n_new[b] : p.n_new_max;
  n_new = min(n_new, p.n_new_max);
  if (n_new <= 0) return;
  const long long pos0 = p.append_pos[b];
  const long long blkg = (pos0 >= 0 ? pos0 / 128 : -((-pos0 + 127) / 128)) + blockIdx.x;  // floor(pos0 / 128) + x
  const long long t_lo = max(blkg * 128, pos0);                  // first cache row of this block that is appended
  const long long t_hi = min(blkg * 128 + 128, pos0 + n_new);    // one past the last
  if (t_lo >= t_hi) return;
  const bool in_cache = blkg >= 0 && blkg * 128 + 128 <= p.t_cap;  // t_cap is a multiple of 128
  if (!in_cache) {
    if (tid == 0 && p.status) {
      atomicOr(&p.status[0], IQ_STATUS_ROW_OUT_OF_RANGE);
      atomicAdd(&p.status[2], (unsigned)(t_hi - t_lo));
    }
    return;
  }
  size_t block_row0;  // the block's first row in the cache arrays
  if (!cache_row_for_write(p.pm, b, h, blkg * 128, p.status, block_row0)) {  // no such page: the block's rows are skipped and counted
    if (tid == 0 && p.status) atomicAdd(&p.status[2], (unsigned)(t_hi - t_lo));
    return;
  }

  RQ::fill_matrices(p.rot + (size_t)h * (D / 4) * 8, m_s, tid, 128);
  __syncthreads();
  RQ rq;
  rq.init(p.rot + (size_t)h * (D / 4) * 8, p.thresholds_v, lane, m_s);
  const int li = lane % LPR, sub = lane / LPR;
  const __half* src_base = p.v_new + (size_t)b * p.stride_b + (size_t)h * p.stride_h + li * 16;
  const int n_rows = (int)(t_hi - t_lo);
  // the warps take the block's new rows RPW at a time, interleaved; the next rows are in flight during the math
  auto fetch = [&](int i0, uint4& r0, uint4& r1, bool& active) {
    const int i = i0 + sub;
    active = i < n_rows;
    r0 = r1 = make_uint4(0u, 0u, 0u, 0u);
    if (active) {
      const uint4* src = reinterpret_cast<const uint4*>(src_base + (size_t)(t_lo + i - pos0) * p.stride_t);
      r0 = __ldg(src);
      r1 = __ldg(src + 1);
    }
  };
  uint4 n0, n1;
  bool n_active;
  fetch(warp * RPW, n0, n1, n_active);
  for (int i0 = warp * RPW; i0 < n_rows; i0 += 4 * RPW) {
    const uint4 r0 = n0, r1 = n1;
    const bool active = n_active;
    if (i0 + 4 * RPW < n_rows) fetch(i0 + 4 * RPW, n0, n1, n_active);
    const long long t = t_lo + i0 + sub;
    int code[16];
    const float s = rq.template run<SYM>(r0, r1, active, lane, code, p.status);
    if (active) {
      uint32_t pk[4];
#pragma unroll
      for (int q = 0; q < 4; q++)
        pk[q] = (uint32_t)code[4 * q] | ((uint32_t)code[4 * q + 1] << 8) | ((uint32_t)code[4 * q + 2] << 16) | ((uint32_t)code[4 * q + 3] << 24);
      *reinterpret_cast<uint4*>(&codes_s[t & 127][li * 16]) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
      if (li == 0) store_scale(p.v_scales, block_row0 + (size_t)(t & 127), s, p.scale_f16, p.status);
    }
  }
  __syncthreads();

  // Thread c assembles the record of coordinate c: four packing units of three words, the row-in-block as the entry.
  const int c_lo = (int)(t_lo & 127), c_hi = (int)(t_hi - blkg * 128);  // rows [c_lo, c_hi) of the block are new
#pragma unroll
  for (int j = 0; j < D / 128; j++) {
    const int c = tid + 128 * j;  // coordinate
    uint32_t* rec = reinterpret_cast<uint32_t*>(p.v_codes + ((block_row0 / 128) * D + c) * 48);
    if (c_lo == 0 && c_hi == 128) {  // the whole block is new: the record is written with three 16-byte stores
      uint32_t w[12];
#pragma unroll
      for (int u = 0; u < 4; u++) {
        uint32_t w0 = 0u, w1 = 0u, w2 = 0u;
#pragma unroll
        for (int r = 0; r < 8; r++) {
          w0 |= (uint32_t)codes_s[32 * u + r][c] << (4 * r);
          w1 |= (uint32_t)codes_s[32 * u + 8 + r][c] << (4 * r);
          w2 |= (uint32_t)codes_s[32 * u + 16 + r][c] << (4 * r);
        }
#pragma unroll
        for (int r = 0; r < 8; r++) {  // entries 24..31: bit k of the code into the top bit of nibble r of word k
          const uint32_t cd = codes_s[32 * u + 24 + r][c];
          w0 |= (cd & 1u) << (4 * r + 3);
          w1 |= ((cd >> 1) & 1u) << (4 * r + 3);
          w2 |= ((cd >> 2) & 1u) << (4 * r + 3);
        }
        w[3 * u] = w0; w[3 * u + 1] = w1; w[3 * u + 2] = w2;
      }
      uint4* dst = reinterpret_cast<uint4*>(rec);
      dst[0] = make_uint4(w[0], w[1], w[2], w[3]);
      dst[1] = make_uint4(w[4], w[5], w[6], w[7]);
      dst[2] = make_uint4(w[8], w[9], w[10], w[11]);
      continue;
    }
    for (int u = 0; u < 4; u++) {  // partly covered block: unit by unit, words that keep old entries are merged
      const int lo = max(c_lo, 32 * u) - 32 * u, hi = min(c_hi, 32 * u + 32) - 32 * u;
      if (lo >= hi) continue;
      uint32_t w[3] = {0u, 0u, 0u}, m[3] = {0u, 0u, 0u};
      for (int r = lo; r < hi; r++) {
        const uint32_t cd = codes_s[32 * u + r][c];
        if (r < 24) {
          w[r >> 3] |= cd << (4 * (r & 7));
          m[r >> 3] |= 7u << (4 * (r & 7));
        } else {
          const int sh = 4 * (r - 24) + 3;
#pragma unroll
          for (int k = 0; k < 3; k++) {
            w[k] |= ((cd >> k) & 1u) << sh;
            m[k] |= 1u << sh;
          }
        }
      }
      uint32_t* dst = rec + 3 * u;
#pragma unroll
      for (int k = 0; k < 3; k++) {
        if (m[k] == 0u) continue;
        dst[k] = (m[k] == 0xFFFFFFFFu) ? w[k] : ((dst[k] & ~m[k]) | w[k]);
      }
    }
  }
}

// ---------------------------------------------------------------------------------------------------------
// Few new rows per sequence (the decode step appends one): latency matters, not throughput. One warp per
// (sequence, KV head, tensor) with the whole warp on a row -- lane l owns coordinates l*d/32 .. (one or two SO(4)
// blocks), five shuffle stages of the butterfly -- a short instruction stream and no shared memory. The V row goes
// straight into its transposed records with one read-modify-write per touched word.
// ---------------------------------------------------------------------------------------------------------
template <int D, int BITS>
__global__ void __launch_bounds__(32) quantize_append_few_kernel(const __grid_constant__ QuantizeParams p) {
  constexpr int E = D / 32;
  grid_dependency_wait();
  allow_dependent_launch();
  const int lane = threadIdx.x;
  const bool is_v = (blockIdx.x & 1) != 0;
  const int chunk = blockIdx.x >> 1;  // the warp takes the rows that fall into one 128-row block of the cache
  const int h = blockIdx.y, b = blockIdx.z;
  int n_new = p.n_new ? p.n_new[b] : p.n_new_max;
  n_new = min(n_new, p.n_new_max);
  if (n_new <= 0) return;
  const long long pos0 = p.append_pos[b];
  // rows i with floor((pos0 + i) / 128) == floor(pos0 / 128) + chunk (rows at negative positions: chunk 0, they are refused below)
  const long long blk0 = pos0 >= 0 ? pos0 / 128 : 0;
  const long long lo = max(0ll, (blk0 + chunk) * 128 - pos0), hi = min((long long)n_new, (blk0 + chunk + 1) * 128 - pos0);
  const int i_lo = (int)((chunk == 0) ? 0 : lo), i_hi = (int)hi;
  if (i_lo >= i_hi) return;
  const __half* src_base = (is_v ? p.v_new : p.k_new) + (size_t)b * p.stride_b + (size_t)h * p.stride_h + lane * E;
  __half2 raw[E / 2];  // the first row is requested before the rotation blocks are set up: two latencies in one
#pragma unroll
  for (int k = 0; k < E / 2; k++) raw[k] = reinterpret_cast<const __half2*>(src_base + (size_t)i_lo * p.stride_t)[k];
  WarpRowQuantizer<D, BITS> rq;
  const RowSink sink{p.k_codes, p.k_scales, p.v_codes, p.v_scales, p.status, p.scale_f16};
  rq.init(p.rot + (size_t)h * (D / 4) * 8, is_v ? p.thresholds_v : p.thresholds_k, lane);
  // 2 and 4 bits, V rows: the codes of consecutive rows that share a word of the records (8 or 16 rows) are collected in
  // registers and the word is written once -- whole when every entry of it is new, merged with the old word otherwise --
  // instead of one read-modify-write per row (this kernel is also the bulk path of those widths).
  uint32_t pend[E];
  uint32_t pend_mask = 0u;
  int pend_word = -1;
  size_t pend_blk = 0;
#pragma unroll
  for (int e = 0; e < E; e++) pend[e] = 0u;
  auto flush_pending = [&]() {
    if constexpr (BITS != 3) {
      if (pend_word >= 0 && pend_mask != 0u) {
#pragma unroll
        for (int e = 0; e < E; e++) {
          uint32_t* dst = reinterpret_cast<uint32_t*>(p.v_codes + (pend_blk * D + lane * E + e) * (size_t)(16 * BITS)) + pend_word;
          *dst = (pend_mask == 0xFFFFFFFFu) ? pend[e] : ((*dst & ~pend_mask) | pend[e]);
          pend[e] = 0u;
        }
      }
      pend_mask = 0u;
      pend_word = -1;
    }
  };
  for (int i = i_lo; i < i_hi; i++) {
    __half2 nxt[E / 2];  // the next row is requested before this one is worked on
    if (i + 1 < i_hi) {
#pragma unroll
      for (int k = 0; k < E / 2; k++) nxt[k] = reinterpret_cast<const __half2*>(src_base + (size_t)(i + 1) * p.stride_t)[k];
    }
    const long long t = pos0 + i;
    bool ok = true;
    size_t row = 0;  // the row's place in the cache arrays
    if (t < 0 || t >= p.t_cap) {
      if (lane == 0 && p.status) {  // counted per (row, KV head, tensor), like the bulk kernels
        atomicOr(&p.status[0], IQ_STATUS_ROW_OUT_OF_RANGE);
        atomicAdd(&p.status[2], 1u);
      }
      ok = false;
    } else if (!cache_row_for_write(p.pm, b, h, t, p.status, row)) {  // no such page: skipped and counted
      if (lane == 0 && p.status) atomicAdd(&p.status[2], 1u);
      ok = false;
    }
    if (ok) {
      int code[E];
      const float s = rq.run(raw, lane, code, p.status);
      if (!is_v) {
        warp_store_k_row<D, BITS>(sink, row, code, s, lane);
      } else if constexpr (BITS == 3) {
        warp_store_v_row<D, BITS>(sink, row, t, code, s, lane);
      } else {
        int word, sh;
        packed_place<BITS>((int)(t % 128), word, sh);
        if (word != pend_word || row / 128 != pend_blk) {
          flush_pending();
          pend_word = word;
          pend_blk = row / 128;
        }
#pragma unroll
        for (int e = 0; e < E; e++) pend[e] |= (uint32_t)code[e] << sh;
        pend_mask |= ((1u << BITS) - 1u) << sh;
        if (lane == 0) store_scale(p.v_scales, row, s, p.scale_f16, p.status);
      }
    }
    if (i + 1 < i_hi) {
#pragma unroll
      for (int k = 0; k < E / 2; k++) raw[k] = nxt[k];
    }
  }
  flush_pending();
}

// ---------------------------------------------------------------------------------------------------------
// Calibration: histogram of the rotated, normalised coordinates u = sqrt(d) R x^ of a set of rows -- the empirical
// marginal that Step 3's Lloyd-Max codebook is fitted to. Same row mapping as the K kernel; the CTA counts into a
// histogram in shared memory and adds its non-empty bins to the caller's at the end. Zero rows are left out.
// ---------------------------------------------------------------------------------------------------------
// The row quantiser the histogram shares with the append kernels loads seven thresholds; the histogram has none.
__device__ const float g_no_thresholds[7] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};

template <int D>
__global__ void __launch_bounds__(QA_WARPS * 32, 4) rotated_histogram_kernel(const __grid_constant__ HistogramParams p) {
  using RQ = RowQuantizer<D>;
  constexpr int LPR = RQ::LPR, RPW = RQ::RPW;
  __shared__ uint32_t hist_s[HIST_MAX_BINS];
  __shared__ __align__(16) float m_s[RQ::M_FLOATS];
  grid_dependency_wait();
  allow_dependent_launch();
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int b = blockIdx.z, h = blockIdx.y;
  int n_rows = p.n_rows ? p.n_rows[b] : p.n_rows_max;
  n_rows = min(n_rows, p.n_rows_max);
  const int cta_begin = blockIdx.x * QA_WARPS * HIST_ROWS_PER_WARP;
  if (cta_begin >= n_rows) return;
  for (int i = tid; i < p.bins; i += QA_WARPS * 32) hist_s[i] = 0u;
  RQ::fill_matrices(p.rot + (size_t)h * (D / 4) * 8, m_s, tid, QA_WARPS * 32);
  __syncthreads();
  RQ rq;
  rq.init(p.rot + (size_t)h * (D / 4) * 8, g_no_thresholds, lane, m_s);  // (the histogram takes u itself, no codes)
  const int li = lane % LPR, sub = lane / LPR;
  const __half* src_base = p.x + (size_t)b * p.stride_b + (size_t)h * p.stride_h + li * 16;
  const int row_begin = cta_begin + warp * HIST_ROWS_PER_WARP, row_end = min(n_rows, row_begin + HIST_ROWS_PER_WARP);
  const float to_bin = (float)p.bins / (2.f * p.range);
  for (int i0 = row_begin; i0 < row_end; i0 += RPW) {
    const int i = i0 + sub;
    const bool active = i < row_end;
    uint4 r0 = make_uint4(0u, 0u, 0u, 0u), r1 = r0;
    if (active) {
      const uint4* src = reinterpret_cast<const uint4*>(src_base + (size_t)i * p.stride_t);
      r0 = __ldg(src);
      r1 = __ldg(src + 1);
    }
    float x[16];
    double ss;
    const float s = rq.rotate(r0, r1, lane, x, ss);
    if (active && s > 0.f) {
      const float inv_s = __frcp_rn(s);
#pragma unroll
      for (int e = 0; e < 16; e++) {
        const int bin = (int)floorf((x[e] * inv_s + p.range) * to_bin);
        atomicAdd(&hist_s[min(max(bin, 0), p.bins - 1)], 1u);
      }
    }
  }
  __syncthreads();
  for (int i = tid; i < p.bins; i += QA_WARPS * 32)
    if (hist_s[i]) atomicAdd(&p.hist[i], hist_s[i]);
}

cudaError_t launch_rotated_histogram(const HistogramParams& p, int head_dim, int batch, cudaStream_t stream) {
  if (p.n_rows_max <= 0 || batch <= 0) return cudaSuccess;
  const int rows_per_cta = QA_WARPS * HIST_ROWS_PER_WARP;
  dim3 grid((p.n_rows_max + rows_per_cta - 1) / rows_per_cta, p.n_kv_heads, batch);
  return head_dim == 128 ? launch_after_predecessor(rotated_histogram_kernel<128>, grid, dim3(QA_WARPS * 32), 0, stream, p)
                         : launch_after_predecessor(rotated_histogram_kernel<256>, grid, dim3(QA_WARPS * 32), 0, stream, p);
}

// Calibration of the rotation: z = sqrt(d) H_d x^ (Algorithm 1, lines 1-2, in the unit-variance units of the codebook) of
// a set of rows, written out as fp32. One warp per row, lane l holds coordinates l E .. l E + E - 1.
template <int D>
__global__ void __launch_bounds__(QA_WARPS * 32) wht_coordinates_kernel(const __grid_constant__ WhtParams p) {
  constexpr int E = D / 32;
  grid_dependency_wait();
  allow_dependent_launch();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int b = blockIdx.z, h = blockIdx.y;
  const int t = blockIdx.x * QA_WARPS + warp;
  int n_rows = p.n_rows ? p.n_rows[b] : p.n_rows_max;
  n_rows = min(n_rows, p.n_rows_max);
  if (t >= n_rows) return;
  const __half* src = p.x + (size_t)b * p.stride_b + (size_t)t * p.stride_t + (size_t)h * p.stride_h + lane * E;
  float v[E];
  double ss = 0.0;  // squares of fp16 values are exact in fp32
#pragma unroll
  for (int e = 0; e < E; e++) {
    v[e] = __half2float(src[e]);
    ss += (double)(v[e] * v[e]);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(FULL, ss, o);
  wht_warp<float, E>(v, lane);  // unnormalised: the 1/sqrt(d) of H_d and the sqrt(d) of the units cancel
  const float inv_s = ss > 0.0 ? (float)(1.0 / sqrt(ss)) : 0.f;
  float* dst = p.z + (((size_t)b * p.n_rows_max + t) * p.n_kv_heads + h) * D + lane * E;
#pragma unroll
  for (int e = 0; e < E; e++) dst[e] = v[e] * inv_s;
}

cudaError_t launch_wht_coordinates(const WhtParams& p, int head_dim, int batch, cudaStream_t stream) {
  if (p.n_rows_max <= 0 || batch <= 0) return cudaSuccess;
  dim3 grid((p.n_rows_max + QA_WARPS - 1) / QA_WARPS, p.n_kv_heads, batch);
  return head_dim == 128 ? launch_after_predecessor(wht_coordinates_kernel<128>, grid, dim3(QA_WARPS * 32), 0, stream, p)
                         : launch_after_predecessor(wht_coordinates_kernel<256>, grid, dim3(QA_WARPS * 32), 0, stream, p);
}

template <int D, int BITS>
static cudaError_t launch_few(const QuantizeParams& p, int batch, cudaStream_t stream) {
  // x = 2 * chunk + (0: the K rows, 1: the V rows) of (sequence, KV head); a chunk is the part of the new rows inside
  // one 128-row block of the cache (+1: the first row may sit in the middle of a block)
  dim3 grid(2 * ((p.n_new_max + 127) / 128 + 1), p.n_kv_heads, batch);
  return launch_after_predecessor(quantize_append_few_kernel<D, BITS>, grid, dim3(32), 0, stream, p);
}

cudaError_t launch_quantize_append(const QuantizeParams& p, int head_dim, int batch, cudaStream_t stream) {
  if (p.n_new_max <= 0 || batch <= 0) return cudaSuccess;
  // 2 and 4 bits: one warp per row throughout (the row-tiled kernels below are written for the 3-bit layout)
  if (p.bits == 2) return head_dim == 128 ? launch_few<128, 2>(p, batch, stream) : launch_few<256, 2>(p, batch, stream);
  if (p.bits == 4) return head_dim == 128 ? launch_few<128, 4>(p, batch, stream) : launch_few<256, 4>(p, batch, stream);
  const int rows_per_cta = QA_WARPS * QA_ROWS_PER_WARP;
  dim3 kgrid((p.n_new_max + rows_per_cta - 1) / rows_per_cta, p.n_kv_heads, batch);
  dim3 vgrid((p.n_new_max + 127) / 128 + 1, p.n_kv_heads, batch);  // +1: the first row may sit in the middle of a block
  if (p.n_new_max <= QA_FEW_ROWS) return head_dim == 128 ? launch_few<128, 3>(p, batch, stream) : launch_few<256, 3>(p, batch, stream);
  // (the V kernel may start under the K kernel: they write different arrays)
  auto symmetric = [](const float* t) { return t[3] == 0.f && t[0] == -t[6] && t[1] == -t[5] && t[2] == -t[4]; };  // two compares per coordinate instead of three
  const bool sym_k = symmetric(p.thresholds_k), sym_v = symmetric(p.thresholds_v);
  const dim3 kblock(QA_WARPS * 32), vblock(128);
  cudaError_t e;
  if (head_dim == 128)
    e = sym_k ? launch_after_predecessor(quantize_append_k_kernel<128, true>, kgrid, kblock, 0, stream, p)
              : launch_after_predecessor(quantize_append_k_kernel<128, false>, kgrid, kblock, 0, stream, p);
  else
    e = sym_k ? launch_after_predecessor(quantize_append_k_kernel<256, true>, kgrid, kblock, 0, stream, p)
              : launch_after_predecessor(quantize_append_k_kernel<256, false>, kgrid, kblock, 0, stream, p);
  if (e != cudaSuccess) return e;
  if (head_dim == 128)
    return sym_v ? launch_after_predecessor(quantize_append_v_kernel<128, true>, vgrid, vblock, 0, stream, p)
                 : launch_after_predecessor(quantize_append_v_kernel<128, false>, vgrid, vblock, 0, stream, p);
  return sym_v ? launch_after_predecessor(quantize_append_v_kernel<256, true>, vgrid, vblock, 0, stream, p)
               : launch_after_predecessor(quantize_append_v_kernel<256, false>, vgrid, vblock, 0, stream, p);
}

}  // namespace iq
