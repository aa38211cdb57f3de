// Reconstruct-then-compute, first half (Figure 1, top): every cached row dequantised and rotated back to the original
// space, x_hat = R^T x~ = H_d blockdiag(M_b^T) (scale * level[code] / sqrt(d)) / sqrt(d), written as binary16 K/V
// tensors for a standard attention kernel. This is the execution model the fused decode path replaces; it exists so that
// the two can be measured against each other on the same packed cache.
#include "iq_common.cuh"
#include "iq_format.cuh"
#include "iq_kernels.h"

namespace iq {

// One CTA per (128-row block, KV head, sequence): the block's packed K rows and its token-transposed V records are
// staged in shared memory once; a row is shared by d/16 lanes, 16 consecutive coordinates (4 whole SO(4) blocks) per
// lane, so a warp holds 4 rows at a time at d = 128 (2 at d = 256): 4 butterfly stages inside the lane, log2(d/16)
// across the row's lanes.
constexpr int RC_WARPS = 8;

template <int D, int BITS>
__global__ void __launch_bounds__(RC_WARPS * 32) reconstruct_kernel(const ReconstructParams p) {
  constexpr int ROWB = BITS * D / 8, VREC = 16 * BITS, LPR = D / 16, RPW = 32 / LPR, TB = 128;
  __shared__ __align__(16) uint8_t k_s[TB * ROWB];
  __shared__ __align__(16) uint8_t v_s[D * VREC];
  __shared__ float ks_s[TB], vs_s[TB], lv_s[16], lvv_s[16];

  grid_dependency_wait();
  allow_dependent_launch();
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int b = blockIdx.z, g = blockIdx.y;
  const int len = max(0, min(p.seq_lens[b], min(p.t_cap, p.out_rows)));
  const int r_begin = blockIdx.x * TB;
  if (r_begin >= len) return;
  const int n = min(TB, len - r_begin);
  const size_t row0 = cache_row(p.pm, b, g, r_begin, p.status);  // the block's first row in the cache arrays

  {  // stage the block: n packed K rows, the whole V record set of the block (128 * ROWB = D * 16 b bytes), the scales
    const uint4* ksrc = reinterpret_cast<const uint4*>(p.k_codes + row0 * ROWB);
    const uint4* vsrc = reinterpret_cast<const uint4*>(p.v_codes + row0 * ROWB);
    for (int i = tid; i < n * ROWB / 16; i += RC_WARPS * 32) reinterpret_cast<uint4*>(k_s)[i] = ksrc[i];
    for (int i = tid; i < D * VREC / 16; i += RC_WARPS * 32) reinterpret_cast<uint4*>(v_s)[i] = vsrc[i];
    if (tid < n) {
      ks_s[tid] = load_scale(p.k_scales, row0 + tid, p.scale_f16);
      vs_s[tid] = load_scale(p.v_scales, row0 + tid, p.scale_f16);
    }
    if (tid < 16) { lv_s[tid] = p.levels_k[tid]; lvv_s[tid] = p.levels_v[tid]; }
  }
  const int li = lane % LPR, sub = lane / LPR;  // lane within the row, row within the warp
  float M[4][4][4];
  {
    const float* qb = p.rot + ((size_t)g * (D / 4) + (size_t)li * 4) * 8;
#pragma unroll
    for (int j = 0; j < 4; j++) so4_matrix<float>(qb + 8 * j, M[j]);
  }
  __syncthreads();

  // x (16 coordinates of this lane, dequantised levels) -> 16 binary16 values of the reconstructed row at dst
  auto rotate_back_and_store = [&](float (&x)[16], float scale, __half* dst, bool active) {
    so4_apply<float, 16, true>(M, x);
#pragma unroll
    for (int s = 1; s < 16; s <<= 1)
#pragma unroll
      for (int i = 0; i < 16; i++)
        if ((i & s) == 0) {
          const float a = x[i], c = x[i + s];
          x[i] = a + c;
          x[i + s] = a - c;
        }
#pragma unroll
    for (int o = 1; o < LPR; o <<= 1) {
      const float sgn = (lane & o) ? -1.f : 1.f;  // the upper lane of a pair keeps (other - own)
#pragma unroll
      for (int i = 0; i < 16; i++) x[i] = fmaf(sgn, x[i], __shfl_xor_sync(FULL, x[i], o));
    }
    if (active) {
      const float f = scale * (1.0f / (float)D);  // 1/sqrt(d) of the dequantisation times 1/sqrt(d) of H_d
      uint32_t h[8];
#pragma unroll
      for (int i = 0; i < 8; i++) h[i] = pack_half2(x[2 * i] * f, x[2 * i + 1] * f);
      reinterpret_cast<uint4*>(dst)[0] = make_uint4(h[0], h[1], h[2], h[3]);
      reinterpret_cast<uint4*>(dst)[1] = make_uint4(h[4], h[5], h[6], h[7]);
    }
  };

  for (int r0 = warp * RPW; r0 < n; r0 += RC_WARPS * RPW) {
    const int r = r0 + sub;
    const bool active = r < n;  // the lanes of a row beyond the block still take part in the shuffles
    const int rr = active ? r : 0;
    const size_t out_off = (size_t)b * p.stride_b + (size_t)(r_begin + rr) * p.stride_t + (size_t)g * p.stride_h + (size_t)li * 16;
    float x[16];
    if constexpr (BITS != 3) {  // K row rr: the lane's 16 entries
      const uint32_t* w = reinterpret_cast<const uint32_t*>(k_s + rr * ROWB);
#pragma unroll
      for (int e = 0; e < 16; e++) x[e] = lv_s[packed_code<BITS>(w, li * 16 + e)];
    } else {  // K row rr: this lane's half of packing unit li / 2
      const uint32_t* w = reinterpret_cast<const uint32_t*>(k_s + rr * ROWB) + 3 * (li >> 1);
      const uint32_t w0 = w[0], w1 = w[1], w2 = w[2];
      uint32_t sa, sb;  // eight codes each, one per nibble
      if (li & 1) {
        sa = w2 & 0x77777777u;
        sb = ((w0 >> 3) & 0x11111111u) | ((w1 >> 2) & 0x22222222u) | ((w2 >> 1) & 0x44444444u);
      } else {
        sa = w0 & 0x77777777u;
        sb = w1 & 0x77777777u;
      }
#pragma unroll
      for (int e = 0; e < 8; e++) {
        x[e] = lv_s[(sa >> (4 * e)) & 7u];
        x[8 + e] = lv_s[(sb >> (4 * e)) & 7u];
      }
    }
    rotate_back_and_store(x, ks_s[rr], p.k_out + out_off, active);
    {  // V row rr: one record per coordinate, the row-in-block is the entry
#pragma unroll
      for (int e = 0; e < 16; e++) {
        const uint32_t* w = reinterpret_cast<const uint32_t*>(v_s + (size_t)(li * 16 + e) * VREC);
        x[e] = lvv_s[packed_code<BITS>(w, rr)];
      }
    }
    rotate_back_and_store(x, vs_s[rr], p.v_out + out_off, active);
  }
}

template <int BITS>
static cudaError_t launch_reconstruct_bits(const ReconstructParams& p, int head_dim, dim3 grid, cudaStream_t stream) {
  if (head_dim == 128) return launch_after_predecessor(reconstruct_kernel<128, BITS>, grid, dim3(RC_WARPS * 32), 0, stream, p);
  return launch_after_predecessor(reconstruct_kernel<256, BITS>, grid, dim3(RC_WARPS * 32), 0, stream, p);
}
cudaError_t launch_reconstruct_rows(const ReconstructParams& p, int head_dim, int batch, cudaStream_t stream) {
  if (batch <= 0 || p.t_cap <= 0 || p.out_rows <= 0) return cudaSuccess;
  dim3 grid((unsigned)((min(p.t_cap, p.out_rows) + 127) / 128), (unsigned)p.n_kv_heads, (unsigned)batch);
  if (p.bits == 2) return launch_reconstruct_bits<2>(p, head_dim, grid, stream);
  if (p.bits == 4) return launch_reconstruct_bits<4>(p, head_dim, grid, stream);
  return launch_reconstruct_bits<3>(p, head_dim, grid, stream);
}

}  // namespace iq
