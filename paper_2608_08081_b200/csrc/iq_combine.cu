// Merge of the context-split partials and the single inverse rotation o = R^T o~ (Table 2, kernel D;
// Appendix A), plus the small kernels that prepare the rotation parameters (Appendix B).
#include "iq_common.cuh"
#include "iq_kernels.h"

namespace iq {

constexpr int CMB_WARPS = 4;

// WPH = 1: one warp per (sequence, query head), CMB_WARPS heads per CTA. WPH > 1 (many slots): one CTA of WPH warps
// per head; warp w merges slots w, w + WPH, ... and warp 0 merges the warps' results. Lane l owns rotated
// coordinates l*E .. l*E+E-1, i.e. whole SO(4) blocks, so M_b^T is applied in registers and H_d by the warp butterfly.
template <int D, int WPH>
__global__ void __launch_bounds__(WPH == 1 ? CMB_WARPS * 32 : WPH * 32) combine_kernel(const CombineParams p) {
  constexpr int E = D / 32;
  grid_dependency_wait();
  allow_dependent_launch();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int bh = WPH == 1 ? blockIdx.x * CMB_WARPS + warp : blockIdx.x;
  if (bh >= p.batch * p.n_q_heads) return;
  const int h = bh % p.n_q_heads;
  const int kvh = h / (p.n_q_heads / p.n_kv_heads);
  const int S1 = p.splits, S = p.splits * p.shards;  // slots of one shard, of all shards
  const size_t shard_heads = (size_t)p.batch * p.n_q_heads;
  // slot s of this head: shard s / S1, its slot s % S1 (one shard: s itself)
  auto slot_index = [&](int s) { return p.shards == 1 ? (size_t)bh * S1 + s : ((size_t)(s / S1) * shard_heads + bh) * S1 + (s % S1); };
  auto slot_argmax = [&](int s, size_t o) {
    int idx = p.part_argmax ? p.part_argmax[o] : -1;
    if (idx >= 0 && p.row_offsets) idx += p.row_offsets[(size_t)(s / S1) * p.batch + bh / p.n_q_heads];
    return idx;
  };
  const int s0 = WPH == 1 ? 0 : warp;

  // the rotation block of this lane first: its loads do not depend on the partials and overlap with theirs
  float M[E / 4][4][4];
  if (WPH == 1 || warp == 0) {
    const float* qb = p.rot + ((size_t)kvh * (D / 4) + (size_t)lane * (E / 4)) * 8;
#pragma unroll
    for (int j = 0; j < E / 4; j++) so4_matrix<float>(qb + 8 * j, M[j]);
  }

  float m = -INFINITY;
  int best = -1;
  float l = 0.f;
  float v[E];
#pragma unroll
  for (int e = 0; e < E; e++) v[e] = 0.f;
  // The warp's run of slots: all of them (WPH = 1), else an equal share of consecutive slots.
  const int chunk = WPH == 1 ? S : (S + WPH - 1) / WPH;
  const int c0 = WPH == 1 ? 0 : warp * chunk;
  const int cn = max(0, min(chunk, S - c0));
  if (chunk <= 32) {
    // at most 32 slots per warp: lane j takes (m, l, argmax) of slot c0 + j, the reference and the weights come from warp
    // reductions, and the acc rows are then loaded eight at a time (their addresses do not depend on one another)
    float ms = -INFINITY, ls = 0.f;
    int idx = -1;
    size_t o = 0;
    if (lane < cn) {
      o = slot_index(c0 + lane);
      ms = p.part_ml[2 * o];
      ls = p.part_ml[2 * o + 1];
      if (ls > 0.f) idx = slot_argmax(c0 + lane, o);
      else ms = -INFINITY;
    }
    m = ms;
    best = idx;
#pragma unroll
    for (int d2 = 16; d2 > 0; d2 >>= 1) {
      const float om = __shfl_xor_sync(FULL, m, d2);
      const int ob = __shfl_xor_sync(FULL, best, d2);
      if (om > m) { m = om; best = ob; }
      else if (om == m && ob >= 0 && (best < 0 || ob < best)) best = ob;
    }
    const float w = (ls > 0.f) ? __expf(ms - m) : 0.f;
    l = ls * w;
#pragma unroll
    for (int d2 = 16; d2 > 0; d2 >>= 1) l += __shfl_xor_sync(FULL, l, d2);
    constexpr int NF = 8;  // rows in flight
    for (int sb = 0; sb < cn; sb += NF) {
      float4 f[NF][E / 4];
      float ws[NF];
#pragma unroll
      for (int k = 0; k < NF; k++) {
        ws[k] = __shfl_sync(FULL, w, (sb + k) & 31);
        const size_t ok = __shfl_sync(FULL, o, (sb + k) & 31);
        if (sb + k >= cn) ws[k] = 0.f;
#pragma unroll
        for (int e4 = 0; e4 < E / 4; e4++)
          f[k][e4] = ws[k] != 0.f ? *reinterpret_cast<const float4*>(p.part_acc + ok * D + lane * E + 4 * e4) : make_float4(0.f, 0.f, 0.f, 0.f);
      }
#pragma unroll
      for (int k = 0; k < NF; k++)
#pragma unroll
        for (int e4 = 0; e4 < E / 4; e4++) {
          v[4 * e4] += ws[k] * f[k][e4].x; v[4 * e4 + 1] += ws[k] * f[k][e4].y; v[4 * e4 + 2] += ws[k] * f[k][e4].z; v[4 * e4 + 3] += ws[k] * f[k][e4].w;
        }
    }
  } else {
  for (int s = s0; s < S; s += WPH) {
    const size_t o = slot_index(s);
    const float ms = p.part_ml[2 * o], ls = p.part_ml[2 * o + 1];
    if (!(ls > 0.f)) continue;
    const int idx = slot_argmax(s, o);
    if (ms > m) { m = ms; best = idx; }
    else if (ms == m && idx >= 0 && (best < 0 || idx < best)) best = idx;
  }
  for (int s = s0; s < S; s += WPH) {
    const size_t o = slot_index(s);
    const float ms = p.part_ml[2 * o], ls = p.part_ml[2 * o + 1];
    if (!(ls > 0.f)) continue;
    const float w = __expf(ms - m);
    l += ls * w;
    const float* a = p.part_acc + o * D + lane * E;
#pragma unroll
    for (int e4 = 0; e4 < E; e4 += 4) {
      const float4 f = *reinterpret_cast<const float4*>(a + e4);
      v[e4] += w * f.x; v[e4 + 1] += w * f.y; v[e4 + 2] += w * f.z; v[e4 + 3] += w * f.w;
    }
  }
  }
  if constexpr (WPH > 1) {  // the warps' results (relative to their own maxima) merged by warp 0
    __shared__ float sv[WPH][D];
    __shared__ float sm[WPH], sl[WPH];
    __shared__ int sb[WPH];
#pragma unroll
    for (int e = 0; e < E; e++) sv[warp][lane * E + e] = v[e];
    if (lane == 0) { sm[warp] = m; sl[warp] = l; sb[warp] = best; }
    __syncthreads();
    if (warp != 0) return;
    m = -INFINITY;
    best = -1;
    for (int w2 = 0; w2 < WPH; w2++) {
      if (!(sl[w2] > 0.f)) continue;
      if (sm[w2] > m) { m = sm[w2]; best = sb[w2]; }
      else if (sm[w2] == m && sb[w2] >= 0 && (best < 0 || sb[w2] < best)) best = sb[w2];
    }
    l = 0.f;
#pragma unroll
    for (int e = 0; e < E; e++) v[e] = 0.f;
    for (int w2 = 0; w2 < WPH; w2++) {
      if (!(sl[w2] > 0.f)) continue;
      const float w = __expf(sm[w2] - m);
      l += sl[w2] * w;
#pragma unroll
      for (int e = 0; e < E; e++) v[e] += w * sv[w2][lane * E + e];
    }
  }
  if (p.new_ml) {  // the step's new row: one more slot (its row index is the highest of the sequence: it wins no tie)
    const float mn = p.new_ml[2 * (size_t)bh], ln = p.new_ml[2 * (size_t)bh + 1];
    if (ln > 0.f) {
      const bool had = l > 0.f;
      const float m2 = had ? fmaxf(m, mn) : mn;
      const float wa = had ? __expf(m - m2) : 0.f, wn = __expf(mn - m2);
      const float4* a = reinterpret_cast<const float4*>(p.new_acc + (size_t)bh * D + lane * E);
#pragma unroll
      for (int e4 = 0; e4 < E / 4; e4++) {
        const float4 f = a[e4];
        v[4 * e4] = fmaf(wn, f.x, wa * v[4 * e4]);
        v[4 * e4 + 1] = fmaf(wn, f.y, wa * v[4 * e4 + 1]);
        v[4 * e4 + 2] = fmaf(wn, f.z, wa * v[4 * e4 + 2]);
        v[4 * e4 + 3] = fmaf(wn, f.w, wa * v[4 * e4 + 3]);
      }
      l = fmaf(ln, wn, wa * l);
      if (!had || mn > m) best = p.new_rows[bh / p.n_q_heads];
      m = m2;
    }
  }
  const bool empty = !(l > 0.f);
  const float inv = empty ? 0.f : 1.f / l;
#pragma unroll
  for (int e = 0; e < E; e++) v[e] *= inv;

  // o = H_d * blockdiag(M_b^T) * o~   (H_d symmetric, R^T = H_d^T R_SO4^T)
  so4_apply<float, E, true>(M, v);
  wht_warp<float, E>(v, lane);
  const float inv_root_d = rsqrtf((float)D);
#pragma unroll
  for (int e = 0; e < E; e++) v[e] *= inv_root_d;

  if (p.out_is_fp16) {
    __half* o = reinterpret_cast<__half*>(p.out) + (size_t)bh * D + lane * E;
#pragma unroll
    for (int e = 0; e < E; e += 2) *reinterpret_cast<__half2*>(o + e) = __floats2half2_rn(v[e], v[e + 1]);
  } else {
    float* o = reinterpret_cast<float*>(p.out) + (size_t)bh * D + lane * E;
#pragma unroll
    for (int e4 = 0; e4 < E; e4 += 4) *reinterpret_cast<float4*>(o + e4) = make_float4(v[e4], v[e4 + 1], v[e4 + 2], v[e4 + 3]);
  }
  if (lane == 0) {
    if (p.lse) p.lse[bh] = empty ? -INFINITY : m + __logf(l);
    if (p.argmax) p.argmax[bh] = empty ? -1 : best;
  }
}

constexpr int CMB_WIDE = 8;  // warps per head when there are many slots

cudaError_t launch_combine_splits(const CombineParams& p, int head_dim, cudaStream_t stream) {
  const int n = p.batch * p.n_q_heads;
  if (n <= 0) return cudaSuccess;
  if (p.splits * p.shards > 16) {  // many slots per head (small batches cut into many pieces): the slots of a head spread over a CTA
    dim3 grid(n), block(CMB_WIDE * 32);
    if (head_dim == 128) return launch_after_predecessor(combine_kernel<128, CMB_WIDE>, grid, block, 0, stream, p);
    return launch_after_predecessor(combine_kernel<256, CMB_WIDE>, grid, block, 0, stream, p);
  }
  dim3 grid((n + CMB_WARPS - 1) / CMB_WARPS), block(CMB_WARPS * 32);
  if (head_dim == 128) return launch_after_predecessor(combine_kernel<128, 1>, grid, block, 0, stream, p);
  return launch_after_predecessor(combine_kernel<256, 1>, grid, block, 0, stream, p);
}

// ------------------------------------------------------------------------------------------------
// Rotation parameters: unit quaternion pairs (Appendix B). Counter-based generator: splitmix64 of
// (seed, quaternion index, component) -> two uniforms -> Box-Muller normal.
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ uint64_t splitmix64(uint64_t x) {
  x += 0x9E3779B97F4A7C15ull;
  x = (x ^ (x >> 30)) * 0xBF58476D1CE4E5B9ull;
  x = (x ^ (x >> 27)) * 0x94D049BB133111EBull;
  return x ^ (x >> 31);
}

__global__ void make_rotation_kernel(float* rot, int n_quats, uint64_t seed) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n_quats) return;
  float q[4];
  float nn = 0.f;
#pragma unroll
  for (int c = 0; c < 4; c++) {
    const uint64_t r = splitmix64(splitmix64(seed) ^ ((uint64_t)i * 4 + c));
    const float u1 = ((float)(uint32_t)(r >> 40) + 0.5f) * (1.0f / 16777216.0f);
    const float u2 = ((float)(uint32_t)((r >> 8) & 0xFFFFFFu) + 0.5f) * (1.0f / 16777216.0f);
    q[c] = sqrtf(-2.f * logf(u1)) * cospif(2.f * u2);
    nn += q[c] * q[c];
  }
  const float inv = rsqrtf(nn);
#pragma unroll
  for (int c = 0; c < 4; c++) rot[(size_t)i * 4 + c] = q[c] * inv;
}

__global__ void normalize_rotation_kernel(float* rot, int n_quats) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n_quats) return;
  float4 q = *reinterpret_cast<float4*>(rot + (size_t)i * 4);
  const float inv = rsqrtf(q.x * q.x + q.y * q.y + q.z * q.z + q.w * q.w);
  q.x *= inv; q.y *= inv; q.z *= inv; q.w *= inv;
  *reinterpret_cast<float4*>(rot + (size_t)i * 4) = q;
}

cudaError_t launch_make_rotation(float* rot, int n_quats, uint64_t seed, cudaStream_t stream) {
  make_rotation_kernel<<<(n_quats + 127) / 128, 128, 0, stream>>>(rot, n_quats, seed);
  return cudaGetLastError();
}
cudaError_t launch_normalize_rotation(float* rot, int n_quats, cudaStream_t stream) {
  normalize_rotation_kernel<<<(n_quats + 127) / 128, 128, 0, stream>>>(rot, n_quats);
  return cudaGetLastError();
}

}  // namespace iq
