// Shared device helpers of the IsoQuant CUDA library: warp-level Walsh-Hadamard butterfly, SO(4) blocks
// from quaternion pairs (Eq. 2; Section 3.3; Appendix B), PTX wrappers. Device code only.
#pragma once
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/isoquant.h"
#include "iq_kernels.h"

namespace iq {

constexpr unsigned FULL = 0xffffffffu;

// ------------------------------------------------------------------------------------------------
// SO(4) block: the 4x4 matrix of v -> q_L v conj(q_R), as the product of the left-multiplication matrix
// of q_L and the right-multiplication matrix of conj(q_R) (Section 3.3, "SO(4) parameterization").
// q8 = (q_L.wxyz, q_R.wxyz); both are rescaled to unit length in the working precision T.
// ------------------------------------------------------------------------------------------------
template <typename T>
__device__ __forceinline__ void so4_matrix(const float* q8, T (&M)[4][4]) {
  T a = q8[0], b = q8[1], c = q8[2], d = q8[3];
  T e = q8[4], f = q8[5], g = q8[6], h = q8[7];
  T nl = T(1) / sqrt(a * a + b * b + c * c + d * d);
  T nr = T(1) / sqrt(e * e + f * f + g * g + h * h);
  a *= nl; b *= nl; c *= nl; d *= nl;
  e *= nr; f *= nr; g *= nr; h *= nr;
  const T L[4][4] = {{a, -b, -c, -d}, {b, a, -d, c}, {c, d, a, -b}, {d, -c, b, a}};
  const T R[4][4] = {{e, f, g, h}, {-f, e, -h, g}, {-g, h, e, -f}, {-h, -g, f, e}};
#pragma unroll
  for (int i = 0; i < 4; i++)
#pragma unroll
    for (int j = 0; j < 4; j++) {
      T s = 0;
#pragma unroll
      for (int k = 0; k < 4; k++) s += L[i][k] * R[k][j];
      M[i][j] = s;
    }
}

template <typename T>
__device__ __forceinline__ T shfl_xor_t(T v, int mask);
template <>
__device__ __forceinline__ float shfl_xor_t<float>(float v, int mask) { return __shfl_xor_sync(FULL, v, mask); }
template <>
__device__ __forceinline__ double shfl_xor_t<double>(double v, int mask) { return __shfl_xor_sync(FULL, v, mask); }

// ------------------------------------------------------------------------------------------------
// Unnormalised Walsh-Hadamard transform (natural order) of a vector of 32*E coordinates spread over a
// warp: lane l holds coordinates l*E .. l*E+E-1. Strides 1 .. E/2 are butterflies inside the lane,
// strides E .. 16E are xor-shuffles (lane bit b <-> stride E << b). d log2 d adds in total (Section 3.2,
// rotation cost analysis).
// ------------------------------------------------------------------------------------------------
template <typename T, int E>
__device__ __forceinline__ void wht_warp(T (&v)[E], int lane) {
#pragma unroll
  for (int s = 1; s < E; s <<= 1) {
#pragma unroll
    for (int i = 0; i < E; i++) {
      if ((i & s) == 0) {
        T x = v[i], y = v[i + s];
        v[i] = x + y;
        v[i + s] = x - y;
      }
    }
  }
#pragma unroll
  for (int b = 0; b < 5; b++) {
    const bool upper = (lane >> b) & 1;
#pragma unroll
    for (int i = 0; i < E; i++) {
      T o = shfl_xor_t<T>(v[i], 1 << b);
      v[i] = upper ? (o - v[i]) : (v[i] + o);
    }
  }
}

// y = M x (or M^T x) for the E/4 blocks a lane owns.
template <typename T, int E, bool TRANSPOSE>
__device__ __forceinline__ void so4_apply(const T (&M)[E / 4][4][4], T (&v)[E]) {
#pragma unroll
  for (int j = 0; j < E / 4; j++) {
    T x0 = v[4 * j], x1 = v[4 * j + 1], x2 = v[4 * j + 2], x3 = v[4 * j + 3];
#pragma unroll
    for (int r = 0; r < 4; r++) {
      if (TRANSPOSE)
        v[4 * j + r] = M[j][0][r] * x0 + M[j][1][r] * x1 + M[j][2][r] * x2 + M[j][3][r] * x3;
      else
        v[4 * j + r] = M[j][r][0] * x0 + M[j][r][1] * x1 + M[j][r][2] * x2 + M[j][r][3] * x3;
    }
  }
}

// ------------------------------------------------------------------------------------------------
// PTX wrappers
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
  uint32_t d;
  asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
  return d;
}

__device__ __forceinline__ float ex2f(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ uint32_t pack_half2(float lo, float hi) {
  uint32_t d;
  asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
  return d;
}

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
// One poll of the barrier phase. The hint lets the hardware keep the thread suspended (it is woken when the phase
// completes) instead of returning early, so that waiting warps do not spend issue slots on the polling loop.
// Programmatic dependent launch. Every kernel of the library is launched so that it may start while the kernel
// before it on the stream is still finishing (launch_after_predecessor below) and therefore begins with
// grid_dependency_wait(): nothing that a predecessor may have written -- lengths, queries, new rows, the cache, the
// partials -- is read before it. The wait returns once the preceding grid has completed and its writes are visible
// (at once for a launch without the attribute). allow_dependent_launch() lets the next kernel's CTAs become resident
// and block in their own wait. It is called after the wait (the decode kernel: after its main loop), so at most the
// tail of one kernel overlaps the start of the next: calling it first thing, which lets the launches of a whole
// step pile up behind a running decode kernel, measured 2-9 % slower per step. Since each kernel waits for its
// direct predecessor and cannot complete before its own wait has returned, kernels further back have completed too.
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void allow_dependent_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename Params>
inline cudaError_t launch_after_predecessor(void (*kernel)(Params), dim3 grid, dim3 block, size_t smem_bytes, cudaStream_t stream,
                                            const Params& p) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem_bytes;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, p);
}

// Where cache row t of (sequence b, KV head g) sits in the cache arrays, in rows. Contiguous cache: the arrays are
// [batch][n_kv_heads][t_cap]. Paged cache: a pool [num_pages][n_kv_heads][page_rows] and a table [batch][t_cap /
// page_rows] of page numbers; page_rows is a multiple of 128, so a 128-row block never straddles two pages and the
// row index of a block's first row, times the row size, is also where its token-transposed V records start.
__device__ __forceinline__ size_t cache_row(const PageMap& m, int b, int g, long long t, uint32_t* status) {
  if (m.table == nullptr) return ((size_t)b * m.n_kv_heads + g) * (size_t)m.t_cap + (size_t)t;
  const int j = (int)t / m.page_rows;  // (t < t_cap: 32-bit arithmetic)
  int page = m.table[(size_t)b * (m.t_cap / m.page_rows) + j];
  if ((unsigned)page >= (unsigned)m.num_pages) {  // never turned into an address: flagged and read as page 0
    if (status) atomicOr(&status[0], IQ_STATUS_BAD_PAGE);
    page = 0;
  }
  return ((size_t)page * m.n_kv_heads + g) * (size_t)m.page_rows + (size_t)(t - (long long)j * m.page_rows);
}

// The same for a kernel that WRITES the row. A block-table entry outside the pool must not redirect the write to
// another page (page 0 may belong to another sequence): the function then returns false and sets IQ_STATUS_BAD_PAGE;
// the caller skips the row and counts it.
__device__ __forceinline__ bool cache_row_for_write(const PageMap& m, int b, int g, long long t, uint32_t* status, size_t& row) {
  if (m.table != nullptr) {
    const int page = m.table[(size_t)b * (m.t_cap / m.page_rows) + (int)t / m.page_rows];
    if ((unsigned)page >= (unsigned)m.num_pages) {
      if (status) atomicOr(&status[0], IQ_STATUS_BAD_PAGE);
      return false;
    }
  }
  row = cache_row(m, b, g, t, status);
  return true;
}

// The scale arrays hold fp32 values or (f16 != 0) binary16 values of the same shape.
__device__ __forceinline__ void store_scale(float* arr, size_t row, float s, int f16, uint32_t* status) {
  if (!f16) {
    arr[row] = s;
  } else {
    if (s > 65504.f) {
      if (status) atomicOr(&status[0], IQ_STATUS_SCALE_OVERFLOW);
      s = 65504.f;
    }
    reinterpret_cast<__half*>(arr)[row] = __float2half_rn(s);
  }
}
__device__ __forceinline__ float load_scale(const void* arr, size_t row, int f16) {
  return f16 ? __half2float(reinterpret_cast<const __half*>(arr)[row]) : reinterpret_cast<const float*>(arr)[row];
}

#ifndef IQ_MBAR_SUSPEND_NS
#define IQ_MBAR_SUSPEND_NS 20000
#endif
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity), "r"((uint32_t)IQ_MBAR_SUSPEND_NS)
      : "memory");
  return ok != 0;
}
// Bounded wait: gives up after `limit` polls and reports false (the caller flags the error and unwinds). A poll that
// does not find the phase complete suspends the thread for at most IQ_MBAR_SUSPEND_NS, so `limit` polls last at most
// limit * IQ_MBAR_SUSPEND_NS (plus the polls' own latency) and at least limit times the latency of a poll (tens of
// nanoseconds). The loop is kept this plain on purpose: a timer read or an out-of-line call in it measurably slows
// the kernels that wait, whose waits all succeed.
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity, uint32_t limit) {
  for (uint32_t i = 0; i < limit; i++)
    if (mbar_try_wait(bar, parity)) return true;
  return false;
}
// 1-D bulk asynchronous copy global -> shared, completion counted in bytes on an mbarrier. Both addresses
// 16-byte aligned, size a multiple of 16 bytes.
__device__ __forceinline__ void bulk_g2s(void* dst_smem, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                   smem_u32(dst_smem)),
               "l"(src), "r"(bytes), "r"(smem_u32(bar))
               : "memory");
}
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void fence_mbar_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }

}  // namespace iq
