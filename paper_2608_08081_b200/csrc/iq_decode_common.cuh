// Device helpers shared by the decode kernels: tcgen05 / tensor-memory wrappers, the byte-lookup dequantisation of
// a packing unit, named barriers.
#pragma once
#include "iq_common.cuh"

namespace iq {

// Polls one mbarrier wait of the decode kernel may take before the kernel gives up (IQ_STATUS_WAIT_TIMEOUT): with the
// 20 us suspend hint of a poll that is at most 65536 * 20 us = 1.3 s (and a few milliseconds at least). Waits that
// work last microseconds. A thread that has given up skips every later wait, so a CTA returns within about that time
// after its first failed wait.
constexpr uint32_t DEC_WAIT_LIMIT = 1u << 16;

// ---------------------------------------------------------------------------------------------- tcgen05 wrappers
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ void tc_st16(uint32_t taddr, const uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};" ::"r"(taddr),
      "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]), "r"(r[10]),
      "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
}
__device__ __forceinline__ void tc_ld16(uint32_t taddr, float (&o)[16]) {
  uint32_t r[16];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
        "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
  tc_wait_ld();
#pragma unroll
  for (int i = 0; i < 16; i++) o[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tc_st8(uint32_t taddr, const uint32_t (&r)[8]) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]),
               "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7])
               : "memory");
}
// The same load without the wait: the registers are valid after tc_wait_ld().
__device__ __forceinline__ void tc_ld16_issue(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
        "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem descriptor]; fp16 operands, fp32 accumulate, M = 128, N and majors in idesc.
__device__ __forceinline__ void tc_mma_f16(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, {%5, %6, %7, %8}, p;\n\t}" ::"r"(d_tmem),
      "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(0), "r"(0), "r"(0), "r"(0)
      : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem descriptor]; int8 operands, int32 accumulate, K = 32 per instruction.
__device__ __forceinline__ void tc_mma_i8(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::i8 [%0], [%1], %2, %3, {%5, %6, %7, %8}, p;\n\t}" ::"r"(d_tmem),
      "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(0), "r"(0), "r"(0), "r"(0)
      : "memory");
}
__device__ __forceinline__ void tc_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// Shared-memory operand descriptor, MN-major, no swizzle: element (n, k) of a 16-bit operand sits at
// (n % 8) * 2 + (n / 8) * sbo + (k % 8) * 16 + (k / 8) * lbo bytes from the start address.
__device__ __forceinline__ uint64_t smem_desc_mn(uint32_t addr, uint32_t lbo, uint32_t sbo) {
  return (uint64_t)((addr >> 4) & 0x3FFFu) | ((uint64_t)(lbo >> 4) << 16) | ((uint64_t)(sbo >> 4) << 32) | (1ull << 46);
}
// Instruction descriptor: D = f32, A = B = f16, A K-major (TMEM), B MN-major, N = 16, M = 128.
constexpr uint32_t DEC_IDESC = (1u << 4) | (1u << 16) | ((16u >> 3) << 17) | ((128u >> 4) << 24);
// Integer path: D = s32, A = s8 (K-major, TMEM), B MN-major, N = 32, M = 128; B = s8 (query digits) or u8 (probability digits).
constexpr uint32_t DEC_IDESC_I8_SS = (2u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((32u >> 3) << 17) | ((128u >> 4) << 24);
constexpr uint32_t DEC_IDESC_I8_SU = (2u << 4) | (1u << 7) | (0u << 10) | (1u << 16) | ((32u >> 3) << 17) | ((128u >> 4) << 24);

// ---------------------------------------------------------------------------------------------- dequantisation
// x >> s for a compile-time s, computed as the high word of x * 2^(32-s): the multiply issues on the integer
// multiply-add pipe, which idles here, instead of the shift/logic pipe that carries the byte lookups.
template <int SH>
__device__ __forceinline__ uint32_t shr_mul(uint32_t x) {
  uint32_t hi;
  asm("{\n\t.reg .b64 t;\n\t.reg .b32 lo;\n\tmul.wide.u32 t, %1, %2;\n\tmov.b64 {lo, %0}, t;\n\t}" : "=r"(hi) : "r"(x), "n"(1u << (32 - SH)));
  return hi;
}
// Selectors of the 8 entries whose code bits sit in bit 3 of the nibbles of the unit's three words.
__device__ __forceinline__ uint32_t sliced_selectors(uint32_t w0, uint32_t w1, uint32_t w2) {
  return (shr_mul<3>(w0) & 0x11111111u) | (shr_mul<2>(w1) & 0x22222222u) | (shr_mul<1>(w2) & 0x44444444u);
}
// One packing unit (32 codes in 3 words) -> 16 registers of two fp16 levels each, entries in natural order:
// out[r] = (level[code 2r], level[code 2r+1]). Byte lookups with prmt: 8 levels x (low byte, high byte).
__device__ __forceinline__ void dequant_unit(uint32_t w0, uint32_t w1, uint32_t w2, uint32_t lo0, uint32_t lo1, uint32_t hi0,
                                             uint32_t hi1, uint32_t (&out)[16]) {
  const uint32_t sel[4] = {w0 & 0x77777777u, w1 & 0x77777777u, w2 & 0x77777777u, sliced_selectors(w0, w1, w2)};
#pragma unroll
  for (int k = 0; k < 4; k++)
#pragma unroll
    for (int hh = 0; hh < 2; hh++) {
      const uint32_t x = hh ? shr_mul<16>(sel[k]) : sel[k];
      const uint32_t l = prmt(lo0, lo1, x), h = prmt(hi0, hi1, x);
      out[4 * k + 2 * hh] = prmt(l, h, 0x5140u);
      out[4 * k + 2 * hh + 1] = prmt(l, h, 0x7362u);
    }
}

// Integer path: one packing unit -> 8 registers of four int8 levels each, entries in natural order (one prmt per 4 codes).
__device__ __forceinline__ void dequant_unit8(uint32_t w0, uint32_t w1, uint32_t w2, uint32_t l0, uint32_t l1, uint32_t* out) {
  const uint32_t sel[4] = {w0 & 0x77777777u, w1 & 0x77777777u, w2 & 0x77777777u, sliced_selectors(w0, w1, w2)};
#pragma unroll
  for (int k = 0; k < 4; k++) {
    out[2 * k] = prmt(l0, l1, sel[k]);
    out[2 * k + 1] = prmt(l0, l1, shr_mul<16>(sel[k]));
  }
}
// ---- the same for every bit width: 32 consecutive entries of a packed run (BITS words at w) -> natural order.
// b = 2: 16 entries per word, codes in the low (entries 0..7) and high (8..15) bit pair of the nibbles: one 4-byte table.
// b = 4: 8 entries per word; a byte permute selects among 8 bytes, so the 16 levels are two tables of 8, looked up with
// the low three bits of the code and chosen byte by byte with a mask made from its top bit.
__device__ __forceinline__ uint32_t byte_select(uint32_t lo, uint32_t hi, uint32_t mask) { return (hi & mask) | (lo & ~mask); }

template <int BITS>
__device__ __forceinline__ void dequant32_i8(const uint32_t* w, const uint32_t (&t)[4], uint32_t* out) {
  if constexpr (BITS == 3) {
    dequant_unit8(w[0], w[1], w[2], t[0], t[1], out);
  } else if constexpr (BITS == 2) {
#pragma unroll
    for (int j = 0; j < 2; j++) {
      const uint32_t a = w[j] & 0x33333333u, b = shr_mul<2>(w[j]) & 0x33333333u;
      out[4 * j] = prmt(t[0], t[0], a);
      out[4 * j + 1] = prmt(t[0], t[0], shr_mul<16>(a));
      out[4 * j + 2] = prmt(t[0], t[0], b);
      out[4 * j + 3] = prmt(t[0], t[0], shr_mul<16>(b));
    }
  } else {
#pragma unroll
    for (int j = 0; j < 4; j++) {
      const uint32_t s7 = w[j] & 0x77777777u, s3 = shr_mul<3>(w[j]) & 0x11111111u;
#pragma unroll
      for (int hh = 0; hh < 2; hh++) {
        const uint32_t x = hh ? shr_mul<16>(s7) : s7, mx = hh ? shr_mul<16>(s3) : s3;
        out[2 * j + hh] = byte_select(prmt(t[0], t[1], x), prmt(t[2], t[3], x), prmt(0x0000FF00u, 0u, mx));
      }
    }
  }
}

// fp16 levels: out[r] = (level[code 2r], level[code 2r+1]), 16 registers for the 32 entries.
template <int BITS>
__device__ __forceinline__ void dequant32_f16(const uint32_t* w, const uint32_t (&lo)[4], const uint32_t (&hi)[4], uint32_t (&out)[16]) {
  if constexpr (BITS == 3) {
    dequant_unit(w[0], w[1], w[2], lo[0], lo[1], hi[0], hi[1], out);
  } else {
    uint32_t sel[4], top[4];  // four selectors of 8 entries each (b = 4: and the top bits of their codes)
    if constexpr (BITS == 2) {
      sel[0] = w[0] & 0x33333333u; sel[1] = shr_mul<2>(w[0]) & 0x33333333u;
      sel[2] = w[1] & 0x33333333u; sel[3] = shr_mul<2>(w[1]) & 0x33333333u;
      top[0] = top[1] = top[2] = top[3] = 0u;
    } else {
#pragma unroll
      for (int k = 0; k < 4; k++) { sel[k] = w[k] & 0x77777777u; top[k] = shr_mul<3>(w[k]) & 0x11111111u; }
    }
#pragma unroll
    for (int k = 0; k < 4; k++)
#pragma unroll
      for (int hh = 0; hh < 2; hh++) {
        const uint32_t x = hh ? shr_mul<16>(sel[k]) : sel[k];
        uint32_t l, h;
        if constexpr (BITS == 2) {
          l = prmt(lo[0], lo[0], x);
          h = prmt(hi[0], hi[0], x);
        } else {
          const uint32_t m = prmt(0x0000FF00u, 0u, hh ? shr_mul<16>(top[k]) : top[k]);
          l = byte_select(prmt(lo[0], lo[1], x), prmt(lo[2], lo[3], x), m);
          h = byte_select(prmt(hi[0], hi[1], x), prmt(hi[2], hi[3], x), m);
        }
        out[4 * k + 2 * hh] = prmt(l, h, 0x5140u);
        out[4 * k + 2 * hh + 1] = prmt(l, h, 0x7362u);
      }
  }
}

// int32 -> float for |x| < 2^22, on the integer and FMA pipes (the conversion instruction runs at a quarter of their rate).
__device__ __forceinline__ float i2f_small(uint32_t x) { return __uint_as_float(x + 0x4B400000u) - 12582912.0f; }

// One lane of a converged warp. Issuing the MMAs / bulk copies from an elected lane of a converged warp keeps
// their operands in uniform registers; a lone divergent thread issues the same sequence about 3x slower.
__device__ __forceinline__ bool elect_one() {
  uint32_t pred;
  asm volatile("{\n\t.reg .pred p;\n\telect.sync _|p, 0xffffffff;\n\tselp.u32 %0, 1, 0, p;\n\t}" : "=r"(pred));
  return pred != 0;
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// Named barrier `id` over the 128 compute threads of one group, with an OR reduction.
__device__ __forceinline__ bool group_bar_or(int id, bool pred) {
  uint32_t r;
  asm volatile("{\n\t.reg .pred p, q;\n\tsetp.ne.u32 q, %2, 0;\n\tbarrier.red.or.pred p, %1, 128, q;\n\tselp.u32 %0, 1, 0, p;\n\t}"
               : "=r"(r) : "r"(id), "r"((uint32_t)pred) : "memory");
  return r != 0;
}
// Barrier 0 over the whole CTA, for the places where the control and the compute warps arrive from different code.
__device__ __forceinline__ void cta_bar_sync() { asm volatile("barrier.sync 0;" ::: "memory"); }
// Named barrier `id` over `count` threads (a multiple of 32).
__device__ __forceinline__ void cta_bar_sync_n(int id, int count) { asm volatile("barrier.sync %0, %1;" ::"r"(id), "r"(count) : "memory"); }
__device__ __forceinline__ void group_bar_sync(int id) { asm volatile("barrier.sync %0, 128;" ::"r"(id) : "memory"); }

__device__ __forceinline__ float max3f(float a, float b, float c) {
  float r;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
  return r;
}
// Reduction of 8 values per lane over the 32 lanes of a warp with 9 shuffles instead of 40: the lanes first trade
// halves of their value sets (xor 16: four values each way, xor 8: two, xor 4: one), so that lane l ends up with one
// value of head warp_reduce8_head(l), which two more butterfly steps complete. Every lane gets the result of its head.
__device__ __forceinline__ int warp_reduce8_head(int lane) { return ((lane >> 4) & 1) * 4 + ((lane >> 3) & 1) * 2 + ((lane >> 2) & 1); }
template <typename OP>
__device__ __forceinline__ float warp_reduce8(const float (&v)[8], int lane, OP op) {
  const bool b4 = lane & 16, b3 = lane & 8, b2 = lane & 4;
  float a[4], c[2];
#pragma unroll
  for (int i = 0; i < 4; i++) a[i] = op(b4 ? v[i + 4] : v[i], __shfl_xor_sync(FULL, b4 ? v[i] : v[i + 4], 16));
#pragma unroll
  for (int i = 0; i < 2; i++) c[i] = op(b3 ? a[i + 2] : a[i], __shfl_xor_sync(FULL, b3 ? a[i] : a[i + 2], 8));
  float r = op(b2 ? c[1] : c[0], __shfl_xor_sync(FULL, b2 ? c[0] : c[1], 4));
  r = op(r, __shfl_xor_sync(FULL, r, 2));
  return op(r, __shfl_xor_sync(FULL, r, 1));
}
// The same for (value, row) pairs: the larger value wins, the lower row among equal values (rows < 0 mean "none").
__device__ __forceinline__ void argmax_merge(float& bv, int& bi, float ov, int oi) {
  if (ov > bv || (ov == bv && oi >= 0 && (bi < 0 || oi < bi))) { bv = ov; bi = oi; }
}
__device__ __forceinline__ void warp_argmax8(const float (&v)[8], const int (&ix)[8], int lane, float& rv, int& ri) {
  const bool b4 = lane & 16, b3 = lane & 8, b2 = lane & 4;
  float a[4], c[2];
  int ai[4], ci[2];
#pragma unroll
  for (int i = 0; i < 4; i++) {
    a[i] = b4 ? v[i + 4] : v[i];
    ai[i] = b4 ? ix[i + 4] : ix[i];
    argmax_merge(a[i], ai[i], __shfl_xor_sync(FULL, b4 ? v[i] : v[i + 4], 16), __shfl_xor_sync(FULL, b4 ? ix[i] : ix[i + 4], 16));
  }
#pragma unroll
  for (int i = 0; i < 2; i++) {
    c[i] = b3 ? a[i + 2] : a[i];
    ci[i] = b3 ? ai[i + 2] : ai[i];
    argmax_merge(c[i], ci[i], __shfl_xor_sync(FULL, b3 ? a[i] : a[i + 2], 8), __shfl_xor_sync(FULL, b3 ? ai[i] : ai[i + 2], 8));
  }
  rv = b2 ? c[1] : c[0];
  ri = b2 ? ci[1] : ci[0];
  argmax_merge(rv, ri, __shfl_xor_sync(FULL, b2 ? c[0] : c[1], 4), __shfl_xor_sync(FULL, b2 ? ci[0] : ci[1], 4));
  argmax_merge(rv, ri, __shfl_xor_sync(FULL, rv, 2), __shfl_xor_sync(FULL, ri, 2));
  argmax_merge(rv, ri, __shfl_xor_sync(FULL, rv, 1), __shfl_xor_sync(FULL, ri, 1));
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(FULL, v, o));
  return v;
}

}  // namespace iq
