// Fused decode kernel (Appendix A; Table 2 kernels A, B, C): scores on packed K codes, split-K online
// softmax, value accumulation on packed V codes, on the 5th-generation tensor cores (tcgen05) with the
// dequantised operands resident in tensor memory (TMEM).
//
// One CTA of 128 threads per (context split, KV head x head group, sequence); the CTA walks its chunk in
// blocks of 128 cached rows. Per block:
//   1. thread r dequantises packed K row r (its own 3d/8 bytes from the staged tile) into fp16 and stores it
//      to TMEM lane r: A_K[128 rows x d].
//   2. one thread issues tcgen05.mma (M = 128 rows, N = 16, K = 16 per instruction):
//         S[row][n] = sum_i A_K[row][i] * B_Q[n][i],  B_Q = q~ of the <= 8 heads as fp16 hi (n < 8) and lo (n >= 8)
//   3. every thread reads its row of S back, applies the K scale, joins the block-wide running maximum and
//      writes its probabilities (times the V scale, again as fp16 hi / lo) into the shared-memory operand
//      B_P[n][row].
//   4. thread c dequantises coordinate c of the token-transposed V block (128 codes = one 48-byte row) into
//      TMEM lane c: A_V[d coords x 128 rows]; one thread issues
//         O[c][n] = sum_row A_V[c][row] * B_P[n][row]
//   5. thread c folds O (hi + lo columns) into its running accumulator for coordinate c.
// Packed tiles arrive through a 1-D bulk-copy (TMA) pipeline; every wait is bounded.
#include "iq_common.cuh"
#include "iq_kernels.h"

namespace iq {

// Tuning knob: 1 = the K and V operand tiles share TMEM columns at d = 128 (4 CTAs per SM, measured fastest),
// 0 = separate tiles (3 CTAs per SM, the dequantisation of one tile overlaps the MMAs on the other).
#ifndef IQ_DEC_SHARED128
#define IQ_DEC_SHARED128 1
#endif
constexpr int DEC_COMPUTE_THREADS = 128;  // 4 warps: dequantisation, softmax, accumulation (thread = TMEM lane)
constexpr int DEC_THREADS = 160;          // + 1 control warp: issues the bulk copies and the MMAs
constexpr uint32_t DEC_WAIT_LIMIT = 1u << 22;
constexpr int DEC_HDR_BYTES = 1024;  // barriers, TMEM base, cross-warp scratch
constexpr float DEC_MAX_SLACK = 4.0f;  // log2 units a score may exceed the running reference before it is raised

template <int D>
struct DecLayout {
  static constexpr int DJ = D / 128;
  static constexpr int WPR = 3 * D / 32;  // 32-bit words per packed K row
  static constexpr int ROWB = WPR * 4;
  static constexpr int K_BYTES = DEC_BLOCK_TOKENS * ROWB;
  static constexpr int VT_BYTES = D * 48;  // token-transposed V block: one 48-byte row (128 codes) per coordinate
  static constexpr int SC_BYTES = DEC_BLOCK_TOKENS * 4;
  static constexpr int STAGE_BYTES = K_BYTES + VT_BYTES + 2 * SC_BYTES;
  static constexpr int BQ_BYTES = 16 * D * 2;
  static constexpr int BP_BYTES = 16 * DEC_BLOCK_TOKENS * 2;
  // TMEM. Separate tiles (d = 128 default): the K tile and the V tile have their own 64 columns each (allocation
  // 0, 128 columns) and the fp32 results live in a second allocation of 32 columns, so that 3 CTAs fit the SM's
  // 512 columns and the dequantisation of one tile overlaps the MMAs on the other. Shared tile (d = 256): one
  // allocation, the K and V tiles share columns (the kernel then waits for the MMAs that read a tile before
  // overwriting it).
  static constexpr bool SHARED_A = (D != 128) || (IQ_DEC_SHARED128 != 0);
  static constexpr int CTAS_PER_SM = (D == 128) ? (SHARED_A ? 4 : 3) : 2;
  static constexpr int STAGES = (D == 128 && !SHARED_A) ? 4 : 3;
  static constexpr int SMEM_BYTES = DEC_HDR_BYTES + BQ_BYTES + BP_BYTES + STAGES * STAGE_BYTES;
  static constexpr int ALLOC0_COLS = SHARED_A ? D : 128;
  static constexpr int ALLOC1_COLS = SHARED_A ? 0 : 32;
  static constexpr int AK_COL = 0;
  static constexpr int AV_COL = SHARED_A ? 0 : 64;
  static constexpr int S_COL = SHARED_A ? D / 2 : 0;    // in allocation 1 when it exists
  static constexpr int O_COL = SHARED_A ? D / 2 + 16 : 16;
};
static_assert(DEC_BLOCK_TOKENS == 128, "the TMEM operand layout assumes 128-row blocks");

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
// D[tmem] (+)= A[tmem] * B[smem descriptor]; fp16 operands, fp32 accumulate, M = 128, N and majors in idesc.
__device__ __forceinline__ void tc_mma_f16(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, {%5, %6, %7, %8}, p;\n\t}" ::"r"(d_tmem),
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
// Named barrier 1 over the 128 compute threads (the control warp does not take part), with an OR reduction.
__device__ __forceinline__ bool compute_bar_or(bool pred) {
  uint32_t r;
  asm volatile("{\n\t.reg .pred p, q;\n\tsetp.ne.u32 q, %1, 0;\n\tbarrier.red.or.pred p, 1, 128, q;\n\tselp.u32 %0, 1, 0, p;\n\t}"
               : "=r"(r) : "r"((uint32_t)pred) : "memory");
  return r != 0;
}
__device__ __forceinline__ void compute_bar_sync() { asm volatile("barrier.sync 1, 128;" ::: "memory"); }

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(FULL, v, o));
  return v;
}

template <int D, bool ARGMAX>
__global__ void __launch_bounds__(DEC_THREADS, DecLayout<D>::CTAS_PER_SM) decode_kernel(const DecodeParams p) {
  using L = DecLayout<D>;
  constexpr int DJ = L::DJ;
  constexpr int E = D / 32;
  constexpr int TB = DEC_BLOCK_TOKENS;
  constexpr int NST = L::STAGES;
  constexpr float LOG2E = 1.4426950408889634f;
  constexpr float LN2 = 0.6931471805599453f;

  extern __shared__ __align__(1024) uint8_t smem[];
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem);     // [stages]
  uint64_t* s_bar = reinterpret_cast<uint64_t*>(smem + 64);   // scores ready
  uint64_t* o_bar = reinterpret_cast<uint64_t*>(smem + 72);   // values ready
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + 80);  // [2] bases of the TMEM allocations
  uint64_t* k_ready = reinterpret_cast<uint64_t*>(smem + 88);   // K tile in TMEM (128 arrivals)
  uint64_t* p_ready = reinterpret_cast<uint64_t*>(smem + 96);   // V tile in TMEM + probabilities in smem (128 arrivals)
  uint64_t* empty_bar = reinterpret_cast<uint64_t*>(smem + 32);  // [stages] staged tile consumed (128 arrivals)
  float* red = reinterpret_cast<float*>(smem + 128);          // [4 warps][8 heads] cross-warp scratch
  float* red2 = red + 32;                                     // second scratch (maxima)
  int* redi = reinterpret_cast<int*>(red2 + 32);              // argmax rows
  uint8_t* bq = smem + DEC_HDR_BYTES;                         // B_Q: (n, i) MN-major
  uint8_t* bp = bq + L::BQ_BYTES;                             // B_P: (n, row) MN-major
  uint8_t* stages = bp + L::BP_BYTES;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int split = blockIdx.x;
  const int kvh = blockIdx.y / p.head_groups;
  const int hg = blockIdx.y - kvh * p.head_groups;
  const int S = p.splits;
  // Longest sequences first: CTAs are dispatched in order of blockIdx (z slowest), so slice z of the grid takes the
  // sequence with the z-th largest length and the short chunks fill the tail of the launch. Every thread ranks one
  // sequence (ties by index); batches larger than the CTA keep the identity order.
  int b = blockIdx.z;
  if (p.batch > 1 && p.batch <= DEC_THREADS) {
    int* b_slot = reinterpret_cast<int*>(smem + 120);
    if (tid < p.batch) {
      const int mine = p.seq_lens[tid];
      int rank = 0;
      for (int o = 0; o < p.batch; o++) {
        const int other = p.seq_lens[o];
        rank += (other > mine) || (other == mine && o < tid);
      }
      if (rank == (int)blockIdx.z) *b_slot = tid;
    }
    __syncthreads();
    b = *b_slot;
  }

  const int len = max(0, min(p.seq_lens[b], p.t_cap));
  const int per = (len + S - 1) / S;
  const int chunk = ((per + TB - 1) / TB) * TB;
  const int start = split * chunk;
  const int end = min(len, start + chunk);
  const int h0 = kvh * p.group + hg * DEC_HEADS;
  const int nh = min(DEC_HEADS, p.group - hg * DEC_HEADS);

  if (start >= end) {  // empty chunk: (m, l) = (-inf, 0), acc = 0
    for (int idx = tid; idx < nh * D; idx += DEC_THREADS) {
      const int head = idx / D, c = idx - head * D;
      p.part_acc[(((size_t)b * p.n_q_heads + h0 + head) * S + split) * D + c] = 0.f;
    }
    if (tid < nh) {
      const size_t o = ((size_t)b * p.n_q_heads + h0 + tid) * S + split;
      p.part_ml[2 * o] = -INFINITY;
      p.part_ml[2 * o + 1] = 0.f;
      if (ARGMAX) p.part_argmax[o] = -1;
    }
    return;
  }

  // ---------------------------------------------------------------- set-up: barriers, TMEM, tile pipeline
  const size_t slab = ((size_t)b * p.n_kv_heads + kvh) * (size_t)p.t_cap;  // row index of this (sequence, KV head)
  const int nblk = (end - start + TB - 1) / TB;
  const bool control = (warp == 4);
  auto issue = [&](int blk) {  // elected lane of the control warp only
    const int st = blk % NST;
    const int r0 = start + blk * TB;
    const int n = min(TB, end - r0);
    const int n4 = (n + 3) & ~3;
    uint8_t* sp = stages + st * L::STAGE_BYTES;
    mbar_expect_tx(&full_bar[st], (uint32_t)(n * L::ROWB + L::VT_BYTES + 2 * n4 * 4));
    bulk_g2s(sp, p.k_codes + (slab + r0) * L::ROWB, (uint32_t)(n * L::ROWB), &full_bar[st]);
    bulk_g2s(sp + L::K_BYTES, p.v_codes + (slab + r0) * L::ROWB, (uint32_t)L::VT_BYTES, &full_bar[st]);  // whole 128-row V block
    bulk_g2s(sp + L::K_BYTES + L::VT_BYTES, p.k_scales + slab + r0, (uint32_t)(n4 * 4), &full_bar[st]);
    bulk_g2s(sp + L::K_BYTES + L::VT_BYTES + L::SC_BYTES, p.v_scales + slab + r0, (uint32_t)(n4 * 4), &full_bar[st]);
  };
  if (control && elect_one()) {
#pragma unroll
    for (int st = 0; st < NST; st++) { mbar_init(&full_bar[st], 1); mbar_init(&empty_bar[st], DEC_COMPUTE_THREADS); }
    mbar_init(s_bar, 1);
    mbar_init(o_bar, 1);
    mbar_init(k_ready, DEC_COMPUTE_THREADS);
    mbar_init(p_ready, DEC_COMPUTE_THREADS);
    fence_mbar_init();
    fence_proxy_async();
    for (int blk = 0; blk < NST && blk < nblk; blk++) issue(blk);
  }
  if (control) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(L::ALLOC0_COLS));
    if (L::ALLOC1_COLS > 0)
      asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot + 1)), "r"(L::ALLOC1_COLS));
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::);
  }

  // ---------------------------------------------------------------- d1: q~ = R q, written as the operand B_Q
  if (!control) {
    float M[E / 4][4][4];
    const float* qb = p.rot + ((size_t)kvh * (D / 4) + (size_t)lane * (E / 4)) * 8;
#pragma unroll
    for (int j = 0; j < E / 4; j++) so4_matrix<float>(qb + 8 * j, M[j]);
    const float inv_root_d = rsqrtf((float)D);
    for (int hh = warp; hh < DEC_HEADS; hh += 4) {
      float v[E];
      if (hh < nh) {
        const __half* src = p.q + ((size_t)b * p.n_q_heads + h0 + hh) * D + lane * E;
#pragma unroll
        for (int e = 0; e < E; e++) v[e] = __half2float(src[e]);
        wht_warp<float, E>(v, lane);
        so4_apply<float, E, false>(M, v);
      } else {
#pragma unroll
        for (int e = 0; e < E; e++) v[e] = 0.f;
      }
#pragma unroll
      for (int e = 0; e < E; e++) {
        const float x = v[e] * inv_root_d;
        const __half xh = __float2half_rn(x);
        const __half xl = __float2half_rn(x - __half2float(xh));
        const int i = lane * E + e;  // contraction index = rotated coordinate
        const int off = (i & 7) * 16 + (i >> 3) * 128;
        *reinterpret_cast<__half*>(bq + (hh & 7) * 2 + off) = xh;                  // n = head (hi part)
        *reinterpret_cast<__half*>(bq + (hh & 7) * 2 + (D / 8) * 128 + off) = xl;  // n = 8 + head (lo part)
      }
    }
  }
  fence_proxy_async();  // B_Q was written through the generic proxy, the tensor core reads it through the async proxy
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_a = tmem_slot[0];
  const uint32_t tmem_r = (L::ALLOC1_COLS > 0) ? tmem_slot[1] : tmem_slot[0];  // base of the fp32 result columns
  const uint32_t lane_sel = (uint32_t)((warp & 3) * 32) << 16;  // this warp's 32 TMEM lanes

  float acc[DJ][8];  // thread c: coordinates c (+128), 8 heads
#pragma unroll
  for (int j = 0; j < DJ; j++)
#pragma unroll
    for (int h = 0; h < 8; h++) acc[j][h] = 0.f;
  float m_run[8], l_run[8], best_v[8], alpha[8];
  int best_i[8];
#pragma unroll
  for (int h = 0; h < 8; h++) { m_run[h] = -INFINITY; l_run[h] = 0.f; best_v[h] = -INFINITY; best_i[h] = -1; alpha[h] = 1.f; }
  bool failed = false;

  if (control) {
    // ================================================================ control warp: issues MMAs and tile refills.
    // All 32 lanes run the loop and the waits; an elected lane issues.
    const uint32_t bq_addr = smem_u32(bq), bp_addr = smem_u32(bp);
    for (int blk = 0; blk < nblk; blk++) {
      // scores of block blk: S = A_K * B_Q^T once all 128 rows are in TMEM
      if (!failed) failed = !mbar_wait_bounded(k_ready, (uint32_t)blk & 1u, DEC_WAIT_LIMIT);
      tc_fence_after();
      if (elect_one()) {
#pragma unroll
        for (int kk = 0; kk < D / 16; kk++)
          tc_mma_f16(tmem_r + L::S_COL, tmem_a + L::AK_COL + 8 * kk, smem_desc_mn(bq_addr + kk * 256, 128, (D / 8) * 128), DEC_IDESC, kk > 0);
        tc_commit(s_bar);
      }
      __syncwarp();
      // values of block blk: O = A_V * B_P^T once the V tile is in TMEM and the probabilities are in shared memory
      if (!failed) failed = !mbar_wait_bounded(p_ready, (uint32_t)blk & 1u, DEC_WAIT_LIMIT);
      tc_fence_after();
      if (elect_one()) {
#pragma unroll
        for (int j = 0; j < DJ; j++)
#pragma unroll
          for (int kk = 0; kk < TB / 16; kk++)
            tc_mma_f16(tmem_r + L::O_COL + 16 * j, tmem_a + L::AV_COL + 64 * j + 8 * kk,
                       smem_desc_mn(bp_addr + kk * 256, 128, (TB / 8) * 128), DEC_IDESC, kk > 0);
        tc_commit(o_bar);
      }
      __syncwarp();
      // the compute threads released the stage when they signalled p_ready: refill it
      if (blk + NST < nblk) {
        if (!failed) failed = !mbar_wait_bounded(&empty_bar[blk % NST], (uint32_t)(blk / NST) & 1u, DEC_WAIT_LIMIT);
        if (elect_one()) {
          fence_proxy_async();
          issue(blk + NST);
        }
        __syncwarp();
      }
    }
  } else {
    // ================================================================ compute warps
    const uint32_t lut_lo0 = p.lut_lo[0], lut_lo1 = p.lut_lo[1], lut_hi0 = p.lut_hi[0], lut_hi1 = p.lut_hi[1];
    const float kfac = p.sm_scale * LOG2E * rsqrtf((float)D);  // scores in log2 units: z2 = S_raw * scale_K * kfac
    const float vfac = rsqrtf((float)D);

    // K row tid of the staged tile -> TMEM lane tid (A_K), then signal the control warp.
    auto k_phase = [&](int blk) {
      const uint8_t* sp = stages + (blk % NST) * L::STAGE_BYTES;
      if (!failed) failed = !mbar_wait_bounded(&full_bar[blk % NST], (uint32_t)(blk / NST) & 1u, DEC_WAIT_LIMIT);
      uint32_t w[L::WPR];
      const uint4* krow = reinterpret_cast<const uint4*>(sp + tid * L::ROWB);
#pragma unroll
      for (int i = 0; i < L::WPR / 4; i++) {
        const uint4 t4 = krow[i];
        w[4 * i] = t4.x; w[4 * i + 1] = t4.y; w[4 * i + 2] = t4.z; w[4 * i + 3] = t4.w;
      }
#pragma unroll
      for (int u = 0; u < 4 * DJ; u++) {
        uint32_t f[16];
        dequant_unit(w[3 * u], w[3 * u + 1], w[3 * u + 2], lut_lo0, lut_lo1, lut_hi0, lut_hi1, f);
        tc_st16(tmem_a + lane_sel + L::AK_COL + 16 * u, f);
      }
      tc_wait_st();
      tc_fence_before();
      mbar_arrive(k_ready);
    };
    // Fold the value product of block `blk` (ready on o_bar) into the running accumulator.
    auto fold = [&](int blk) {
      if (!failed) failed = !mbar_wait_bounded(o_bar, (uint32_t)blk & 1u, DEC_WAIT_LIMIT);
      tc_fence_after();
#pragma unroll
      for (int j = 0; j < DJ; j++) {
        float o[16];
        tc_ld16(tmem_r + lane_sel + L::O_COL + 16 * j, o);
#pragma unroll
        for (int h = 0; h < 8; h++) acc[j][h] = acc[j][h] * alpha[h] + (o[h] + o[8 + h]);
      }
      tc_fence_before();
    };

    k_phase(0);
    bool folded = true;  // is the value product of the previous block already in acc?
    for (int blk = 0; blk < nblk; blk++) {
      const uint8_t* sp = stages + (blk % NST) * L::STAGE_BYTES;
      const int r0 = start + blk * TB;
      const int n = min(TB, end - r0);
      if (L::SHARED_A) {  // the score MMAs read the tile that the V dequantisation is about to overwrite
        if (!failed) failed = !mbar_wait_bounded(s_bar, (uint32_t)blk & 1u, DEC_WAIT_LIMIT);
      }
      if (!folded) { fold(blk - 1); folded = true; }  // also: the value MMAs of the previous block have released A_V and B_P

      // ---- V coordinate tid (+128) of this block -> TMEM lane tid (A_V), while the score MMAs run
#pragma unroll
      for (int j = 0; j < DJ; j++) {
        const uint4* vrow = reinterpret_cast<const uint4*>(sp + L::K_BYTES + (tid + 128 * j) * 48);
        uint32_t w[12];
#pragma unroll
        for (int i = 0; i < 3; i++) {
          const uint4 t4 = vrow[i];
          w[4 * i] = t4.x; w[4 * i + 1] = t4.y; w[4 * i + 2] = t4.z; w[4 * i + 3] = t4.w;
        }
#pragma unroll
        for (int u = 0; u < 4; u++) {
          uint32_t f[16];
          dequant_unit(w[3 * u], w[3 * u + 1], w[3 * u + 2], lut_lo0, lut_lo1, lut_hi0, lut_hi1, f);
          tc_st16(tmem_a + lane_sel + L::AV_COL + 64 * j + 16 * u, f);
        }
      }
      const float ksc = reinterpret_cast<const float*>(sp + L::K_BYTES + L::VT_BYTES)[tid];
      const float vsc = reinterpret_cast<const float*>(sp + L::K_BYTES + L::VT_BYTES + L::SC_BYTES)[tid];

      // ---- online softmax (log2 units); thread tid owns row r0 + tid, all 8 heads
      if (!L::SHARED_A) {
        if (!failed) failed = !mbar_wait_bounded(s_bar, (uint32_t)blk & 1u, DEC_WAIT_LIMIT);
      }
      tc_fence_after();
      float s[8];
      {
        float raw[16];
        tc_ld16(tmem_r + lane_sel + L::S_COL, raw);
        const bool valid = tid < n;  // rows >= n of the last block hold stale bytes
        const float kf = valid ? ksc * kfac : 0.f;
#pragma unroll
        for (int h = 0; h < 8; h++) s[h] = valid ? (raw[h] + raw[8 + h]) * kf : -INFINITY;
      }
#pragma unroll
      for (int h = 0; h < 8; h++) {  // exact maximum seen by this thread (the partial's m) and, optionally, its row
        if (ARGMAX) {
          if (s[h] > best_v[h]) { best_v[h] = s[h]; best_i[h] = r0 + tid; }
        } else {
          best_v[h] = fmaxf(best_v[h], s[h]);
        }
      }
      // The running reference m_run is raised only when some score of the block exceeds it by more than
      // DEC_MAX_SLACK (log2 units): exp2(s - m_run) then stays below 2^DEC_MAX_SLACK and nothing has to be
      // exchanged between the warps in the common case (one barrier with an OR reduction).
      bool exceed = false;
#pragma unroll
      for (int h = 0; h < 8; h++) exceed |= (s[h] - m_run[h] > DEC_MAX_SLACK);
      if (compute_bar_or(exceed)) {
#pragma unroll
        for (int h = 0; h < 8; h++) {
          const float wm = warp_max(s[h]);
          if (lane == h) red[warp * 8 + h] = wm;
        }
        compute_bar_sync();
#pragma unroll
        for (int h = 0; h < 8; h++) {
          const float bm = fmaxf(fmaxf(red[h], red[8 + h]), fmaxf(red[16 + h], red[24 + h]));
          const float mn = fmaxf(m_run[h], bm);
          alpha[h] = ex2f(m_run[h] - mn);
          m_run[h] = mn;
          l_run[h] *= alpha[h];
        }
      } else {
#pragma unroll
        for (int h = 0; h < 8; h++) alpha[h] = 1.f;
      }
      {
        const float vf = (tid < n) ? vsc * vfac : 0.f;
        float wv[8];
#pragma unroll
        for (int h = 0; h < 8; h++) {
          const float pr = ex2f(s[h] - m_run[h]);
          l_run[h] += pr;
          wv[h] = pr * vf;
        }
        // probabilities (times scale_V / sqrt(d)) as fp16 hi + lo: B_P[n][row], n = head (hi) or 8 + head (lo)
        uint4 hi4, lo4;
        uint32_t* hp = reinterpret_cast<uint32_t*>(&hi4);
        uint32_t* lp = reinterpret_cast<uint32_t*>(&lo4);
#pragma unroll
        for (int h2 = 0; h2 < 4; h2++) {
          const uint32_t hpk = pack_half2(wv[2 * h2], wv[2 * h2 + 1]);
          const float2 back = __half22float2(*reinterpret_cast<const __half2*>(&hpk));
          hp[h2] = hpk;
          lp[h2] = pack_half2(wv[2 * h2] - back.x, wv[2 * h2 + 1] - back.y);
        }
        const int off = (tid & 7) * 16 + (tid >> 3) * 128;
        *reinterpret_cast<uint4*>(bp + off) = hi4;
        *reinterpret_cast<uint4*>(bp + (TB / 8) * 128 + off) = lo4;
        fence_proxy_async();
      }
      tc_wait_st();
      tc_fence_before();
      mbar_arrive(p_ready);                 // V tile in TMEM, probabilities in shared memory
      mbar_arrive(&empty_bar[blk % NST]);   // this thread is done with the staged tile
      folded = false;
      // ---- next block's K tile, while the value MMAs run
      if (blk + 1 < nblk) {
        if (L::SHARED_A) { fold(blk); folded = true; }  // the value MMAs read the tile that K is about to overwrite
        k_phase(blk + 1);
      }
    }
    if (!folded) fold(nblk - 1);
  }

  if (__syncthreads_or(failed) && tid == 0 && p.status) atomicOr(&p.status[0], IQ_STATUS_WAIT_TIMEOUT);

  // ---------------------------------------------------------------- reduce l, the exact maximum (and argmax) over the 128 rows
  if (!control) {
#pragma unroll
  for (int h = 0; h < 8; h++) {
    float v = l_run[h];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(FULL, v, o);
    float bv = best_v[h];
    int bi = best_i[h];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float ov = __shfl_xor_sync(FULL, bv, o);
      const int oi = ARGMAX ? __shfl_xor_sync(FULL, bi, o) : -1;
      if (ov > bv || (ARGMAX && ov == bv && oi >= 0 && (bi < 0 || oi < bi))) { bv = ov; bi = oi; }
    }
    if (lane == h) { red[warp * 8 + h] = v; red2[warp * 8 + h] = bv; redi[warp * 8 + h] = bi; }
  }
  }
  __syncthreads();
  if (!control) {
  // The partial is reported relative to the exact maximum m = max_j z_j: rescale from the running reference.
  float fix[8];
#pragma unroll
  for (int h = 0; h < 8; h++) {
    const float mt = fmaxf(fmaxf(red2[h], red2[8 + h]), fmaxf(red2[16 + h], red2[24 + h]));
    fix[h] = ex2f(m_run[h] - mt);
    if (h < nh) {
#pragma unroll
      for (int j = 0; j < DJ; j++)
        p.part_acc[(((size_t)b * p.n_q_heads + h0 + h) * S + split) * D + tid + 128 * j] = acc[j][h] * fix[h];
    }
  }
  if (tid < nh) {
    const int h = tid;
    float mt = -INFINITY;
    int bi = -1;
    for (int w = 0; w < 4; w++) {
      const float ov = red2[w * 8 + h];
      const int oi = redi[w * 8 + h];
      if (ov > mt || (ov == mt && oi >= 0 && (bi < 0 || oi < bi))) { mt = ov; bi = oi; }
    }
    const float l = (red[h] + red[8 + h] + red[16 + h] + red[24 + h]) * ex2f(m_run[h] - mt);
    const size_t o = ((size_t)b * p.n_q_heads + h0 + h) * S + split;
    p.part_ml[2 * o] = mt * LN2;
    p.part_ml[2 * o + 1] = l;
    if (ARGMAX) p.part_argmax[o] = bi;
  }
  }
  tc_fence_before();
  __syncthreads();
  if (control) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_a), "r"(L::ALLOC0_COLS));
    if (L::ALLOC1_COLS > 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_r), "r"(L::ALLOC1_COLS));
  }
}

template <int D, bool ARGMAX>
static cudaError_t launch_one(const DecodeParams& p, cudaStream_t stream) {
  using L = DecLayout<D>;
  static bool configured[64] = {};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  auto kern = decode_kernel<D, ARGMAX>;
  if (dev < 0 || dev >= 64 || !configured[dev]) {
    e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, L::SMEM_BYTES);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64) configured[dev] = true;
  }
  dim3 grid(p.splits, p.n_kv_heads * p.head_groups, p.batch);
  kern<<<grid, DEC_THREADS, L::SMEM_BYTES, stream>>>(p);
  return cudaGetLastError();
}

cudaError_t launch_decode_attention(const DecodeParams& p, int head_dim, cudaStream_t stream) {
  const bool am = p.part_argmax != nullptr;
  if (head_dim == 128) return am ? launch_one<128, true>(p, stream) : launch_one<128, false>(p, stream);
  return am ? launch_one<256, true>(p, stream) : launch_one<256, false>(p, stream);
}

int decode_ctas_per_sm(int head_dim) { return head_dim == 128 ? DecLayout<128>::CTAS_PER_SM : DecLayout<256>::CTAS_PER_SM; }

}  // namespace iq
