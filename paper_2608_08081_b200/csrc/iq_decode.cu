// Fused decode kernel (Appendix A; Table 2 kernels A, B, C): scores on packed K codes, split-K online
// softmax, value accumulation on packed V codes. One CTA per (context split, KV head x head group,
// sequence); every warp streams 64-row tiles of packed codes through its own bulk-copy pipeline,
// dequantises them straight into tensor-core operand registers and keeps a private (m, l, acc) state that
// is merged across the CTA's warps at the end.
//
// Tensor-core shapes (mma.sync m16n8k16, fp16 in, fp32 accumulate), G <= 8 query heads on N:
//   scores   S[16 rows x 8 heads]   += Kdeq[16 rows x 16 coords] * q~^T[16 coords x 8 heads]
//   values   O^T[16 coords x 8 heads] += Vdeq^T[16 coords x 16 rows] * P[16 rows x 8 heads]
// The contraction over coordinates (scores) and the output rows (values) may be visited in any fixed
// order, so each thread takes whole 32-bit words of the packed rows: thread (g, t) of a warp
// (g = lane / 4, t = lane % 4) owns packing unit t of a K row and half of packing unit g / 2 of a V row.
#include "iq_common.cuh"
#include "iq_kernels.h"

namespace iq {

#ifndef IQ_DEC_WARPS
#define IQ_DEC_WARPS 4
#endif
#ifndef IQ_DEC_STAGES
#define IQ_DEC_STAGES 2
#endif
#ifndef IQ_DEC_MINB128
#define IQ_DEC_MINB128 4
#endif
constexpr int DEC_WARPS = IQ_DEC_WARPS;
constexpr int DEC_STAGES = IQ_DEC_STAGES;
constexpr uint32_t DEC_WAIT_LIMIT = 1u << 22;
constexpr int DEC_HDR_BYTES = 512;  // barriers + cross-warp merge scalars

template <int D>
struct DecLayout {
  static constexpr int WPR = 3 * D / 32;  // 32-bit words per packed row
  static constexpr int ROWB = WPR * 4;
  static constexpr int KC_BYTES = DEC_BLOCK_TOKENS * ROWB;
  static constexpr int SC_BYTES = DEC_BLOCK_TOKENS * 4;
  static constexpr int STAGE_BYTES = 2 * KC_BYTES + 2 * SC_BYTES;
  static constexpr int PIPE_BYTES = DEC_WARPS * DEC_STAGES * STAGE_BYTES;
  static constexpr int Q_BYTES = DEC_HEADS * D * 4;
  static constexpr int MERGE_BYTES = DEC_WARPS * DEC_HEADS * D * 4;
  // the rotated-query staging and the cross-warp merge buffer alias the pipeline stages (used before / after them)
  static constexpr int SMEM_BYTES = DEC_HDR_BYTES + (PIPE_BYTES > MERGE_BYTES ? PIPE_BYTES : MERGE_BYTES);
};

// Selectors of the 8 coordinates whose code bits sit in bit 3 of the nibbles of the unit's three words.
__device__ __forceinline__ uint32_t sliced_selectors(uint32_t w0, uint32_t w1, uint32_t w2) {
  return ((w0 >> 3) & 0x11111111u) | ((w1 >> 2) & 0x22222222u) | ((w2 >> 1) & 0x44444444u);
}

static_assert(DecLayout<128>::Q_BYTES <= DecLayout<128>::PIPE_BYTES && DecLayout<256>::Q_BYTES <= DecLayout<256>::PIPE_BYTES, "q staging must fit");

template <int D, bool QSPLIT, bool PSPLIT, bool ARGMAX>
__global__ void __launch_bounds__(DEC_WARPS * 32, (D == 128) ? IQ_DEC_MINB128 : 2) decode_kernel(const DecodeParams p) {
  using L = DecLayout<D>;
  constexpr int DJ = D / 128;
  constexpr int E = D / 32;
  constexpr int WPR = L::WPR;
  constexpr float LOG2E = 1.4426950408889634f;
  constexpr float LN2 = 0.6931471805599453f;

  extern __shared__ __align__(128) uint8_t smem[];
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem);         // [warps][stages]
  float* wm = reinterpret_cast<float*>(smem + 128);           // [warps][8] running max (log2 units)
  float* wl = wm + DEC_WARPS * DEC_HEADS;                     // [warps][8] running sum
  int* wi = reinterpret_cast<int*>(wl + DEC_WARPS * DEC_HEADS);  // [warps][8] argmax row
  uint8_t* pipe = smem + DEC_HDR_BYTES;
  float* qs = reinterpret_cast<float*>(pipe);  // [8][D] rotated queries, consumed before the first tile copy is issued

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int g = lane >> 2, t = lane & 3;
  const int split = blockIdx.x;
  const int kvh = blockIdx.y / p.head_groups;
  const int hg = blockIdx.y - kvh * p.head_groups;
  const int b = blockIdx.z;
  const int S = p.splits;

  const int len = max(0, min(p.seq_lens[b], p.t_cap));
  const int per = (len + S - 1) / S;
  const int chunk = ((per + DEC_BLOCK_TOKENS - 1) / DEC_BLOCK_TOKENS) * DEC_BLOCK_TOKENS;
  const int start = split * chunk;
  const int end = min(len, start + chunk);
  const int h0 = kvh * p.group + hg * DEC_HEADS;       // first query head of this CTA
  const int nh = min(DEC_HEADS, p.group - hg * DEC_HEADS);  // query heads of this CTA

  if (start >= end) {  // empty chunk: (m, l) = (-inf, 0), acc = 0
    for (int idx = tid; idx < nh * D; idx += DEC_WARPS * 32) {
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

  // ---------------------------------------------------------------- pipeline set-up (per warp)
  uint64_t* mybar = bars + warp * DEC_STAGES;
  uint8_t* mypipe = pipe + warp * DEC_STAGES * L::STAGE_BYTES;
  const size_t slab = ((size_t)b * p.n_kv_heads + kvh) * (size_t)p.t_cap;
  const int nblk = (end - start + DEC_BLOCK_TOKENS - 1) / DEC_BLOCK_TOKENS;

  auto issue = [&](int blk, int st) {
    const int r0 = start + blk * DEC_BLOCK_TOKENS;
    const int n = min(DEC_BLOCK_TOKENS, end - r0);
    const int n4 = (n + 3) & ~3;  // scale copies move whole 16-byte groups; t_cap % 4 == 0 keeps them in bounds
    uint8_t* sp = mypipe + st * L::STAGE_BYTES;
    const size_t row = slab + (size_t)r0;
    mbar_expect_tx(&mybar[st], (uint32_t)(2 * n * L::ROWB + 2 * n4 * 4));
    bulk_g2s(sp, p.k_codes + row * L::ROWB, (uint32_t)(n * L::ROWB), &mybar[st]);
    bulk_g2s(sp + L::KC_BYTES, p.v_codes + row * L::ROWB, (uint32_t)(n * L::ROWB), &mybar[st]);
    bulk_g2s(sp + 2 * L::KC_BYTES, p.k_scales + row, (uint32_t)(n4 * 4), &mybar[st]);
    bulk_g2s(sp + 2 * L::KC_BYTES + L::SC_BYTES, p.v_scales + row, (uint32_t)(n4 * 4), &mybar[st]);
  };

  if (lane == 0) {
#pragma unroll
    for (int st = 0; st < DEC_STAGES; st++) mbar_init(&mybar[st], 1);
    fence_mbar_init();
  }

  // ---------------------------------------------------------------- d1: q~ = R q for the CTA's heads
  {
    float M[E / 4][4][4];
    const float* qb = p.rot + ((size_t)kvh * (D / 4) + (size_t)lane * (E / 4)) * 8;
#pragma unroll
    for (int j = 0; j < E / 4; j++) so4_matrix<float>(qb + 8 * j, M[j]);
    const float inv_root_d = rsqrtf((float)D);
    for (int hh = warp; hh < DEC_HEADS; hh += DEC_WARPS) {
      float v[E];
      if (hh < nh) {
        const __half* src = p.q + ((size_t)b * p.n_q_heads + h0 + hh) * D + lane * E;
#pragma unroll
        for (int e = 0; e < E; e++) v[e] = __half2float(src[e]);
        wht_warp<float, E>(v, lane);
        so4_apply<float, E, false>(M, v);
#pragma unroll
        for (int e = 0; e < E; e++) v[e] *= inv_root_d;
      } else {
#pragma unroll
        for (int e = 0; e < E; e++) v[e] = 0.f;
      }
#pragma unroll
      for (int e = 0; e < E; e++) qs[hh * D + lane * E + e] = v[e];
    }
  }
  __syncthreads();

  // B fragments of q~: lane (g, t) keeps head g, coordinates of packing units t + 4j, as fp16 hi (+ lo).
  uint32_t qhi[DJ][8][2];
  uint32_t qlo[QSPLIT ? DJ : 1][8][2];
#pragma unroll
  for (int j = 0; j < DJ; j++)
#pragma unroll
    for (int i = 0; i < 8; i++) {
      const float4 f = *reinterpret_cast<const float4*>(qs + g * D + 32 * (t + 4 * j) + 4 * i);
      const __half2 h01 = __floats2half2_rn(f.x, f.y), h23 = __floats2half2_rn(f.z, f.w);
      qhi[j][i][0] = *reinterpret_cast<const uint32_t*>(&h01);
      qhi[j][i][1] = *reinterpret_cast<const uint32_t*>(&h23);
      if (QSPLIT) {
        const float2 b01 = __half22float2(h01), b23 = __half22float2(h23);
        qlo[j][i][0] = pack_half2(f.x - b01.x, f.y - b01.y);
        qlo[j][i][1] = pack_half2(f.z - b23.x, f.w - b23.y);
      }
    }

  __syncthreads();  // every warp has read its q~ fragments: the staging area becomes pipeline memory
  if (lane == 0) {
    fence_proxy_async();
#pragma unroll
    for (int st = 0; st < DEC_STAGES; st++)
      if (warp + st * DEC_WARPS < nblk) issue(warp + st * DEC_WARPS, st);
  }

  const uint32_t lut_lo0 = p.lut_lo[0], lut_lo1 = p.lut_lo[1], lut_hi0 = p.lut_hi[0], lut_hi1 = p.lut_hi[1];
  const float kfac = p.sm_scale * LOG2E * rsqrtf((float)D);  // scores in log2 units: z2 = S_raw * scale_K * kfac
  const float vfac = rsqrtf((float)D);
  const uint32_t vsel = (g & 1) ? 0x7362u : 0x5140u;  // which 16-bit half of a V word this lane decodes

  float acc[DJ][8][4];
#pragma unroll
  for (int j = 0; j < DJ; j++)
#pragma unroll
    for (int i = 0; i < 8; i++)
#pragma unroll
      for (int r = 0; r < 4; r++) acc[j][i][r] = 0.f;
  float m_run[2] = {-INFINITY, -INFINITY};
  float l_run[2] = {0.f, 0.f};
  float best_v[2] = {-INFINITY, -INFINITY};
  int best_i[2] = {-1, -1};
  bool failed = false;

  // ---------------------------------------------------------------- main loop over this warp's tiles
  for (int it = 0;; it++) {
    const int blk = warp + it * DEC_WARPS;
    if (blk >= nblk) break;
    const int st = it % DEC_STAGES;
    const uint32_t parity = (uint32_t)(it / DEC_STAGES) & 1u;
    const bool ok = mbar_wait_bounded(&mybar[st], parity, DEC_WAIT_LIMIT);
    if (__any_sync(FULL, !ok)) {
      failed = true;
      break;
    }
    const uint8_t* sp = mypipe + st * L::STAGE_BYTES;
    const uint32_t* Kw = reinterpret_cast<const uint32_t*>(sp);
    const uint32_t* Vw = reinterpret_cast<const uint32_t*>(sp + L::KC_BYTES);
    const float* Ksc = reinterpret_cast<const float*>(sp + 2 * L::KC_BYTES);
    const float* Vsc = Ksc + DEC_BLOCK_TOKENS;
    const int r0 = start + blk * DEC_BLOCK_TOKENS;
    const int n = min(DEC_BLOCK_TOKENS, end - r0);

    // ---- d2: raw scores on the codes
    float s[4][4];
#pragma unroll
    for (int mt = 0; mt < 4; mt++) {
#pragma unroll
      for (int r = 0; r < 4; r++) s[mt][r] = 0.f;
      const uint32_t* ka = Kw + (16 * mt + g) * WPR;
      const uint32_t* kb = ka + 8 * WPR;
#pragma unroll
      for (int j = 0; j < DJ; j++) {
        const int u = t + 4 * j;
        const uint32_t a0w = ka[3 * u], a1w = ka[3 * u + 1], a2w = ka[3 * u + 2];
        const uint32_t b0w = kb[3 * u], b1w = kb[3 * u + 1], b2w = kb[3 * u + 2];
        const uint32_t sa[4] = {a0w & 0x77777777u, a1w & 0x77777777u, a2w & 0x77777777u, sliced_selectors(a0w, a1w, a2w)};
        const uint32_t sb[4] = {b0w & 0x77777777u, b1w & 0x77777777u, b2w & 0x77777777u, sliced_selectors(b0w, b1w, b2w)};
#pragma unroll
        for (int k = 0; k < 4; k++)
#pragma unroll
          for (int hh = 0; hh < 2; hh++) {
            const uint32_t xa = hh ? (sa[k] >> 16) : sa[k];
            const uint32_t xb = hh ? (sb[k] >> 16) : sb[k];
            const uint32_t la = prmt(lut_lo0, lut_lo1, xa), ha = prmt(lut_hi0, lut_hi1, xa);
            const uint32_t lb = prmt(lut_lo0, lut_lo1, xb), hb = prmt(lut_hi0, lut_hi1, xb);
            const uint32_t f0 = prmt(la, ha, 0x5140u), f2 = prmt(la, ha, 0x7362u);
            const uint32_t f1 = prmt(lb, hb, 0x5140u), f3 = prmt(lb, hb, 0x7362u);
            mma_16816(s[mt], f0, f1, f2, f3, qhi[j][2 * k + hh][0], qhi[j][2 * k + hh][1]);
            if (QSPLIT) mma_16816(s[mt], f0, f1, f2, f3, qlo[j][2 * k + hh][0], qlo[j][2 * k + hh][1]);
          }
      }
    }

    // ---- d3: online softmax (log2 units). Lane (g, t) holds rows g, g+8 of each 16-row tile, heads 2t, 2t+1.
    float vs[4][2];
#pragma unroll
    for (int mt = 0; mt < 4; mt++) {
      float ka_s = Ksc[16 * mt + g] * kfac, kb_s = Ksc[16 * mt + g + 8] * kfac;
      vs[mt][0] = Vsc[16 * mt + g] * vfac;
      vs[mt][1] = Vsc[16 * mt + g + 8] * vfac;
      s[mt][0] *= ka_s; s[mt][1] *= ka_s; s[mt][2] *= kb_s; s[mt][3] *= kb_s;
    }
    if (n < DEC_BLOCK_TOKENS) {  // last tile of the chunk: rows >= n hold stale bytes
#pragma unroll
      for (int mt = 0; mt < 4; mt++) {
        if (16 * mt + g >= n) { s[mt][0] = -INFINITY; s[mt][1] = -INFINITY; vs[mt][0] = 0.f; }
        if (16 * mt + g + 8 >= n) { s[mt][2] = -INFINITY; s[mt][3] = -INFINITY; vs[mt][1] = 0.f; }
      }
    }
    if (ARGMAX) {
#pragma unroll
      for (int mt = 0; mt < 4; mt++) {
        const int ra = r0 + 16 * mt + g;
        if (s[mt][0] > best_v[0]) { best_v[0] = s[mt][0]; best_i[0] = ra; }
        if (s[mt][1] > best_v[1]) { best_v[1] = s[mt][1]; best_i[1] = ra; }
        if (s[mt][2] > best_v[0]) { best_v[0] = s[mt][2]; best_i[0] = ra + 8; }
        if (s[mt][3] > best_v[1]) { best_v[1] = s[mt][3]; best_i[1] = ra + 8; }
      }
    }
    float mx0 = fmaxf(fmaxf(s[0][0], s[0][2]), fmaxf(s[1][0], s[1][2]));
    float mx1 = fmaxf(fmaxf(s[0][1], s[0][3]), fmaxf(s[1][1], s[1][3]));
    mx0 = fmaxf(mx0, fmaxf(fmaxf(s[2][0], s[2][2]), fmaxf(s[3][0], s[3][2])));
    mx1 = fmaxf(mx1, fmaxf(fmaxf(s[2][1], s[2][3]), fmaxf(s[3][1], s[3][3])));
#pragma unroll
    for (int o = 4; o < 32; o <<= 1) {
      mx0 = fmaxf(mx0, __shfl_xor_sync(FULL, mx0, o));
      mx1 = fmaxf(mx1, __shfl_xor_sync(FULL, mx1, o));
    }
    const float mn0 = fmaxf(m_run[0], mx0), mn1 = fmaxf(m_run[1], mx1);
    if (__any_sync(FULL, (mn0 > m_run[0]) || (mn1 > m_run[1]))) {
      const float c0 = ex2f(m_run[0] - mn0), c1 = ex2f(m_run[1] - mn1);
      l_run[0] *= c0;
      l_run[1] *= c1;
#pragma unroll
      for (int j = 0; j < DJ; j++)
#pragma unroll
        for (int i = 0; i < 8; i++) {
          acc[j][i][0] *= c0; acc[j][i][1] *= c1; acc[j][i][2] *= c0; acc[j][i][3] *= c1;
        }
      m_run[0] = mn0;
      m_run[1] = mn1;
    }
    // probabilities -> B fragments of the value product (transposed across the warp by movmatrix)
    // Each weight p * scale_V / sqrt(d) is carried as a two-term fp16 sum (hi + lo): a single fp16 would leave
    // a 2^-11 relative error on every term, which is isotropic in the rotated space and too large for rows
    // whose norm is dominated by a few outlier channels.
    uint32_t pb[4][2];
    uint32_t pl[PSPLIT ? 4 : 1][2];
#pragma unroll
    for (int mt = 0; mt < 4; mt++) {
      const float p0 = ex2f(s[mt][0] - mn0), p1 = ex2f(s[mt][1] - mn1);
      const float p2 = ex2f(s[mt][2] - mn0), p3 = ex2f(s[mt][3] - mn1);
      l_run[0] += p0 + p2;
      l_run[1] += p1 + p3;
      const float w0 = p0 * vs[mt][0], w1 = p1 * vs[mt][0], w2 = p2 * vs[mt][1], w3 = p3 * vs[mt][1];
      const uint32_t h01 = pack_half2(w0, w1), h23 = pack_half2(w2, w3);
      pb[mt][0] = movmatrix_trans(h01);
      pb[mt][1] = movmatrix_trans(h23);
      if (PSPLIT) {
        const float2 b01 = __half22float2(*reinterpret_cast<const __half2*>(&h01));
        const float2 b23 = __half22float2(*reinterpret_cast<const __half2*>(&h23));
        pl[mt][0] = movmatrix_trans(pack_half2(w0 - b01.x, w1 - b01.y));
        pl[mt][1] = movmatrix_trans(pack_half2(w2 - b23.x, w3 - b23.y));
      }
    }

    // ---- d4: value accumulation on the codes. Lane (g, t) decodes rows 2t, 2t+1, 2t+8, 2t+9 of each
    // 16-row step, 16 coordinates: the (g & 1) half of packing unit (g >> 1) + 4j.
#pragma unroll
    for (int mt = 0; mt < 4; mt++) {
      const uint32_t* va = Vw + (16 * mt + 2 * t) * WPR;
#pragma unroll
      for (int j = 0; j < DJ; j++) {
        const int u = (g >> 1) + 4 * j;
        uint32_t mab[3], mcd[3];
#pragma unroll
        for (int k = 0; k < 3; k++) {
          mab[k] = prmt(va[3 * u + k], va[WPR + 3 * u + k], vsel);
          mcd[k] = prmt(va[8 * WPR + 3 * u + k], va[9 * WPR + 3 * u + k], vsel);
        }
        const uint32_t sab[4] = {mab[0] & 0x77777777u, mab[1] & 0x77777777u, mab[2] & 0x77777777u, sliced_selectors(mab[0], mab[1], mab[2])};
        const uint32_t scd[4] = {mcd[0] & 0x77777777u, mcd[1] & 0x77777777u, mcd[2] & 0x77777777u, sliced_selectors(mcd[0], mcd[1], mcd[2])};
#pragma unroll
        for (int k = 0; k < 4; k++)
#pragma unroll
          for (int hh = 0; hh < 2; hh++) {
            const uint32_t x1 = hh ? (sab[k] >> 16) : sab[k];
            const uint32_t x2 = hh ? (scd[k] >> 16) : scd[k];
            const uint32_t l1 = prmt(lut_lo0, lut_lo1, x1), h1 = prmt(lut_hi0, lut_hi1, x1);
            const uint32_t l2 = prmt(lut_lo0, lut_lo1, x2), h2 = prmt(lut_hi0, lut_hi1, x2);
            const uint32_t f0 = prmt(l1, h1, 0x6240u), f1 = prmt(l1, h1, 0x7351u);
            const uint32_t f2 = prmt(l2, h2, 0x6240u), f3 = prmt(l2, h2, 0x7351u);
            mma_16816(acc[j][2 * k + hh], f0, f1, f2, f3, pb[mt][0], pb[mt][1]);
            if (PSPLIT) mma_16816(acc[j][2 * k + hh], f0, f1, f2, f3, pl[mt][0], pl[mt][1]);
          }
      }
    }

    // ---- refill this stage
    __syncwarp();
    if (lane == 0) {
      const int nb = blk + DEC_STAGES * DEC_WARPS;
      if (nb < nblk) {
        fence_proxy_async();
        issue(nb, st);
      }
    }
  }

  if (failed) {
    if (lane == 0 && p.status) atomicOr(&p.status[0], IQ_STATUS_WAIT_TIMEOUT);
  }

  // ---------------------------------------------------------------- merge the warps of this CTA
#pragma unroll
  for (int o = 4; o < 32; o <<= 1) {
    l_run[0] += __shfl_xor_sync(FULL, l_run[0], o);
    l_run[1] += __shfl_xor_sync(FULL, l_run[1], o);
    if (ARGMAX) {
#pragma unroll
      for (int c = 0; c < 2; c++) {
        const float ov = __shfl_xor_sync(FULL, best_v[c], o);
        const int oi = __shfl_xor_sync(FULL, best_i[c], o);
        if (ov > best_v[c] || (ov == best_v[c] && oi >= 0 && (best_i[c] < 0 || oi < best_i[c]))) { best_v[c] = ov; best_i[c] = oi; }
      }
    }
  }
  __syncthreads();  // every warp has consumed all of its tiles: the pipeline memory is free
  float* wacc = reinterpret_cast<float*>(pipe) + (size_t)warp * DEC_HEADS * D;
#pragma unroll
  for (int j = 0; j < DJ; j++)
#pragma unroll
    for (int i = 0; i < 8; i++) {
      const int c = 32 * ((g >> 1) + 4 * j) + 8 * (i >> 1) + 4 * (g & 1) + 2 * (i & 1);
      wacc[(2 * t) * D + c] = acc[j][i][0];
      wacc[(2 * t + 1) * D + c] = acc[j][i][1];
      wacc[(2 * t) * D + c + 1] = acc[j][i][2];
      wacc[(2 * t + 1) * D + c + 1] = acc[j][i][3];
    }
  if (g == 0) {
    wm[warp * DEC_HEADS + 2 * t] = m_run[0];
    wm[warp * DEC_HEADS + 2 * t + 1] = m_run[1];
    wl[warp * DEC_HEADS + 2 * t] = l_run[0];
    wl[warp * DEC_HEADS + 2 * t + 1] = l_run[1];
    wi[warp * DEC_HEADS + 2 * t] = best_i[0];
    wi[warp * DEC_HEADS + 2 * t + 1] = best_i[1];
  }
  __syncthreads();
  const float* allacc = reinterpret_cast<const float*>(pipe);
  for (int idx = tid; idx < nh * D; idx += DEC_WARPS * 32) {
    const int head = idx / D, c = idx - head * D;
    float mm = -INFINITY;
#pragma unroll
    for (int w = 0; w < DEC_WARPS; w++) mm = fmaxf(mm, wm[w * DEC_HEADS + head]);
    float a = 0.f;
#pragma unroll
    for (int w = 0; w < DEC_WARPS; w++) a += allacc[((size_t)w * DEC_HEADS + head) * D + c] * ex2f(wm[w * DEC_HEADS + head] - mm);
    p.part_acc[(((size_t)b * p.n_q_heads + h0 + head) * S + split) * D + c] = a;
  }
  if (tid < nh) {
    const int head = tid;
    float mm = -INFINITY;
#pragma unroll
    for (int w = 0; w < DEC_WARPS; w++) mm = fmaxf(mm, wm[w * DEC_HEADS + head]);
    float l = 0.f;
    int bi = -1;
#pragma unroll
    for (int w = 0; w < DEC_WARPS; w++) {
      l += wl[w * DEC_HEADS + head] * ex2f(wm[w * DEC_HEADS + head] - mm);
      if (ARGMAX && wm[w * DEC_HEADS + head] == mm) {
        const int ci = wi[w * DEC_HEADS + head];
        if (ci >= 0 && (bi < 0 || ci < bi)) bi = ci;
      }
    }
    const size_t o = ((size_t)b * p.n_q_heads + h0 + head) * S + split;
    p.part_ml[2 * o] = mm * LN2;
    p.part_ml[2 * o + 1] = l;
    if (ARGMAX) p.part_argmax[o] = bi;
  }
}

template <int D, bool QSPLIT, bool PSPLIT, bool ARGMAX>
static cudaError_t launch_one(const DecodeParams& p, cudaStream_t stream) {
  using L = DecLayout<D>;
  static bool configured[64] = {};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  auto kern = decode_kernel<D, QSPLIT, PSPLIT, ARGMAX>;
  if (dev < 0 || dev >= 64 || !configured[dev]) {
    e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, L::SMEM_BYTES);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64) configured[dev] = true;
  }
  dim3 grid(p.splits, p.n_kv_heads * p.head_groups, p.batch);
  kern<<<grid, DEC_WARPS * 32, L::SMEM_BYTES, stream>>>(p);
  return cudaGetLastError();
}

cudaError_t launch_decode_attention(const DecodeParams& p, int head_dim, cudaStream_t stream) {
  const bool am = p.part_argmax != nullptr;
  if (head_dim == 128) return am ? launch_one<128, true, true, true>(p, stream) : launch_one<128, true, true, false>(p, stream);
  return am ? launch_one<256, true, true, true>(p, stream) : launch_one<256, true, true, false>(p, stream);
}

int decode_ctas_per_sm(int head_dim) { return head_dim == 128 ? IQ_DEC_MINB128 : 2; }

}  // namespace iq
