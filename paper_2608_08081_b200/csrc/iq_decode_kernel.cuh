// Fused decode kernel (Appendix A; Table 2 kernels A, B, C): scores on packed K codes, split-K online
// softmax, value accumulation on packed V codes, on the 5th-generation tensor cores (tcgen05) with the
// dequantised operands resident in tensor memory (TMEM).
//
// Work decomposition. A CTA -- one per SM -- holds NG independent workers ("groups": 4 compute warps + 1 control
// warp, their own TMEM columns, tile pipeline, query operand and softmax state). After the set-up there is no
// CTA-wide synchronisation: a group never waits for another group.
//   Range mode (num_splits >= 2 NG). The 128-row blocks of all (sequence, KV head, head group) items of the launch
//   are laid end to end and every CTA takes an equal, contiguous range of that sequence, whatever the length mix of
//   the batch. The groups of the CTA draw the blocks of the range one at a time from a shared-memory counter, so they
//   stay busy although the warp schedulers do not serve them evenly. The part of one item inside a range is a
//   "segment"; piece k of an item (its k-th CTA) reports to partial slots k NG .. k NG + NG - 1, one per group. A
//   group that crosses into another segment writes its partial of the old one straight to its slot, rotates the
//   queries of the new item into its own operand buffer and goes on, while its tiles keep streaming in.
//   Unit mode (fewer slots). Every item is cut into num_splits consecutive runs of blocks, run k reports to slot
//   k, and the runs are dealt out to the groups of all CTAs in turn.
// Every partial slot of every head is written on every launch: by the group that worked on it, else by the
// control warp that is responsible for it (unused slots hold m = -inf, l = 0; their acc is not written).
//
// Per block, in group g (thread r of the group = TMEM lane r):
//   1. thread r dequantises packed K row r (its own 3d/8 bytes from the staged tile) and stores it to TMEM lane r.
//   2. the control warp issues tcgen05.mma (M = 128 rows): S[row][n] = sum_i A_K[row][i] * B_Q[n][i], the columns n
//      holding q~ of the <= 8 heads (fp16 hi | lo, or three int8 digits per head).
//   3. every thread reads its row of S back, applies the K scale, joins the group-wide running reference and
//      writes its probabilities (times the V scale) into the shared-memory operand B_P[n][row].
//   4. thread c dequantises coordinate c of the token-transposed V block (128 codes = one 48-byte row) into
//      TMEM lane c; the control warp issues O[c][n] = sum_row A_V[c][row] * B_P[n][row].
//   5. thread c folds O into its running accumulator for coordinate c.
// Packed tiles arrive through a 1-D bulk-copy (TMA) pipeline; every mbarrier wait is bounded (a poll count).
//
// Template parameters of the kernel: head_dim D; ARGMAX (exact slot maxima and their rows); I8 (levels on an 8-bit grid:
// int8 operands, int32 accumulation; otherwise fp16 operands); APPEND (the launch also appends the step's new rows: a few
// CTAs at the start of the grid do only that, see dec_aux_work); BITS (2, 3 or 4 bits per code: tile sizes and lookups).
#pragma once
#include <climits>

#include "iq_append_row.cuh"
#include "iq_decode_common.cuh"
#include "iq_kernels.h"

namespace iq {

constexpr int DEC_GROUP_THREADS = 128;  // 4 warps: dequantisation, softmax, accumulation (thread = TMEM lane)
constexpr int DEC_HDR_BYTES = 4096;    // barriers, TMEM base, work counter, block descriptors, scratch
constexpr int DEC_NPRE = 4;             // query operands prepared at the start of a CTA: those of its range's first segments
constexpr int DEC_PRE_BAR = 9;          // named barrier of all compute threads (used while those operands are built)
constexpr int DEC_SEG_COST = 8;          // what an item entering a CTA's range costs the CTA, in blocks (range partition)
constexpr float DEC_RAISE_MARGIN = 3.0f;  // log2 units a raised reference is put above the block's maximum
constexpr float DEC_MAX_SLACK = 4.0f;  // log2 units a score may exceed the running reference before it is raised
#ifndef IQ_SLACK_I8
#define IQ_SLACK_I8 4
#endif
constexpr float DEC_MAX_SLACK_I8 = (float)IQ_SLACK_I8;  // the same on the integer path, where the probabilities are fixed-point numbers

// What the control warp tells the compute warps about a staged tile.
struct DecDesc {
  int n;        // valid rows of the block; n < 0: end marker, the group is done
  int flags;    // bit 0: first block this group gets of a segment: close the open one, open (b, y, slot)
  int r0;       // first row of the block in its sequence
  int slot;     // partial slot of the item this group reports the segment to
  int b, y;     // sequence, item within it (KV head x head group)
  int len;      // cached rows of the sequence (unused by the compute warps; kept for diagnosis)
  int bqbuf;    // which prepared query operand the segment uses, -1: the group builds its own
};
static_assert(sizeof(DecDesc) == 32, "descriptor layout");

template <int D, int BITS = 3>
struct DecLayout {
  static constexpr int DJ = D / 128;
  static constexpr int WPR = BITS * D / 32;  // 32-bit words per packed K row
  static constexpr int ROWB = WPR * 4;
  static constexpr int K_BYTES = DEC_BLOCK_TOKENS * ROWB;
  static constexpr int VREC = 16 * BITS;      // bytes of one V record: the 128 codes of one coordinate
  static constexpr int VT_BYTES = D * VREC;   // token-transposed V block: one record per coordinate
  static constexpr int SC_BYTES = DEC_BLOCK_TOKENS * 4;
  static constexpr int STAGE_BYTES = K_BYTES + VT_BYTES + 2 * SC_BYTES;
  static constexpr int STAGES = BITS == 4 ? 2 : 3;  // (what fits: a 4-bit tile is a third larger)
  static constexpr int BQ_BYTES = 16 * D * 2;  // per group: 16 fp16 columns or 32 int8 columns over d contraction steps
  static constexpr int BP_BYTES = 16 * DEC_BLOCK_TOKENS * 2;
  // TMEM columns of one group, fp16 path: the operand tile (K rows, then V coordinates: d fp16 = d/2 columns), 16
  // columns of scores, 16 * DJ columns of values. The CTA owns all 512 columns of the SM.
  static constexpr int GROUP_COLS = D;
  static constexpr int A_COL = 0;
  static constexpr int S_COL = D / 2;
  static constexpr int O_COL = D / 2 + 16;
  static constexpr int V_COL = O_COL + 16 * (D / 128);  // rows 0..63 of the V tile (32 columns per 128 coordinates)
  // Integer path (int8 operands: 4 elements per column, separate K and V tiles, 32 result columns = 8 heads x 4 digits)
  static constexpr int I8_K_COL = 0;                   // K tile: d/4 columns
  static constexpr int I8_V_COL = D / 4;               // V tile: 32 columns per 128 coordinates
  static constexpr int I8_S_COL = D / 4 + 32 * (D / 128);
  static constexpr int I8_O_COL = I8_S_COL + 32;       // 32 columns per 128 coordinates
  static constexpr int NG = 512 / GROUP_COLS;  // groups per CTA: 4 at d = 128, 2 at d = 256
  static constexpr int COMPUTE_THREADS = NG * DEC_GROUP_THREADS;
  static constexpr int THREADS = COMPUTE_THREADS + NG * 32;  // + one control warp per group
  static constexpr int GROUP_SMEM = BQ_BYTES + BP_BYTES + STAGES * STAGE_BYTES;
  static constexpr int PRE_BYTES = DEC_NPRE * BQ_BYTES;  // the prepared query operands, shared by the groups
  static constexpr int SMEM_BYTES = DEC_HDR_BYTES + PRE_BYTES + NG * GROUP_SMEM;
  // header offsets
  static constexpr int BAR_STRIDE = 96;  // per group: full[3], empty[3], s_bar, o_bar, k_ready, p_ready
  static constexpr int OFF_TMEM = 384, OFF_NEXT = 388, OFF_ACCF = 400, OFF_START = 448, OFF_DESC = 512, OFF_QFAC = 896, OFF_SEGID = 960, OFF_RED = 1024, OFF_PRE = 2560;
  // OFF_PRE: count, [DEC_NPRE] (sequence, item), [DEC_NPRE] score factors, [DEC_NPRE][8] per-head maxima
  static constexpr int DESC_STRIDE = STAGES * 32;  // per group
  static constexpr int RED_STRIDE = 384;            // per group: 3 x [4 warps][8 heads] words
};
static_assert(DEC_BLOCK_TOKENS == 128, "the TMEM operand layout assumes 128-row blocks");
static_assert(DecLayout<128>::OFF_DESC + 4 * DecLayout<128>::DESC_STRIDE <= DecLayout<128>::OFF_QFAC, "header overflow");
static_assert(DecLayout<128>::OFF_RED + 4 * DecLayout<128>::RED_STRIDE <= DecLayout<128>::OFF_PRE, "header overflow");
static_assert(DecLayout<128>::OFF_PRE + 8 + 8 * DEC_NPRE + 4 * DEC_NPRE + 32 * DEC_NPRE <= DEC_HDR_BYTES, "header overflow");
static_assert(DecLayout<128>::V_COL + 32 * DecLayout<128>::DJ <= DecLayout<128>::GROUP_COLS, "TMEM group overflow");
static_assert(DecLayout<256>::V_COL + 32 * DecLayout<256>::DJ <= DecLayout<256>::GROUP_COLS, "TMEM group overflow");
static_assert(DecLayout<128>::I8_O_COL + 32 * DecLayout<128>::DJ <= DecLayout<128>::GROUP_COLS, "TMEM group overflow");
static_assert(DecLayout<256>::I8_O_COL + 32 * DecLayout<256>::DJ <= DecLayout<256>::GROUP_COLS, "TMEM group overflow");
static_assert(DecLayout<128>::SMEM_BYTES <= 227 * 1024 && DecLayout<256>::SMEM_BYTES <= 227 * 1024, "shared memory overflow");
static_assert(DecLayout<128, 2>::SMEM_BYTES <= 227 * 1024 && DecLayout<256, 2>::SMEM_BYTES <= 227 * 1024, "shared memory overflow");
static_assert(DecLayout<128, 4>::SMEM_BYTES <= 227 * 1024 && DecLayout<256, 4>::SMEM_BYTES <= 227 * 1024, "shared memory overflow");
static_assert((2 * DecLayout<128, 2>::THREADS + DecLayout<128, 2>::THREADS / 32) * 4 <= DecLayout<128, 2>::BP_BYTES + DecLayout<128, 2>::STAGE_BYTES, "set-up scratch must fit group 0's B_P region and first stage");
static_assert((2 * DecLayout<128>::THREADS + DecLayout<128>::THREADS / 32) * 4 <= DecLayout<128>::BP_BYTES + DecLayout<128>::STAGE_BYTES, "set-up scratch must fit group 0's B_P region and first stage");

// Marks one partial slot of nh consecutive heads unused: (m, l) = (-inf, 0), argmax = -1 (the merge skips a slot with
// l = 0 without reading its acc, which is left as it is). ml / argmax point at the slot of the first head; consecutive
// heads are S slots apart. Thread t of the caller writes head t.
__device__ __forceinline__ void dec_fill_slot(float* ml, int32_t* argmax, int nh, int S, int t) {
  if (t < nh) {
    ml[2 * (size_t)t * S] = -INFINITY;
    ml[2 * (size_t)t * S + 1] = 0.f;
    if (argmax) argmax[(size_t)t * S] = -1;
  }
}

// The control warp's position in its work, and the block it has drawn. All lanes hold the same values.
struct DecWalk {
  int range_mode, grp, ng, ips, count;
  // range mode: item (b, y) of the CTA's range the walk is in, blocks of its sequence, which piece of the item lies in
  // this range, whether this group has staged a block of the segment
  int b, y, nb, len, piece, touched;  // (len: cached rows of sequence b)
  int sidx, n_pre;                    // ordinal of the segment in the range; segments below n_pre have a prepared query operand
  long long item_g, g0, g_end;  // launch-wide index of block 0 of the item; the range [g0, g_end)
  // unit mode: run k of item i is unit i * S + k; the walk is in run uk of item (ub, uy), at block ublk of [.., uhi)
  int n_units, unit_step, unit;  // (the host refuses launches whose unit count does not fit 31 bits)
  int ub, uy, uk, ublk, uhi, unew, ulen;
};
struct DecDrawn {
  int kind;  // -1: nothing drawn, 0: a block, 1: the work has run out
  int b, y, blk, slot, len, is_new, bqbuf;
  size_t row0;  // first row of the block in the cache arrays
};

// Draws the group's next block. Range mode: the next block of the CTA's range from the shared counter; on the way the
// walk passes over the segments of the range, and the partial slots this group owes -- its slot of a segment it got
// no block of, the slots of an item beyond its last piece (those with index = grp mod ng) -- are marked unused. Unit
// mode: the next block of the worker's current run, else of its next run with blocks (runs without blocks are marked
// unused). Nothing is loaded from global memory unless the walk moves to another sequence (or the cache is paged).
template <int D>
__device__ __forceinline__ void dec_draw(const DecodeParams& p, DecWalk& w, DecDrawn& d, int* next_s, int lane, int with_argmax) {
  constexpr int TB = DEC_BLOCK_TOKENS;
  const int S = p.splits, B = p.batch;
  auto len_of = [&](int b) { return max(0, min(p.seq_lens[b] + p.len_bias, p.t_cap)); };
  auto warp_fill = [&](int b, int y, int slot) {
    const int kvh = y / p.head_groups, hg = y - kvh * p.head_groups;
    const int h0 = kvh * p.group + hg * DEC_HEADS, nh = min(DEC_HEADS, p.group - hg * DEC_HEADS);
    const size_t o = ((size_t)b * p.n_q_heads + h0) * S + slot;
    dec_fill_slot(p.part_ml + 2 * o, with_argmax ? p.part_argmax + o : nullptr, nh, S, lane);
  };
  if (w.range_mode) {
    auto leave_segment = [&](bool item_ends) {
      if (!w.touched) warp_fill(w.b, w.y, w.piece * w.ng + w.grp);
      if (item_ends)
        for (int sl = (w.piece + 1) * w.ng + w.grp; sl < S; sl += w.ng) warp_fill(w.b, w.y, sl);
    };
    auto next_item = [&]() {
      w.item_g += w.nb;
      w.touched = 0;
      w.piece = 0;  // the next item starts inside this range
      w.sidx++;
      if (++w.y == w.ips) {
        w.y = 0;
        do { w.b++; w.len = (w.b < B) ? len_of(w.b) : 0; w.nb = (w.len + TB - 1) / TB; } while (w.b < B && w.nb == 0);
      }
    };
    int n = 0;
    if (lane == 0) n = atomicAdd(next_s, 1);
    n = __shfl_sync(FULL, n, 0);
    if (n >= w.count) {  // walk to the end of the range: the slots this group still owes
      while (w.b < B && w.item_g + w.nb <= w.g_end) { leave_segment(true); next_item(); }
      if (w.b < B && max(w.item_g, w.g0) < w.g_end) leave_segment(false);
      w.b = B;
      d.kind = 1;
      return;
    }
    const long long g = w.g0 + n;
    while (g >= w.item_g + w.nb) { leave_segment(true); next_item(); }
    d.is_new = w.touched ? 0 : 1;
    w.touched = 1;
    d.b = w.b;
    d.y = w.y;
    d.blk = (int)(g - w.item_g);
    d.slot = w.piece * w.ng + w.grp;
    d.len = w.len;
    d.bqbuf = w.sidx < w.n_pre ? w.sidx : -1;
  } else {
    while (w.ublk >= w.uhi) {  // the next run with blocks
      if (w.unit >= w.n_units) { d.kind = 1; return; }
      const int item = w.unit / S;
      const int k = w.unit - item * S;
      w.unit = (w.unit_step > w.n_units - w.unit) ? w.n_units : w.unit + w.unit_step;  // (no overflow)
      const int b = item / w.ips, y = item - b * w.ips;
      const int len = len_of(b), nb = (len + TB - 1) / TB;
      if (nb == 0) continue;  // an empty sequence: its slots were written during the set-up
      const int cb = (nb + S - 1) / S, lo = k * cb, hi = min(nb, lo + cb);
      if (lo >= hi) { warp_fill(b, y, k); continue; }
      w.ub = b; w.uy = y; w.uk = k; w.ublk = lo; w.uhi = hi; w.unew = 1; w.ulen = len;
    }
    d.b = w.ub; d.y = w.uy; d.blk = w.ublk++; d.slot = w.uk; d.is_new = w.unew; d.len = w.ulen; d.bqbuf = -1;
    w.unew = 0;
  }
  d.row0 = cache_row(p.pm, d.b, d.y / p.head_groups, (long long)d.blk * TB, p.status);
  d.kind = 0;
}

// d1 (App. A): q~ = R q of one head times 1/sqrt(d), as the lane's E = D / 32 coordinates (lane l holds l E .. l E + E - 1).
// Out of line, like dec_write_operand: both run once per segment at most, and the kernel's code should stay small
// (a launch over a short context spends a good part of its time fetching instructions it executes once).
template <int D>
struct DecHeadCoords { float v[D / 32]; };
template <int D>
static __device__ __noinline__ DecHeadCoords<D> dec_rotate_head(const __half* q_head, const float* rot_head, int lane) {
  constexpr int E = D / 32;
  DecHeadCoords<D> r;
  if (q_head == nullptr) {
#pragma unroll
    for (int e = 0; e < E; e++) r.v[e] = 0.f;
    return r;
  }
  float M[E / 4][4][4];
  const float* qb = rot_head + (size_t)lane * (E / 4) * 8;
#pragma unroll
  for (int j = 0; j < E / 4; j++) so4_matrix<float>(qb + 8 * j, M[j]);
  const __half* src = q_head + lane * E;
#pragma unroll
  for (int e = 0; e < E; e++) r.v[e] = __half2float(src[e]);
  wht_warp<float, E>(r.v, lane);
  so4_apply<float, E, false>(M, r.v);
  const float inv_root_d = rsqrtf((float)D);
#pragma unroll
  for (int e = 0; e < E; e++) r.v[e] *= inv_root_d;
  return r;
}
// Column block hh (one head) of the operand B_Q in buffer `dst`. Integer path: q~ as three balanced base-128 digits
// (int8) of round(q~ * (2^20 - 1) / qmax), qmax = max |q~| over the item's heads: one scale for all heads, so that
// the score read-back needs a single factor. (Two base-256 digits would halve the read-back, but 16 bits are not
// enough for lse at the logit magnitudes of outlier rows.) fp16 path: q~ as hi + lo.
template <int D, bool I8>
static __device__ __noinline__ void dec_write_operand(uint8_t* dst, int hh, DecHeadCoords<D> c, float qmax, int lane) {
  constexpr int E = D / 32;
  if constexpr (I8) {
    const float qs = qmax > 0.f ? 1048575.0f / qmax : 0.f;
#pragma unroll
    for (int e = 0; e < E; e++) {
      const int Q = __float2int_rn(c.v[e] * qs);
      const int d2 = (Q + 8192) >> 14;
      const int r = Q - (d2 << 14);
      const int d1 = (r + 64) >> 7;
      const int d0 = r - (d1 << 7);
      const int i = lane * E + e;  // contraction index = rotated coordinate; column n = 4 * head + digit
      const uint32_t word = (uint32_t)(d0 & 0xff) | ((uint32_t)(d1 & 0xff) << 8) | ((uint32_t)(d2 & 0xff) << 16);
      *reinterpret_cast<uint32_t*>(dst + 4 * (hh & 3) + (hh >> 2) * ((D / 8) * 128) + (i & 7) * 16 + (i >> 3) * 128) = word;
    }
  } else {
#pragma unroll
    for (int e = 0; e < E; e++) {
      const float x = c.v[e];
      const __half xh = __float2half_rn(x);
      const __half xl = __float2half_rn(x - __half2float(xh));
      const int i = lane * E + e;  // contraction index = rotated coordinate
      const int off = (i & 7) * 16 + (i >> 3) * 128;
      *reinterpret_cast<__half*>(dst + hh * 2 + off) = xh;                  // n = head (hi part)
      *reinterpret_cast<__half*>(dst + hh * 2 + (D / 8) * 128 + off) = xl;  // n = 8 + head (lo part)
    }
  }
}

// Decode with append: the step's new K and V rows are quantised and appended (Algorithm 1) by the launch that attends
// to them. The first aux_ctas CTAs of the grid do nothing else: their warps take the tasks of the (sequence, KV head)
// units in turn; a unit's rows are quantised and written to the cache, and with them the new row's own partial (m, l) = (z, 1), acc = v~ -- computed from the row's codes and stored
// scale, like a cached row's -- which the merge reads as one more slot. The blocks of the cache are read WITHOUT that
// row (rows below seq_lens[b]), so nothing the other warps load depends on these writes.
template <int D>
static __device__ __noinline__ void dec_aux_work(const DecodeParams& p, int lane, int first_task, int task_stride) {
  constexpr int E = D / 32;
  // A (sequence, KV head) unit is 1 + group tasks, one warp each: task 0 quantises and stores the two rows and writes
  // the value part of the partial; task 1 + j quantises the K row again (in registers) and writes head j's score.
  const int per_unit = 1 + p.group;
  const int n_tasks = p.batch * p.n_kv_heads * per_unit;
  for (int t = first_task; t < n_tasks; t += task_stride) {
    const int u = t / per_unit, part = t - u * per_unit;
    const int b = u / p.n_kv_heads, kvh = u - b * p.n_kv_heads;
    const int raw_len = p.seq_lens[b];
    bool have_new = false;
    size_t row = 0;
    if (raw_len < 0 || raw_len >= p.t_cap) {
      if (part == 0 && lane == 0 && p.status) {  // counted per (row, KV head, tensor)
        atomicOr(&p.status[0], IQ_STATUS_ROW_OUT_OF_RANGE);
        atomicAdd(&p.status[2], 2u);
      }
    } else if (!cache_row_for_write(p.pm, b, kvh, raw_len, part == 0 ? p.status : nullptr, row)) {  // no such page: skipped and counted
      if (part == 0 && lane == 0 && p.status) atomicAdd(&p.status[2], 2u);
    } else {
      have_new = true;
    }
    if (!have_new) {
      if (part == 0)
        for (int j = lane; j < p.group; j += 32) {
          const size_t bh = (size_t)b * p.n_q_heads + kvh * p.group + j;
          p.new_ml[2 * bh] = -INFINITY;
          p.new_ml[2 * bh + 1] = 0.f;
        }
      continue;
    }
    const size_t src = ((size_t)b * p.n_kv_heads + kvh) * D + lane * E;
    __half2 raw[E / 2];
#pragma unroll
    for (int k = 0; k < E / 2; k++) raw[k] = reinterpret_cast<const __half2*>(p.k_new + src)[k];
    WarpRowQuantizer<D> rq;
    rq.init(p.rot + (size_t)kvh * (D / 4) * 8, p.thresholds_k, lane);
    int code[E];
    if (part == 0) {
      const RowSink sink{const_cast<uint8_t*>(p.k_codes), const_cast<float*>(p.k_scales), const_cast<uint8_t*>(p.v_codes),
                         const_cast<float*>(p.v_scales), p.status, p.scale_f16};
      const float sk = rq.run(raw, lane, code, p.status);
      warp_store_k_row<D>(sink, row, code, sk, lane);
#pragma unroll
      for (int k = 0; k < E / 2; k++) raw[k] = reinterpret_cast<const __half2*>(p.v_new + src)[k];
      rq.set_thresholds(p.thresholds_v);
      float sv = rq.run(raw, lane, code, p.status);
      warp_store_v_row<D>(sink, row, raw_len, code, sv, lane);
      if (p.scale_f16) sv = __half2float(__float2half_rn(fminf(sv, 65504.f)));  // the scale as the cache holds it
      const float vf = sv * rsqrtf((float)D);
      float lv[E];
#pragma unroll
      for (int e = 0; e < E; e++) lv[e] = p.levels_v[code[e]] * vf;
      for (int j = 0; j < p.group; j++) {  // acc = v~, the same for every head of the KV head
        float4* a = reinterpret_cast<float4*>(p.new_acc + ((size_t)b * p.n_q_heads + kvh * p.group + j) * D + lane * E);
#pragma unroll
        for (int e4 = 0; e4 < E / 4; e4++) a[e4] = make_float4(lv[4 * e4], lv[4 * e4 + 1], lv[4 * e4 + 2], lv[4 * e4 + 3]);
      }
    } else {  // z = sm_scale q~ . k~ of the new row for one head; (m, l) = (z, 1)
      const size_t bh = (size_t)b * p.n_q_heads + kvh * p.group + (part - 1);
      float sk = rq.run(raw, lane, code, nullptr);
      if (p.scale_f16) sk = __half2float(__float2half_rn(fminf(sk, 65504.f)));
      const DecHeadCoords<D> c = dec_rotate_head<D>(p.q + bh * D, p.rot + (size_t)kvh * (D / 4) * 8, lane);
      float dot = 0.f;
#pragma unroll
      for (int e = 0; e < E; e++) dot = fmaf(c.v[e], p.levels_k[code[e]], dot);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) dot += __shfl_xor_sync(FULL, dot, o);
      if (lane == 0) {
        p.new_ml[2 * bh] = dot * sk * p.sm_scale * rsqrtf((float)D);  // z = sm_scale q~ . (s level / sqrt d)
        p.new_ml[2 * bh + 1] = 1.f;
      }
    }
  }
}

// Where the CTA's range starts (thread 0, set-up).
struct DecStart {
  int b, y, len, piece;  // sequence, item within it, rows of the sequence, which piece of the item the range starts in
  long long item_g;     // launch-wide index of block 0 of that item (<= the range's first block)
  long long g0;         // launch-wide index of the range's first block
  int count, pad;       // blocks of the range
};

template <int D, bool ARGMAX, bool I8, bool APPEND, int BITS>
__global__ void __launch_bounds__(DecLayout<D, BITS>::THREADS, 1) decode_kernel(const __grid_constant__ DecodeParams p) {
  static_assert(!APPEND || BITS == 3, "the append inside the decode launch is built for the 3-bit layout");
  using L = DecLayout<D, BITS>;
  constexpr int DJ = L::DJ;
  constexpr int E = D / 32;
  constexpr int TB = DEC_BLOCK_TOKENS;
  constexpr int NST = L::STAGES;
  constexpr int NG = L::NG;
  constexpr float LOG2E = 1.4426950408889634f;
  constexpr float LN2 = 0.6931471805599453f;

  extern __shared__ __align__(1024) uint8_t smem[];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const bool control = warp >= NG * 4;
  const int grp = control ? warp - NG * 4 : warp >> 2;  // group of this warp
  // Decode with append: the first aux_ctas CTAs append the new rows (every warp of them takes units) while the others
  // work on the blocks; those see a grid of n_cta CTAs in which they are CTA number cta.
  const int n_aux = APPEND ? p.aux_ctas : 0;
  const int cta = (int)blockIdx.x - n_aux, n_cta = (int)gridDim.x - n_aux;
  if constexpr (APPEND) {
    if (cta < 0) {
      grid_dependency_wait();
      dec_aux_work<D>(p, lane, (int)blockIdx.x * (L::THREADS / 32) + warp, n_aux * (L::THREADS / 32));
      return;
    }
  }
  const int gt = tid & (DEC_GROUP_THREADS - 1);         // compute thread within its group = TMEM lane
  const int bar_id = 1 + grp;                           // named barrier of the group's compute threads

  uint64_t* gbar = reinterpret_cast<uint64_t*>(smem + grp * L::BAR_STRIDE);
  uint64_t* full_bar = gbar;        // [stages] tile landed (or end marker)
  uint64_t* empty_bar = gbar + 3;   // [stages] staged tile consumed (128 arrivals)
  uint64_t* s_bar = gbar + 6;       // scores ready
  uint64_t* o_bar = gbar + 7;       // values ready
  uint64_t* k_ready = gbar + 8;     // K tile in TMEM (128 arrivals)
  uint64_t* p_ready = gbar + 9;     // V tile in TMEM + probabilities in smem (128 arrivals)
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + L::OFF_TMEM);
  int* next_s = reinterpret_cast<int*>(smem + L::OFF_NEXT);            // next block of the CTA's range
  DecStart* start_s = reinterpret_cast<DecStart*>(smem + L::OFF_START);
  DecDesc* desc = reinterpret_cast<DecDesc*>(smem + L::OFF_DESC + grp * L::DESC_STRIDE);  // [stages]
  float* qtmp = reinterpret_cast<float*>(smem + L::OFF_QFAC + grp * 16);  // [4] per-warp maxima of |q~|
  float* red = reinterpret_cast<float*>(smem + L::OFF_RED + grp * L::RED_STRIDE);  // [4 warps][8 heads] cross-warp scratch
  float* red2 = red + 32;
  int* redi = reinterpret_cast<int*>(red2 + 32);
  int* n_pre_s = reinterpret_cast<int*>(smem + L::OFF_PRE);
  int2* pre_tab = reinterpret_cast<int2*>(smem + L::OFF_PRE + 8);
  float* pre_sfac = reinterpret_cast<float*>(smem + L::OFF_PRE + 8 + 8 * DEC_NPRE);
  float* pre_hmax = pre_sfac + DEC_NPRE;
  uint8_t* bq_pre = smem + DEC_HDR_BYTES;                                    // B_Q of the range's first segments
  uint8_t* bq = bq_pre + L::PRE_BYTES + grp * L::GROUP_SMEM;                 // B_Q: (n, i) MN-major, this group's own
  uint8_t* bp = bq + L::BQ_BYTES;                            // B_P: (n, row) MN-major
  uint8_t* stages = bp + L::BP_BYTES;
  // Set-up scratch in group 0's B_P region and first stage: [THREADS] blocks per slice of the batch, the per-warp maxima,
  // [THREADS] non-empty sequences per slice. It is last read before the barrier that ends the set-up.
  int* scan_s = reinterpret_cast<int*>(smem + DEC_HDR_BYTES + L::PRE_BYTES + L::BQ_BYTES);

  const int S = p.splits;
  const int B = p.batch;
  const int ips = p.n_kv_heads * p.head_groups;  // items per sequence
  const bool range_mode = S >= 2 * NG;
  auto len_of = [&](int b) { return max(0, min(p.seq_lens[b] + p.len_bias, p.t_cap)); };
  auto nb_of = [&](int b) { return (len_of(b) + TB - 1) / TB; };
  auto item_heads = [&](int y, int& kvh, int& h0, int& nh) {
    kvh = y / p.head_groups;
    const int hg = y - kvh * p.head_groups;
    h0 = kvh * p.group + hg * DEC_HEADS;
    nh = min(DEC_HEADS, p.group - hg * DEC_HEADS);
  };
  // Partial slot `slot` of the heads of item (b, y) marked unused: (m, l) = (-inf, 0). Thread t writes head t.
  auto fill_slot = [&](int b, int y, int slot, int t) {
    int kvh, h0, nh;
    item_heads(y, kvh, h0, nh);
    const size_t o = ((size_t)b * p.n_q_heads + h0) * S + slot;
    dec_fill_slot(p.part_ml + 2 * o, ARGMAX ? p.part_argmax + o : nullptr, nh, S, t);
  };

  // Everything up to grid_dependency_wait() below runs while the kernel before this one on the stream may still be
  // running (programmatic dependent launch): it reads seq_lens only -- which no kernel of this library writes and the
  // caller must have written before that kernel started -- and writes nothing outside shared and tensor memory.

  // ---------------------------------------------------------------- range mode: the block sequence of the launch and this CTA's range
  // The ranges are cut at equal COST, not at equal block counts: a block costs 1 and every item a range enters costs
  // DEC_SEG_COST more (its groups close one partial and open another: measured at 8 - 10 block times per segment and
  // CTA). Block blk of item y of sequence b (nb blocks per item, ips items) sits at cost position
  //   C = C_b + y (nb + W) + W + blk,   C_b = sum over the non-empty sequences before b of ips (nb + W),
  // strictly increasing along the block sequence; CTA c owns the blocks with c * cper <= C < (c + 1) * cper.
  long long g0 = 0;
  int count = 0;  // blocks of this CTA's range (read from shared memory after the set-up barrier)
  bool no_work = false;
  int n_work = n_cta;  // CTAs of the grid that have blocks (they share the slots of the sequences without cached rows)
  if (range_mode) {
    constexpr long long W = DEC_SEG_COST;
    int* cnt_s = scan_s + L::THREADS + L::THREADS / 32;  // [THREADS] non-empty sequences per slice of the batch
    const int per_thread = (B + L::THREADS - 1) / L::THREADS;
    {
      int sum = 0, mx = 0, cnt = 0;
      for (int b = tid * per_thread; b < min(B, (tid + 1) * per_thread); b++) {
        const int n = nb_of(b);
        sum += n;
        cnt += n > 0;
        mx = max(mx, n);
      }
      scan_s[tid] = sum;
      cnt_s[tid] = cnt;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) mx = max(mx, __shfl_xor_sync(FULL, mx, o));
      if (lane == 0) scan_s[L::THREADS + warp] = mx;
    }
    __syncthreads();
    long long c_total, n_cols;  // cost of the whole launch; blocks per item column (all sequences)
    int nb_max = 0;
    {
      int v = 0, c = 0;
      for (int i = lane; i < L::THREADS; i += 32) { v += scan_s[i]; c += cnt_s[i]; }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) { v += __shfl_xor_sync(FULL, v, o); c += __shfl_xor_sync(FULL, c, o); }
      c_total = ((long long)v + W * c) * ips;
      n_cols = v;
      for (int i = 0; i < L::THREADS / 32; i++) nb_max = max(nb_max, scan_s[L::THREADS + i]);
    }
    long long cper = (c_total + n_cta - 1) / n_cta;
    cper = max(cper, (long long)((nb_max + W - 1) / (S / NG - 1) + 1));  // an item then spans at most S / NG ranges
    cper = max(cper, W + 1);                                              // and no range between two ranges of blocks is empty
    const long long t_lo = (long long)cta * cper;
    if (t_lo >= c_total) no_work = true;
    n_work = (int)min((long long)n_cta, (c_total + cper - 1) / cper);  // 0: no sequence has a cached row
    if (tid == 0 && !no_work) {
      // the first block at or after cost position t: its sequence, item, block, and launch-wide block index
      auto locate = [&](long long t, int& b, int& nb, int& y, int& blk, long long& before_nb, long long& c_b) {
        before_nb = 0;  // blocks (per item column) of the sequences before b
        long long before_cnt = 0;
        int i = 0;
        if (t >= c_total) { b = B; nb = 0; y = 0; blk = 0; before_nb = n_cols; c_b = c_total; return; }  // past the last block
        while (i < L::THREADS - 1 && ((before_nb + scan_s[i]) + W * (before_cnt + cnt_s[i])) * ips <= t) { before_nb += scan_s[i]; before_cnt += cnt_s[i]; i++; }
        b = i * per_thread;
        c_b = (before_nb + W * before_cnt) * ips;
        for (;; b++) {
          nb = (b < B) ? nb_of(b) : 0;
          if (b >= B) break;
          if (nb == 0) continue;
          if (c_b + (long long)ips * (nb + W) > t) break;
          c_b += (long long)ips * (nb + W);
          before_nb += nb;
        }
        if (b >= B) { y = 0; blk = 0; return; }  // past the last block
        const long long rel = t - c_b;
        y = (int)(rel / (nb + W));
        const long long r = rel - (long long)y * (nb + W);
        blk = (int)max(0ll, r - W);
      };
      int b = 0, nb = 0, y = 0, blk = 0, b1 = 0, nb1 = 0, y1 = 0, blk1 = 0;
      long long before = 0, c_b = 0, before1 = 0, c_b1 = 0;
#pragma unroll 1
      for (int k = 0; k < 2; k++) {  // (a loop so that the search exists once in the code)
        b = b1; nb = nb1; y = y1; blk = blk1; before = before1; c_b = c_b1;
        locate(k == 0 ? t_lo + cper : t_lo, b1, nb1, y1, blk1, before1, c_b1);
      }
      {  // the first pass found the end of the range, the second its start: swap them into place
        int ti; long long tl;
        ti = b; b = b1; b1 = ti; ti = nb; nb = nb1; nb1 = ti; ti = y; y = y1; y1 = ti; ti = blk; blk = blk1; blk1 = ti;
        tl = before; before = before1; before1 = tl; tl = c_b; c_b = c_b1; c_b1 = tl;
      }
      DecStart s0;
      s0.b = b;
      s0.len = len_of(b);
      s0.y = y;
      s0.item_g = before * ips + (long long)y * nb;
      s0.g0 = s0.item_g + blk;
      s0.count = (int)((b1 < B ? before1 * ips + (long long)y1 * nb1 + blk1 : before1 * ips) - s0.g0);
      s0.piece = (int)((long long)cta - (c_b + (long long)y * (nb + W) + W) / cper);  // CTAs since the one that holds the item's first block
      *start_s = s0;
      *next_s = 0;
      // the range's first segments: their query operands are prepared once for all groups
      int np = 0;
      long long item_g = s0.item_g;
      while (np < DEC_NPRE && b < B && max(item_g, s0.g0) < s0.g0 + s0.count) {
        pre_tab[np++] = make_int2(b, y);
        item_g += nb;
        if (++y == ips) {
          y = 0;
          do { b++; nb = (b < B) ? nb_of(b) : 0; } while (b < B && nb == 0);
        }
      }
      *n_pre_s = np;
    }
  } else {
    // unit mode: worker w = grp * grid + CTA takes units w, w + NG * grid, ...; a CTA none of whose groups has a unit leaves
    if ((long long)cta >= (long long)B * ips * S) no_work = true;
    n_work = (int)min((long long)n_cta, (long long)B * ips * S);
    if (tid == 0) *n_pre_s = 0;
  }
  if (no_work) {
    if (n_work == 0 && cta == 0) {  // not one cached row in the whole batch: this CTA marks every slot unused
      grid_dependency_wait();
      for (int b = 0; b < B; b++)
        for (int i = tid / DEC_HEADS; i < ips * S; i += L::THREADS / DEC_HEADS) fill_slot(b, i / S, i % S, tid % DEC_HEADS);
    }
    return;
  }

  // ---------------------------------------------------------------- set-up: barriers, TMEM
  if (control && elect_one()) {  // every control warp initialises the barriers of its group
#pragma unroll
    for (int st = 0; st < NST; st++) { mbar_init(&full_bar[st], 1); mbar_init(&empty_bar[st], DEC_GROUP_THREADS); }
    mbar_init(s_bar, 1);
    mbar_init(o_bar, 1);
    mbar_init(k_ready, DEC_GROUP_THREADS);
    mbar_init(p_ready, DEC_GROUP_THREADS);
    fence_mbar_init();
    fence_proxy_async();
  }
  if (warp == NG * 4) {  // the whole tensor memory of the SM: one CTA per SM
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(512));
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::);
  }
  grid_dependency_wait();  // queries, cache rows and the partial buffers are not touched above this line

  // sequences without cached rows belong to no range and no unit: the CTAs that have blocks define their partial slots, CTA c
  // those of sequences c, c + n_work, ...
  for (int b = cta; b < B; b += n_work)
    if (len_of(b) == 0)
      for (int i = tid / DEC_HEADS; i < ips * S; i += L::THREADS / DEC_HEADS) fill_slot(b, i / S, i % S, tid % DEC_HEADS);

  tc_fence_before();
  __syncthreads();  // the last CTA-wide barrier before the end of the kernel
  tc_fence_after();
  if (range_mode) { g0 = start_s->g0; count = start_s->count; }
  const uint32_t tmem_base = tmem_slot[0];
  const uint32_t tmem_g = tmem_base + (uint32_t)(grp * L::GROUP_COLS);        // this group's columns
  const uint32_t lane_sel = (uint32_t)((warp & 3) * 32) << 16;                // this warp's 32 TMEM lanes
  bool failed = false;  // a bounded wait gave up; every later wait of this thread is skipped

  if (control) {
    // ================================================================ control warp of group grp: walks the work, fetches blocks, issues MMAs.
    // All 32 lanes run the loop and the waits (the walk is uniform over the warp); an elected lane issues.
    const uint32_t bq_addr = smem_u32(bq), bp_addr = smem_u32(bp);
    // operand descriptors of the first k-step, built before the waits: a k-step further on adds its byte offset / 16
    const uint64_t bq_desc_own = smem_desc_mn(bq_addr, 128, (D / 8) * 128), bp_desc0 = smem_desc_mn(bp_addr, 128, (TB / 8) * 128);
    const uint64_t bq_desc_pre = smem_desc_mn(smem_u32(bq_pre), 128, (D / 8) * 128);
    int it = 0;         // staged slots consumed so far (tile pipeline phases), the end marker included
    int it_issue = 0;   // slots staged so far
    int nbk = 0;        // blocks processed (phases of k_ready, s_bar, p_ready, o_bar)
    bool ended = false; // the work ran out and the end marker has been staged
    // The walk over the CTA's work lives in a struct and advances in an out-of-line function (dec_draw).
    DecWalk wk;
    wk.range_mode = range_mode ? 1 : 0;
    wk.grp = grp;
    wk.ng = NG;
    wk.ips = ips;
    wk.count = count;
    wk.g0 = g0;
    wk.g_end = g0 + count;
    wk.touched = 0;
    wk.sidx = 0;
    wk.n_pre = *n_pre_s;
    if (range_mode) { wk.b = start_s->b; wk.y = start_s->y; wk.len = start_s->len; wk.nb = (wk.len + TB - 1) / TB; wk.piece = start_s->piece; wk.item_g = start_s->item_g; }
    else { wk.b = wk.y = wk.nb = wk.len = wk.piece = 0; wk.item_g = 0; }
    wk.n_units = B * ips * S;
    wk.unit_step = NG * n_cta;
    wk.unit = min(wk.n_units, grp * n_cta + cta);
    wk.ub = wk.uy = wk.uk = wk.ublk = wk.uhi = wk.unew = wk.ulen = 0;
    // The next block is drawn (shared counter; with a paged cache also its block-table entry, a load from global
    // memory) while the compute warps are busy with the softmax of the current one, and staged after the value MMAs.
    DecDrawn dr;
    dr.kind = -1;
    auto draw = [&]() {
      dec_draw<D>(p, wk, dr, next_s, lane, ARGMAX ? 1 : 0);
    };
    auto stage_next = [&]() {  // the drawn (or next) block into slot it_issue, or the end marker
      const int st = it_issue % NST;
      if (it_issue >= NST && !failed)  // the slot's previous occupant has been consumed
        failed = !mbar_wait_bounded(&empty_bar[st], (uint32_t)(it_issue / NST - 1) & 1u, DEC_WAIT_LIMIT);
      if (dr.kind < 0 && !failed) draw();
      if (dr.kind == 0 && !failed) {
        const int r0 = dr.blk * TB;
        const int n = min(TB, dr.len - r0);
        if (elect_one()) {
          DecDesc dd;
          dd.n = n; dd.flags = dr.is_new; dd.r0 = r0; dd.slot = dr.slot; dd.b = dr.b; dd.y = dr.y; dd.len = dr.len; dd.bqbuf = dr.bqbuf;
          desc[st] = dd;
          const uint32_t sc_bytes = p.scale_f16 ? (uint32_t)(((n + 7) & ~7) * 2) : (uint32_t)(((n + 3) & ~3) * 4);  // whole 16-byte pieces
          uint8_t* sp = stages + st * L::STAGE_BYTES;
          const size_t row0 = dr.row0;
          fence_proxy_async();
          mbar_expect_tx(&full_bar[st], (uint32_t)(n * L::ROWB + L::VT_BYTES) + 2 * sc_bytes);  // also publishes desc[st]
          bulk_g2s(sp, p.k_codes + row0 * L::ROWB, (uint32_t)(n * L::ROWB), &full_bar[st]);
          bulk_g2s(sp + L::K_BYTES, p.v_codes + row0 * L::ROWB, (uint32_t)L::VT_BYTES, &full_bar[st]);  // whole 128-row V block
          bulk_g2s(sp + L::K_BYTES + L::VT_BYTES, reinterpret_cast<const uint8_t*>(p.k_scales) + row0 * (p.scale_f16 ? 2 : 4), sc_bytes, &full_bar[st]);
          bulk_g2s(sp + L::K_BYTES + L::VT_BYTES + L::SC_BYTES, reinterpret_cast<const uint8_t*>(p.v_scales) + row0 * (p.scale_f16 ? 2 : 4), sc_bytes, &full_bar[st]);
        }
        dr.kind = -1;
      } else {
        ended = true;
        if (elect_one()) {
          desc[st].n = -1;  // end marker: no tile, the group closes what it has open and leaves
          mbar_arrive(&full_bar[st]);
        }
      }
      __syncwarp();
      it_issue++;
    };
    for (;;) {
#pragma unroll 1
      while (!ended && it_issue - it < NST) stage_next();  // keep the pipeline full (at the start: tiles in flight while the compute warps open their first segment)
      if (ended && it == it_issue - 1) { it++; break; }  // slot `it` holds the end marker
      // scores of the block in slot `it`: S = A_K * B_Q^T once all 128 rows are in TMEM (and B_Q of its segment is complete)
      if (!failed) failed = !mbar_wait_bounded(k_ready, (uint32_t)nbk & 1u, DEC_WAIT_LIMIT);
      if (failed) break;
      tc_fence_after();
      const int bqbuf = desc[it % NST].bqbuf;  // the query operand of the block's segment (the start address field counts 16-byte units)
      const uint64_t bq_desc0 = bqbuf < 0 ? bq_desc_own : bq_desc_pre + (uint64_t)(bqbuf * (L::BQ_BYTES / 16));
      if (elect_one()) {
        if constexpr (I8) {
#pragma unroll
          for (int kk = 0; kk < D / 32; kk++)
            tc_mma_i8(tmem_g + L::I8_S_COL, tmem_g + L::I8_K_COL + 8 * kk, bq_desc0 + 32 * kk, DEC_IDESC_I8_SS, kk > 0);
        } else {
#pragma unroll
          for (int kk = 0; kk < D / 16; kk++)
            tc_mma_f16(tmem_g + L::S_COL, tmem_g + L::A_COL + 8 * kk, bq_desc0 + 16 * kk, DEC_IDESC, kk > 0);
        }
        tc_commit(s_bar);
      }
      __syncwarp();
      if (!ended && dr.kind < 0) draw();
      // values: O = A_V * B_P^T once the V tile is in TMEM and the probabilities are in shared memory
      failed = !mbar_wait_bounded(p_ready, (uint32_t)nbk & 1u, DEC_WAIT_LIMIT);
      if (failed) break;
      tc_fence_after();
      const bool keep_values = I8 && *reinterpret_cast<volatile int*>(smem + L::OFF_ACCF + 4 * grp) != 0;
      if (elect_one()) {
        if constexpr (I8) {
#pragma unroll
          for (int j = 0; j < DJ; j++)
#pragma unroll
            for (int kk = 0; kk < TB / 32; kk++)  // the values stay in TMEM (int32) over the blocks until the compute threads read them
              tc_mma_i8(tmem_g + L::I8_O_COL + 32 * j, tmem_g + L::I8_V_COL + 32 * j + 8 * kk, bp_desc0 + 32 * kk, DEC_IDESC_I8_SU,
                        (kk > 0) || keep_values);
        } else {
#pragma unroll
          for (int j = 0; j < DJ; j++)
#pragma unroll
            for (int kk = 0; kk < TB / 16; kk++)
              tc_mma_f16(tmem_g + L::O_COL + 16 * j,  // rows 0..63 of the V tile sit in V_COL, rows 64..127 in the operand columns
                         tmem_g + (kk < 4 ? L::V_COL + 32 * j + 8 * kk : L::A_COL + 64 * j + 8 * (kk - 4)),
                         bp_desc0 + 16 * kk, DEC_IDESC, kk > 0);
        }
        tc_commit(o_bar);
      }
      __syncwarp();
      it++;
      nbk++;  // the compute threads released the slot when they signalled p_ready: the loop stages the next block into it
    }
    if (failed) {
      // Give-up path. Tiles staged and not consumed may still be landing: wait (bounded) for each of them, so that no
      // bulk copy targets this CTA's shared memory after it has left. Tensor-core work in flight is covered by the
      // fence before the TMEM release at the end of the kernel.
      for (int s = it; s < it_issue; s++) mbar_wait_bounded(&full_bar[s % NST], (uint32_t)(s / NST) & 1u, DEC_WAIT_LIMIT);
    }
  }
  if (!control) {
    // ================================================================ compute warps of group grp
    const float inv_root_d = rsqrtf((float)D);
    const float kfac = p.sm_scale * LOG2E * inv_root_d;  // scores in log2 units: z2 = S_raw * scale_K * kfac
    const float vfac = inv_root_d;
    float acc[DJ][8];  // thread c: coordinates c (+128), 8 heads
    float m_run[8], l_run[8], best_v[8];
    int best_i[8];
    float sfac = 0.f;  // integer path: score digits -> log2-domain score per unit K scale (set when a segment is opened)
    int it = 0;        // staged slots of this group consumed so far (tile pipeline phases), the end marker included
    int nbk = 0;       // blocks this group has processed (phases of k_ready, s_bar, p_ready, o_bar)
    int* seg_id = reinterpret_cast<int*>(smem + L::OFF_SEGID + 16 * grp);  // the open segment: (sequence, item, slot); kept in shared memory between open and close

    auto rotate_head = [&](int b, int kvh, int h_abs, bool present, float (&v)[E]) {
      const DecHeadCoords<D> c = dec_rotate_head<D>(present ? p.q + ((size_t)b * p.n_q_heads + h_abs) * D : nullptr,
                                                    p.rot + (size_t)kvh * (D / 4) * 8, lane);
#pragma unroll
      for (int e = 0; e < E; e++) v[e] = c.v[e];
    };
    auto abs_max = [&](const float (&v)[E]) {
      float m = 0.f;
#pragma unroll
      for (int e = 0; e < E; e++) m = fmaxf(m, fabsf(v[e]));
      return warp_max(m);
    };
    auto write_operand = [&](uint8_t* dst, int hh, const float (&v)[E], float qmax) {
      DecHeadCoords<D> c;
#pragma unroll
      for (int e = 0; e < E; e++) c.v[e] = v[e];
      dec_write_operand<D, I8>(dst, hh, c, qmax, lane);
    };
    auto score_factor = [&](float qmax) { return (qmax * (1.0f / 1048575.0f)) * p.delta * kfac; };  // digits -> log2-domain score per unit K scale

    // ---- the operands of the range's first segments, built once for all groups of the CTA by all compute warps
    // (a group that meets a later segment, or works in unit mode, builds the operand itself in open_segment)
    {
      const int n_pre = *n_pre_s;
      if (n_pre > 0) {
        constexpr int NCW = NG * 4, JOBS = (8 * DEC_NPRE + NCW - 1) / NCW;
        float v[JOBS][E];
#pragma unroll
        for (int t = 0; t < JOBS; t++) {
          const int job = warp + t * NCW, sg = job >> 3, hh = job & 7;
          int kvh = 0, h0 = 0, nh = 0, b = 0;
          if (sg < n_pre) { b = pre_tab[sg].x; item_heads(pre_tab[sg].y, kvh, h0, nh); }
          rotate_head(b, kvh, h0 + hh, sg < n_pre && hh < nh, v[t]);
          if (I8 && sg < DEC_NPRE) {
            const float m = abs_max(v[t]);
            if (lane == 0) pre_hmax[sg * 8 + hh] = m;
          }
        }
        if (I8) cta_bar_sync_n(DEC_PRE_BAR, L::COMPUTE_THREADS);
#pragma unroll
        for (int t = 0; t < JOBS; t++) {
          const int job = warp + t * NCW, sg = job >> 3, hh = job & 7;
          if (sg < n_pre) {
            float qmax = 0.f;
            if (I8) {
#pragma unroll
              for (int h2 = 0; h2 < 8; h2++) qmax = fmaxf(qmax, pre_hmax[sg * 8 + h2]);
              if (hh == 0 && lane == 0) pre_sfac[sg] = score_factor(qmax);
            }
            write_operand(bq_pre + sg * L::BQ_BYTES, hh, v[t], qmax);
          }
        }
        fence_proxy_async();  // the operands are written through the generic proxy and read by the tensor core through the async proxy
        cta_bar_sync_n(DEC_PRE_BAR, L::COMPUTE_THREADS);
      }
    }

    // ---- open a segment: reset the softmax state; the operand B_Q is either one of the prepared ones (dd.bqbuf >= 0)
    // or written here into the group's own buffer, warp w of the group rotating heads w and w + 4. The operand is read
    // by the score MMAs of the segment's blocks, which the control warp issues after every thread of the group has
    // signalled k_ready, i.e. after this function.
    auto open_segment = [&](const DecDesc& dd) {
      const int seg_b = dd.b, seg_y = dd.y, bqbuf = dd.bqbuf;
      if (gt == 0) { seg_id[0] = seg_b; seg_id[1] = seg_y; seg_id[2] = dd.slot; }  // read back in close_segment, barriers in between
#pragma unroll
      for (int j = 0; j < DJ; j++)
#pragma unroll
        for (int h = 0; h < 8; h++) acc[j][h] = 0.f;
#pragma unroll
      for (int h = 0; h < 8; h++) { m_run[h] = -INFINITY; l_run[h] = 0.f; best_v[h] = -INFINITY; best_i[h] = -1; }
      if (bqbuf >= 0) {
        if (I8) sfac = pre_sfac[bqbuf];
        return;
      }
      int kvh, h0, nh;
      item_heads(seg_y, kvh, h0, nh);
      const int wq = warp & 3;
      float v[2][E];
#pragma unroll
      for (int t = 0; t < 2; t++) rotate_head(seg_b, kvh, h0 + wq + 4 * t, wq + 4 * t < nh, v[t]);
      float qmax = 0.f;
      if constexpr (I8) {
        qmax = fmaxf(abs_max(v[0]), abs_max(v[1]));
        if (lane == 0) qtmp[wq] = qmax;
        group_bar_sync(bar_id);
        qmax = fmaxf(fmaxf(qtmp[0], qtmp[1]), fmaxf(qtmp[2], qtmp[3]));
        sfac = score_factor(qmax);
      }
#pragma unroll
      for (int t = 0; t < 2; t++) write_operand(bq, wq + 4 * t, v[t], qmax);
      fence_proxy_async();  // B_Q is written through the generic proxy and read by the tensor core through the async proxy
    };

    // ---- close the open segment: reduce l and the exact maximum (and argmax) over the group's 128 rows and write the
    // group's partial to its slot of the item (d5 merges the slots). Called with the group's value MMAs complete and
    // acc up to date.
    auto close_segment = [&]() {
      const int seg_b = seg_id[0], seg_y = seg_id[1], seg_slot = seg_id[2];
      int kvh, h0, nh;
      item_heads(seg_y, kvh, h0, nh);
      if constexpr (!ARGMAX) {
        // without the argmax output the partial is reported relative to the running reference as it stands
        float* dst = p.part_acc + (((size_t)seg_b * p.n_q_heads + h0) * S + seg_slot) * D + gt;
        const size_t hstride = (size_t)S * D;
#pragma unroll
        for (int h = 0; h < 8; h++)
          if (h < nh) {
#pragma unroll
            for (int j = 0; j < DJ; j++) dst[h * hstride + 128 * j] = acc[j][h];
          }
        const int hr = warp_reduce8_head(lane);  // the head whose sum this lane ends up with
        const float lsum = warp_reduce8(l_run, lane, [](float x, float y) { return x + y; });
        float msel = m_run[0];  // m_run[hr] (every thread of the group holds the same references)
#pragma unroll
        for (int h = 1; h < 8; h++) msel = (hr == h) ? m_run[h] : msel;
        if ((lane & 3) == 0) {
          red[(warp & 3) * 8 + hr] = lsum;
          if ((warp & 3) == 0) red2[hr] = msel;
        }
        group_bar_sync(bar_id);
        if (gt < nh) {
          const size_t o = ((size_t)seg_b * p.n_q_heads + h0 + gt) * S + seg_slot;
          p.part_ml[2 * o] = red2[gt] * LN2;
          p.part_ml[2 * o + 1] = red[gt] + red[8 + gt] + red[16 + gt] + red[24 + gt];
        }
        return;  // (the scratch is written next after the group barrier of the next block's vote)
      }
      {
        const int hr = warp_reduce8_head(lane);  // the head whose sums this lane ends up with
        const float lsum = warp_reduce8(l_run, lane, [](float x, float y) { return x + y; });
        if ((lane & 3) == 0) red[(warp & 3) * 8 + hr] = lsum;
        if (ARGMAX) {
          float bv;
          int bi;
          warp_argmax8(best_v, best_i, lane, bv, bi);
          if ((lane & 3) == 0) { red2[(warp & 3) * 8 + hr] = bv; redi[(warp & 3) * 8 + hr] = bi; }
        }
      }
      group_bar_sync(bar_id);
      float scale[8];  // the partial is reported relative to the exact maximum where that is tracked
#pragma unroll
      for (int h = 0; h < 8; h++) {
        float mt = m_run[h];  // every thread of the group holds the same reference
        int bi = -1;
        if (ARGMAX) {
          mt = -INFINITY;
#pragma unroll
          for (int wq = 0; wq < 4; wq++) {
            argmax_merge(mt, bi, red2[wq * 8 + h], redi[wq * 8 + h]);
          }
        }
        scale[h] = ARGMAX ? ex2f(m_run[h] - mt) : 1.f;
        if (gt == h && h < nh) {
          const size_t o = ((size_t)seg_b * p.n_q_heads + h0 + h) * S + seg_slot;
          p.part_ml[2 * o] = mt * LN2;
          p.part_ml[2 * o + 1] = (red[h] + red[8 + h] + red[16 + h] + red[24 + h]) * scale[h];
          if (ARGMAX) p.part_argmax[o] = bi;
        }
      }
#pragma unroll
      for (int h = 0; h < 8; h++)
        if (h < nh) {
#pragma unroll
          for (int j = 0; j < DJ; j++)
            p.part_acc[(((size_t)seg_b * p.n_q_heads + h0 + h) * S + seg_slot) * D + gt + 128 * j] = acc[j][h] * scale[h];
        }
      // (the scratch is written next after the group barrier of the next block's vote)
    };

    int st = 0;          // stage of slot `it` and its phase, kept incrementally
    uint32_t st_ph = 0;
    int2 dsc = make_int2(-1, 0);  // (valid rows | end marker, flags) of slot `it`; the rest of its descriptor is read where it is needed
    auto next_slot = [&]() {      // wait for slot `it` and read its descriptor
      if (!failed) failed = !mbar_wait_bounded(&full_bar[st], st_ph, DEC_WAIT_LIMIT);
      if (failed) { dsc.x = -1; return; }
      dsc = *reinterpret_cast<const int2*>(&desc[st]);
    };
    auto advance_slot = [&]() {
      it++;
      if (++st == NST) { st = 0; st_ph ^= 1u; }
    };
    next_slot();

    if constexpr (I8) {
      // Integer path. The group's TMEM columns: K tile (d/4), V tile (32 per 128 coordinates), scores (32 = 8 heads x 4
      // digit columns), values (32 per 128 coordinates). The tiles do not share columns: the V tile of a block is
      // dequantised while its score MMAs run, the K tile of the next block while its value MMAs run.
      constexpr int NLR = BITS == 4 ? 4 : (BITS == 3 ? 2 : 1);  // registers of a level table
      uint32_t lk8[4], lv8[4];  // the int8 levels of the K and of the V codebook
#pragma unroll
      for (int i = 0; i < 4; i++) { lk8[i] = i < NLR ? p.lut8[i] : 0u; lv8[i] = i < NLR ? p.lut8_v[i] : 0u; }
      float vref = 0.f;    // power of two >= every V scale (x 1/sqrt d) seen by the group in this segment
      float pscale = 0.f;  // probabilities are written as round(p * vscale * pscale) <= 2^30: pscale = 2^(30 - slack) / vref
      // The value products of consecutive blocks accumulate in TMEM as int32 (exact) for as long as the references they are
      // relative to (m_run, vref) stand; nacc counts the blocks in there. A block adds at most 128 * 127 * 255 < 2^22 per
      // column, so 384 blocks stay below 2^31. flush() adds the accumulated digits to the float accumulator.
      int nacc = 0;
      int* accf = reinterpret_cast<int*>(smem + L::OFF_ACCF + 4 * grp);  // tells the control warp to accumulate onto TMEM
      auto flush = [&]() {
        const float ofac = p.delta_v * vref * ((float)(1 << IQ_SLACK_I8) / 1073741824.0f);  // value digits -> real units: delta / pscale
        tc_fence_after();
#pragma unroll
        for (int j = 0; j < DJ; j++)
#pragma unroll
          for (int half = 0; half < 2; half++) {
            uint32_t o_u[16];
            tc_ld16_issue(tmem_g + lane_sel + L::I8_O_COL + 32 * j + 16 * half, o_u);
            tc_wait_ld();
#pragma unroll
            for (int hq = 0; hq < 4; hq++) {
              const float of = fmaf(fmaf(fmaf(__int2float_rn((int)o_u[4 * hq + 3]), 256.f, __int2float_rn((int)o_u[4 * hq + 2])), 256.f,
                                         __int2float_rn((int)o_u[4 * hq + 1])), 256.f, __int2float_rn((int)o_u[4 * hq]));
              acc[j][4 * half + hq] = fmaf(of, ofac, acc[j][4 * half + hq]);
            }
          }
        tc_fence_before();
        nacc = 0;
      };
      auto k_tile = [&](const uint8_t* sp_) {  // K row gt of the staged tile -> TMEM lane gt, then signal the control warp
        uint32_t kw[L::WPR];
        const uint4* krow = reinterpret_cast<const uint4*>(sp_ + gt * L::ROWB);
#pragma unroll
        for (int i = 0; i < L::WPR / 4; i++) {
          const uint4 t4 = krow[i];
          kw[4 * i] = t4.x; kw[4 * i + 1] = t4.y; kw[4 * i + 2] = t4.z; kw[4 * i + 3] = t4.w;
        }
#pragma unroll
        for (int u = 0; u < 4 * DJ; u += 2) {  // twice 32 coordinates per TMEM store
          uint32_t f[16];
          dequant32_i8<BITS>(kw + BITS * u, lk8, f);
          dequant32_i8<BITS>(kw + BITS * (u + 1), lk8, f + 8);
          tc_st16(tmem_g + lane_sel + L::I8_K_COL + 8 * u, f);
        }
        tc_wait_st();
        tc_fence_before();
        mbar_arrive(k_ready);
      };
#pragma unroll 1
      while (dsc.x >= 0) {  // one segment per pass: slot `it` holds the first block this group gets of it
        open_segment(desc[st]);
        vref = 0.f;
        pscale = 0.f;
        nacc = 0;
        k_tile(stages + st * L::STAGE_BYTES);
        bool more = true;
#pragma unroll 1
      while (more) {  // the blocks of the segment
        const uint8_t* sp = stages + st * L::STAGE_BYTES;
        const int n = dsc.x;
        const int r0 = ARGMAX ? desc[st].r0 : 0;
        (void)r0;
        // ---- V coordinate gt (+128) of this block -> TMEM lane gt, while the score MMAs run
#pragma unroll
        for (int j = 0; j < DJ; j++) {
          const uint4* vrow = reinterpret_cast<const uint4*>(sp + L::K_BYTES + (gt + 128 * j) * L::VREC);
          uint32_t wd[4 * BITS];
#pragma unroll
          for (int i = 0; i < BITS; i++) {
            const uint4 t4 = vrow[i];
            wd[4 * i] = t4.x; wd[4 * i + 1] = t4.y; wd[4 * i + 2] = t4.z; wd[4 * i + 3] = t4.w;
          }
#pragma unroll
          for (int u = 0; u < 4; u += 2) {  // twice 32 rows per TMEM store
            uint32_t f[16];
            dequant32_i8<BITS>(wd + BITS * u, lv8, f);
            dequant32_i8<BITS>(wd + BITS * (u + 1), lv8, f + 8);
            tc_st16(tmem_g + lane_sel + L::I8_V_COL + 32 * j + 8 * u, f);
          }
        }
        const float ksc = load_scale(sp + L::K_BYTES + L::VT_BYTES, gt, p.scale_f16);
        const float vsc = load_scale(sp + L::K_BYTES + L::VT_BYTES + L::SC_BYTES, gt, p.scale_f16);
        const bool valid = gt < n;  // rows >= n of the last block hold stale bytes
        const float kfs = valid ? ksc * sfac : 0.f;
        const float mask = valid ? 0.f : -INFINITY;  // stale rows: 0 * finite - inf = -inf
        const float vf = valid ? vsc * vfac : 0.f;

        // ---- scores: three int32 digit columns per head -> log2-domain score of row gt
        if (!failed) failed = !mbar_wait_bounded(s_bar, (uint32_t)nbk & 1u, DEC_WAIT_LIMIT);
        if (failed) break;
        tc_fence_after();
        float s[8];
        {
          auto digits_to_scores = [&](const uint32_t (&raw_u)[16], int half) {
#pragma unroll
            for (int hq = 0; hq < 4; hq++) {  // S = (S0 + 128 S1) + 16384 S2: the lower two digits combine in an int32 (< 2^28)
              const float lo = __int2float_rn((int)raw_u[4 * hq + 1] * 128 + (int)raw_u[4 * hq]);
              s[4 * half + hq] = fmaf(fmaf(__int2float_rn((int)raw_u[4 * hq + 2]), 16384.f, lo), kfs, mask);
            }
          };
          uint32_t raw0[16], raw1[16];
          tc_ld16_issue(tmem_g + lane_sel + L::I8_S_COL, raw0);
          tc_wait_ld();
          tc_ld16_issue(tmem_g + lane_sel + L::I8_S_COL + 16, raw1);  // heads 4..7 in flight while heads 0..3 are converted
          digits_to_scores(raw0, 0);
          tc_wait_ld();
          digits_to_scores(raw1, 1);
        }
        if (ARGMAX) {  // exact maximum seen by this thread and its row (a group sees the blocks of a segment in ascending order)
#pragma unroll
          for (int h = 0; h < 8; h++)
            if (s[h] > best_v[h]) { best_v[h] = s[h]; best_i[h] = r0 + gt; }
        }
        // The running reference m_run is raised when a score exceeds it by more than DEC_MAX_SLACK_I8 log2 units, the
        // V-scale bound vref when a row exceeds it: both are rare after the first blocks (one barrier with an OR reduction
        // otherwise).
        float over[8];
#pragma unroll
        for (int h = 0; h < 8; h++) over[h] = s[h] - m_run[h];  // NaN (-inf - -inf) for a stale row of an unopened reference: max ignores it
        const bool exceed = max3f(max3f(over[0], over[1], over[2]), max3f(over[3], over[4], over[5]), fmaxf(over[6], over[7])) > DEC_MAX_SLACK_I8 ||
                            vf > vref || nacc >= 384;
        
        if (group_bar_or(bar_id, exceed)) {
          if (nacc > 0) flush();  // what TMEM holds is relative to the old references (the previous value MMAs have completed)
          {
            const float wm = warp_reduce8(s, lane, [](float x, float y) { return fmaxf(x, y); });
            if ((lane & 3) == 0) red[(warp & 3) * 8 + warp_reduce8_head(lane)] = wm;
          }
          const float wv_max = warp_max(vf);
          if (lane == 0) red2[warp & 3] = wv_max;
          group_bar_sync(bar_id);
#pragma unroll
          for (int h = 0; h < 8; h++) {
            const float bm = fmaxf(fmaxf(red[h], red[8 + h]), fmaxf(red[16 + h], red[24 + h]));
            const float mn = fmaxf(m_run[h], bm + DEC_RAISE_MARGIN);  // every head goes above its block maximum whichever head asked: fewer raises later
            const float alpha = ex2f(m_run[h] - mn);  // the accumulator holds the blocks before this one: rescale it now
            m_run[h] = mn;
            l_run[h] *= alpha;
#pragma unroll
            for (int j = 0; j < DJ; j++) acc[j][h] *= alpha;
            over[h] = s[h] - mn;
          }
          const float bv = fmaxf(fmaxf(red2[0], red2[1]), fmaxf(red2[2], red2[3]));
          if (bv > vref) vref = __uint_as_float((__float_as_uint(bv) + 0x007FFFFFu) & 0x7F800000u);  // next power of two
          pscale = vref > 0.f ? (1073741824.0f / (float)(1 << IQ_SLACK_I8)) / vref : 0.f;  // p * vscale * pscale <= 2^30
        }
        {
          // probabilities (times scale_V / sqrt(d)) as 30-bit fixed point: the bytes of round(p * vscale * pscale) are its four
          // base-256 digits. B_P[n][row], n = 4 head + digit.
          uint32_t pb[8];
          const float vfp = vf * pscale;
#pragma unroll
          for (int h = 0; h < 8; h++) {
            const float pr = ex2f(over[h]);
            l_run[h] += pr;
            pb[h] = __float2uint_rn(pr * vfp);
          }
          const int off = (gt & 7) * 16 + (gt >> 3) * 128;
          *reinterpret_cast<uint4*>(bp + off) = make_uint4(pb[0], pb[1], pb[2], pb[3]);
          *reinterpret_cast<uint4*>(bp + (TB / 8) * 128 + off) = make_uint4(pb[4], pb[5], pb[6], pb[7]);
          fence_proxy_async();
        }
        if (gt == 0) *accf = nacc;     // 0: this block's value product starts a new accumulation
        nacc++;
        tc_wait_st();
        tc_fence_before();
        mbar_arrive(p_ready);          // V tile in TMEM, probabilities in shared memory
        mbar_arrive(&empty_bar[st]);   // this thread is done with the staged tile

        // ---- next slot: if it continues the segment, its K tile now, while the value MMAs run
        advance_slot();
        next_slot();
        more = dsc.x >= 0 && !(dsc.y & 1);
        if (more) k_tile(stages + st * L::STAGE_BYTES);

        // ---- the value MMAs of this block must have completed before its V tile and B_P are overwritten; their result stays in TMEM
        if (!failed) failed = !mbar_wait_bounded(o_bar, (uint32_t)nbk & 1u, DEC_WAIT_LIMIT);
        nbk++;
      }
        if (failed) break;
        if (nacc > 0) flush();
        close_segment();
      }
    } else {
      // fp16 path. The group's 128 TMEM columns: [0, 64 DJ) operand tile, then scores, values, and V_COL.. a second home for
      // the first half of the V tile. Schedule of one block (K tile complete, k_ready signalled):
      //   V rows 0..63 -> V_COL columns               while the score MMAs read the K tile
      //   wait for the scores; V rows 64..127 -> lower half of the operand columns, interleaved with the softmax
      //   signal p_ready; next block's K coordinates 32..63 (+64..) -> upper half of the operand columns
      //                                                while the value MMAs read the lower half and V_COL
      //   wait for the values, fold them; next block's other K coordinates -> lower half; signal k_ready
      uint32_t lk_lo[4], lk_hi[4], lv_lo[4], lv_hi[4];  // low / high bytes of the fp16 levels of the K and of the V codebook
#pragma unroll
      for (int i = 0; i < 4; i++) {
        constexpr int NLR = BITS == 4 ? 4 : (BITS == 3 ? 2 : 1);
        lk_lo[i] = i < NLR ? p.lut_lo[i] : 0u; lk_hi[i] = i < NLR ? p.lut_hi[i] : 0u;
        lv_lo[i] = i < NLR ? p.lut_v_lo[i] : 0u; lv_hi[i] = i < NLR ? p.lut_v_hi[i] : 0u;
      }
      uint32_t kw[L::WPR];                    // packed K row of the block being staged into TMEM
      auto k_load = [&](const uint8_t* sp_) {
        const uint4* krow = reinterpret_cast<const uint4*>(sp_ + gt * L::ROWB);
#pragma unroll
        for (int i = 0; i < L::WPR / 4; i++) {
          const uint4 t4 = krow[i];
          kw[4 * i] = t4.x; kw[4 * i + 1] = t4.y; kw[4 * i + 2] = t4.z; kw[4 * i + 3] = t4.w;
        }
      };
      auto k_unit = [&](int u) {
        uint32_t f[16];
        dequant32_f16<BITS>(kw + BITS * u, lk_lo, lk_hi, f);
        tc_st16(tmem_g + lane_sel + L::A_COL + 16 * u, f);
      };
#pragma unroll 1
      while (dsc.x >= 0) {  // one segment per pass: slot `it` holds the first block this group gets of it
        open_segment(desc[st]);
        k_load(stages + st * L::STAGE_BYTES);  // the whole K tile
#pragma unroll
        for (int u = 0; u < 4 * DJ; u++) k_unit(u);
        tc_wait_st();
        tc_fence_before();
        mbar_arrive(k_ready);
        bool more = true;
#pragma unroll 1
      while (more) {  // the blocks of the segment
        const uint8_t* sp = stages + st * L::STAGE_BYTES;
        const int n = dsc.x;
        const int r0 = ARGMAX ? desc[st].r0 : 0;
        (void)r0;
        // ---- V coordinate gt (+128): rows 0..63 now, rows 64..127 with the softmax
        uint32_t wd[DJ][4 * BITS];
#pragma unroll
        for (int j = 0; j < DJ; j++) {
          const uint4* vrow = reinterpret_cast<const uint4*>(sp + L::K_BYTES + (gt + 128 * j) * L::VREC);
#pragma unroll
          for (int i = 0; i < BITS; i++) {
            const uint4 t4 = vrow[i];
            wd[j][4 * i] = t4.x; wd[j][4 * i + 1] = t4.y; wd[j][4 * i + 2] = t4.z; wd[j][4 * i + 3] = t4.w;
          }
        }
        const float ksc = load_scale(sp + L::K_BYTES + L::VT_BYTES, gt, p.scale_f16);
        const float vsc = load_scale(sp + L::K_BYTES + L::VT_BYTES + L::SC_BYTES, gt, p.scale_f16);
        auto v_unit = [&](int j, int u) {  // rows 32u .. 32u+31 of coordinate gt + 128 j
          uint32_t f[16];
          dequant32_f16<BITS>(wd[j] + BITS * u, lv_lo, lv_hi, f);
          const uint32_t col = (u < 2) ? (uint32_t)(L::V_COL + 32 * j + 16 * u) : (uint32_t)(L::A_COL + 64 * j + 16 * (u - 2));
          tc_st16(tmem_g + lane_sel + col, f);
        };
#pragma unroll
        for (int j = 0; j < DJ; j++) { v_unit(j, 0); v_unit(j, 1); }

        // the score MMAs read the K tile that the rest of the V tile is about to overwrite
        if (!failed) failed = !mbar_wait_bounded(s_bar, (uint32_t)nbk & 1u, DEC_WAIT_LIMIT);
        if (failed) break;
        tc_fence_after();
        uint32_t raw_u[16];
        tc_ld16_issue(tmem_g + lane_sel + L::S_COL, raw_u);  // scores of row gt: in flight during the next unit
#pragma unroll
        for (int j = 0; j < DJ; j++) v_unit(j, 2);

        // ---- online softmax (log2 units); thread gt owns row r0 + gt, all 8 heads
        tc_wait_ld();
        float s[8];
        {
          const bool valid = gt < n;  // rows >= n of the last block hold stale bytes
          const float kf = valid ? ksc * kfac : 0.f;
          const float mask = valid ? 0.f : -INFINITY;  // stale rows: 0 * finite - inf = -inf
#pragma unroll
          for (int h = 0; h < 8; h++) s[h] = fmaf(__uint_as_float(raw_u[h]) + __uint_as_float(raw_u[8 + h]), kf, mask);
        }
        if (ARGMAX) {  // exact maximum seen by this thread and its row (a group sees the blocks of a segment in ascending order)
#pragma unroll
          for (int h = 0; h < 8; h++)
            if (s[h] > best_v[h]) { best_v[h] = s[h]; best_i[h] = r0 + gt; }
        }
        // The running reference m_run is raised only when some score of the block exceeds it by more than
        // DEC_MAX_SLACK (log2 units): exp2(s - m_run) then stays below 2^DEC_MAX_SLACK and nothing has to be
        // exchanged between the warps in the common case (one barrier with an OR reduction).
        float over[8];
#pragma unroll
        for (int h = 0; h < 8; h++) over[h] = s[h] - m_run[h];  // NaN (-inf - -inf) for a stale row of an unopened reference: max ignores it
        const bool exceed = max3f(max3f(over[0], over[1], over[2]), max3f(over[3], over[4], over[5]), fmaxf(over[6], over[7])) > DEC_MAX_SLACK;
        if (group_bar_or(bar_id, exceed)) {
          {
            const float wm = warp_reduce8(s, lane, [](float x, float y) { return fmaxf(x, y); });
            if ((lane & 3) == 0) red[(warp & 3) * 8 + warp_reduce8_head(lane)] = wm;
          }
          group_bar_sync(bar_id);
#pragma unroll
          for (int h = 0; h < 8; h++) {
            const float bm = fmaxf(fmaxf(red[h], red[8 + h]), fmaxf(red[16 + h], red[24 + h]));
            const float mn = fmaxf(m_run[h], bm + DEC_RAISE_MARGIN);  // every head goes above its block maximum whichever head asked: fewer raises later
            const float alpha = ex2f(m_run[h] - mn);  // the accumulator holds the blocks before this one: rescale it now
            m_run[h] = mn;
            l_run[h] *= alpha;
#pragma unroll
            for (int j = 0; j < DJ; j++) acc[j][h] *= alpha;
            over[h] = s[h] - mn;
          }
        }
#pragma unroll
        for (int j = 0; j < DJ; j++) v_unit(j, 3);  // the last V unit, next to the exponentials
        {
          const float vf = (gt < n) ? vsc * vfac : 0.f;
          float wv[8];
#pragma unroll
          for (int h = 0; h < 8; h++) {
            const float pr = ex2f(over[h]);
            l_run[h] += pr;
            wv[h] = pr * vf;
          }
          // probabilities (times scale_V / sqrt(d)) as fp16 hi + lo: B_P[n][row], n = head (hi) or 8 + head (lo)
          uint32_t hp[4], lp[4];
#pragma unroll
          for (int h2 = 0; h2 < 4; h2++) {
            const uint32_t hpk = pack_half2(wv[2 * h2], wv[2 * h2 + 1]);
            const float2 back = __half22float2(*reinterpret_cast<const __half2*>(&hpk));
            hp[h2] = hpk;
            lp[h2] = pack_half2(wv[2 * h2] - back.x, wv[2 * h2 + 1] - back.y);
          }
          const int off = (gt & 7) * 16 + (gt >> 3) * 128;
          *reinterpret_cast<uint4*>(bp + off) = make_uint4(hp[0], hp[1], hp[2], hp[3]);
          *reinterpret_cast<uint4*>(bp + (TB / 8) * 128 + off) = make_uint4(lp[0], lp[1], lp[2], lp[3]);
          fence_proxy_async();
        }
        tc_wait_st();
        tc_fence_before();
        mbar_arrive(p_ready);          // V tile in TMEM, probabilities in shared memory
        mbar_arrive(&empty_bar[st]);   // this thread is done with the staged tile

        // ---- next slot: if it continues the segment, its K coordinates that live in the upper half of the operand
        // columns, while the value MMAs run
        advance_slot();
        next_slot();
        more = dsc.x >= 0 && !(dsc.y & 1);
        if (more) {
          k_load(stages + st * L::STAGE_BYTES);
#pragma unroll
          for (int u = 0; u < 4 * DJ; u++)
            if (u & 2) k_unit(u);
        }

        // ---- fold the value product into the running accumulator (the value MMAs also release the lower half)
        if (!failed) failed = !mbar_wait_bounded(o_bar, (uint32_t)nbk & 1u, DEC_WAIT_LIMIT);
        if (failed) break;
        tc_fence_after();
#pragma unroll
        for (int j = 0; j < DJ; j++) {
          float o[16];
          tc_ld16(tmem_g + lane_sel + L::O_COL + 16 * j, o);
#pragma unroll
          for (int h = 0; h < 8; h++) acc[j][h] += o[h] + o[8 + h];
        }
        tc_fence_before();
        nbk++;
        if (more) {
#pragma unroll
          for (int u = 0; u < 4 * DJ; u++)
            if (!(u & 2)) k_unit(u);
          tc_wait_st();
          tc_fence_before();
          mbar_arrive(k_ready);
        }
      }
        if (failed) break;
        close_segment();
      }
    }
    if (!failed && dsc.x < 0) mbar_arrive(&empty_bar[st]);  // the end marker's slot
  }

  allow_dependent_launch();
  if (__syncthreads_or(failed) && tid == 0 && p.status) atomicOr(&p.status[0], IQ_STATUS_WAIT_TIMEOUT);
  tc_fence_before();
  __syncthreads();
  if (warp == NG * 4) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512));
}

template <int D, bool ARGMAX, bool I8, bool APPEND, int BITS>
static cudaError_t launch_one(const DecodeParams& p, cudaStream_t stream) {
  using L = DecLayout<D, BITS>;
  static bool configured[64] = {};
  static int n_sm[64] = {};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  auto kern = decode_kernel<D, ARGMAX, I8, APPEND, BITS>;
  if (!configured[dev]) {
    e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, L::SMEM_BYTES);
    if (e != cudaSuccess) return e;
    e = cudaDeviceGetAttribute(&n_sm[dev], cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    configured[dev] = true;
  }
  // One CTA per SM; each takes an equal share of the launch's 128-row blocks. No more CTAs than blocks.
  const long long max_blocks = (long long)p.batch * p.n_kv_heads * p.head_groups * ((p.t_cap + DEC_BLOCK_TOKENS - 1) / DEC_BLOCK_TOKENS);
  long long ctas = n_sm[dev];
  if (ctas > max_blocks) ctas = max_blocks;
  if (ctas < 1) ctas = 1;
  if (APPEND) {
    // A few CTAs of the grid only append: a warp takes ~5 us per task (a (sequence, KV head) unit is 1 + group tasks);
    // enough CTAs for one round of tasks, never more than a sixteenth of the SMs.
    const long long tasks = (long long)p.batch * p.n_kv_heads * (1 + p.group);
    const int warps = L::THREADS / 32;
    long long aux = (tasks + warps - 1) / warps;
    if (aux > n_sm[dev] / 16) aux = n_sm[dev] / 16;
    if (aux < 1) aux = 1;
    if (ctas + aux > n_sm[dev] && ctas > 1) ctas = n_sm[dev] - aux;  // still one CTA per SM
    DecodeParams q = p;
    q.aux_ctas = (int)aux;
    return launch_after_predecessor(kern, dim3((unsigned)(ctas + aux)), dim3(L::THREADS), L::SMEM_BYTES, stream, q);
  }
  return launch_after_predecessor(kern, dim3((unsigned)ctas), dim3(L::THREADS), L::SMEM_BYTES, stream, p);
}

template <bool APPEND, int BITS>
static cudaError_t launch_decode_variant(const DecodeParams& p, int head_dim, cudaStream_t stream) {
  const bool am = p.part_argmax != nullptr;
  if (p.use_i8) {  // levels on an 8-bit grid: int8 operands, int32 accumulation
    if (head_dim == 128) return am ? launch_one<128, true, true, APPEND, BITS>(p, stream) : launch_one<128, false, true, APPEND, BITS>(p, stream);
    return am ? launch_one<256, true, true, APPEND, BITS>(p, stream) : launch_one<256, false, true, APPEND, BITS>(p, stream);
  }
  if (head_dim == 128) return am ? launch_one<128, true, false, APPEND, BITS>(p, stream) : launch_one<128, false, false, APPEND, BITS>(p, stream);
  return am ? launch_one<256, true, false, APPEND, BITS>(p, stream) : launch_one<256, false, false, APPEND, BITS>(p, stream);
}

}  // namespace iq
