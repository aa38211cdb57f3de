// Fused decode kernel (Appendix A; Table 2 kernels A, B, C): scores on packed K codes, split-K online
// softmax, value accumulation on packed V codes, on the 5th-generation tensor cores (tcgen05) with the
// dequantised operands resident in tensor memory (TMEM).
//
// Work decomposition. The 128-row blocks of all (sequence, KV head, head group) items of the launch are laid
// end to end and every CTA -- one per SM -- takes an equal, contiguous range of that sequence, whatever the length
// mix of the batch. A range is processed item piece by item piece ("segment"); each segment ends in one partial
// result (slot) of the item. Inside the CTA, NG groups of 4 compute warps + 1 control warp each run their own
// tile pipeline and draw the segment's blocks one at a time from a shared-memory counter, so the groups stay
// busy until the segment is exhausted even though the warp schedulers do not serve them evenly; their partial
// softmax states are merged in shared memory at the end of the segment.
//
// Per block, in group g (thread r of the group = TMEM lane r):
//   1. thread r dequantises packed K row r (its own 3d/8 bytes from the staged tile) into fp16 and stores it
//      to TMEM lane r: A_K[128 rows x d].
//   2. the control warp issues tcgen05.mma (M = 128 rows, N = 16, K = 16 per instruction):
//         S[row][n] = sum_i A_K[row][i] * B_Q[n][i],  B_Q = q~ of the <= 8 heads as fp16 hi (n < 8) and lo (n >= 8)
//   3. every thread reads its row of S back, applies the K scale, joins the group-wide running maximum and
//      writes its probabilities (times the V scale, again as fp16 hi / lo) into the shared-memory operand
//      B_P[n][row].
//   4. thread c dequantises coordinate c of the token-transposed V block (128 codes = one 48-byte row) into
//      TMEM lane c: A_V[d coords x 128 rows] (same columns as A_K, once the score MMAs have read them); the
//      control warp issues   O[c][n] = sum_row A_V[c][row] * B_P[n][row]
//   5. thread c folds O (hi + lo columns) into its running accumulator for coordinate c.
// Packed tiles arrive through a 1-D bulk-copy (TMA) pipeline; every mbarrier wait is bounded.
#include <climits>

#include "iq_decode_common.cuh"
#include "iq_kernels.h"

namespace iq {

constexpr int DEC_GROUP_THREADS = 128;  // 4 warps: dequantisation, softmax, accumulation (thread = TMEM lane)
constexpr int DEC_HDR_BYTES = 4096;    // barriers, TMEM base, work counter, segment and block descriptors, scratch
constexpr float DEC_MAX_SLACK = 4.0f;  // log2 units a score may exceed the running reference before it is raised
#ifndef IQ_SLACK_I8
#define IQ_SLACK_I8 4
#endif
constexpr float DEC_MAX_SLACK_I8 = (float)IQ_SLACK_I8;  // the same on the integer path, where the probabilities are fixed-point numbers

template <int D>
struct DecLayout {
  static constexpr int DJ = D / 128;
  static constexpr int WPR = 3 * D / 32;  // 32-bit words per packed K row
  static constexpr int ROWB = WPR * 4;
  static constexpr int K_BYTES = DEC_BLOCK_TOKENS * ROWB;
  static constexpr int VT_BYTES = D * 48;  // token-transposed V block: one 48-byte row (128 codes) per coordinate
  static constexpr int SC_BYTES = DEC_BLOCK_TOKENS * 4;
  static constexpr int STAGE_BYTES = K_BYTES + VT_BYTES + 2 * SC_BYTES;
  static constexpr int STAGES = 3;
  static constexpr int BQ_BYTES = 16 * D * 2;
  static constexpr int BP_BYTES = 16 * DEC_BLOCK_TOKENS * 2;
  // TMEM columns of one group: the operand tile (K rows, then V coordinates: d fp16 = d/2 columns), 16 columns of
  // scores, 16 * DJ columns of values. The CTA owns all 512 columns of the SM.
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
  static constexpr int GROUP_SMEM = BP_BYTES + STAGES * STAGE_BYTES;
  static constexpr int SMEM_BYTES = DEC_HDR_BYTES + BQ_BYTES + NG * GROUP_SMEM;
  // header offsets
  static constexpr int BAR_STRIDE = 96;  // per group: full[3], empty[3], s_bar, o_bar, k_ready, p_ready
  static constexpr int OFF_TMEM = 384, OFF_NEXT = 388, OFF_SEG = 400, OFF_DESC = 448, OFF_ACCF = 544, OFF_QFAC = 576, OFF_RED = 640, OFF_WALK = 2176;
  static constexpr int RED_STRIDE = 384;  // per group: 3 x [4 warps][8 heads] words
};
static_assert(DEC_BLOCK_TOKENS == 128, "the TMEM operand layout assumes 128-row blocks");
static_assert(DecLayout<128>::OFF_RED + 4 * DecLayout<128>::RED_STRIDE <= DEC_HDR_BYTES, "header overflow");
static_assert(DecLayout<128>::V_COL + 32 * DecLayout<128>::DJ <= DecLayout<128>::GROUP_COLS, "TMEM group overflow");
static_assert(DecLayout<256>::V_COL + 32 * DecLayout<256>::DJ <= DecLayout<256>::GROUP_COLS, "TMEM group overflow");
static_assert(DecLayout<128>::I8_O_COL + 32 * DecLayout<128>::DJ <= DecLayout<128>::GROUP_COLS, "TMEM group overflow");
static_assert(DecLayout<256>::I8_O_COL + 32 * DecLayout<256>::DJ <= DecLayout<256>::GROUP_COLS, "TMEM group overflow");
static_assert(DecLayout<128>::SMEM_BYTES <= 227 * 1024 && DecLayout<256>::SMEM_BYTES <= 227 * 1024, "shared memory overflow");
static_assert((DecLayout<128>::THREADS + DecLayout<128>::THREADS / 32) * 4 <= DecLayout<128>::BP_BYTES, "set-up scratch must fit one B_P region");

template <int D, bool ARGMAX, bool I8>
__global__ void __launch_bounds__(DecLayout<D>::THREADS, 1) decode_kernel(const DecodeParams p) {
  using L = DecLayout<D>;
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
  const int gt = tid & (DEC_GROUP_THREADS - 1);         // compute thread within its group = TMEM lane
  const int bar_id = 1 + grp;                           // named barrier of the group's compute threads
  constexpr int HEADS_BAR = 8;                          // named barrier of the eight warps that rotate the query heads

  uint64_t* gbar = reinterpret_cast<uint64_t*>(smem + grp * L::BAR_STRIDE);
  uint64_t* full_bar = gbar;        // [stages] tile landed (or end marker)
  uint64_t* empty_bar = gbar + 3;   // [stages] staged tile consumed (128 arrivals)
  uint64_t* s_bar = gbar + 6;       // scores ready
  uint64_t* o_bar = gbar + 7;       // values ready
  uint64_t* k_ready = gbar + 8;     // K tile in TMEM (128 arrivals)
  uint64_t* p_ready = gbar + 9;     // V tile in TMEM + probabilities in smem (128 arrivals)
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + L::OFF_TMEM);
  int* next_s = reinterpret_cast<int*>(smem + L::OFF_NEXT);            // next block of the open segment
  DecSegment* seg_s = reinterpret_cast<DecSegment*>(smem + L::OFF_SEG);
  int2* desc = reinterpret_cast<int2*>(smem + L::OFF_DESC) + grp * NST;  // [stages] (first row, rows | end marker) of the staged block
  float* red = reinterpret_cast<float*>(smem + L::OFF_RED + grp * L::RED_STRIDE);  // [4 warps][8 heads] cross-warp scratch
  float* red2 = red + 32;
  int* redi = reinterpret_cast<int*>(red2 + 32);
  uint8_t* bq = smem + DEC_HDR_BYTES;                                  // B_Q: (n, i) MN-major, shared by the groups
  uint8_t* bp = bq + L::BQ_BYTES + grp * L::GROUP_SMEM;                // B_P: (n, row) MN-major
  uint8_t* stages = bp + L::BP_BYTES;
  // Set-up scratch in group 0's B_P region: [THREADS] blocks per slice of the batch, then the per-warp maxima. It is
  // last read before the first segment opens.
  int* scan_s = reinterpret_cast<int*>(bq + L::BQ_BYTES);

  const int S = p.splits;
  const int B = p.batch;
  const int ips = p.n_kv_heads * p.head_groups;  // items per sequence
  auto len_of = [&](int b) { return max(0, min(p.seq_lens[b], p.t_cap)); };
  auto nb_of = [&](int b) { return (len_of(b) + TB - 1) / TB; };
  // Unused partial slots [slot_lo, S) of the heads [h_lo, h_lo + n_h) of sequence b: (m, l) = (-inf, 0), acc = 0.
  auto fill_slots = [&](int b, int h_lo, int n_h, int slot_lo, int n_threads, int t) {
    const int n_slots = S - slot_lo;
    if (n_slots <= 0) return;
    for (int idx = t; idx < n_h * n_slots * D; idx += n_threads) {
      const int c = idx % D, sl = (idx / D) % n_slots, h = idx / (D * n_slots);
      p.part_acc[(((size_t)b * p.n_q_heads + h_lo + h) * S + slot_lo + sl) * D + c] = 0.f;
    }
    for (int idx = t; idx < n_h * n_slots; idx += n_threads) {
      const int sl = idx % n_slots, h = idx / n_slots;
      const size_t o = ((size_t)b * p.n_q_heads + h_lo + h) * S + slot_lo + sl;
      p.part_ml[2 * o] = -INFINITY;
      p.part_ml[2 * o + 1] = 0.f;
      if (ARGMAX) p.part_argmax[o] = -1;
    }
  };

  grid_dependency_wait();  // nothing written by an earlier kernel (lengths, queries, cache rows) is read above this line

  // ---------------------------------------------------------------- the block sequence of the launch and this CTA's range
  const int per_thread = (B + L::THREADS - 1) / L::THREADS;
  {
    int sum = 0, mx = 0;
    for (int b = tid * per_thread; b < min(B, (tid + 1) * per_thread); b++) {
      const int n = nb_of(b);
      sum += n;
      mx = max(mx, n);
    }
    scan_s[tid] = sum;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = max(mx, __shfl_xor_sync(FULL, mx, o));
    if (lane == 0) scan_s[L::THREADS + warp] = mx;
  }
  // sequences without cached rows belong to no range: CTA c defines the partial slots of sequences c, c + grid, ...
  for (int b = blockIdx.x; b < B; b += gridDim.x)
    if (len_of(b) == 0) fill_slots(b, 0, p.n_q_heads, 0, L::THREADS, tid);
  __syncthreads();
  long long n_total;
  int nb_max = 0;
  {
    int v = 0;
    for (int i = lane; i < L::THREADS; i += 32) v += scan_s[i];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(FULL, v, o);
    n_total = (long long)v * ips;
    for (int i = 0; i < L::THREADS / 32; i++) nb_max = max(nb_max, scan_s[L::THREADS + i]);
  }
  const bool whole_items = (S == 1);  // one slot per head: an item cannot be shared between CTAs
  long long per = (n_total + gridDim.x - 1) / gridDim.x;
  if (!whole_items) per = max(per, (long long)((nb_max - 1) / (S - 1) + 1));  // an item then spans at most S ranges
  per = max(per, 1ll);
  const long long g0 = (long long)blockIdx.x * per;
  if (n_total == 0 || (!whole_items && g0 >= n_total) || (whole_items && (long long)blockIdx.x >= (long long)B * ips)) return;

  // Thread 0 walks the range segment by segment; the walk lives in shared memory between segments. Range mode:
  // position (b, y, blk) and `left` blocks to go; whole-item mode: items blockIdx.x, blockIdx.x + grid, ... with rows.
  DecWalk* walk_s = reinterpret_cast<DecWalk*>(smem + L::OFF_WALK);
  auto next_item_with_rows = [&](DecWalk& w) {  // whole-item mode: settle on the next item that has rows, or b = B
    for (;; w.item += gridDim.x) {
      if (w.item >= (long long)B * ips) { w.b = B; w.nb = 0; return; }
      w.b = (int)(w.item / ips);
      w.y = (int)(w.item % ips);
      w.nb = nb_of(w.b);
      w.blk = 0;
      if (w.nb > 0) return;
    }
  };
  {
    DecWalk w = {0, 0, 0, 0, 0, g0, (long long)blockIdx.x};
    if (whole_items) {
      next_item_with_rows(w);  // every thread: the CTA leaves together when none of its items has rows
      if (w.b >= B) return;
    } else if (tid == 0) {
      long long before = 0;  // blocks (per item column) of the sequences before w.b
      int t = 0;
      while (t < L::THREADS - 1 && (before + scan_s[t]) * ips <= g0) { before += scan_s[t]; t++; }
      w.b = t * per_thread;
      w.nb = (w.b < B) ? nb_of(w.b) : 0;
      while (w.b < B - 1 && (before + w.nb) * ips <= g0) { before += w.nb; w.b++; w.nb = nb_of(w.b); }
      const long long r = g0 - before * ips;  // offset inside sequence b's blocks (nb per item, ips items)
      w.y = (int)(r / w.nb);
      w.blk = (int)(r % w.nb);
      w.left = min(per, n_total - g0);
    }
    if (tid == 0) *walk_s = w;
  }
  // thread 0: describe the next segment in seg_s, open its block counter, advance the walk
  auto open_segment = [&]() {
    DecWalk w = *walk_s;
    const int take = whole_items ? w.nb : (int)min((long long)(w.nb - w.blk), w.left);
    DecSegment sg;
    sg.b = w.b;
    sg.y = w.y;
    sg.blk0 = w.blk;
    sg.blk1 = w.blk + take;
    sg.slot = whole_items ? 0 : (int)((long long)blockIdx.x - (w.g - w.blk) / per);
    sg.len = len_of(w.b);
    const bool item_end = (sg.blk1 == w.nb);
    w.g += take;
    w.left -= take;
    bool cta_end;
    if (whole_items) {
      w.item += gridDim.x;
      next_item_with_rows(w);
      cta_end = (w.b >= B);
    } else {
      if (item_end) {
        w.blk = 0;
        if (++w.y == ips) {
          w.y = 0;
          do { w.b++; w.nb = (w.b < B) ? nb_of(w.b) : 0; } while (w.b < B && w.nb == 0);
        }
      } else {
        w.blk = sg.blk1;
      }
      cta_end = (w.left <= 0) || (w.b >= B);
    }
    sg.flags = (item_end ? 1 : 0) | (cta_end ? 2 : 0);
    sg.pad = 0;
    *seg_s = sg;
    *next_s = sg.blk0;
    *walk_s = w;
  };

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
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_slot[0];
  const uint32_t tmem_g = tmem_base + (uint32_t)(grp * L::GROUP_COLS);        // this group's columns
  const uint32_t lane_sel = (uint32_t)((warp & 3) * 32) << 16;                // this warp's 32 TMEM lanes
  bool failed = false;  // a bounded wait gave up; assumed to hit all threads of a group alike (they wait on the same barriers)
  int it = 0;           // staged slots of this group consumed so far (tile pipeline phases), end markers included
  int nbk = 0;          // blocks this group has processed (phases of k_ready, s_bar, p_ready, o_bar)

  for (;;) {
    // ================================================================ one segment: blocks [blk0, blk1) of one item
    if (tid == 0) open_segment();
    __syncthreads();  // segment published; the previous segment's merge has finished reading the staging buffers
    if (!control && warp < DEC_HEADS) {
      // ---- d1: q~ = R q of head `warp`, written as the operand B_Q (shared by the groups)
      const int b = seg_s->b;
      const int kvh = seg_s->y / p.head_groups;
      const int hg = seg_s->y - kvh * p.head_groups;
      const int h0 = kvh * p.group + hg * DEC_HEADS;
      const int nh = min(DEC_HEADS, p.group - hg * DEC_HEADS);
      const int hh = warp;
      float v[E];
      if (hh < nh) {
        float M[E / 4][4][4];
        const float* qb = p.rot + ((size_t)kvh * (D / 4) + (size_t)lane * (E / 4)) * 8;
#pragma unroll
        for (int j = 0; j < E / 4; j++) so4_matrix<float>(qb + 8 * j, M[j]);
        const __half* src = p.q + ((size_t)b * p.n_q_heads + h0 + hh) * D + lane * E;
#pragma unroll
        for (int e = 0; e < E; e++) v[e] = __half2float(src[e]);
        wht_warp<float, E>(v, lane);
        so4_apply<float, E, false>(M, v);
      } else {
#pragma unroll
        for (int e = 0; e < E; e++) v[e] = 0.f;
      }
      const float inv_root_d = rsqrtf((float)D);
      if constexpr (I8) {
        // q~ as three balanced base-128 digits (int8) of round(q~ * (2^20 - 1) / qmax), qmax = max |q~| over the item's
        // heads: one scale for all heads, so that the score read-back needs a single factor. (Two base-256 digits would
        // halve the read-back, but 16 bits are not enough for lse at the logit magnitudes of outlier rows.)
        float qmax = 0.f;
#pragma unroll
        for (int e = 0; e < E; e++) qmax = fmaxf(qmax, fabsf(v[e] * inv_root_d));
        qmax = warp_max(qmax);
        float* qtmp = reinterpret_cast<float*>(smem + L::OFF_QFAC);  // [8] per-head maxima, then [8] = the common factor
        if (lane == 0) qtmp[hh] = qmax;
        cta_bar_sync_n(HEADS_BAR, DEC_HEADS * 32);
#pragma unroll
        for (int h2 = 0; h2 < DEC_HEADS; h2++) qmax = fmaxf(qmax, qtmp[h2]);
        const float qs = qmax > 0.f ? 1048575.0f / qmax : 0.f;
#pragma unroll
        for (int e = 0; e < E; e++) {
          const int Q = __float2int_rn(v[e] * inv_root_d * qs);
          const int d2 = (Q + 8192) >> 14;
          const int r = Q - (d2 << 14);
          const int d1 = (r + 64) >> 7;
          const int d0 = r - (d1 << 7);
          const int i = lane * E + e;  // contraction index = rotated coordinate; column n = 4 * head + digit
          const uint32_t word = (uint32_t)(d0 & 0xff) | ((uint32_t)(d1 & 0xff) << 8) | ((uint32_t)(d2 & 0xff) << 16);
          *reinterpret_cast<uint32_t*>(bq + 4 * (hh & 3) + (hh >> 2) * ((D / 8) * 128) + (i & 7) * 16 + (i >> 3) * 128) = word;
        }
        if (hh == 0 && lane == 0)  // digits -> log2-domain score per unit K scale
          qtmp[8] = (qmax * (1.0f / 1048575.0f)) * p.delta * (p.sm_scale * LOG2E * inv_root_d);
      } else {
#pragma unroll
        for (int e = 0; e < E; e++) {
          const float x = v[e] * inv_root_d;
          const __half xh = __float2half_rn(x);
          const __half xl = __float2half_rn(x - __half2float(xh));
          const int i = lane * E + e;  // contraction index = rotated coordinate
          const int off = (i & 7) * 16 + (i >> 3) * 128;
          *reinterpret_cast<__half*>(bq + hh * 2 + off) = xh;                  // n = head (hi part)
          *reinterpret_cast<__half*>(bq + hh * 2 + (D / 8) * 128 + off) = xl;  // n = 8 + head (lo part)
        }
      }
      fence_proxy_async();  // B_Q is written through the generic proxy and read by the tensor core through the async proxy
    }
    // (the control warps stage their first tiles below before they join the barrier that completes B_Q)
    if (control) {
      // ================================================================ control warp of group grp: fetches blocks, issues MMAs.
      // All 32 lanes run the loop and the waits; an elected lane issues.
      const int blk1 = seg_s->blk1, len = seg_s->len;
      const int seg_b = seg_s->b, seg_kvh = seg_s->y / p.head_groups;
      const uint32_t bq_addr = smem_u32(bq), bp_addr = smem_u32(bp);
      // operand descriptors of the first k-step, built before the waits: a k-step further on adds its byte offset / 16
      const uint64_t bq_desc0 = smem_desc_mn(bq_addr, 128, (D / 8) * 128), bp_desc0 = smem_desc_mn(bp_addr, 128, (TB / 8) * 128);
      bool ended = false;   // the segment's counter ran out and the end marker has been staged
      int it_issue = it;    // slots staged so far (the pipeline is empty between segments)
      // The next block is drawn (shared counter; with a paged cache also its block-table entry, a load from global
      // memory) while the compute warps are busy with the softmax of the current one, and staged after the value MMAs.
      int drawn_j = -1;        // block drawn ahead of its staging, -1: none
      size_t drawn_row0 = 0;   // its first row in the cache arrays
      auto draw = [&]() {
        int j = 0;
        if (lane == 0) j = atomicAdd(next_s, 1);
        drawn_j = __shfl_sync(FULL, j, 0);
        if (drawn_j < blk1) drawn_row0 = cache_row(p.pm, seg_b, seg_kvh, drawn_j * TB, p.status);
      };
      auto stage_next = [&]() {  // the next block of the segment into slot it_issue, or the end marker
        const int st = it_issue % NST;
        if (it_issue >= NST && !failed)  // the slot's previous occupant has been consumed
          failed = !mbar_wait_bounded(&empty_bar[st], (uint32_t)(it_issue / NST - 1) & 1u, DEC_WAIT_LIMIT);
        if (drawn_j < 0) draw();
        const int j = drawn_j;
        const size_t row0 = drawn_row0;
        drawn_j = -1;
        if (j < blk1) {
          const int r0 = j * TB;
          const int n = min(TB, len - r0);
          if (elect_one()) {
            desc[st] = make_int2(r0, n);
            const uint32_t sc_bytes = p.scale_f16 ? (uint32_t)(((n + 7) & ~7) * 2) : (uint32_t)(((n + 3) & ~3) * 4);  // whole 16-byte pieces
            uint8_t* sp = stages + st * L::STAGE_BYTES;
            fence_proxy_async();
            mbar_expect_tx(&full_bar[st], (uint32_t)(n * L::ROWB + L::VT_BYTES) + 2 * sc_bytes);  // also publishes desc[st]
            bulk_g2s(sp, p.k_codes + row0 * L::ROWB, (uint32_t)(n * L::ROWB), &full_bar[st]);
            bulk_g2s(sp + L::K_BYTES, p.v_codes + row0 * L::ROWB, (uint32_t)L::VT_BYTES, &full_bar[st]);  // whole 128-row V block
            bulk_g2s(sp + L::K_BYTES + L::VT_BYTES, reinterpret_cast<const uint8_t*>(p.k_scales) + row0 * (p.scale_f16 ? 2 : 4), sc_bytes, &full_bar[st]);
            bulk_g2s(sp + L::K_BYTES + L::VT_BYTES + L::SC_BYTES, reinterpret_cast<const uint8_t*>(p.v_scales) + row0 * (p.scale_f16 ? 2 : 4), sc_bytes, &full_bar[st]);
          }
        } else {
          ended = true;
          if (elect_one()) {
            desc[st] = make_int2(0, -1);  // end marker: no tile, the group closes its part of the segment
            mbar_arrive(&full_bar[st]);
          }
        }
        __syncwarp();
        it_issue++;
      };
      while (!ended && it_issue - it < NST) stage_next();  // tiles in flight while q~ is being rotated
      cta_bar_sync();  // B_Q complete
      for (;;) {
        if (it == it_issue) stage_next();  // nothing staged ahead (end of a segment): draw now
        if (ended && it == it_issue - 1) { it++; break; }  // slot `it` holds the end marker
        // scores of the block in slot `it`: S = A_K * B_Q^T once all 128 rows are in TMEM
        if (!failed) failed = !mbar_wait_bounded(k_ready, (uint32_t)nbk & 1u, DEC_WAIT_LIMIT);
        tc_fence_after();
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
        if (!ended) draw();
        // values: O = A_V * B_P^T once the V tile is in TMEM and the probabilities are in shared memory
        if (!failed) failed = !mbar_wait_bounded(p_ready, (uint32_t)nbk & 1u, DEC_WAIT_LIMIT);
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
        nbk++;
        // the compute threads released the slot when they signalled p_ready
        if (!ended) stage_next();
      }
    }
    float* gacc = reinterpret_cast<float*>(stages);                 // group partial for the merge: acc [DJ][8][128]
    float* gml = gacc + DJ * 8 * DEC_GROUP_THREADS;                 // then per head: reference, l, exact maximum, its row
    if (!control) {
      cta_bar_sync();  // B_Q complete
      // ================================================================ compute warps of group grp
      const uint32_t lut_lo0 = p.lut_lo[0], lut_lo1 = p.lut_lo[1], lut_hi0 = p.lut_hi[0], lut_hi1 = p.lut_hi[1];
      const float kfac = p.sm_scale * LOG2E * rsqrtf((float)D);  // scores in log2 units: z2 = S_raw * scale_K * kfac
      const float vfac = rsqrtf((float)D);
      float acc[DJ][8];  // thread c: coordinates c (+128), 8 heads
      float m_run[8], l_run[8], best_v[8];
      int best_i[8];
#pragma unroll
      for (int j = 0; j < DJ; j++)
#pragma unroll
        for (int h = 0; h < 8; h++) acc[j][h] = 0.f;
#pragma unroll
      for (int h = 0; h < 8; h++) { m_run[h] = -INFINITY; l_run[h] = 0.f; best_v[h] = -INFINITY; best_i[h] = -1; }

      if constexpr (I8) {
      // Integer path. The group's TMEM columns: K tile (d/4), V tile (32 per 128 coordinates), scores (32 = 8 heads x 4
      // digit columns), values (32 per 128 coordinates). The tiles do not share columns: the V tile of a block is
      // dequantised while its score MMAs run, the K tile of the next block while its value MMAs run.
      int st = it % NST;                      // stage of slot `it` and its phase, kept incrementally
      uint32_t st_ph = (uint32_t)(it / NST) & 1u;
      const uint32_t l8_0 = p.lut8[0], l8_1 = p.lut8[1];
      const float sfac = reinterpret_cast<const float*>(smem + L::OFF_QFAC)[8];  // score digits -> log2-domain score per unit K scale
      float vref = 0.f;    // power of two >= every V scale (x 1/sqrt d) seen by the group in this segment
      float pscale = 0.f;  // probabilities are written as round(p * vscale * pscale) <= 2^30: pscale = 2^(30 - slack) / vref
      // The value products of consecutive blocks accumulate in TMEM as int32 (exact) for as long as the references they are
      // relative to (m_run, vref) stand; nacc counts the blocks in there. A block adds at most 128 * 127 * 255 < 2^22 per
      // column, so 384 blocks stay below 2^31. flush() adds the accumulated digits to the float accumulator.
      int nacc = 0;
      int* accf = reinterpret_cast<int*>(smem + L::OFF_ACCF + 4 * grp);  // tells the control warp to accumulate onto TMEM
      auto flush = [&]() {
        const float ofac = p.delta * vref * ((float)(1 << IQ_SLACK_I8) / 1073741824.0f);  // value digits -> real units: delta / pscale
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
        for (int u = 0; u < 4 * DJ; u++) {
          uint32_t f[8];
          dequant_unit8(kw[3 * u], kw[3 * u + 1], kw[3 * u + 2], l8_0, l8_1, f);
          tc_st8(tmem_g + lane_sel + L::I8_K_COL + 8 * u, f);
        }
        tc_wait_st();
        tc_fence_before();
        mbar_arrive(k_ready);
      };
      bool have_block = false;
      int2 dsc = make_int2(0, -1);
      if (!failed) {
        failed = !mbar_wait_bounded(&full_bar[st], st_ph, DEC_WAIT_LIMIT);
        dsc = desc[st];
        if (dsc.y < 0) {  // end marker: the segment has no blocks for this group
          mbar_arrive(&empty_bar[st]);
          it++;
        } else {
          have_block = true;
          k_tile(stages + st * L::STAGE_BYTES);
        }
      }
      while (have_block) {
        const uint8_t* sp = stages + st * L::STAGE_BYTES;
        const int r0 = dsc.x, n = dsc.y;
        (void)r0;
        // ---- V coordinate gt (+128) of this block -> TMEM lane gt, while the score MMAs run
#pragma unroll
        for (int j = 0; j < DJ; j++) {
          const uint4* vrow = reinterpret_cast<const uint4*>(sp + L::K_BYTES + (gt + 128 * j) * 48);
          uint32_t wd[12];
#pragma unroll
          for (int i = 0; i < 3; i++) {
            const uint4 t4 = vrow[i];
            wd[4 * i] = t4.x; wd[4 * i + 1] = t4.y; wd[4 * i + 2] = t4.z; wd[4 * i + 3] = t4.w;
          }
#pragma unroll
          for (int u = 0; u < 4; u++) {
            uint32_t f[8];
            dequant_unit8(wd[3 * u], wd[3 * u + 1], wd[3 * u + 2], l8_0, l8_1, f);
            tc_st8(tmem_g + lane_sel + L::I8_V_COL + 32 * j + 8 * u, f);
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
        tc_fence_after();
        float s[8];
        {
          auto digits_to_scores = [&](const uint32_t (&raw_u)[16], int half) {
#pragma unroll
            for (int hq = 0; hq < 4; hq++) {  // S = S0 + 128 (S1 + 128 S2): the upper two digits combine in an int32
              const float hi = __int2float_rn((int)raw_u[4 * hq + 2] * 128 + (int)raw_u[4 * hq + 1]);
              s[4 * half + hq] = fmaf(fmaf(hi, 128.f, i2f_small(raw_u[4 * hq])), kfs, mask);
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
        if (ARGMAX) {  // exact maximum seen by this thread and its row (a group sees its blocks in ascending order)
#pragma unroll
          for (int h = 0; h < 8; h++)
            if (s[h] > best_v[h]) { best_v[h] = s[h]; best_i[h] = r0 + gt; }
        }
        // The running reference m_run is raised when a score exceeds it by more than one log2 unit, the V-scale bound vref
        // when a row exceeds it: both are rare after the first blocks (one barrier with an OR reduction otherwise).
        float over[8];
#pragma unroll
        for (int h = 0; h < 8; h++) over[h] = s[h] - m_run[h];  // NaN (-inf - -inf) for a stale row of an unopened reference: max ignores it
        const bool exceed = max3f(max3f(over[0], over[1], over[2]), max3f(over[3], over[4], over[5]), fmaxf(over[6], over[7])) > DEC_MAX_SLACK_I8 ||
                            vf > vref || nacc >= 384;
        if (group_bar_or(bar_id, exceed)) {
          if (nacc > 0) flush();  // what TMEM holds is relative to the old references (the previous value MMAs have completed)
#pragma unroll
          for (int h = 0; h < 8; h++) {
            const float wm = warp_max(s[h]);
            if (lane == h) red[(warp & 3) * 8 + h] = wm;
          }
          const float wv_max = warp_max(vf);
          if (lane == 0) red2[warp & 3] = wv_max;
          group_bar_sync(bar_id);
#pragma unroll
          for (int h = 0; h < 8; h++) {
            const float bm = fmaxf(fmaxf(red[h], red[8 + h]), fmaxf(red[16 + h], red[24 + h]));
            const float mn = fmaxf(m_run[h], bm);
            const float alpha = ex2f(m_run[h] - mn);  // the accumulator holds the blocks before this one: rescale it now
            m_run[h] = mn;
            l_run[h] *= alpha;
#pragma unroll
            for (int j = 0; j < DJ; j++) acc[j][h] *= alpha;
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
            const float pr = ex2f(s[h] - m_run[h]);
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

        // ---- next slot: its K tile, while the value MMAs run
        it++;
        if (++st == NST) { st = 0; st_ph ^= 1u; }
        if (!failed) failed = !mbar_wait_bounded(&full_bar[st], st_ph, DEC_WAIT_LIMIT);
        dsc = failed ? make_int2(0, -1) : desc[st];
        have_block = dsc.y >= 0;
        if (have_block) k_tile(stages + st * L::STAGE_BYTES);

        // ---- the value MMAs of this block must have completed before its V tile and B_P are overwritten; their result stays in TMEM
        if (!failed) failed = !mbar_wait_bounded(o_bar, (uint32_t)nbk & 1u, DEC_WAIT_LIMIT);
        nbk++;
        if (!have_block && !failed) {
          mbar_arrive(&empty_bar[st]);  // the end marker's slot
          it++;
        }
      }
      if (nacc > 0) flush();

      } else {
      // The group's 128 TMEM columns: [0, 64 DJ) operand tile, then scores, values, and V_COL.. a second home for the first
      // half of the V tile. Schedule of one block (K tile complete, k_ready signalled):
      //   V rows 0..63 -> V_COL columns               while the score MMAs read the K tile
      //   wait for the scores; V rows 64..127 -> lower half of the operand columns, interleaved with the softmax
      //   signal p_ready; next block's K coordinates 32..63 (+64..) -> upper half of the operand columns
      //                                                while the value MMAs read the lower half and V_COL
      //   wait for the values, fold them; next block's other K coordinates -> lower half; signal k_ready
      int st = it % NST;                      // stage of slot `it` and its phase, kept incrementally
      uint32_t st_ph = (uint32_t)(it / NST) & 1u;
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
        dequant_unit(kw[3 * u], kw[3 * u + 1], kw[3 * u + 2], lut_lo0, lut_lo1, lut_hi0, lut_hi1, f);
        tc_st16(tmem_g + lane_sel + L::A_COL + 16 * u, f);
      };
      // first block of the group in this segment: the whole K tile
      bool have_block = false;
      int2 dsc = make_int2(0, -1);
      if (!failed) {
        failed = !mbar_wait_bounded(&full_bar[st], st_ph, DEC_WAIT_LIMIT);
        dsc = desc[st];
        if (dsc.y < 0) {  // end marker: the segment has no blocks for this group
          mbar_arrive(&empty_bar[st]);
          it++;
        } else {
          have_block = true;
          k_load(stages + st * L::STAGE_BYTES);
#pragma unroll
          for (int u = 0; u < 4 * DJ; u++) k_unit(u);
          tc_wait_st();
          tc_fence_before();
          mbar_arrive(k_ready);
        }
      }
      while (have_block) {
        const uint8_t* sp = stages + st * L::STAGE_BYTES;
        const int r0 = dsc.x, n = dsc.y;
        (void)r0;
        // ---- V coordinate gt (+128): rows 0..63 now, rows 64..127 with the softmax
        uint32_t wd[DJ][12];
#pragma unroll
        for (int j = 0; j < DJ; j++) {
          const uint4* vrow = reinterpret_cast<const uint4*>(sp + L::K_BYTES + (gt + 128 * j) * 48);
#pragma unroll
          for (int i = 0; i < 3; i++) {
            const uint4 t4 = vrow[i];
            wd[j][4 * i] = t4.x; wd[j][4 * i + 1] = t4.y; wd[j][4 * i + 2] = t4.z; wd[j][4 * i + 3] = t4.w;
          }
        }
        const float ksc = load_scale(sp + L::K_BYTES + L::VT_BYTES, gt, p.scale_f16);
        const float vsc = load_scale(sp + L::K_BYTES + L::VT_BYTES + L::SC_BYTES, gt, p.scale_f16);
        auto v_unit = [&](int j, int u) {  // rows 32u .. 32u+31 of coordinate gt + 128 j
          uint32_t f[16];
          dequant_unit(wd[j][3 * u], wd[j][3 * u + 1], wd[j][3 * u + 2], lut_lo0, lut_lo1, lut_hi0, lut_hi1, f);
          const uint32_t col = (u < 2) ? (uint32_t)(L::V_COL + 32 * j + 16 * u) : (uint32_t)(L::A_COL + 64 * j + 16 * (u - 2));
          tc_st16(tmem_g + lane_sel + col, f);
        };
#pragma unroll
        for (int j = 0; j < DJ; j++) { v_unit(j, 0); v_unit(j, 1); }

        // the score MMAs read the K tile that the rest of the V tile is about to overwrite
        if (!failed) failed = !mbar_wait_bounded(s_bar, (uint32_t)nbk & 1u, DEC_WAIT_LIMIT);
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
        if (ARGMAX) {  // exact maximum seen by this thread and its row (a group sees its blocks in ascending order)
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
#pragma unroll
          for (int h = 0; h < 8; h++) {
            const float wm = warp_max(s[h]);
            if (lane == h) red[(warp & 3) * 8 + h] = wm;
          }
          group_bar_sync(bar_id);
#pragma unroll
          for (int h = 0; h < 8; h++) {
            const float bm = fmaxf(fmaxf(red[h], red[8 + h]), fmaxf(red[16 + h], red[24 + h]));
            const float mn = fmaxf(m_run[h], bm);
            const float alpha = ex2f(m_run[h] - mn);  // the accumulator holds the blocks before this one: rescale it now
            m_run[h] = mn;
            l_run[h] *= alpha;
#pragma unroll
            for (int j = 0; j < DJ; j++) acc[j][h] *= alpha;
          }
        }
#pragma unroll
        for (int j = 0; j < DJ; j++) v_unit(j, 3);  // the last V unit, next to the exponentials
        {
          const float vf = (gt < n) ? vsc * vfac : 0.f;
          float wv[8];
#pragma unroll
          for (int h = 0; h < 8; h++) {
            const float pr = ex2f(s[h] - m_run[h]);
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

        // ---- next slot: its K coordinates that live in the upper half of the operand columns, while the value MMAs run
        it++;
        if (++st == NST) { st = 0; st_ph ^= 1u; }
        if (!failed) failed = !mbar_wait_bounded(&full_bar[st], st_ph, DEC_WAIT_LIMIT);
        dsc = failed ? make_int2(0, -1) : desc[st];
        have_block = dsc.y >= 0;
        if (have_block) {
          k_load(stages + st * L::STAGE_BYTES);
#pragma unroll
          for (int u = 0; u < 4 * DJ; u++)
            if (u & 2) k_unit(u);
        }

        // ---- fold the value product into the running accumulator (the value MMAs also release the lower half)
        if (!failed) failed = !mbar_wait_bounded(o_bar, (uint32_t)nbk & 1u, DEC_WAIT_LIMIT);
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
        if (have_block) {
#pragma unroll
          for (int u = 0; u < 4 * DJ; u++)
            if (!(u & 2)) k_unit(u);
          tc_wait_st();
          tc_fence_before();
          mbar_arrive(k_ready);
        } else if (!failed) {
          mbar_arrive(&empty_bar[st]);  // the end marker's slot
          it++;
        }
      }

      }
      // ---- close the group's part of the segment: reduce l and the exact maximum (and argmax) over the 128 rows and
      // leave the group partial in the group's (drained) staging buffer for the merge
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
        if (lane == h) { red[(warp & 3) * 8 + h] = v; red2[(warp & 3) * 8 + h] = bv; redi[(warp & 3) * 8 + h] = bi; }
      }
#pragma unroll
      for (int j = 0; j < DJ; j++)
#pragma unroll
        for (int h = 0; h < 8; h++) gacc[(j * 8 + h) * DEC_GROUP_THREADS + gt] = acc[j][h];
      group_bar_sync(bar_id);
      if (gt < 8) {
        const int h = gt;
        float mt = -INFINITY;
        int bi = -1;
        for (int wq = 0; wq < 4; wq++) {
          const float ov = red2[wq * 8 + h];
          const int oi = redi[wq * 8 + h];
          if (ov > mt || (ov == mt && oi >= 0 && (bi < 0 || oi < bi))) { mt = ov; bi = oi; }
        }
        gml[4 * h] = m_run[h];  // every thread of the group holds the same reference
        gml[4 * h + 1] = red[h] + red[8 + h] + red[16 + h] + red[24 + h];
        gml[4 * h + 2] = ARGMAX ? mt : m_run[h];  // without the argmax output the reference stands in for the maximum
        reinterpret_cast<int*>(gml)[4 * h + 3] = bi;
      }
    }
    // ================================================================ merge the groups' partials into the item's partial slot
    const int seg_b = seg_s->b, seg_y = seg_s->y, seg_slot = seg_s->slot, seg_flags = seg_s->flags;  // before thread 0 reopens seg_s
    __syncthreads();  // every group has closed its part
    if (!control) {
      const int kvh = seg_y / p.head_groups;
      const int hg = seg_y - kvh * p.head_groups;
      const int h0 = kvh * p.group + hg * DEC_HEADS;
      const int nh = min(DEC_HEADS, p.group - hg * DEC_HEADS);
      const uint8_t* group0 = bq + L::BQ_BYTES + L::BP_BYTES;  // staging buffer of group 0; the others follow at GROUP_SMEM
      auto gacc_of = [&](int g) { return reinterpret_cast<const float*>(group0 + (size_t)g * L::GROUP_SMEM); };
      auto gml_of = [&](int g) { return gacc_of(g) + DJ * 8 * DEC_GROUP_THREADS; };
      // thread (c, hsel): coordinate c (+128), heads hsel, hsel + NG, ...
      const int c = tid & (DEC_GROUP_THREADS - 1);
      for (int h = tid >> 7; h < nh; h += NG) {
        float mt = -INFINITY;  // the exact maximum of the segment: the partial is reported relative to it
#pragma unroll
        for (int g = 0; g < NG; g++) mt = fmaxf(mt, gml_of(g)[4 * h + 2]);
        float sc[NG];
#pragma unroll
        for (int g = 0; g < NG; g++) sc[g] = ex2f(gml_of(g)[4 * h] - mt);  // a group without blocks: exp2(-inf) = 0
#pragma unroll
        for (int j = 0; j < DJ; j++) {
          float v = 0.f;
#pragma unroll
          for (int g = 0; g < NG; g++) v += gacc_of(g)[(j * 8 + h) * DEC_GROUP_THREADS + c] * sc[g];
          p.part_acc[(((size_t)seg_b * p.n_q_heads + h0 + h) * S + seg_slot) * D + c + 128 * j] = v;
        }
      }
      if (tid < nh) {
        const int h = tid;
        float mt = -INFINITY;
        int bi = -1;
#pragma unroll
        for (int g = 0; g < NG; g++) {
          const float ov = gml_of(g)[4 * h + 2];
          const int oi = reinterpret_cast<const int*>(gml_of(g))[4 * h + 3];
          if (ov > mt || (ov == mt && oi >= 0 && (bi < 0 || oi < bi))) { mt = ov; bi = oi; }
        }
        float l = 0.f;
#pragma unroll
        for (int g = 0; g < NG; g++) l += gml_of(g)[4 * h + 1] * ex2f(gml_of(g)[4 * h] - mt);
        const size_t o = ((size_t)seg_b * p.n_q_heads + h0 + h) * S + seg_slot;
        p.part_ml[2 * o] = mt * LN2;
        p.part_ml[2 * o + 1] = l;
        if (ARGMAX) p.part_argmax[o] = bi;
      }
      if (seg_flags & 1) fill_slots(seg_b, h0, nh, seg_slot + 1, L::COMPUTE_THREADS, tid);  // end of the item: its unused slots
    }
    if (seg_flags & 2) break;  // last segment of this CTA
  }

  allow_dependent_launch();
  if (__syncthreads_or(failed) && tid == 0 && p.status) atomicOr(&p.status[0], IQ_STATUS_WAIT_TIMEOUT);
  tc_fence_before();
  __syncthreads();
  if (warp == NG * 4) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512));
}

template <int D, bool ARGMAX, bool I8>
static cudaError_t launch_one(const DecodeParams& p, cudaStream_t stream) {
  using L = DecLayout<D>;
  static bool configured[64] = {};
  static int n_sm[64] = {};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  auto kern = decode_kernel<D, ARGMAX, I8>;
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
  return launch_after_predecessor(kern, dim3((unsigned)ctas), dim3(L::THREADS), L::SMEM_BYTES, stream, p);
}

cudaError_t launch_decode_attention(const DecodeParams& p, int head_dim, cudaStream_t stream) {
  const bool am = p.part_argmax != nullptr;
  if (p.use_i8) {  // levels on an 8-bit grid: int8 operands, int32 accumulation
    if (head_dim == 128) return am ? launch_one<128, true, true>(p, stream) : launch_one<128, false, true>(p, stream);
    return am ? launch_one<256, true, true>(p, stream) : launch_one<256, false, true>(p, stream);
  }
  if (head_dim == 128) return am ? launch_one<128, true, false>(p, stream) : launch_one<128, false, false>(p, stream);
  return am ? launch_one<256, true, false>(p, stream) : launch_one<256, false, false>(p, stream);
}

// CTAs the decode kernel keeps resident per SM (it sizes its grid as one CTA per SM).
int decode_ctas_per_sm(int head_dim) { (void)head_dim; return 1; }

}  // namespace iq
