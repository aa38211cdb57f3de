// Internal interface between the C ABI (iq_api.cu) and the kernel translation units.
#pragma once
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace iq {

// Addressing of the cache arrays: contiguous per sequence (table == nullptr) or a pool of pages with a block table
// (see cache_row in iq_common.cuh).
struct PageMap {
  const int32_t* table;
  int page_rows, num_pages, n_kv_heads, t_cap;
};

// ---- quantize-append
constexpr int QA_WARPS = 4;
constexpr int QA_FEW_ROWS = 4;        // calls with at most this many new rows per sequence take the one-warp-per-row latency path
constexpr int QA_ROWS_PER_WARP = 16;  // K rows per warp and launch (a warp holds 4 rows at a time at head_dim 128)

struct QuantizeParams {
  const __half* k_new;
  const __half* v_new;
  long long stride_b, stride_t, stride_h;
  const int32_t* append_pos;
  const int32_t* n_new;
  int n_new_max;
  const float* rot;
  int bits;                 // 2, 3 or 4
  float thresholds_k[15];   // the first 2^bits - 1 are read
  float thresholds_v[15];
  uint8_t* k_codes;
  float* k_scales;
  uint8_t* v_codes;
  float* v_scales;
  uint32_t* status;
  int n_kv_heads, t_cap;
  PageMap pm;
  int scale_f16;
};
cudaError_t launch_quantize_append(const QuantizeParams& p, int head_dim, int batch, cudaStream_t stream);

// ---- calibration: histogram of the rotated, normalised coordinates of a set of rows
constexpr int HIST_MAX_BINS = 4096;
constexpr int HIST_ROWS_PER_WARP = 128;
struct HistogramParams {
  const __half* x;
  long long stride_b, stride_t, stride_h;
  const int32_t* n_rows;
  int n_rows_max;
  const float* rot;
  uint32_t* hist;
  int bins;
  float range;
  int n_kv_heads;
};
cudaError_t launch_rotated_histogram(const HistogramParams& p, int head_dim, int batch, cudaStream_t stream);

// ---- calibration of the rotation: z = sqrt(d) H x^ of a set of rows
struct WhtParams {
  const __half* x;
  long long stride_b, stride_t, stride_h;
  const int32_t* n_rows;
  int n_rows_max;
  float* z;  // [batch][n_rows_max][n_kv_heads][head_dim]
  int n_kv_heads;
};
cudaError_t launch_wht_coordinates(const WhtParams& p, int head_dim, int batch, cudaStream_t stream);

// ---- fused decode
constexpr int DEC_BLOCK_TOKENS = 128;  // cached rows per block of the decode kernel = rows of one transposed V block
constexpr int DEC_HEADS = 8;          // query heads of one KV head that a work item covers (they share the N columns of one MMA)

struct DecodeParams {
  const uint8_t* k_codes;
  const float* k_scales;
  const uint8_t* v_codes;
  const float* v_scales;
  const __half* q;
  const float* rot;
  const int32_t* seq_lens;
  float* part_acc;
  float* part_ml;
  int32_t* part_argmax;
  uint32_t* status;
  int batch, n_q_heads, n_kv_heads, group, head_groups, t_cap, splits;
  PageMap pm;
  int scale_f16;
  float sm_scale;
  int bits;  // 2, 3 or 4
  // fp16 path: low / high bytes of the fp16 levels of the K and V codebooks, 4 per register (2^bits / 4 registers used)
  uint32_t lut_lo[4], lut_hi[4], lut_v_lo[4], lut_v_hi[4];
  // integer path (levels on an 8-bit grid): level_j = lut8 byte j (int8) * delta, per side
  uint32_t lut8[4], lut8_v[4];
  float delta, delta_v;
  int use_i8;
  // Decode with append (k_new != nullptr; otherwise none of the following is read): the step's new K and V rows
  // [batch][n_kv_heads][head_dim] are quantised and appended at row seq_lens[b] by one warp per (sequence, KV head),
  // which also writes the new row's own partial (new_acc [batch][n_q_heads][head_dim], new_ml [batch][n_q_heads][2]);
  // the blocks of the cache are read up to row seq_lens[b] - 1.
  const __half* k_new;
  const __half* v_new;
  float* new_acc;
  float* new_ml;
  int aux_ctas;  // CTAs at the start of the grid that only append (set by the launcher)
  int len_bias;  // added to every sequence length before it is clamped to [0, t_cap] (1: the lengths given are those before an append that has been enqueued)
  float thresholds_k[15], thresholds_v[15];
  float levels_k[16], levels_v[16];
};
cudaError_t launch_decode_attention(const DecodeParams& p, int head_dim, cudaStream_t stream);
int decode_ctas_per_sm(int head_dim);
int decode_groups_per_cta(int head_dim);
cudaError_t launch_bounded_wait_selftest(uint32_t* status, uint32_t polls, cudaStream_t stream);

// ---- combine + inverse rotation
struct CombineParams {
  const float* part_acc;
  const float* part_ml;
  const int32_t* part_argmax;
  const float* rot;
  void* out;
  float* lse;
  int32_t* argmax;
  int batch, n_q_heads, n_kv_heads, splits, out_is_fp16;
  // Context sharding: the partials of `shards` ranks laid out rank after rank (each [batch][n_q_heads][splits][..]);
  // a head then has shards * splits slots. row_offsets [shards][batch] (or nullptr) turns a shard's argmax rows into
  // rows of the whole sequence. shards = 1 is the plain layout.
  int shards;
  const int32_t* row_offsets;
  // Decode with append: the partial of the step's new row, one more slot per head (nullptr: none); its row is new_rows[b].
  const float* new_acc;
  const float* new_ml;
  const int32_t* new_rows;
};
cudaError_t launch_combine_splits(const CombineParams& p, int head_dim, cudaStream_t stream);

// ---- reconstruction of fp16 K/V rows from the packed cache (the reconstruct-then-compute model)
struct ReconstructParams {
  const uint8_t* k_codes;
  const float* k_scales;
  const uint8_t* v_codes;
  const float* v_scales;
  const float* rot;
  const int32_t* seq_lens;
  __half* k_out;
  __half* v_out;
  long long stride_b, stride_t, stride_h;  // in elements
  int n_kv_heads, t_cap, out_rows;
  PageMap pm;
  int scale_f16;
  uint32_t* status;
  int bits;
  float levels_k[16], levels_v[16];
};
cudaError_t launch_reconstruct_rows(const ReconstructParams& p, int head_dim, int batch, cudaStream_t stream);

// ---- rotation parameters
cudaError_t launch_make_rotation(float* rot, int n_quats, uint64_t seed, cudaStream_t stream);
cudaError_t launch_normalize_rotation(float* rot, int n_quats, cudaStream_t stream);

}  // namespace iq
