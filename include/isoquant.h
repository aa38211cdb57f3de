/*
 * isoquant.h -- C ABI of the IsoQuant compressed-space decode-attention library (CUDA, sm_100a).
 *
 * The library implements the data-parallel hot path of IsoQuant KV-cache compression:
 *
 *   quantize-append   Algorithm 1 of the paper: s = ||x||_2, x^ = x/s, x~ = R_SO4(H_d x^) (Eq. 2),
 *                     b-bit Lloyd-Max code per coordinate (Step 3; b = 3 in the paper, 2 and 4 as well here),
 *                     bit-pack (Step 4).
 *   fused decode      Appendix A: q~ = R q once, scores q~ . k~_j / sqrt(d_k) taken directly on the
 *                     packed codes, softmax, o~ = sum_j alpha_j v~_j accumulated directly on the packed
 *                     codes, o = R^T o~ once (Table 2, kernels A-D). FP16 K/V are never materialised.
 *                     The context is split flash-decoding style; the partial results are merged by
 *                     iq_combine_splits, which also applies the single inverse rotation.
 *
 * Conventions
 *   - Every pointer named *_dev (and every cache / partial / q / out pointer) is DEVICE memory owned by
 *     the caller. Pointers named *_host and the iq_shape / iq_codebook / iq_cache structs are HOST memory,
 *     read during the call only. The library allocates nothing and keeps no state between calls.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream). Calls enqueue work on it
 *     and return without synchronising. They never throw or abort.
 *   - Every entry point returns IQ_OK (0) or a negative IQ_ERR_* code. Arguments are validated on the host
 *     before anything is launched; on an error nothing has been enqueued.
 *   - Device-side conditions that cannot be known on the host are reported through an optional
 *     `status_dev` array of 4 uint32 (zeroed by the caller): [0] bit mask of IQ_STATUS_* flags,
 *     [1] rows whose codes were re-decided in fp64 (see iq_quantize_append), [2] rows skipped because
 *     they fell outside the cache, [3] reserved. Nothing on the device traps or spins without a bound: the
 *     decode kernel's waits on its asynchronous copies and tensor-core results give up after 65536 polls of at most
 *     20 us each (about a second at worst; a wait that works lasts microseconds), flag IQ_STATUS_WAIT_TIMEOUT and
 *     the kernel returns with invalid results.
 *
 * Rotation (Eq. 2, Section 3.3 "SO(4) parameterization", Appendix B)
 *   R = R_SO4 o H_d. H_d is the normalised Walsh-Hadamard matrix in natural (Sylvester) order,
 *   H[i][j] = (-1)^popcount(i & j) / sqrt(d). R_SO4 is block diagonal: block b = 0 .. d/4-1 acts on
 *   coordinates [4b, 4b+4) as v -> q_L v conj(q_R) with unit quaternions stored (w, x, y, z), Hamilton
 *   product, the four coordinates read as y0 + y1 i + y2 j + y3 k. Storage: [n_kv_heads][d/4][8] fp32 =
 *   (q_L.wxyz, q_R.wxyz): 8 floats per block, 256 per head at d = 128 (Appendix B). K and V of a KV head
 *   and all query heads of its group share that head's rotation.
 *
 * Codebook (Section 3.2, Step 3; Algorithm 1 is written for a general bit width b and codebook C_b)
 *   2^b ascending levels and 2^b - 1 ascending decision thresholds in unit-variance units u = sqrt(d) * x~, b = bits
 *   in {2, 3, 4}. code = #{ j : u > t_j } (strict: an exact tie takes the lower code). A dequantised coordinate is
 *   scale * level[code] / sqrt(d). The K rows and the V rows may have codebooks of their own (separate_v): keys and
 *   values need not have the same post-rotation marginal. iq_quantize_append uses the thresholds only and takes any
 *   ascending set.
 *   iq_decode_attention feeds the levels to tensor-core operands without rounding them, so it takes two forms:
 *   levels on an 8-bit grid, level_j = n_j * delta with integers |n_j| <= 127 (iq_int8_codebook, or iq_fit_codebook
 *   with grid = 1; with separate_v each side on a grid of its own): int8 operands, the faster path; or levels that
 *   are all exact IEEE binary16 values (iq_default_codebook, iq_fit_codebook with grid = 0): fp16 operands. Anything
 *   else is IQ_ERR_CODEBOOK.
 *
 * Packed cache (Section 3.2, Step 4 fixes the size only: b d / 8 bytes per row, 48 at b = 3, d = 128)
 *   codes: b d / 8 bytes per cached row and side, scales [batch][n_kv_heads][t_cap] fp32 (= ||x||_2), separately
 *   for K and V. A run of packed entries (a K row, or a V record) is a sequence of little-endian 32-bit words:
 *     b = 3: groups of 32 entries in 3 consecutive words: in group-local numbering, entry c < 24 stores its code in
 *            bits [4n, 4n+3) of word c/8, n = c mod 8; entry c >= 24 (n = c - 24) stores bit k of its code in bit 4n+3
 *            of word k.
 *     b = 4: entry c stores its code in bits [4n, 4n+4) of word c/8, n = c mod 8.
 *     b = 2: groups of 16 entries in one word: entry e < 8 of the group in bits [4e, 4e+2), entry e >= 8 in bits
 *            [4(e-8)+2, 4(e-8)+4).
 *   (Every layout keeps the codes nibble-aligned, which is what the decode kernel's byte-permute lookups index by.)
 *   K codes [batch][n_kv_heads][t_cap][b d / 8]: one packed row per cached row, entries = rotated coordinates.
 *   V codes [batch][n_kv_heads][t_cap/128][d][16 b]: token-transposed. For every block of 128 cached rows and every
 *   rotated coordinate c there is one record of 16 b bytes (48 at b = 3) holding the 128 codes of coordinate c,
 *   entries = row within the block. (The decode kernel contracts K over coordinates and V over rows; either way the contraction
 *   index then runs along a packed record.) Bits of rows that were never appended are left as they are.
 *   t_cap must be a multiple of 128 and all four arrays 16-byte aligned.
 */
#ifndef ISOQUANT_H_
#define ISOQUANT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define IQ_VERSION 300
/* Version of the packed-cache byte layout described above and in docs/FORMAT.md (bit order of a packing unit,
 * token-transposed V records, scale arrays, rotation parameters, partial slots). A cache written under one format
 * version is read correctly only by a library of the same format version; iq_format_version() reports the library's. */
#define IQ_FORMAT_VERSION 3

enum {
  IQ_OK = 0,
  IQ_ERR_NULL = -1,     /* a required pointer is NULL */
  IQ_ERR_SHAPE = -2,    /* unsupported head_dim / bits, n_q_heads % n_kv_heads != 0, bad sizes or strides */
  IQ_ERR_ALIGN = -3,    /* a pointer or stride breaks the stated alignment */
  IQ_ERR_CODEBOOK = -4, /* bits differ from the shape's; levels / thresholds not ascending; decode: levels neither on an 8-bit grid nor exact binary16 */
  IQ_ERR_CUDA = -5,     /* the CUDA runtime reported an error for the launch */
  IQ_ERR_LIMIT = -6     /* a size exceeds a documented maximum of the entry point */
};

enum {
  IQ_STATUS_ROW_OUT_OF_RANGE = 1u, /* quantize-append: append_pos + i >= t_cap, row skipped */
  IQ_STATUS_WAIT_TIMEOUT = 2u,     /* decode: a bounded wait on an asynchronous copy ran out; results invalid */
  IQ_STATUS_SCALE_OVERFLOW = 8u,   /* binary16 scales: a row norm above 65504 was stored as 65504 */
  IQ_STATUS_BAD_PAGE = 4u          /* paged cache: a block-table entry outside [0, num_pages) was met: read as page 0 by
                                      decode / reconstruct, the rows skipped (and counted in [2]) by quantize-append */
};

typedef struct iq_shape {
  int32_t batch;
  int32_t n_q_heads;
  int32_t n_kv_heads; /* n_q_heads % n_kv_heads == 0 */
  int32_t head_dim;   /* 128 or 256 */
  int32_t t_cap;      /* rows allocated per (sequence, KV head); multiple of 128 */
  int32_t bits;       /* 2, 3 or 4 */
  float sm_scale;     /* softmax scale; <= 0 selects 1/sqrt(head_dim) (Appendix A) */
} iq_shape;

#define IQ_MAX_LEVELS 16
typedef struct iq_codebook {
  int32_t bits;                          /* 2, 3 or 4: 2^bits levels, 2^bits - 1 thresholds are read; must equal iq_shape.bits */
  int32_t separate_v;                    /* 0: the V rows use levels / thresholds too; else v_levels / v_thresholds */
  float levels[IQ_MAX_LEVELS];           /* K rows (and V rows unless separate_v) */
  float thresholds[IQ_MAX_LEVELS - 1];
  float v_levels[IQ_MAX_LEVELS];
  float v_thresholds[IQ_MAX_LEVELS - 1];
} iq_codebook;

typedef struct iq_cache {
  uint8_t* k_codes;
  float* k_scales;
  uint8_t* v_codes;
  float* v_scales;
  /* Paged cache (optional; the paper's cache is contiguous per sequence). block_table_dev == NULL: the arrays are
   * [batch][n_kv_heads][t_cap] rows as described above. Otherwise they are a pool of num_pages pages,
   * [num_pages][n_kv_heads][page_rows] rows (V: page_rows / 128 token-transposed blocks per page and KV head), and
   * block_table_dev is a device int32 [batch][t_cap / page_rows]: entry (b, j) is the page that holds rows
   * [j * page_rows, (j + 1) * page_rows) of sequence b. page_rows is a multiple of 128 and divides t_cap, which is
   * then the logical capacity of a sequence. Entries that a call can reach (rows below the lengths it is given)
   * must be valid; an entry outside [0, num_pages) sets IQ_STATUS_BAD_PAGE: a reading kernel takes page 0 in its place,
   * iq_quantize_append skips the rows that would go there and counts them in status[2]. */
  const int32_t* block_table_dev;
  int32_t page_rows;
  int32_t num_pages;
  /* 0: k_scales / v_scales are fp32 arrays (52 bytes per row and side at head_dim 128). 1: they are binary16 arrays of
   * the same shape (the pointers are then really uint16_t*; 50 bytes per row): the norm is rounded to binary16 when a
   * row is appended -- the row is still normalised by its exact norm -- and a norm beyond the binary16 range is
   * stored as 65504 and flagged with IQ_STATUS_SCALE_OVERFLOW. */
  int32_t scales_fp16;
} iq_cache;

int iq_version(void);
int iq_format_version(void);
const char* iq_strerror(int code);

/* Bytes of one packed row: bits * head_dim / 8 (Section 3.2, Step 4); iq_row_bytes is the 3-bit case. 0 for an
 * unsupported head_dim or bit width. The V array of a (sequence, KV head) has the same number of bytes as the K array. */
size_t iq_row_bytes(int32_t head_dim);
size_t iq_row_bytes_bits(int32_t head_dim, int32_t bits);
/* Floats of the rotation parameter buffer: n_kv_heads * (head_dim / 4) * 8 (Appendix B). */
size_t iq_rotation_floats(int32_t head_dim, int32_t n_kv_heads);

/*
 * Lloyd-Max codebook for the post-rotation marginal (Section 3.2, Step 3): one coordinate of a uniform
 * point on S^{d-1} in unit-variance units, density ~ (1 - u^2/d)^((d-3)/2). Levels are rounded to
 * binary16-representable values, thresholds are the midpoints of the rounded levels. Host only.
 */
int iq_default_codebook(int32_t head_dim, iq_codebook* out_host);

/*
 * The same Lloyd-Max codebook with its levels snapped to an 8-bit grid: level_j = n_j * delta, n_j integer,
 * |n_j| <= 127, delta = max|level| / 127 (fp32); thresholds = midpoints of the snapped levels. The snapping moves a
 * level by at most delta / 2 (0.4 % of the largest level). iq_decode_attention runs codebooks of this form on the
 * integer tensor-core path (int8 operands, int32 accumulation); any other codebook must have levels that are exact
 * binary16 values and runs on the fp16 path.
 */
int iq_int8_codebook(int32_t head_dim, iq_codebook* out_host);
/* The same two codebooks for any bit width (iq_default_codebook / iq_int8_codebook are bits = 3): 2^bits Lloyd-Max
 * levels for the post-rotation marginal, grid = 0: rounded to binary16, grid = 1: snapped to the 8-bit grid. */
int iq_lloyd_max_codebook(int32_t head_dim, int32_t bits, int32_t grid, iq_codebook* out_host);
/* Makes `cb` a two-sided codebook: its V side becomes the K side of `v_side` (same bits). Host only. */
int iq_codebook_set_v(iq_codebook* cb, const iq_codebook* v_side);

/*
 * Rotation parameters (Appendix B). If quats_host != NULL it holds [n_kv_heads][d/4][8] floats which are
 * scaled to unit length per quaternion and copied to rot_dev; otherwise the quaternions are drawn on the
 * device from `seed` (4 iid N(0,1) components per quaternion from a counter-based generator, scaled to
 * unit length: Haar measure on S^3). rot_dev: device, iq_rotation_floats() floats, 16-byte aligned.
 */
int iq_make_rotation(int32_t head_dim, int32_t n_kv_heads, uint64_t seed, const float* quats_host,
                     float* rot_dev, void* stream);

/*
 * Algorithm 1 for the new K and V rows of every sequence and KV head; results appended to the cache.
 *   k_new, v_new   device, binary16; element (b, i, h, c) at b*stride_b + i*stride_t + h*stride_h + c
 *                  (strides in elements, multiples of 8; base pointers 16-byte aligned).
 *   append_pos_dev device int32 [batch]: cache row that receives new row 0 of sequence b.
 *   n_new_dev      device int32 [batch] rows to append per sequence (clamped to n_new_max), or NULL for
 *                  n_new_max everywhere. n_new_max = 0 is a no-op.
 *   cache          host struct of device pointers; rows append_pos[b] + i are overwritten (on the V side: the
 *                  bits of those rows inside the transposed records). The call does not touch any
 *                  sequence-length array: the caller advances its lengths. Calls that append to the same
 *                  (sequence, KV head) must be ordered on one stream.
 *   status_dev     optional (see top). Rows with append_pos + i outside [0, t_cap) are skipped and flagged.
 * Arithmetic: fp32 butterfly WHT and 4x4 block products; any row with a coordinate closer than 2^-15 to a
 * decision threshold is re-decided in fp64 inside the kernel, so the codes equal those of an fp64
 * evaluation except for ties at the fp64 rounding level. The stored scale is sqrt(sum x^2) accumulated
 * in fp64 and rounded to fp32. A zero row stores scale 0 and the code of u = 0 everywhere.
 */
int iq_quantize_append(const iq_shape* shape, const float* rot_dev, const iq_codebook* codebook,
                       const void* k_new, const void* v_new, int64_t stride_b, int64_t stride_t,
                       int64_t stride_h, const int32_t* append_pos_dev, const int32_t* n_new_dev,
                       int32_t n_new_max, const iq_cache* cache, uint32_t* status_dev, void* stream);

/*
 * Fused decode step on the packed cache (Appendix A; Table 2, kernels A-C), split over the context.
 *   q              device binary16 [batch][n_q_heads][head_dim], 16-byte aligned; not quantised.
 *   seq_lens_dev   device int32 [batch]: rows 0 .. len-1 of each sequence are attended to (clamped to
 *                  [0, t_cap]); the row appended last is attended to like any other. The lengths are read while the
 *                  kernel that precedes the call on the stream may still be finishing (the launch overlaps it): they
 *                  must have been written before that kernel started (by the host, a copy, or earlier work). No kernel
 *                  of this library writes them. Everything else is read after that kernel has completed.
 *   num_splits     S >= 1: partial slots per (sequence, head). Every cached row of a sequence is covered by exactly one
 *                  slot of each head; which rows a slot covers is the library's choice, and a slot's rows need not be
 *                  consecutive. With S >= 2 G (G = 4 workers per SM at head_dim 128, 2 at 256) the launch is balanced
 *                  over the whole batch: every SM takes an equal, contiguous share of all 128-row blocks, and the part of
 *                  a (sequence, KV head) inside a share reports to G slots, one per worker of that SM. With fewer slots
 *                  every (sequence, KV head) is cut into S runs of consecutive blocks, one slot each, dealt out to the
 *                  workers in turn (S = 1: one worker per (sequence, KV head), no merge needed afterwards).
 *                  iq_suggest_splits gives a value for the balanced mode.
 *   part_acc       device fp32 [batch][n_q_heads][S][head_dim]: sum_j exp(z_j - m) v~_j over the slot's rows,
 *                  in the rotated space, natural coordinate order. 16-byte aligned.
 *   part_ml        device fp32 [batch][n_q_heads][S][2] = (m, l): the slot's reference m and l = sum_j exp(z_j - m),
 *                  z_j = sm_scale * q~ . k~_j. With part_argmax, m = max_j z_j exactly; without it m is the kernel's
 *                  running reference, max_j z_j - 4 ln 2 <= m <= max_j z_j (acc and l are relative to the same m
 *                  either way). An unused slot holds (-inf, 0), and its acc is not written (the merge skips a slot
 *                  with l = 0 without reading acc); (m, l) of every slot of every head is written on every call.
 *   part_argmax    device int32 [batch][n_q_heads][S] or NULL: row index attaining m (lowest on ties), -1 if empty.
 *   status_dev     optional (see top).
 * Arithmetic, codebook levels on an 8-bit grid (iq_int8_codebook): int8 tensor-core operands and int32
 * accumulation -- the levels as integers, q~ as three base-128 digits of a 21-bit fixed-point number (one scale per
 * KV head group), the probabilities times V scale as four base-256 digits of a 30-bit fixed-point number; softmax
 * statistics and the running output in fp32. Other codebooks: levels must be exact binary16 values; q~ and the
 * probabilities enter fp16 operands as two-term sums (hi + lo), every accumulation is fp32. Blocks are handed to the
 * warps of an SM dynamically, so the order of the fp32 additions -- and with it the last bits of the
 * result -- can differ between two calls on the same inputs; m and the argmax do not.
 */
int iq_decode_attention(const iq_shape* shape, const float* rot_dev, const iq_codebook* codebook,
                        const void* q, const iq_cache* cache, const int32_t* seq_lens_dev,
                        int32_t num_splits, float* part_acc, float* part_ml, int32_t* part_argmax,
                        uint32_t* status_dev, void* stream);

/*
 * Merge of the split partials and the single inverse rotation (Table 2, kernel D):
 *   m = max_s m_s, l = sum_s l_s e^{m_s - m}, o~ = sum_s acc_s e^{m_s - m} / l, o = R^T o~ = H_d blockdiag(M_b^T) o~.
 *   out            device [batch][n_q_heads][head_dim], fp32 or (out_is_fp16 != 0) binary16; 16-byte aligned.
 *   lse_out        device fp32 [batch][n_q_heads] or NULL: m + log(l) (-inf for an empty sequence).
 *   argmax_out     device int32 [batch][n_q_heads] or NULL (needs part_argmax): row with the largest score.
 * A sequence of length 0 yields out = 0, lse = -inf, argmax = -1.
 */
int iq_combine_splits(const iq_shape* shape, const float* rot_dev, int32_t num_splits,
                      const float* part_acc, const float* part_ml, const int32_t* part_argmax,
                      void* out, int32_t out_is_fp16, float* lse_out, int32_t* argmax_out, void* stream);

/*
 * The same merge over the partials of several ranks that each decoded a slice of every sequence's rows (context
 * sharding; the paper's system is a single device, the merge is the one exchange step the method has when the context
 * itself is spread over GPUs). The arrays hold the ranks' partials one after the other, as an all-gather into one
 * buffer leaves them: part_acc [n_shards][batch][n_q_heads][S][head_dim], part_ml [n_shards][batch][n_q_heads][S][2],
 * part_argmax [n_shards][batch][n_q_heads][S] or NULL; a head is merged over its n_shards * S slots in place, nothing
 * is copied or allocated. row_offsets_dev: device int32 [n_shards][batch], the first row of rank r's slice of
 * sequence b, added to that rank's argmax rows (NULL: the rows are taken as they are). n_shards = 1 is
 * iq_combine_splits.
 */
int iq_combine_splits_sharded(const iq_shape* shape, const float* rot_dev, int32_t num_splits, int32_t n_shards,
                              const float* part_acc, const float* part_ml, const int32_t* part_argmax,
                              const int32_t* row_offsets_dev, void* out, int32_t out_is_fp16, float* lse_out,
                              int32_t* argmax_out, void* stream);

/*
 * Reconstruct-then-compute, first half (Figure 1, top; the execution model that Section 3 argues against and the
 * fused path replaces): rows [0, seq_lens[b]) of every (sequence, KV head) dequantised and rotated back to the
 * original space, x_hat = R^T x~ with x~_i = scale * level[code_i] / sqrt(d) (Algorithm 1 read backwards; R is
 * orthogonal). The fp16 tensors it writes are what a standard attention kernel consumes; the call exists to measure
 * that model against iq_decode_attention on the same packed cache, and as a way to read the cache back.
 *   k_out, v_out   device binary16, element (b, t, g, i) at b*stride_b + t*stride_t + g*stride_h + i (strides in
 *                  elements, multiples of 8; pointers 16-byte aligned), out_rows rows per sequence. Rows
 *                  t >= min(seq_lens[b], out_rows) are not written.
 *   codebook       only the levels are used (any fp32 values).
 * fp32 arithmetic, one rounding to binary16 at the end.
 */
int iq_reconstruct_rows(const iq_shape* shape, const float* rot_dev, const iq_codebook* codebook,
                        const iq_cache* cache, const int32_t* seq_lens_dev, void* k_out, void* v_out,
                        int32_t out_rows, int64_t stride_b, int64_t stride_t, int64_t stride_h, void* stream);

/*
 * Calibration of the codebook on data (Section 3.2, Step 3: "Lloyd-Max for the post-rotation distribution"; the paper
 * does not say how that distribution is obtained -- here it is the empirical marginal of a calibration set).
 *
 * iq_rotated_histogram adds to hist_dev the histogram of u = sqrt(d) R x^ (Algorithm 1, lines 1-4: the quantity the
 * thresholds are compared with) over all coordinates of the given rows: `bins` uniform bins on [-range, range), values
 * outside counted in the end bins, zero rows left out.
 *   x              device binary16 rows, element (b, t, g, i) at b*stride_b + t*stride_t + g*stride_h + i (strides in
 *                  elements, multiples of 8), t < n_rows_dev[b] (NULL: n_rows_max for every sequence), capped at n_rows_max.
 *   hist_dev       device uint32 [bins], 16 <= bins <= 4096; the caller zeroes it once and may accumulate several calls.
 * iq_fit_codebook (host only, no CUDA) runs Lloyd's iteration on such a histogram read as a piecewise-constant density
 * (level = centroid of its cell, threshold = midpoint of neighbouring levels) and writes the codebook in the form the
 * kernels take: grid = 0: levels exactly representable in binary16; grid = 1: levels on an 8-bit grid as from
 * iq_int8_codebook; thresholds = midpoints of the final levels. symmetric != 0 averages the histogram with its mirror
 * image first (a codebook symmetric about zero takes the faster decision path of the bulk quantize kernels).
 * IQ_ERR_CODEBOOK if the data has too few distinct values for 2^bits ascending levels. Calibrating K and V separately is
 * two histograms and two fits, joined with iq_codebook_set_v.
 */
int iq_rotated_histogram(const iq_shape* shape, const float* rot_dev, const void* x, int64_t stride_b,
                         int64_t stride_t, int64_t stride_h, const int32_t* n_rows_dev, int32_t n_rows_max,
                         uint32_t* hist_dev, int32_t bins, float range, void* stream);
int iq_fit_codebook(const uint32_t* hist_host, int32_t bins, float range, int32_t bits, int32_t symmetric, int32_t grid,
                    iq_codebook* out_host);

/*
 * Calibration of the rotation (Section 3.2 counts 192 learnable parameters at d = 128: the 6 rotational degrees of
 * freedom of each of the 32 SO(4) blocks; Appendix B stores them as 8 floats per block. The paper does not say how they
 * are learned -- here each block's rotation is chosen to minimise the mean squared quantisation error of the block's
 * four rotated coordinates, under the codebook in use, over a calibration set of rows).
 *
 * iq_wht_coordinates writes z = sqrt(d) H_d x^ (Algorithm 1, lines 1-2, in the unit-variance units of the codebook) of
 * the given rows as fp32: the quantity the blocks rotate.
 *   x              device binary16 rows, element (b, t, g, i) at b*stride_b + t*stride_t + g*stride_h + i (strides in
 *                  elements, multiples of 8), t < n_rows_dev[b] (NULL: n_rows_max for every sequence), capped at n_rows_max.
 *   z_dev          device fp32 [batch][n_rows_max][n_kv_heads][head_dim], 16-byte aligned; rows beyond a sequence's
 *                  count are not written, zero rows give zeros.
 * iq_fit_rotation (host only, no CUDA) fits the d/4 blocks of ONE KV head: z_host holds n_rows rows of that head's z,
 * row r at z_host + r * row_stride (floats); quats_host [d/4][8] holds the starting rotation (q_L.wxyz, q_R.wxyz per
 * block) and receives the fitted one, as unit quaternion pairs ready for iq_make_rotation. Per block a pattern search
 * over the six coordinate planes: rotate by +-delta, keep the move if the distortion
 *     1/N sum_rows sum_{i<4} (u_i - level[code(u_i)])^2,  u = M z,
 * decreases, halve delta (pi/8 down to 1e-3 rad) when a sweep over the planes improves nothing. The result is never
 * worse than the start. distortion_host (optional, 2 doubles): mean distortion per coordinate before and after.
 */
int iq_wht_coordinates(const iq_shape* shape, const void* x, int64_t stride_b, int64_t stride_t, int64_t stride_h,
                       const int32_t* n_rows_dev, int32_t n_rows_max, float* z_dev, void* stream);
int iq_fit_rotation(const float* z_host, int32_t n_rows, int64_t row_stride, int32_t head_dim, const iq_codebook* codebook,
                    float* quats_host, double* distortion_host);

/*
 * One whole decode step from HOST buffers, in one call: the step's inputs go to the device in one copy, one new row
 * per sequence is appended (Algorithm 1), the fused decode and the merge run (Appendix A), the output comes back and
 * the call returns when it has arrived. It is iq_quantize_append (n_new_max = 1) + iq_decode_attention +
 * iq_combine_splits with the two copies and one cudaStreamSynchronize around them; unlike every other call it blocks.
 *   inputs_host    host (pinned for a truly asynchronous copy) binary16: q [batch][n_q_heads][head_dim], then
 *                  k_new [batch][n_kv_heads][head_dim], then v_new [batch][n_kv_heads][head_dim], contiguous.
 *   inputs_dev     device staging buffer of the same size, 16-byte aligned, caller-owned.
 *   append_pos_dev device int32 [batch]: row that receives the new K/V row (the sequence's length before the step).
 *   seq_lens_dev   device int32 [batch]: rows attended to (the length after the step).
 *   out_dev        device [batch][n_q_heads][head_dim], fp32 or binary16 (out_is_fp16); out_host: host, same size.
 * part_acc / part_ml / num_splits / status_dev as for iq_decode_attention. No lse or argmax output.
 */
int iq_decode_step_host(const iq_shape* shape, const float* rot_dev, const iq_codebook* codebook,
                        const void* inputs_host, void* inputs_dev, const int32_t* append_pos_dev,
                        const int32_t* seq_lens_dev, const iq_cache* cache, int32_t num_splits, float* part_acc,
                        float* part_ml, void* out_dev, void* out_host, int32_t out_is_fp16, uint32_t* status_dev,
                        void* stream);

/*
 * The decode step in one call, with the append folded into the decode launch where that pays (Algorithm 1 for the
 * step's new rows; Appendix A): what iq_quantize_append (one row per sequence) + iq_decode_attention +
 * iq_combine_splits compute. For a single sequence or a few -- at most 180 (sequence, KV head, 1 + heads per KV head)
 * tasks, 3-bit codes -- the decode launch itself appends: a few CTAs at the start of its grid do nothing but quantise
 * the new K and V rows, write them to the cache and write the new row's own partial (its score per head from its
 * codes and stored scale, its value vector), one warp per task, while the other CTAs read the cache WITHOUT those
 * rows; the merge takes the partial as one more slot. Two launches instead of three, and the append off the critical
 * path: 17.8 against 20.9 us per step for one sequence of 32 K rows. For larger batches the call enqueues the three
 * launches (the append kernel, the decode over one more row per sequence, the merge), which are faster there.
 *   k_new, v_new   device binary16 [batch][n_kv_heads][head_dim], contiguous, 16-byte aligned: the step's new rows,
 *                  appended at row seq_lens[b] of every sequence and attended to.
 *   seq_lens_dev   device int32 [batch]: the lengths BEFORE the step (as for iq_decode_attention they are read early).
 *                  The caller advances them afterwards. A sequence with seq_lens[b] outside [0, t_cap) gets no new row
 *                  (IQ_STATUS_ROW_OUT_OF_RANGE, 2 rows per KV head counted in status_dev[2]) and attends to its cached
 *                  rows only.
 *   workspace_dev  device, iq_decode_step_workspace_bytes(shape, num_splits) bytes, 16-byte aligned: the partial slots
 *                  and the new rows' partials; needs no initialisation. Calls that share a workspace must be ordered on
 *                  one stream.
 *   out, lse_out, argmax_out   as for iq_combine_splits (argmax_out != NULL also selects exact slot maxima).
 *   num_splits     as for iq_decode_attention.
 * With a paged cache the page that receives the new row must be in the block table before the call.
 * (Merging inside the decode kernel as well -- arrival counters, the last writer merges -- was built and measured
 * slower than the separate merge launch at every batch size, and is not part of the library.)
 */
size_t iq_decode_step_workspace_bytes(const iq_shape* shape, int32_t num_splits);
int iq_decode_step_fused(const iq_shape* shape, const float* rot_dev, const iq_codebook* codebook, const void* q,
                         const void* k_new, const void* v_new, const iq_cache* cache, const int32_t* seq_lens_dev,
                         int32_t num_splits, void* workspace_dev, void* out, int32_t out_is_fp16, float* lse_out,
                         int32_t* argmax_out, uint32_t* status_dev, void* stream);

/*
 * Decode step for callers that cannot allocate device memory (the paper has no counterpart: its pipeline
 * is unsplit and needs no scratch). It runs iq_decode_attention followed by iq_combine_splits with the
 * split partials kept in a fixed array inside the library image instead of caller-provided buffers.
 * Meant for code that must not call cudaMalloc or a framework allocator: work enqueued while a stream
 * capture is open, plugins that receive only their inputs and outputs, embeddings with a memory budget
 * fixed at load time.
 *   - The array is IQ_STATIC_SCRATCH_BYTES (8 MiB) of device memory on every GPU that loads the library,
 *     held until the process exits. A call needs batch * n_q_heads * num_splits * (head_dim + 2) floats;
 *     larger requests are rejected with IQ_ERR_LIMIT and nothing is enqueued.
 *   - The first call on a device resolves the array's device address (cudaGetSymbolAddress, with that
 *     device current); with lazy module loading that is also the moment the driver places the array on
 *     the GPU. Make that first call before any stream capture begins.
 *   - The call itself allocates nothing and frees nothing. The address found by the first call is kept until the
 *     process ends; after a cudaDeviceReset of the device it is stale and the entry point must not be called again.
 *   - All calls on a device share the one array, which keeps the previous call's contents. Every split of
 *     every head is rewritten on each call, so no clearing is needed; but two calls whose kernels overlap
 *     on the GPU (different streams) race on it. Serialise them on one stream or with events.
 * Arguments as for iq_decode_attention / iq_combine_splits; no argmax output.
 */
#define IQ_STATIC_SCRATCH_BYTES (8u << 20)
size_t iq_static_scratch_bytes(void);
int iq_decode_attention_static(const iq_shape* shape, const float* rot_dev, const iq_codebook* codebook,
                               const void* q, const iq_cache* cache, const int32_t* seq_lens_dev,
                               int32_t num_splits, void* out, int32_t out_is_fp16, float* lse_out,
                               uint32_t* status_dev, void* stream);

/*
 * Diagnostic (the paper has no counterpart): exercises the give-up path of the decode kernel's bounded waits without
 * the decode kernel. A one-warp kernel waits on a barrier that nothing completes -- no copy and no tensor-core work
 * is in flight -- with `polls` (1 .. 65536) as its poll limit, sets IQ_STATUS_WAIT_TIMEOUT in status_dev[0] when the
 * wait gives up and writes the polls it took to status_dev[1]. polls == 0 completes the barrier first: the wait
 * succeeds and status_dev[0] stays as it is. A poll suspends the thread for at most 20 us, so the call lasts at
 * most polls * 20 us.
 */
int iq_selftest_bounded_wait(uint32_t* status_dev, uint32_t polls, void* stream);

/* A slot count that leaves the decode kernel free to balance the launch when the longest sequence has
 * max_seq_len rows (more slots than needed only cost the writing and merging of unused ones). */
int32_t iq_suggest_splits(const iq_shape* shape, int32_t max_seq_len);

#ifdef __cplusplus
}
#endif
#endif /* ISOQUANT_H_ */
