/*
 * IsoQuant oracle: a plain, slow, fp64 CPU statement of what the hot path computes.
 *
 * THIS IS TEST INFRASTRUCTURE. Only the test-suite, the smoke check and the benchmark's CPU
 * baseline may build, load or call it. The product (the CUDA library) shares no code, header,
 * table or helper with this file and never calls it.
 *
 * Everything is written from the paper's definitions, in the paper's order, with dense matrices
 * and plain loops: no butterfly, no blocking, no fusion.
 *   - Algorithm 1 (compression): s = ||x||_2, x^ = x/s, x~ = R_SO4(H_d x^), Lloyd-Max code per
 *     coordinate, bit-pack.
 *   - Eq. 2: R = R_SO4 o H_d, H_d the normalised Walsh-Hadamard matrix, R_SO4 block-diagonal with
 *     one 4x4 block per contiguous group of four coordinates.
 *   - Section 3.3 "SO(4) parameterization" and Appendix B: a block acts as v -> q_L v conj(q_R)
 *     with unit quaternions q_L, q_R; 8 floats per block.
 *   - Appendix A: q~ = R q, alpha = softmax(q~ . k~_j / sqrt(d_k)), o~ = sum_j alpha_j v~_j,
 *     o = R^T o~.
 *
 * Readings taken where the paper is silent (each is also listed in the design notes):
 *   - H_d in natural (Sylvester) order: H[i][j] = (-1)^popcount(i & j) / sqrt(d).
 *   - blocks b = 0 .. d/4-1 cover coordinates [4b, 4b+4) (Algorithm 1 prints 1-based "4i:4i+4").
 *   - quaternion = (w, x, y, z), Hamilton product, block coordinates (y0,y1,y2,y3) <-> y0 + y1 i + y2 j + y3 k.
 *   - quantiser works in unit-variance units u = sqrt(d) * x~; code = #{ j : u > t_j } over the 2^b - 1
 *     ascending thresholds (strict ">", an exact tie takes the lower code); codes 0 .. 2^b - 1 ascend with level.
 *     b = 3 is the paper's setting; Algorithm 1 is written for a general b, and b = 2 and b = 4 are carried too.
 *   - zero row: s = 0, x^ = 0.
 *   - stored scale = s rounded to fp32; dequantised coordinate = scale * level[code] / sqrt(d).
 *   - K and V of one KV head share that head's rotation; each side has its codebook (the same one unless the caller
 *     gives two); all query heads of a group use their KV head's rotation.
 *   - packed row layout (3 bits x d, 3d/8 bytes, the paper fixes only the size): the row is a
 *     sequence of little-endian 32-bit words; coordinates are taken in groups of 32, each group
 *     owning 3 consecutive words. In group-local numbering, coordinate c < 24 puts its 3-bit code in
 *     bits [4n, 4n+3) of word c/8, n = c mod 8; coordinate c >= 24 (n = c - 24) spreads its code
 *     over bit 4n+3 of the three words: bit k of the code goes to word k. K rows are stored this way, one
 *     row after the other. b = 4: entry c puts its code in bits [4n, 4n+4) of word c/8, n = c mod 8 (b d / 8 = d/2
 *     bytes per row). b = 2: entries are taken in groups of 16, one word each; in group-local numbering entry c < 8
 *     puts its code in bits [4c, 4c+2), entry c >= 8 in bits [4(c-8)+2, 4(c-8)+4) (d/4 bytes per row).
 *   - V codes are stored token-transposed (the paper says nothing about the arrangement): the rows of one
 *     (sequence, KV head) are taken in blocks of 128; for block j and coordinate c there is one record of 16 b
 *     bytes (48 at b = 3), at byte ((j * d) + c) * 16 b of that head's V area, holding the 128 codes of coordinate c for the
 *     block's rows, arranged exactly like a packed row of 128 entries with the row-in-block as the entry
 *     index. t_cap is a multiple of 128.
 *
 * Parity pins: every function here is pinned by tests/test_oracle_*.py (invariants, closed forms,
 * library routines, brute force). Not pinned (no published artefact exists): equality of the code
 * values and codebook with the authors' own files -- "parity unpinned" for those two items.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

int iqo_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

void iqo_set_num_threads(int n) {
#ifdef _OPENMP
  if (n > 0) omp_set_num_threads(n);
#else
  (void)n;
#endif
}

/* IEEE binary16 -> double, from the format definition. */
double iqo_half_to_double(uint16_t h) {
  int sign = (h >> 15) & 1, e = (h >> 10) & 31, m = h & 1023;
  double v;
  if (e == 0) v = ldexp((double)m, -24);
  else if (e == 31) v = m ? NAN : INFINITY;
  else v = ldexp((double)(m + 1024), e - 25);
  return sign ? -v : v;
}

/* Hamilton product of quaternions stored (w, x, y, z). */
static void quat_mul(const double* a, const double* b, double* o) {
  o[0] = a[0] * b[0] - a[1] * b[1] - a[2] * b[2] - a[3] * b[3];
  o[1] = a[0] * b[1] + a[1] * b[0] + a[2] * b[3] - a[3] * b[2];
  o[2] = a[0] * b[2] - a[1] * b[3] + a[2] * b[0] + a[3] * b[1];
  o[3] = a[0] * b[3] + a[1] * b[2] - a[2] * b[1] + a[3] * b[0];
}

/* Section 3.3 / Appendix B: the 4x4 matrix of v -> q_L v conj(q_R), built column by column by
 * applying the map to the basis quaternions. q8 = (q_L.wxyz, q_R.wxyz) as stored (fp32); both are
 * renormalised to unit length in fp64 first. M is row-major [4][4]. */
void iqo_so4_block(const float* q8, double* M) {
  double qL[4], qR[4], qRc[4], nL = 0, nR = 0;
  for (int i = 0; i < 4; i++) { qL[i] = q8[i]; qR[i] = q8[4 + i]; nL += qL[i] * qL[i]; nR += qR[i] * qR[i]; }
  nL = sqrt(nL); nR = sqrt(nR);
  for (int i = 0; i < 4; i++) { qL[i] /= nL; qR[i] /= nR; }
  qRc[0] = qR[0]; qRc[1] = -qR[1]; qRc[2] = -qR[2]; qRc[3] = -qR[3];
  for (int c = 0; c < 4; c++) {
    double e[4] = {0, 0, 0, 0}, t[4], r[4];
    e[c] = 1.0;
    quat_mul(qL, e, t);
    quat_mul(t, qRc, r);
    for (int i = 0; i < 4; i++) M[i * 4 + c] = r[i];
  }
}

/* Eq. 2: normalised Walsh-Hadamard matrix, natural order. H is row-major [d][d]. */
void iqo_hadamard(int d, double* H) {
  double s = 1.0 / sqrt((double)d);
  for (int i = 0; i < d; i++)
    for (int j = 0; j < d; j++)
      H[(size_t)i * d + j] = (__builtin_popcount((unsigned)(i & j)) & 1) ? -s : s;
}

/* Eq. 2: R = blockdiag(M_0 .. M_{d/4-1}) * H_d as a dense d x d matrix (row-major).
 * quats = [d/4][8] fp32 for one KV head. */
void iqo_rotation_matrix(int d, const float* quats, double* R) {
  double* H = (double*)malloc(sizeof(double) * d * d);
  iqo_hadamard(d, H);
  for (int b = 0; b < d / 4; b++) {
    double M[16];
    iqo_so4_block(quats + 8 * b, M);
    for (int r = 0; r < 4; r++)
      for (int j = 0; j < d; j++) {
        double acc = 0;
        for (int c = 0; c < 4; c++) acc += M[r * 4 + c] * H[(size_t)(4 * b + c) * d + j];
        R[(size_t)(4 * b + r) * d + j] = acc;
      }
  }
  free(H);
}

/* Algorithm 1, lines 1-4 and Step 3, for one row. x: d binary16 values. codes: one byte per
 * coordinate (0 .. 2^bits - 1; thresholds: 2^bits - 1 of them). Returns the fp32 scale; if u_out != NULL also returns u = sqrt(d) * x~. */
float iqo_quantize_row(int d, int bits, const double* R, const float* thresholds, const uint16_t* x,
                       uint8_t* codes, double* u_out) {
  const int n_th = (1 << bits) - 1;
  double* xh = (double*)malloc(sizeof(double) * d);
  double ss = 0;
  for (int i = 0; i < d; i++) { xh[i] = iqo_half_to_double(x[i]); ss += xh[i] * xh[i]; }
  double s = sqrt(ss);
  for (int i = 0; i < d; i++) xh[i] = (s == 0.0) ? 0.0 : xh[i] / s;
  double rootd = sqrt((double)d);
  for (int i = 0; i < d; i++) {
    double acc = 0;
    for (int j = 0; j < d; j++) acc += R[(size_t)i * d + j] * xh[j];
    double u = rootd * acc;
    int code = 0;
    for (int j = 0; j < n_th; j++) if (u > (double)thresholds[j]) code++;
    codes[i] = (uint8_t)code;
    if (u_out) u_out[i] = u;
  }
  free(xh);
  return (float)s;
}

static int row_bytes(int d, int bits) { return bits * d / 8; }

static void put_word(uint8_t* p, uint32_t w) { p[0] = w & 255; p[1] = (w >> 8) & 255; p[2] = (w >> 16) & 255; p[3] = (w >> 24) & 255; }
static uint32_t get_word(const uint8_t* p) { return (uint32_t)p[0] | ((uint32_t)p[1] << 8) | ((uint32_t)p[2] << 16) | ((uint32_t)p[3] << 24); }

/* Entry e of a packed record (a K row: e = coordinate; a V record: e = row within the block), layouts as described at
 * the top of this file. rec points at the record's first byte. */
static uint32_t record_get(int bits, const uint8_t* rec, int e) {
  if (bits == 4) return (get_word(rec + 4 * (e / 8)) >> (4 * (e % 8))) & 15u;
  if (bits == 2) {
    int c = e % 16;
    int sh = (c < 8) ? 4 * c : 4 * (c - 8) + 2;
    return (get_word(rec + 4 * (e / 16)) >> sh) & 3u;
  }
  const uint8_t* grp = rec + 12 * (e / 32);  /* bits == 3: groups of 32 entries in 3 words */
  int cc = e % 32;
  if (cc < 24) return (get_word(grp + 4 * (cc / 8)) >> (4 * (cc % 8))) & 7u;
  uint32_t code = 0;
  for (int k = 0; k < 3; k++) code |= ((get_word(grp + 4 * k) >> (4 * (cc - 24) + 3)) & 1u) << k;
  return code;
}
static void record_put(int bits, uint8_t* rec, int e, uint32_t code) {
  if (bits == 4) {
    uint8_t* wp = rec + 4 * (e / 8);
    int sh = 4 * (e % 8);
    put_word(wp, (get_word(wp) & ~(15u << sh)) | ((code & 15u) << sh));
    return;
  }
  if (bits == 2) {
    uint8_t* wp = rec + 4 * (e / 16);
    int c = e % 16;
    int sh = (c < 8) ? 4 * c : 4 * (c - 8) + 2;
    put_word(wp, (get_word(wp) & ~(3u << sh)) | ((code & 3u) << sh));
    return;
  }
  uint8_t* grp = rec + 12 * (e / 32);
  int cc = e % 32;
  if (cc < 24) {
    uint8_t* wp = grp + 4 * (cc / 8);
    int sh = 4 * (cc % 8);
    put_word(wp, (get_word(wp) & ~(7u << sh)) | ((code & 7u) << sh));
  } else {
    int sh = 4 * (cc - 24) + 3;
    for (int k = 0; k < 3; k++) {
      uint8_t* wp = grp + 4 * k;
      put_word(wp, (get_word(wp) & ~(1u << sh)) | (((code >> k) & 1u) << sh));
    }
  }
}

/* Step 4 (bit-pack) of one K row, and its inverse. */
void iqo_pack_row(int d, int bits, const uint8_t* codes, uint8_t* row) {
  memset(row, 0, (size_t)row_bytes(d, bits));
  for (int c = 0; c < d; c++) record_put(bits, row, c, codes[c]);
}

void iqo_unpack_row(int d, int bits, const uint8_t* row, uint8_t* codes) {
  for (int c = 0; c < d; c++) codes[c] = (uint8_t)record_get(bits, row, c);
}

/* Token-transposed V area of one (sequence, KV head): the record of (block t / 128, coordinate c) holds 128 entries,
 * the row within the block as the entry. */
static size_t v_record(int d, int bits, int64_t t, int c) { return ((size_t)(t / 128) * (size_t)d + (size_t)c) * (size_t)(16 * bits); }
/* Codes of V row t of one (sequence, KV head) area, one byte per coordinate. */
void iqo_v_row_codes(int d, int bits, const uint8_t* area, int64_t t, uint8_t* codes) {
  for (int c = 0; c < d; c++) codes[c] = (uint8_t)record_get(bits, area + v_record(d, bits, t, c), (int)(t % 128));
}
void iqo_v_row_store(int d, int bits, uint8_t* area, int64_t t, const uint8_t* codes) {
  for (int c = 0; c < d; c++) record_put(bits, area + v_record(d, bits, t, c), (int)(t % 128), codes[c]);
}

/* Algorithm 1 applied to the new K and V rows of every sequence and KV head, appended to the cache.
 * k_new, v_new: binary16, element (b, i, h, c) at b*stride_b + i*stride_t + h*stride_h + c (element strides).
 * Row i < n_new[b] of sequence b goes to cache row append_pos[b] + i (rows >= t_cap are skipped).
 * quats: [H_kv][d/4][8]. codes: [B][H_kv][t_cap][bits d/8], scales: [B][H_kv][t_cap]. thresholds_k / thresholds_v: the
 * 2^bits - 1 thresholds of the K side and of the V side.
 * Returns the number of rows skipped because they fell outside the cache. */
int64_t iqo_quantize_append(int B, int H_kv, int d, int bits, int t_cap, const float* quats, const float* thresholds_k,
                            const float* thresholds_v, const uint16_t* k_new, const uint16_t* v_new,
                            int64_t stride_b, int64_t stride_t, int64_t stride_h,
                            const int32_t* append_pos, const int32_t* n_new, int n_new_max,
                            uint8_t* k_codes, float* k_scales, uint8_t* v_codes, float* v_scales) {
  int P = row_bytes(d, bits);
  int64_t skipped = 0;
  for (int h = 0; h < H_kv; h++) {
    double* R = (double*)malloc(sizeof(double) * d * d);
    iqo_rotation_matrix(d, quats + (size_t)h * (d / 4) * 8, R);
    for (int b = 0; b < B; b++) {
      int n = n_new ? n_new[b] : n_new_max;
      if (n > n_new_max) n = n_new_max;
      int64_t sk = 0;
#pragma omp parallel for schedule(static) reduction(+ : sk)
      for (int i = 0; i < n; i++) {
        int64_t t = (int64_t)append_pos[b] + i;
        if (t < 0 || t >= t_cap) { sk += 2; continue; }
        uint8_t codes[512];
        size_t src = (size_t)(b * stride_b + i * stride_t + h * stride_h);
        size_t row = ((size_t)b * H_kv + h) * t_cap + t;
        k_scales[row] = iqo_quantize_row(d, bits, R, thresholds_k, k_new + src, codes, NULL);
        iqo_pack_row(d, bits, codes, k_codes + row * P);
      }
      /* V rows share words between neighbouring rows (token-transposed records): written one row at a time */
      for (int i = 0; i < n; i++) {
        int64_t t = (int64_t)append_pos[b] + i;
        if (t < 0 || t >= t_cap) continue;
        uint8_t codes[512];
        size_t src = (size_t)(b * stride_b + i * stride_t + h * stride_h);
        size_t area = ((size_t)b * H_kv + h) * t_cap;
        v_scales[area + t] = iqo_quantize_row(d, bits, R, thresholds_v, v_new + src, codes, NULL);
        iqo_v_row_store(d, bits, v_codes + area * P, t, codes);
      }
      skipped += sk;
    }
    free(R);
  }
  return skipped;
}

/* Dequantised rotated vector of cached V row t of a (sequence, KV head) area. */
static void dequant_v_row(int d, int bits, const uint8_t* area, int64_t t, float scale, const float* levels, double* out) {
  uint8_t codes[512];
  iqo_v_row_codes(d, bits, area, t, codes);
  double f = (double)scale / sqrt((double)d);
  for (int i = 0; i < d; i++) out[i] = f * (double)levels[codes[i]];
}

/* Dequantised rotated vector of one cached K row: x~_i = scale * level[code_i] / sqrt(d). */
static void dequant_row(int d, int bits, const uint8_t* row, float scale, const float* levels, double* out) {
  uint8_t codes[512];
  iqo_unpack_row(d, bits, row, codes);
  double f = (double)scale / sqrt((double)d);
  for (int i = 0; i < d; i++) out[i] = f * (double)levels[codes[i]];
}

/* Appendix A, one query head against the first len rows of its KV head's packed cache.
 * z_out (optional, [len]) receives the scaled scores; o_rot (optional, [d]) the rotated-space output. */
static void decode_one(int d, int bits, const double* R, const float* levels_k, const float* levels_v, double sm_scale, const uint16_t* q,
                       const uint8_t* k_codes, const float* k_scales, const uint8_t* v_codes,
                       const float* v_scales, int len, double* out, double* lse, int32_t* argmax,
                       double* z_out, double* o_rot_out) {
  int P = row_bytes(d, bits);
  double* qt = (double*)malloc(sizeof(double) * d);
  double* z = (double*)malloc(sizeof(double) * (len > 0 ? len : 1));
  double* row = (double*)malloc(sizeof(double) * d);
  double* orot = (double*)calloc(d, sizeof(double));
  for (int i = 0; i < d; i++) {           /* q~ = R q */
    double acc = 0;
    for (int j = 0; j < d; j++) acc += R[(size_t)i * d + j] * iqo_half_to_double(q[j]);
    qt[i] = acc;
  }
  int best = -1;
  double zmax = -INFINITY;
  for (int j = 0; j < len; j++) {         /* z_j = sm_scale * q~ . k~_j */
    dequant_row(d, bits, k_codes + (size_t)j * P, k_scales[j], levels_k, row);
    double acc = 0;
    for (int i = 0; i < d; i++) acc += qt[i] * row[i];
    z[j] = sm_scale * acc;
    if (z[j] > zmax) { zmax = z[j]; best = j; }
    if (z_out) z_out[j] = z[j];
  }
  double denom = 0;
  for (int j = 0; j < len; j++) denom += exp(z[j] - zmax);
  for (int j = 0; j < len; j++) {         /* o~ = sum_j alpha_j v~_j */
    double a = exp(z[j] - zmax) / denom;
    dequant_v_row(d, bits, v_codes, j, v_scales[j], levels_v, row);
    for (int i = 0; i < d; i++) orot[i] += a * row[i];
  }
  for (int j = 0; j < d; j++) {           /* o = R^T o~ */
    double acc = 0;
    for (int i = 0; i < d; i++) acc += R[(size_t)i * d + j] * orot[i];
    out[j] = (len > 0) ? acc : 0.0;
  }
  if (o_rot_out) for (int i = 0; i < d; i++) o_rot_out[i] = orot[i];
  if (lse) *lse = (len > 0) ? zmax + log(denom) : -INFINITY;
  if (argmax) *argmax = best;
  free(qt); free(z); free(row); free(orot);
}

/* One decode step for every sequence and query head. q: [B][H_q][d] binary16. out: [B][H_q][d],
 * lse: [B][H_q], argmax: [B][H_q] (lowest row index attaining the maximum score; -1 if len = 0).
 * sm_scale <= 0 selects 1/sqrt(d). o_rot (optional): [B][H_q][d], the output before R^T. */
void iqo_decode_attention(int B, int H_q, int H_kv, int d, int bits, int t_cap, double sm_scale, const float* quats,
                          const float* levels_k, const float* levels_v, const uint16_t* q, const uint8_t* k_codes,
                          const float* k_scales, const uint8_t* v_codes, const float* v_scales,
                          const int32_t* seq_lens, double* out, double* lse, int32_t* argmax, double* o_rot) {
  int P = row_bytes(d, bits), G = H_q / H_kv;
  if (sm_scale <= 0) sm_scale = 1.0 / sqrt((double)d);
  double* Rs = (double*)malloc(sizeof(double) * (size_t)H_kv * d * d);
  for (int g = 0; g < H_kv; g++) iqo_rotation_matrix(d, quats + (size_t)g * (d / 4) * 8, Rs + (size_t)g * d * d);
#pragma omp parallel for schedule(dynamic) collapse(2)
  for (int b = 0; b < B; b++)
    for (int h = 0; h < H_q; h++) {
      int g = h / G;
      int len = seq_lens[b];
      if (len > t_cap) len = t_cap;
      if (len < 0) len = 0;
      size_t base = ((size_t)b * H_kv + g) * t_cap;
      size_t o = ((size_t)b * H_q + h);
      decode_one(d, bits, Rs + (size_t)g * d * d, levels_k, levels_v, sm_scale, q + o * d, k_codes + base * P, k_scales + base,
                 v_codes + base * P, v_scales + base, len, out + o * d, lse ? lse + o : NULL,
                 argmax ? argmax + o : NULL, NULL, o_rot ? o_rot + o * d : NULL);
    }
  free(Rs);
}

/* Reconstruct-then-compute, first half (Figure 1, top; the execution model the fused path replaces): every cached
 * row back in the original space, x_hat = R^T x~ with x~_i = scale * level[code_i] / sqrt(d) (Algorithm 1 read
 * backwards; R is orthogonal, so R^-1 = R^T). k_out, v_out: [B][t_cap][H_kv][d] doubles; rows >= seq_lens[b] are
 * left untouched. */
void iqo_reconstruct_rows(int B, int H_kv, int d, int bits, int t_cap, const float* quats, const float* levels_k, const float* levels_v,
                          const uint8_t* k_codes, const float* k_scales, const uint8_t* v_codes,
                          const float* v_scales, const int32_t* seq_lens, double* k_out, double* v_out) {
  int P = row_bytes(d, bits);
  double* Rs = (double*)malloc(sizeof(double) * (size_t)H_kv * d * d);
  for (int g = 0; g < H_kv; g++) iqo_rotation_matrix(d, quats + (size_t)g * (d / 4) * 8, Rs + (size_t)g * d * d);
#pragma omp parallel for schedule(dynamic) collapse(2)
  for (int b = 0; b < B; b++)
    for (int g = 0; g < H_kv; g++) {
      int len = seq_lens[b];
      if (len > t_cap) len = t_cap;
      const double* R = Rs + (size_t)g * d * d;
      size_t base = ((size_t)b * H_kv + g) * t_cap;
      double xt[512];
      for (int t = 0; t < len; t++)
        for (int which = 0; which < 2; which++) {
          if (which == 0) dequant_row(d, bits, k_codes + (base + t) * P, k_scales[base + t], levels_k, xt);
          else dequant_v_row(d, bits, v_codes + base * P, t, v_scales[base + t], levels_v, xt);
          double* o = (which == 0 ? k_out : v_out) + (((size_t)b * t_cap + t) * H_kv + g) * d;
          for (int i = 0; i < d; i++) {  /* (R^T x~)_i = sum_j R[j][i] x~_j */
            double acc = 0;
            for (int j = 0; j < d; j++) acc += R[(size_t)j * d + i] * xt[j];
            o[i] = acc;
          }
        }
    }
  free(Rs);
}

/* Scaled scores z_j of one (sequence b, query head h): z_out [len]. */
void iqo_scores(int H_q, int H_kv, int d, int bits, int t_cap, double sm_scale, const float* quats, const float* levels_k,
                const uint16_t* q_bh, int b, int h, const uint8_t* k_codes, const float* k_scales, int len,
                double* z_out) {
  int P = row_bytes(d, bits), G = H_q / H_kv, g = h / G;
  if (sm_scale <= 0) sm_scale = 1.0 / sqrt((double)d);
  double* R = (double*)malloc(sizeof(double) * d * d);
  iqo_rotation_matrix(d, quats + (size_t)g * (d / 4) * 8, R);
  size_t base = ((size_t)b * H_kv + g) * t_cap;
  double* qt = (double*)malloc(sizeof(double) * d);
  double* row = (double*)malloc(sizeof(double) * d);
  for (int i = 0; i < d; i++) {
    double acc = 0;
    for (int j = 0; j < d; j++) acc += R[(size_t)i * d + j] * iqo_half_to_double(q_bh[j]);
    qt[i] = acc;
  }
  for (int j = 0; j < len; j++) {
    dequant_row(d, bits, k_codes + (base + j) * P, k_scales[base + j], levels_k, row);
    double acc = 0;
    for (int i = 0; i < d; i++) acc += qt[i] * row[i];
    z_out[j] = sm_scale * acc;
  }
  free(R); free(qt); free(row);
}

/* Merge of split-softmax partials from the definition of softmax (not in the paper: the paper's
 * pipeline is unsplit; the split is the flash-decoding decomposition of the same sums).
 * part_acc [B][H_q][S][d] = sum_{j in split} exp(z_j - m_s) v~_j (rotated space), part_ml [B][H_q][S][2]
 * = (m_s, l_s) with m_s = max z_j (-inf if empty), l_s = sum exp(z_j - m_s); part_argmax [B][H_q][S]
 * (row index attaining m_s, -1 if empty) or NULL.
 * out = R^T ( sum_s acc_s e^{m_s - m} / sum_s l_s e^{m_s - m} ), m = max_s m_s. */
void iqo_combine_splits(int B, int H_q, int H_kv, int d, int S, const float* quats, const float* part_acc,
                        const float* part_ml, const int32_t* part_argmax, double* out, double* lse,
                        int32_t* argmax) {
  int G = H_q / H_kv;
  for (int b = 0; b < B; b++)
    for (int h = 0; h < H_q; h++) {
      size_t o = (size_t)b * H_q + h;
      double m = -INFINITY;
      int best = -1;
      for (int s = 0; s < S; s++) {
        double ms = part_ml[(o * S + s) * 2];
        double ls = part_ml[(o * S + s) * 2 + 1];
        if (!(ls > 0)) continue;
        int idx = part_argmax ? part_argmax[o * S + s] : -1;
        if (ms > m) { m = ms; best = idx; }
        else if (ms == m && idx >= 0 && (best < 0 || idx < best)) best = idx;
      }
      double l = 0;
      double* orot = (double*)calloc(d, sizeof(double));
      for (int s = 0; s < S; s++) {
        double ms = part_ml[(o * S + s) * 2];
        double ls = part_ml[(o * S + s) * 2 + 1];
        if (!(ls > 0)) continue;
        double w = exp(ms - m);
        l += ls * w;
        for (int i = 0; i < d; i++) orot[i] += w * (double)part_acc[(o * S + s) * d + i];
      }
      double* R = (double*)malloc(sizeof(double) * d * d);
      iqo_rotation_matrix(d, quats + (size_t)(h / G) * (d / 4) * 8, R);
      for (int j = 0; j < d; j++) {
        double acc = 0;
        if (l > 0) for (int i = 0; i < d; i++) acc += R[(size_t)i * d + j] * orot[i] / l;
        out[o * d + j] = acc;
      }
      if (lse) lse[o] = (l > 0) ? m + log(l) : -INFINITY;
      if (argmax) argmax[o] = (l > 0) ? best : -1;
      free(R); free(orot);
    }
}
