// C ABI of the IsoQuant library: argument validation and kernel launches. See include/isoquant.h for the
// contract of every entry point. Nothing here allocates device memory or keeps state between calls.
#include <cmath>
#include <cstring>
#include <vector>

#include "iq_common.cuh"
#include "iq_kernels.h"

namespace {

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int check_shape(const iq_shape* s) {
  if (!s) return IQ_ERR_NULL;
  if (s->head_dim != 128 && s->head_dim != 256) return IQ_ERR_SHAPE;
  if (s->bits < 2 || s->bits > 4) return IQ_ERR_SHAPE;
  if (s->batch < 0 || s->batch > 65535) return IQ_ERR_SHAPE;
  if (s->n_kv_heads <= 0 || s->n_q_heads <= 0 || s->n_q_heads % s->n_kv_heads != 0) return IQ_ERR_SHAPE;
  if (s->t_cap <= 0 || (s->t_cap & 127) != 0) return IQ_ERR_SHAPE;
  const int hg = (s->n_q_heads / s->n_kv_heads + iq::DEC_HEADS - 1) / iq::DEC_HEADS;
  if ((long long)s->n_kv_heads * hg > 32767) return IQ_ERR_SHAPE;
  return IQ_OK;
}

bool fp16_exact(float x) { return std::isfinite(x) && __half2float(__float2half_rn(x)) == x; }

// The two sides of a codebook: K rows, V rows (the same unless separate_v).
const float* side_levels(const iq_codebook* cb, int v) { return (v && cb->separate_v) ? cb->v_levels : cb->levels; }
const float* side_thresholds(const iq_codebook* cb, int v) { return (v && cb->separate_v) ? cb->v_thresholds : cb->thresholds; }

int check_codebook(const iq_codebook* cb, int bits, bool need_fp16_levels) {
  if (!cb) return IQ_ERR_NULL;
  if (cb->bits != bits || bits < 2 || bits > 4) return IQ_ERR_CODEBOOK;
  const int n = 1 << bits;
  for (int v = 0; v < (cb->separate_v ? 2 : 1); v++) {
    const float* lv = side_levels(cb, v);
    const float* th = side_thresholds(cb, v);
    for (int i = 0; i < n; i++) {
      if (!std::isfinite(lv[i])) return IQ_ERR_CODEBOOK;
      if (i && !(lv[i] > lv[i - 1])) return IQ_ERR_CODEBOOK;
      if (need_fp16_levels && !fp16_exact(lv[i])) return IQ_ERR_CODEBOOK;
    }
    for (int i = 0; i < n - 1; i++) {
      if (!std::isfinite(th[i])) return IQ_ERR_CODEBOOK;
      if (i && !(th[i] > th[i - 1])) return IQ_ERR_CODEBOOK;
    }
  }
  return IQ_OK;
}

// Levels on an 8-bit grid: level_j = n_j * delta with integer |n_j| <= 127 and delta = max|level| / 127 (to fp32
// rounding). Fills n[] and delta for one side of the codebook.
bool int8_grid_side(const float* lv, int n_levels, int (&n)[16], float& delta) {
  float mx = 0.f;
  for (int i = 0; i < n_levels; i++) mx = std::fmax(mx, std::fabs(lv[i]));
  if (!(mx > 0.f)) return false;
  delta = mx / 127.0f;
  for (int i = 0; i < n_levels; i++) {
    const double r = (double)lv[i] / (double)delta;
    const double ri = std::nearbyint(r);
    if (std::fabs(r - ri) > 1e-4 || std::fabs(ri) > 127.0) return false;
    n[i] = (int)ri;
  }
  return true;
}
// Both sides on 8-bit grids (each its own): the integer decode path.
bool int8_grid(const iq_codebook* cb, int (&nk)[16], float& delta_k, int (&nv)[16], float& delta_v) {
  const int n = 1 << cb->bits;
  return int8_grid_side(side_levels(cb, 0), n, nk, delta_k) && int8_grid_side(side_levels(cb, 1), n, nv, delta_v);
}

int check_cache(const iq_cache* c, const iq_shape* shape) {
  if (!c || !c->k_codes || !c->k_scales || !c->v_codes || !c->v_scales) return IQ_ERR_NULL;
  if (!aligned16(c->k_codes) || !aligned16(c->k_scales) || !aligned16(c->v_codes) || !aligned16(c->v_scales)) return IQ_ERR_ALIGN;
  if (c->block_table_dev) {  // paged: whole 128-row blocks per page, whole pages per sequence
    if (c->page_rows <= 0 || (c->page_rows % 128) != 0 || c->num_pages <= 0 || (shape->t_cap % c->page_rows) != 0) return IQ_ERR_SHAPE;
  }
  return IQ_OK;
}

iq::PageMap page_map(const iq_cache* c, const iq_shape* shape) {
  iq::PageMap m;
  m.table = c->block_table_dev;
  m.page_rows = c->block_table_dev ? c->page_rows : 0;
  m.num_pages = c->block_table_dev ? c->num_pages : 0;
  m.n_kv_heads = shape->n_kv_heads;
  m.t_cap = shape->t_cap;
  return m;
}

// Lloyd's iteration for the marginal of one coordinate of a uniform point on S^{d-1}, unit-variance units:
// density ~ (1 - u^2/d)^((d-3)/2). Cell integrals by composite Simpson on a fixed fine grid.
struct SphereMarginal {
  double d;
  double pdf(double u) const {
    const double b = 1.0 - u * u / d;
    return b > 0.0 ? std::exp(0.5 * (d - 3.0) * std::log(b)) : 0.0;
  }
  void cell(double a, double b, double& mass, double& mom) const {
    const int n = 2048;
    const double hstep = (b - a) / n;
    double m0 = 0, m1 = 0;
    for (int i = 0; i <= n; i++) {
      const double u = a + hstep * i;
      const double w = (i == 0 || i == n) ? 1.0 : ((i & 1) ? 4.0 : 2.0);
      const double f = pdf(u);
      m0 += w * f;
      m1 += w * f * u;
    }
    mass = m0 * hstep / 3.0;
    mom = m1 * hstep / 3.0;
  }
};

void lloyd_max_sphere(int d, int n, double (&lv)[16]) {
  SphereMarginal f{(double)d};
  const double lim = std::sqrt((double)d);
  for (int i = 0; i < n; i++) lv[i] = -2.4 + 4.8 * (i + 0.5) / n;
  for (int iter = 0; iter < 20000; iter++) {
    double edge[17];
    edge[0] = -lim;
    edge[n] = lim;
    for (int i = 1; i < n; i++) edge[i] = 0.5 * (lv[i - 1] + lv[i]);
    double delta = 0;
    for (int i = 0; i < n; i++) {
      double mass, mom;
      f.cell(edge[i], edge[i + 1], mass, mom);
      const double c = mom / mass;
      delta = std::fmax(delta, std::fabs(c - lv[i]));
      lv[i] = c;
    }
    if (delta < 1e-13) break;
  }
}

// Lloyd's iteration on a histogram with uniform bins on [-range, range), read as a piecewise-constant density: a bin
// cut by a threshold contributes to both cells in proportion. mass0 / mom0: mass and first moment below bin edge i.
void lloyd_max_histogram(const std::vector<double>& c, double range, bool symmetric, int n, double (&lv)[16]) {
  const int bins = (int)c.size();
  const double w = 2.0 * range / bins;
  std::vector<double> mass0(bins + 1, 0.0), mom0(bins + 1, 0.0);
  for (int i = 0; i < bins; i++) {
    const double lo = i * w - range, hi = lo + w;
    mass0[i + 1] = mass0[i] + c[i];
    mom0[i + 1] = mom0[i] + c[i] * 0.5 * (lo + hi);
  }
  auto below = [&](double t, double& mass, double& mom) {
    t = std::fmin(std::fmax(t, -range), range);
    int i = (int)((t + range) / w);
    if (i > bins - 1) i = bins - 1;
    const double lo = i * w - range, dens = c[i] / w;
    mass = mass0[i] + dens * (t - lo);
    mom = mom0[i] + dens * 0.5 * (t * t - lo * lo);
  };
  const double total = mass0[bins];
  {  // start: the quantiles (k + 1/2) / n
    int i = 0;
    for (int k = 0; k < n; k++) {
      const double target = total * (k + 0.5) / n;
      while (i < bins - 1 && mass0[i + 1] < target) i++;
      const double frac = c[i] > 0.0 ? (target - mass0[i]) / c[i] : 0.5;
      lv[k] = (i + frac) * w - range;
    }
  }
  for (int iter = 0; iter < 20000; iter++) {
    double cut[17], m[17], f[17];
    cut[0] = -range;
    cut[n] = range;
    for (int i = 1; i < n; i++) cut[i] = 0.5 * (lv[i - 1] + lv[i]);
    for (int i = 0; i <= n; i++) below(cut[i], m[i], f[i]);
    double nl[16];
    for (int i = 0; i < n; i++) {
      const double mass = m[i + 1] - m[i];
      nl[i] = mass > 0.0 ? (f[i + 1] - f[i]) / mass : lv[i];
    }
    if (symmetric)
      for (int i = 0; i < n / 2; i++) {
        const double a = 0.5 * (nl[n - 1 - i] - nl[i]);
        nl[n - 1 - i] = a;
        nl[i] = -a;
      }
    double delta = 0.0;
    for (int i = 0; i < n; i++) {
      delta = std::fmax(delta, std::fabs(nl[i] - lv[i]));
      lv[i] = nl[i];
    }
    if (delta < 1e-13) break;
  }
}

// Levels (fp64, ascending) -> the codebook handed to the kernels: levels exactly representable in binary16 (grid = 0)
// or on an 8-bit grid (grid = 1: level = n * delta, |n| <= 127, delta = max |level| / 127), thresholds = midpoints.
void finish_codebook(const double (&lv)[16], int bits, int grid, iq_codebook* out) {
  const int n = 1 << bits;
  std::memset(out, 0, sizeof(*out));
  out->bits = bits;
  if (grid == 1) {
    double amax = 0.0;
    for (int i = 0; i < n; i++) amax = std::fmax(amax, std::fabs(lv[i]));
    const float delta = (float)(amax / 127.0);
    for (int i = 0; i < n; i++) out->levels[i] = delta > 0.f ? (float)std::nearbyint(lv[i] / (double)delta) * delta : 0.f;
  } else {
    for (int i = 0; i < n; i++) out->levels[i] = __half2float(__float2half_rn((float)lv[i]));
  }
  for (int i = 0; i < n - 1; i++) out->thresholds[i] = (float)(0.5 * ((double)out->levels[i] + (double)out->levels[i + 1]));
}

// ---- fitting the SO(4) blocks (host, fp64) ---------------------------------------------------------------------
// A block matrix from its quaternion pair, M = L(q_L) R(conj q_R) (Section 3.3), both quaternions rescaled to unit length.
void so4_from_pair(const double* q8, double (&M)[4][4]) {
  double a = q8[0], b = q8[1], c = q8[2], d = q8[3], e = q8[4], f = q8[5], g = q8[6], h = q8[7];
  const double nl = 1.0 / std::sqrt(a * a + b * b + c * c + d * d), nr = 1.0 / std::sqrt(e * e + f * f + g * g + h * h);
  a *= nl; b *= nl; c *= nl; d *= nl; e *= nr; f *= nr; g *= nr; h *= nr;
  const double L[4][4] = {{a, -b, -c, -d}, {b, a, -d, c}, {c, d, a, -b}, {d, -c, b, a}};
  const double R[4][4] = {{e, f, g, h}, {-f, e, -h, g}, {-g, h, e, -f}, {-h, -g, f, e}};
  for (int i = 0; i < 4; i++)
    for (int j = 0; j < 4; j++) {
      double s = 0;
      for (int k = 0; k < 4; k++) s += L[i][k] * R[k][j];
      M[i][j] = s;
    }
}
// The pair back from a rotation matrix: M is bilinear in (q_L, q_R) over the 16 matrices T_ab = L(e_a) R(conj e_b), which
// are orthogonal under the Frobenius product with squared norm 4, so <M, T_ab> / 4 = l_a r_b.
void pair_from_so4(const double (&M)[4][4], double* q8) {
  double P[4][4];
  for (int a = 0; a < 4; a++)
    for (int b = 0; b < 4; b++) {
      double e8[8] = {0, 0, 0, 0, 0, 0, 0, 0}, T[4][4];
      e8[a] = 1.0;
      e8[4 + b] = 1.0;
      so4_from_pair(e8, T);
      double s = 0;
      for (int i = 0; i < 4; i++)
        for (int j = 0; j < 4; j++) s += T[i][j] * M[i][j];
      P[a][b] = 0.25 * s;
    }
  int best = 0;
  double bn = -1.0;
  for (int a = 0; a < 4; a++) {
    const double n = P[a][0] * P[a][0] + P[a][1] * P[a][1] + P[a][2] * P[a][2] + P[a][3] * P[a][3];
    if (n > bn) { bn = n; best = a; }
  }
  double r[4], l[4], rn = std::sqrt(bn), ln = 0;
  for (int b = 0; b < 4; b++) r[b] = P[best][b] / rn;
  for (int a = 0; a < 4; a++) {
    l[a] = P[a][0] * r[0] + P[a][1] * r[1] + P[a][2] * r[2] + P[a][3] * r[3];
    ln += l[a] * l[a];
  }
  ln = std::sqrt(ln);
  for (int a = 0; a < 4; a++) { q8[a] = l[a] / ln; q8[4 + a] = r[a]; }
}
// Mean over the rows of the squared quantisation error of u = M z (four coordinates), z = z4[n * stride .. + 4).
double block_distortion(const float* z4, size_t stride, int n, const double (&M)[4][4], const iq_codebook& cb) {
  double total = 0.0;
  for (int i = 0; i < n; i++) {
    const float* z = z4 + (size_t)i * stride;
    for (int r = 0; r < 4; r++) {
      const double u = M[r][0] * z[0] + M[r][1] * z[1] + M[r][2] * z[2] + M[r][3] * z[3];
      int code = 0;
      for (int j = 0; j < (1 << cb.bits) - 1; j++) code += u > (double)cb.thresholds[j];
      const double e = u - (double)cb.levels[code];
      total += e * e;
    }
  }
  return total / n;
}
// Pattern search over the six coordinate planes: rotate by +-delta, keep what lowers the distortion, halve delta when a
// sweep improves nothing (pi/8 down to 1e-3 rad). Returns the distortion reached; M is updated in place.
double fit_block(const float* z4, size_t stride, int n, double (&M)[4][4], const iq_codebook& cb, double& start) {
  static const int planes[6][2] = {{0, 1}, {0, 2}, {0, 3}, {1, 2}, {1, 3}, {2, 3}};
  double best = start = block_distortion(z4, stride, n, M, cb);
  for (double delta = 3.14159265358979323846 / 8; delta >= 1e-3;) {
    bool improved = false;
    for (int pl = 0; pl < 6; pl++) {
      const int i = planes[pl][0], j = planes[pl][1];
      for (int sg = 0; sg < 2; sg++) {
        const double c = std::cos(delta), sn = (sg == 0 ? 1.0 : -1.0) * std::sin(delta);
        double C[4][4];
        for (int r = 0; r < 4; r++)
          for (int k = 0; k < 4; k++) C[r][k] = M[r][k];
        for (int k = 0; k < 4; k++) {  // G(i, j, angle) M: rows i and j mix
          C[i][k] = c * M[i][k] - sn * M[j][k];
          C[j][k] = sn * M[i][k] + c * M[j][k];
        }
        const double dist = block_distortion(z4, stride, n, C, cb);
        if (dist < best) {
          for (int r = 0; r < 4; r++)
            for (int k = 0; k < 4; k++) M[r][k] = C[r][k];
          best = dist;
          improved = true;
          break;
        }
      }
    }
    if (!improved) delta *= 0.5;
  }
  return best;
}

}  // namespace

extern "C" {

int iq_version(void) { return IQ_VERSION; }
int iq_format_version(void) { return IQ_FORMAT_VERSION; }

const char* iq_strerror(int code) {
  switch (code) {
    case IQ_OK: return "ok";
    case IQ_ERR_NULL: return "a required pointer is NULL";
    case IQ_ERR_SHAPE: return "unsupported shape (head_dim 128/256, bits 2/3/4, n_q_heads % n_kv_heads == 0, t_cap % 128 == 0, strides % 8 == 0)";
    case IQ_ERR_ALIGN: return "pointer or stride not 16-byte aligned";
    case IQ_ERR_CODEBOOK: return "codebook bits differ from the shape's, codebook not ascending, or (decode) its levels are neither on an 8-bit grid nor all exact binary16 values";
    case IQ_ERR_CUDA: return "CUDA runtime error at launch";
    case IQ_ERR_LIMIT: return "size exceeds the documented maximum of this entry point";
    default: return "unknown error code";
  }
}

size_t iq_row_bytes_bits(int32_t head_dim, int32_t bits) {
  return ((head_dim == 128 || head_dim == 256) && bits >= 2 && bits <= 4) ? (size_t)(bits * head_dim / 8) : 0;
}
size_t iq_row_bytes(int32_t head_dim) { return iq_row_bytes_bits(head_dim, 3); }

size_t iq_rotation_floats(int32_t head_dim, int32_t n_kv_heads) {
  if ((head_dim != 128 && head_dim != 256) || n_kv_heads <= 0) return 0;
  return (size_t)n_kv_heads * (size_t)(head_dim / 4) * 8;
}

int iq_lloyd_max_codebook(int32_t head_dim, int32_t bits, int32_t grid, iq_codebook* out_host) {
  if (!out_host) return IQ_ERR_NULL;
  if ((head_dim != 128 && head_dim != 256) || bits < 2 || bits > 4 || (grid != 0 && grid != 1)) return IQ_ERR_SHAPE;
  const int n = 1 << bits;
  double lv[16];
  lloyd_max_sphere(head_dim, n, lv);
  std::memset(out_host, 0, sizeof(*out_host));
  out_host->bits = bits;
  double a[8];
  for (int i = 0; i < n / 2; i++) a[i] = 0.5 * (lv[n - 1 - i] - lv[i]);  // exact symmetry; a[0] is the largest magnitude
  const float delta = (float)(a[0] / 127.0);
  for (int i = 0; i < n / 2; i++) {  // rounded to binary16, or snapped to the 8-bit grid
    const float r = grid ? (float)std::nearbyint(a[i] / (double)delta) * delta : __half2float(__float2half_rn((float)a[i]));
    out_host->levels[n - 1 - i] = r;
    out_host->levels[i] = -r;
  }
  for (int i = 0; i < n - 1; i++)
    out_host->thresholds[i] = (float)(0.5 * ((double)out_host->levels[i] + (double)out_host->levels[i + 1]));
  return IQ_OK;
}
int iq_default_codebook(int32_t head_dim, iq_codebook* out_host) { return iq_lloyd_max_codebook(head_dim, 3, 0, out_host); }
int iq_int8_codebook(int32_t head_dim, iq_codebook* out_host) { return iq_lloyd_max_codebook(head_dim, 3, 1, out_host); }

int iq_codebook_set_v(iq_codebook* cb, const iq_codebook* v_side) {
  if (!cb || !v_side) return IQ_ERR_NULL;
  if (cb->bits != v_side->bits || cb->bits < 2 || cb->bits > 4) return IQ_ERR_CODEBOOK;
  cb->separate_v = 1;
  std::memcpy(cb->v_levels, v_side->levels, sizeof(cb->v_levels));
  std::memcpy(cb->v_thresholds, v_side->thresholds, sizeof(cb->v_thresholds));
  return IQ_OK;
}

int iq_make_rotation(int32_t head_dim, int32_t n_kv_heads, uint64_t seed, const float* quats_host, float* rot_dev,
                     void* stream) {
  const size_t nfl = iq_rotation_floats(head_dim, n_kv_heads);
  if (nfl == 0) return IQ_ERR_SHAPE;
  if (!rot_dev) return IQ_ERR_NULL;
  if (!aligned16(rot_dev)) return IQ_ERR_ALIGN;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int n_quats = (int)(nfl / 4);
  cudaError_t e;
  if (quats_host) {
    e = cudaMemcpyAsync(rot_dev, quats_host, nfl * sizeof(float), cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) return IQ_ERR_CUDA;
    e = iq::launch_normalize_rotation(rot_dev, n_quats, st);
  } else {
    e = iq::launch_make_rotation(rot_dev, n_quats, seed, st);
  }
  return e == cudaSuccess ? IQ_OK : IQ_ERR_CUDA;
}

int iq_quantize_append(const iq_shape* shape, const float* rot_dev, const iq_codebook* codebook, const void* k_new,
                       const void* v_new, int64_t stride_b, int64_t stride_t, int64_t stride_h,
                       const int32_t* append_pos_dev, const int32_t* n_new_dev, int32_t n_new_max,
                       const iq_cache* cache, uint32_t* status_dev, void* stream) {
  int rc = check_shape(shape);
  if (rc) return rc;
  if (!rot_dev || !append_pos_dev) return IQ_ERR_NULL;
  if ((rc = check_codebook(codebook, shape->bits, false))) return rc;
  if ((rc = check_cache(cache, shape))) return rc;
  if (n_new_max < 0) return IQ_ERR_SHAPE;
  if (n_new_max == 0 || shape->batch == 0) return IQ_OK;
  if (!k_new || !v_new) return IQ_ERR_NULL;
  if (!aligned16(k_new) || !aligned16(v_new) || !aligned16(rot_dev)) return IQ_ERR_ALIGN;
  if (stride_b < 0 || stride_t < 0 || stride_h < 0) return IQ_ERR_SHAPE;
  if ((stride_b & 7) || (stride_t & 7) || (stride_h & 7)) return IQ_ERR_ALIGN;

  iq::QuantizeParams p;
  p.k_new = static_cast<const __half*>(k_new);
  p.v_new = static_cast<const __half*>(v_new);
  p.stride_b = stride_b;
  p.stride_t = stride_t;
  p.stride_h = stride_h;
  p.append_pos = append_pos_dev;
  p.n_new = n_new_dev;
  p.n_new_max = n_new_max;
  p.rot = rot_dev;
  p.bits = shape->bits;
  std::memcpy(p.thresholds_k, side_thresholds(codebook, 0), sizeof(p.thresholds_k));
  std::memcpy(p.thresholds_v, side_thresholds(codebook, 1), sizeof(p.thresholds_v));
  p.k_codes = cache->k_codes;
  p.k_scales = cache->k_scales;
  p.v_codes = cache->v_codes;
  p.v_scales = cache->v_scales;
  p.status = status_dev;
  p.n_kv_heads = shape->n_kv_heads;
  p.t_cap = shape->t_cap;
  p.pm = page_map(cache, shape);
  p.scale_f16 = cache->scales_fp16 ? 1 : 0;
  const cudaError_t e = iq::launch_quantize_append(p, shape->head_dim, shape->batch, static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? IQ_OK : IQ_ERR_CUDA;
}

// Validation and kernel parameters shared by the decode entry points.
static int decode_params(const iq_shape* shape, const float* rot_dev, const iq_codebook* codebook, const void* q,
                         const iq_cache* cache, const int32_t* seq_lens_dev, int32_t num_splits, float* part_acc,
                         float* part_ml, int32_t* part_argmax, uint32_t* status_dev, iq::DecodeParams& p) {
  int rc = check_shape(shape);
  if (rc) return rc;
  if (!rot_dev || !q || !seq_lens_dev || !part_acc || !part_ml) return IQ_ERR_NULL;
  if ((rc = check_codebook(codebook, shape->bits, false))) return rc;
  int n8[16], n8v[16];
  float delta = 0.f, delta_v = 0.f;
  const bool grid8 = int8_grid(codebook, n8, delta, n8v, delta_v);  // integer tensor-core path; otherwise the levels must be exact fp16 values
  if (!grid8 && (rc = check_codebook(codebook, shape->bits, true))) return rc;
  if ((rc = check_cache(cache, shape))) return rc;
  if (num_splits < 1 || num_splits > 65535) return IQ_ERR_SHAPE;
  {  // the kernel counts (sequence, KV head group, slot) units and 128-row blocks in 31 bits
    const long long items = (long long)shape->batch * shape->n_kv_heads * ((shape->n_q_heads / shape->n_kv_heads + iq::DEC_HEADS - 1) / iq::DEC_HEADS);
    if (items * num_splits >= (1ll << 31) || items * (shape->t_cap / iq::DEC_BLOCK_TOKENS) >= (1ll << 31)) return IQ_ERR_LIMIT;
  }
  if (!aligned16(q) || !aligned16(part_acc) || !aligned16(rot_dev)) return IQ_ERR_ALIGN;

  p.k_codes = cache->k_codes;
  p.k_scales = cache->k_scales;
  p.v_codes = cache->v_codes;
  p.v_scales = cache->v_scales;
  p.q = static_cast<const __half*>(q);
  p.rot = rot_dev;
  p.seq_lens = seq_lens_dev;
  p.part_acc = part_acc;
  p.part_ml = part_ml;
  p.part_argmax = part_argmax;
  p.status = status_dev;
  p.batch = shape->batch;
  p.n_q_heads = shape->n_q_heads;
  p.n_kv_heads = shape->n_kv_heads;
  p.group = shape->n_q_heads / shape->n_kv_heads;
  p.head_groups = (p.group + iq::DEC_HEADS - 1) / iq::DEC_HEADS;
  p.t_cap = shape->t_cap;
  p.pm = page_map(cache, shape);
  p.scale_f16 = cache->scales_fp16 ? 1 : 0;
  p.splits = num_splits;
  p.sm_scale = shape->sm_scale > 0.f ? shape->sm_scale : 1.0f / std::sqrt((float)shape->head_dim);
  p.bits = shape->bits;
  const int n_levels = 1 << shape->bits;
  for (int i = 0; i < 4; i++) p.lut_lo[i] = p.lut_hi[i] = p.lut_v_lo[i] = p.lut_v_hi[i] = p.lut8[i] = p.lut8_v[i] = 0u;
  for (int v = 0; v < 2; v++) {
    const float* lv = side_levels(codebook, v);
    for (int i = 0; i < n_levels; i++) {
      const __half hv = __float2half_rn(lv[i]);
      uint16_t bits;
      std::memcpy(&bits, &hv, 2);
      (v ? p.lut_v_lo : p.lut_lo)[i >> 2] |= (uint32_t)(bits & 0xFFu) << (8 * (i & 3));
      (v ? p.lut_v_hi : p.lut_hi)[i >> 2] |= (uint32_t)(bits >> 8) << (8 * (i & 3));
      if (grid8) (v ? p.lut8_v : p.lut8)[i >> 2] |= (uint32_t)(uint8_t)(int8_t)(v ? n8v : n8)[i] << (8 * (i & 3));
    }
  }
  p.use_i8 = grid8 ? 1 : 0;
  p.delta = delta;
  p.delta_v = delta_v;
  p.k_new = p.v_new = nullptr;
  p.new_acc = p.new_ml = nullptr;
  p.aux_ctas = 0;
  p.len_bias = 0;
  std::memcpy(p.thresholds_k, side_thresholds(codebook, 0), sizeof(p.thresholds_k));
  std::memcpy(p.thresholds_v, side_thresholds(codebook, 1), sizeof(p.thresholds_v));
  std::memcpy(p.levels_k, side_levels(codebook, 0), sizeof(p.levels_k));
  std::memcpy(p.levels_v, side_levels(codebook, 1), sizeof(p.levels_v));
  return IQ_OK;
}

int iq_decode_attention(const iq_shape* shape, const float* rot_dev, const iq_codebook* codebook, const void* q,
                        const iq_cache* cache, const int32_t* seq_lens_dev, int32_t num_splits, float* part_acc,
                        float* part_ml, int32_t* part_argmax, uint32_t* status_dev, void* stream) {
  iq::DecodeParams p;
  const int rc = decode_params(shape, rot_dev, codebook, q, cache, seq_lens_dev, num_splits, part_acc, part_ml, part_argmax, status_dev, p);
  if (rc) return rc;
  if (shape->batch == 0) return IQ_OK;
  const cudaError_t e = iq::launch_decode_attention(p, shape->head_dim, static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? IQ_OK : IQ_ERR_CUDA;
}

// Sections of the decode step's workspace, in bytes from its start (each a multiple of 16).
namespace {
struct StepWorkspace {
  size_t part_acc, part_ml, new_acc, new_ml, part_argmax, total;
};
StepWorkspace step_workspace(const iq_shape* s, int32_t num_splits) {
  auto up = [](size_t x) { return (x + 15) & ~(size_t)15; };
  const size_t bh = (size_t)s->batch * s->n_q_heads, S = (size_t)num_splits, D = (size_t)s->head_dim;
  StepWorkspace w;
  size_t o = 0;
  w.part_acc = o; o += up(bh * S * D * 4);
  w.part_ml = o; o += up(bh * S * 8);
  w.new_acc = o; o += up(bh * D * 4);
  w.new_ml = o; o += up(bh * 8);
  w.part_argmax = o; o += up(bh * S * 4);
  w.total = o;
  return w;
}
}  // namespace

size_t iq_decode_step_workspace_bytes(const iq_shape* shape, int32_t num_splits) {
  if (check_shape(shape) || num_splits < 1 || num_splits > 65535) return 0;
  return step_workspace(shape, num_splits).total;
}

static int combine_with_new_row(const iq_shape* shape, const float* rot_dev, int32_t num_splits, int32_t n_shards, const float* part_acc,
                                const float* part_ml, const int32_t* part_argmax, const int32_t* row_offsets_dev, const float* new_acc,
                                const float* new_ml, const int32_t* new_rows, void* out, int32_t out_is_fp16, float* lse_out,
                                int32_t* argmax_out, void* stream);

int iq_decode_step_fused(const iq_shape* shape, const float* rot_dev, const iq_codebook* codebook, const void* q,
                         const void* k_new, const void* v_new, const iq_cache* cache, const int32_t* seq_lens_dev,
                         int32_t num_splits, void* workspace_dev, void* out, int32_t out_is_fp16, float* lse_out,
                         int32_t* argmax_out, uint32_t* status_dev, void* stream) {
  if (!workspace_dev || !out || !k_new || !v_new) return IQ_ERR_NULL;
  if (!aligned16(workspace_dev) || !aligned16(out) || !aligned16(k_new) || !aligned16(v_new)) return IQ_ERR_ALIGN;
  int rc = check_shape(shape);
  if (rc) return rc;
  if (num_splits < 1 || num_splits > 65535) return IQ_ERR_SHAPE;
  const StepWorkspace w = step_workspace(shape, num_splits);
  uint8_t* ws = static_cast<uint8_t*>(workspace_dev);
  float* part_acc = reinterpret_cast<float*>(ws + w.part_acc);
  float* part_ml = reinterpret_cast<float*>(ws + w.part_ml);
  int32_t* part_argmax = argmax_out ? reinterpret_cast<int32_t*>(ws + w.part_argmax) : nullptr;
  iq::DecodeParams p;
  rc = decode_params(shape, rot_dev, codebook, q, cache, seq_lens_dev, num_splits, part_acc, part_ml, part_argmax, status_dev, p);
  if (rc) return rc;
  if (shape->batch == 0) return IQ_OK;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // The append inside the decode launch pays while its tasks ((sequence, KV head) x (1 + heads per KV head), a warp
  // each) fit the few SMs set aside for them in one round; beyond that the three launches are faster, and the same
  // result is produced by them: append, decode over one more row per sequence, merge.
  const long long tasks = (long long)shape->batch * shape->n_kv_heads * (1 + shape->n_q_heads / shape->n_kv_heads);
  if (tasks > 180 || shape->bits != 3) {  // (the append inside the decode launch is built for the 3-bit layout)
    const int64_t sh = shape->head_dim, sb = (int64_t)shape->n_kv_heads * sh;  // k_new, v_new: [B][1][H_kv][d]
    rc = iq_quantize_append(shape, rot_dev, codebook, k_new, v_new, sb, sb, sh, seq_lens_dev, nullptr, 1, cache, status_dev, stream);
    if (rc) return rc;
    p.len_bias = 1;
    if (iq::launch_decode_attention(p, shape->head_dim, st) != cudaSuccess) return IQ_ERR_CUDA;
    return combine_with_new_row(shape, rot_dev, num_splits, 1, part_acc, part_ml, part_argmax, nullptr, nullptr, nullptr, nullptr, out,
                                out_is_fp16, lse_out, argmax_out, stream);
  }
  p.k_new = static_cast<const __half*>(k_new);
  p.v_new = static_cast<const __half*>(v_new);
  p.new_acc = reinterpret_cast<float*>(ws + w.new_acc);
  p.new_ml = reinterpret_cast<float*>(ws + w.new_ml);
  if (iq::launch_decode_attention(p, shape->head_dim, st) != cudaSuccess) return IQ_ERR_CUDA;
  return combine_with_new_row(shape, rot_dev, num_splits, 1, part_acc, part_ml, part_argmax, nullptr, p.new_acc, p.new_ml, seq_lens_dev,
                              out, out_is_fp16, lse_out, argmax_out, stream);
}

static int combine_with_new_row(const iq_shape* shape, const float* rot_dev, int32_t num_splits, int32_t n_shards, const float* part_acc,
                                const float* part_ml, const int32_t* part_argmax, const int32_t* row_offsets_dev, const float* new_acc,
                                const float* new_ml, const int32_t* new_rows, void* out, int32_t out_is_fp16, float* lse_out,
                                int32_t* argmax_out, void* stream) {
  int rc = check_shape(shape);
  if (rc) return rc;
  if (!rot_dev || !part_acc || !part_ml || !out) return IQ_ERR_NULL;
  if (argmax_out && !part_argmax) return IQ_ERR_NULL;
  if (num_splits < 1 || n_shards < 1) return IQ_ERR_SHAPE;
  if (!aligned16(part_acc) || !aligned16(out) || !aligned16(rot_dev)) return IQ_ERR_ALIGN;
  if (shape->batch == 0) return IQ_OK;

  iq::CombineParams p;
  p.part_acc = part_acc;
  p.part_ml = part_ml;
  p.part_argmax = part_argmax;
  p.rot = rot_dev;
  p.out = out;
  p.lse = lse_out;
  p.argmax = argmax_out;
  p.batch = shape->batch;
  p.n_q_heads = shape->n_q_heads;
  p.n_kv_heads = shape->n_kv_heads;
  p.splits = num_splits;
  p.shards = n_shards;
  p.row_offsets = row_offsets_dev;
  p.out_is_fp16 = out_is_fp16;
  p.new_acc = new_acc;
  p.new_ml = new_ml;
  p.new_rows = new_rows;
  const cudaError_t e = iq::launch_combine_splits(p, shape->head_dim, static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? IQ_OK : IQ_ERR_CUDA;
}

int iq_combine_splits_sharded(const iq_shape* shape, const float* rot_dev, int32_t num_splits, int32_t n_shards,
                              const float* part_acc, const float* part_ml, const int32_t* part_argmax,
                              const int32_t* row_offsets_dev, void* out, int32_t out_is_fp16, float* lse_out,
                              int32_t* argmax_out, void* stream) {
  return combine_with_new_row(shape, rot_dev, num_splits, n_shards, part_acc, part_ml, part_argmax, row_offsets_dev, nullptr, nullptr,
                              nullptr, out, out_is_fp16, lse_out, argmax_out, stream);
}

int iq_combine_splits(const iq_shape* shape, const float* rot_dev, int32_t num_splits, const float* part_acc,
                      const float* part_ml, const int32_t* part_argmax, void* out, int32_t out_is_fp16, float* lse_out,
                      int32_t* argmax_out, void* stream) {
  return iq_combine_splits_sharded(shape, rot_dev, num_splits, 1, part_acc, part_ml, part_argmax, nullptr, out, out_is_fp16,
                                   lse_out, argmax_out, stream);
}

int iq_reconstruct_rows(const iq_shape* shape, const float* rot_dev, const iq_codebook* codebook, const iq_cache* cache,
                        const int32_t* seq_lens_dev, void* k_out, void* v_out, int32_t out_rows, int64_t stride_b,
                        int64_t stride_t, int64_t stride_h, void* stream) {
  int rc = check_shape(shape);
  if (rc) return rc;
  if (!rot_dev || !seq_lens_dev || !k_out || !v_out) return IQ_ERR_NULL;
  if (out_rows < 0) return IQ_ERR_SHAPE;
  if ((rc = check_codebook(codebook, shape->bits, false))) return rc;
  if ((rc = check_cache(cache, shape))) return rc;
  if (!aligned16(k_out) || !aligned16(v_out) || !aligned16(rot_dev)) return IQ_ERR_ALIGN;
  if (stride_b < 0 || stride_t < 0 || stride_h < 0) return IQ_ERR_SHAPE;
  if ((stride_b & 7) || (stride_t & 7) || (stride_h & 7)) return IQ_ERR_ALIGN;
  if (shape->batch == 0 || out_rows == 0) return IQ_OK;

  iq::ReconstructParams p;
  p.k_codes = cache->k_codes;
  p.k_scales = cache->k_scales;
  p.v_codes = cache->v_codes;
  p.v_scales = cache->v_scales;
  p.rot = rot_dev;
  p.seq_lens = seq_lens_dev;
  p.k_out = static_cast<__half*>(k_out);
  p.v_out = static_cast<__half*>(v_out);
  p.stride_b = stride_b;
  p.stride_t = stride_t;
  p.stride_h = stride_h;
  p.n_kv_heads = shape->n_kv_heads;
  p.t_cap = shape->t_cap;
  p.pm = page_map(cache, shape);
  p.scale_f16 = cache->scales_fp16 ? 1 : 0;
  p.status = nullptr;
  p.out_rows = out_rows;
  p.bits = shape->bits;
  std::memcpy(p.levels_k, side_levels(codebook, 0), sizeof(p.levels_k));
  std::memcpy(p.levels_v, side_levels(codebook, 1), sizeof(p.levels_v));
  const cudaError_t e = iq::launch_reconstruct_rows(p, shape->head_dim, shape->batch, static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? IQ_OK : IQ_ERR_CUDA;
}

int iq_decode_step_host(const iq_shape* shape, const float* rot_dev, const iq_codebook* codebook, const void* inputs_host,
                        void* inputs_dev, const int32_t* append_pos_dev, const int32_t* seq_lens_dev, const iq_cache* cache,
                        int32_t num_splits, float* part_acc, float* part_ml, void* out_dev, void* out_host,
                        int32_t out_is_fp16, uint32_t* status_dev, void* stream) {
  int rc = check_shape(shape);
  if (rc) return rc;
  if (!inputs_host || !inputs_dev || !out_dev || !out_host) return IQ_ERR_NULL;
  if (!aligned16(inputs_dev)) return IQ_ERR_ALIGN;
  // everything the three calls below would refuse is refused here, before the copy and the append are enqueued
  if (!rot_dev || !append_pos_dev || !seq_lens_dev || !part_acc || !part_ml) return IQ_ERR_NULL;
  if ((rc = check_codebook(codebook, shape->bits, false))) return rc;
  {
    int n8[16], n8v[16];
    float delta = 0.f, delta_v = 0.f;
    if (!int8_grid(codebook, n8, delta, n8v, delta_v) && (rc = check_codebook(codebook, shape->bits, true))) return rc;
  }
  if ((rc = check_cache(cache, shape))) return rc;
  if (num_splits < 1 || num_splits > 65535) return IQ_ERR_SHAPE;
  if (!aligned16(part_acc) || !aligned16(rot_dev) || !aligned16(out_dev)) return IQ_ERR_ALIGN;
  if (shape->batch == 0) return IQ_OK;
  const size_t d = (size_t)shape->head_dim, B = (size_t)shape->batch;
  const size_t nq = B * (size_t)shape->n_q_heads * d, nk = B * (size_t)shape->n_kv_heads * d;  // elements of q, of k_new
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  __half* in = static_cast<__half*>(inputs_dev);
  if (cudaMemcpyAsync(in, inputs_host, (nq + 2 * nk) * sizeof(__half), cudaMemcpyHostToDevice, st) != cudaSuccess) return IQ_ERR_CUDA;
  const int64_t sh = (int64_t)d, sb = (int64_t)shape->n_kv_heads * sh;  // k_new, v_new: [B][1][H_kv][d]
  rc = iq_quantize_append(shape, rot_dev, codebook, in + nq, in + nq + nk, sb, sb, sh, append_pos_dev, nullptr, 1, cache,
                          status_dev, stream);
  if (rc) return rc;
  rc = iq_decode_attention(shape, rot_dev, codebook, in, cache, seq_lens_dev, num_splits, part_acc, part_ml, nullptr,
                           status_dev, stream);
  if (rc) return rc;
  rc = iq_combine_splits(shape, rot_dev, num_splits, part_acc, part_ml, nullptr, out_dev, out_is_fp16, nullptr, nullptr, stream);
  if (rc) return rc;
  const size_t out_bytes = B * (size_t)shape->n_q_heads * d * (out_is_fp16 ? 2 : 4);
  if (cudaMemcpyAsync(out_host, out_dev, out_bytes, cudaMemcpyDeviceToHost, st) != cudaSuccess) return IQ_ERR_CUDA;
  return cudaStreamSynchronize(st) == cudaSuccess ? IQ_OK : IQ_ERR_CUDA;
}

int iq_rotated_histogram(const iq_shape* shape, const float* rot_dev, const void* x, int64_t stride_b, int64_t stride_t,
                         int64_t stride_h, const int32_t* n_rows_dev, int32_t n_rows_max, uint32_t* hist_dev, int32_t bins,
                         float range, void* stream) {
  int rc = check_shape(shape);
  if (rc) return rc;
  if (!rot_dev || !hist_dev) return IQ_ERR_NULL;
  if (bins < 16 || bins > iq::HIST_MAX_BINS || !(range > 0.f) || n_rows_max < 0) return IQ_ERR_SHAPE;
  if (n_rows_max == 0 || shape->batch == 0) return IQ_OK;
  if (!x) return IQ_ERR_NULL;
  if (!aligned16(x) || !aligned16(rot_dev)) return IQ_ERR_ALIGN;
  if (stride_b < 0 || stride_t < 0 || stride_h < 0) return IQ_ERR_SHAPE;
  if ((stride_b & 7) || (stride_t & 7) || (stride_h & 7)) return IQ_ERR_ALIGN;
  iq::HistogramParams p = {};
  p.x = static_cast<const __half*>(x);
  p.stride_b = stride_b;
  p.stride_t = stride_t;
  p.stride_h = stride_h;
  p.n_rows = n_rows_dev;
  p.n_rows_max = n_rows_max;
  p.rot = rot_dev;
  p.hist = hist_dev;
  p.bins = bins;
  p.range = range;
  p.n_kv_heads = shape->n_kv_heads;
  const cudaError_t e = iq::launch_rotated_histogram(p, shape->head_dim, shape->batch, static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? IQ_OK : IQ_ERR_CUDA;
}

int iq_fit_codebook(const uint32_t* hist_host, int32_t bins, float range, int32_t bits, int32_t symmetric, int32_t grid,
                    iq_codebook* out_host) {
  if (!hist_host || !out_host) return IQ_ERR_NULL;
  if (bins < 16 || bins > iq::HIST_MAX_BINS || !(range > 0.f) || (grid != 0 && grid != 1) || bits < 2 || bits > 4) return IQ_ERR_SHAPE;
  std::vector<double> c((size_t)bins);
  double total = 0.0;
  for (int i = 0; i < bins; i++) total += (double)hist_host[i];
  if (!(total > 0.0)) return IQ_ERR_SHAPE;
  for (int i = 0; i < bins; i++) c[i] = symmetric ? 0.5 * ((double)hist_host[i] + (double)hist_host[bins - 1 - i]) : (double)hist_host[i];
  double lv[16];
  lloyd_max_histogram(c, (double)range, symmetric != 0, 1 << bits, lv);
  finish_codebook(lv, bits, grid, out_host);
  for (int i = 0; i < (1 << bits) - 1; i++)
    if (!(out_host->levels[i] < out_host->levels[i + 1])) return IQ_ERR_CODEBOOK;  // too few distinct values in the data
  return IQ_OK;
}

int iq_wht_coordinates(const iq_shape* shape, const void* x, int64_t stride_b, int64_t stride_t, int64_t stride_h,
                       const int32_t* n_rows_dev, int32_t n_rows_max, float* z_dev, void* stream) {
  int rc = check_shape(shape);
  if (rc) return rc;
  if (n_rows_max < 0) return IQ_ERR_SHAPE;
  if (n_rows_max == 0 || shape->batch == 0) return IQ_OK;
  if (!x || !z_dev) return IQ_ERR_NULL;
  if (!aligned16(x) || !aligned16(z_dev)) return IQ_ERR_ALIGN;
  if (stride_b < 0 || stride_t < 0 || stride_h < 0) return IQ_ERR_SHAPE;
  if ((stride_b & 7) || (stride_t & 7) || (stride_h & 7)) return IQ_ERR_ALIGN;
  iq::WhtParams p = {};
  p.x = static_cast<const __half*>(x);
  p.stride_b = stride_b;
  p.stride_t = stride_t;
  p.stride_h = stride_h;
  p.n_rows = n_rows_dev;
  p.n_rows_max = n_rows_max;
  p.z = z_dev;
  p.n_kv_heads = shape->n_kv_heads;
  const cudaError_t e = iq::launch_wht_coordinates(p, shape->head_dim, shape->batch, static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? IQ_OK : IQ_ERR_CUDA;
}

int iq_fit_rotation(const float* z_host, int32_t n_rows, int64_t row_stride, int32_t head_dim, const iq_codebook* codebook,
                    float* quats_host, double* distortion_host) {
  if (!z_host || !codebook || !quats_host) return IQ_ERR_NULL;
  if ((head_dim != 128 && head_dim != 256) || n_rows < 1 || row_stride < head_dim) return IQ_ERR_SHAPE;
  const int rc = codebook ? check_codebook(codebook, codebook->bits, false) : IQ_ERR_NULL;  // (the K side of the codebook is fitted to)
  if (rc) return rc;
  double before = 0.0, after = 0.0;
  for (int b = 0; b < head_dim / 4; b++) {
    double q8[8], M[4][4], start;
    for (int i = 0; i < 8; i++) q8[i] = (double)quats_host[8 * b + i];
    so4_from_pair(q8, M);
    after += fit_block(z_host + 4 * b, (size_t)row_stride, n_rows, M, *codebook, start);
    before += start;
    pair_from_so4(M, q8);
    for (int i = 0; i < 8; i++) quats_host[8 * b + i] = (float)q8[i];
  }
  if (distortion_host) {
    distortion_host[0] = before / head_dim;
    distortion_host[1] = after / head_dim;
  }
  return IQ_OK;
}

int iq_selftest_bounded_wait(uint32_t* status_dev, uint32_t polls, void* stream) {
  if (!status_dev) return IQ_ERR_NULL;
  if (polls > 65536u) return IQ_ERR_LIMIT;
  return iq::launch_bounded_wait_selftest(status_dev, polls, static_cast<cudaStream_t>(stream)) == cudaSuccess ? IQ_OK : IQ_ERR_CUDA;
}

int32_t iq_suggest_splits(const iq_shape* shape, int32_t max_seq_len) {
  if (check_shape(shape) != IQ_OK || max_seq_len <= 0) return 1;
  static int n_sm_cached[64] = {};
  int dev = 0, n_sm = 148;
  if (cudaGetDevice(&dev) == cudaSuccess && dev >= 0 && dev < 64) {
    if (n_sm_cached[dev] == 0) {
      int v = 0;
      if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && v > 0) n_sm_cached[dev] = v;
    }
    if (n_sm_cached[dev] > 0) n_sm = n_sm_cached[dev];
  }
  const int group = shape->n_q_heads / shape->n_kv_heads;
  const long long items = (long long)(shape->batch > 0 ? shape->batch : 1) * shape->n_kv_heads * ((group + iq::DEC_HEADS - 1) / iq::DEC_HEADS);
  const long long ctas = (long long)n_sm * iq::decode_ctas_per_sm(shape->head_dim);
  const int ng = iq::decode_groups_per_cta(shape->head_dim);
  // The decode kernel gives every CTA an equal, contiguous share of the launch's 128-row blocks; an item of nb blocks
  // then has about nb / share + 1 pieces, and every piece reports to one slot per group of its CTA. With all sequences
  // at full length share = items * nb / ctas; the factor 1.5 leaves room for batches whose mean length is two thirds
  // of the longest. A piece is not worth less than one block per group.
  const long long nb = (max_seq_len + iq::DEC_BLOCK_TOKENS - 1) / iq::DEC_BLOCK_TOKENS;
  long long pieces = (15 * ctas + 10 * items - 1) / (10 * items) + 1;
  const long long cap = (nb + ng - 1) / ng;
  if (pieces > cap) pieces = cap;
  if (pieces < 2) pieces = 2;
  long long s = pieces * ng;
  if (s > 1024) s = 1024;
  return (int32_t)s;
}

}  // extern "C"
