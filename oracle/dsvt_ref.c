/*
 * dsvt_ref.c -- CPU oracle for the DSVT dynamic sparse window attention path.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is a plain, slow, scalar, double-precision
 * restatement of the paper's definitions (arXiv 2301.06051).  It exists so that
 * the CUDA library can be checked against it.  It shares no code, headers,
 * tables or helpers with the CUDA path, and nothing in the product imports it.
 *
 * What is restated, and from where:
 *   - window partition of voxels                         Sec. 3.2 ("Dynamic set partition")
 *   - inner-window voxel id d_i from a sorting strategy  Eq. 1 and the X-/Y-axis main order of Sec. 3.2
 *   - number of sets per window S                        Eq. 2 (also Definition A.1)
 *   - set index rule q^j_k                               Eq. 3 (also Definition A.1)
 *   - INDEX gather of set members                        Eq. 4
 *   - masked-duplicate multi-head self attention         Sec. 3.2 (text after Eq. 3), Eq. 5
 *   - layer = MHSA, residual, LN, 2-layer MLP with GELU,
 *     residual, LN; block = X layer then Y layer         Eq. 5, Appendix B.1.1
 *   - attention-style 3D pooling                         Eq. 6, Eq. 7
 *
 * Pinned by tests (tests/test_oracle_*.py) against: hand-worked Eq. 3 rows and a
 * hand-worked grid, Theorems A.2-A.4, brute-force dense attention written
 * independently in numpy, torch float64 library routines on special cases, and
 * closed forms.  Two conventions have no counterpart the paper fixes and are
 * "parity unpinned" by the paper (pinned only by closed forms): the optional
 * additive positional term `pe`, and the internals of the pooling attention
 * (separate q/k/v/o projections, slot ordering).
 *
 * All pointers are host pointers.  Features and weights are double.
 * Return value: 0 ok, -1 invalid argument, -2 capacity too small, -3 bad input
 * (coordinate outside the grid, or two voxels in the same cell for pooling).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define REF_OK 0
#define REF_ERR_ARG (-1)
#define REF_ERR_CAPACITY (-2)
#define REF_ERR_BAD_INPUT (-3)

static int g_threads = 1;

/* Number of host threads the set / region loops may use (sets and regions are
 * independent of one another, so this changes no arithmetic). */
void dsvt_ref_set_threads(int t) { g_threads = t > 0 ? t : 1; }
int dsvt_ref_get_threads(void) { return g_threads; }
int dsvt_ref_max_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

/* ------------------------------------------------------------------ */
/* Eq. 2: S = floor(N / tau) + [N % tau > 0]                           */
/* ------------------------------------------------------------------ */
int64_t dsvt_ref_num_sets(int64_t N, int64_t tau) { return N / tau + ((N % tau) > 0 ? 1 : 0); }

/* ------------------------------------------------------------------ */
/* Eq. 3: q^j_k = floor( (j*tau + k) / (S*tau) * N ), evaluated as an  */
/* exact integer floor (the theorems of Appendix A assume exact        */
/* arithmetic).  Writes S*tau entries, row j holds q^j_0..q^j_{tau-1}. */
/* ------------------------------------------------------------------ */
int dsvt_ref_set_indices(int64_t N, int64_t tau, int64_t* q_out) {
  if (N < 1 || tau < 1) return REF_ERR_ARG;
  int64_t S = dsvt_ref_num_sets(N, tau);
  for (int64_t j = 0; j < S; ++j)
    for (int64_t k = 0; k < tau; ++k) q_out[j * tau + k] = ((j * tau + k) * N) / (S * tau);
  return REF_OK;
}

/* ------------------------------------------------------------------ */
/* Partition (Sec. 3.2; Eq. 1-3)                                       */
/* ------------------------------------------------------------------ */
typedef struct {
  int64_t win;   /* window id, batch most significant */
  int64_t inner; /* position inside the window under the chosen main order */
  int32_t idx;   /* original voxel index (ties cannot arise for unique cells) */
} ref_key;

static int ref_key_cmp(const void* a, const void* b) {
  const ref_key* p = (const ref_key*)a;
  const ref_key* q = (const ref_key*)b;
  if (p->win != q->win) return p->win < q->win ? -1 : 1;
  if (p->inner != q->inner) return p->inner < q->inner ? -1 : 1;
  if (p->idx != q->idx) return p->idx < q->idx ? -1 : 1;
  return 0;
}

static int64_t ceil_div64(int64_t a, int64_t b) { return (a + b - 1) / b; }

/*
 * coords: [n][4] = (b, x, y, z).  grid = cells per axis (x, y, z).
 * window = (L, W, H).  axis 0: X main order, key (x_in, y_in, z_in);
 * axis 1: Y main order, key (y_in, x_in, z_in).  Windows start at cell 0.
 * Window id = ((b*nWx + wx)*nWy + wy)*nWz + wz.
 * Outputs: set_table [cap_sets][set_size] rows in ascending (window, j);
 * *num_sets; optional perm[n] (voxel indices in sorted order),
 * win_count[num_windows], win_start[num_windows+1], win_setoff[num_windows+1]
 * over ALL windows (empty ones have count 0), num_windows = batch*nWx*nWy*nWz.
 */
/* Window partition displaced by `shift` cells (Sec. 3.2, "Hybrid window partition": the windows are re-cut
 * between consecutive blocks with the window shifting of Swin, and with another window size).  A voxel at
 * cell (x, y, z) lies in the window that holds cell (x + shift_x, y + shift_y, z + shift_z) of the unshifted
 * cut; 0 <= shift < window per axis, so the first window of every axis is the partial one and there are
 * ceil((grid + shift) / window) windows per axis.  Everything else is dsvt_ref_partition. */
int dsvt_ref_partition_shifted(const int32_t* coords, int32_t n, int32_t batch, const int32_t* grid,
                               const int32_t* window, const int32_t* shift, int32_t set_size, int32_t axis,
                               int32_t* set_table, int32_t cap_sets, int32_t* num_sets, int32_t* perm,
                               int32_t* win_start, int32_t* win_count, int32_t* win_setoff) {
  if (n < 0 || batch < 1 || set_size < 1 || (axis != 0 && axis != 1)) return REF_ERR_ARG;
  for (int a = 0; a < 3; ++a)
    if (grid[a] < 1 || window[a] < 1 || shift[a] < 0 || shift[a] >= window[a]) return REF_ERR_ARG;
  const int64_t L = window[0], W = window[1], H = window[2];
  const int64_t nWx = ceil_div64((int64_t)grid[0] + shift[0], L), nWy = ceil_div64((int64_t)grid[1] + shift[1], W),
                nWz = ceil_div64((int64_t)grid[2] + shift[2], H);
  const int64_t num_windows = (int64_t)batch * nWx * nWy * nWz;

  ref_key* keys = (ref_key*)malloc(sizeof(ref_key) * (size_t)(n > 0 ? n : 1));
  int64_t* cnt = (int64_t*)calloc((size_t)num_windows, sizeof(int64_t));
  if (!keys || !cnt) { free(keys); free(cnt); return REF_ERR_ARG; }

  for (int32_t i = 0; i < n; ++i) {
    const int64_t b = coords[4 * i + 0], x = coords[4 * i + 1], y = coords[4 * i + 2], z = coords[4 * i + 3];
    if (b < 0 || b >= batch || x < 0 || x >= grid[0] || y < 0 || y >= grid[1] || z < 0 || z >= grid[2]) {
      free(keys); free(cnt);
      return REF_ERR_BAD_INPUT;
    }
    const int64_t xs = x + shift[0], ys = y + shift[1], zs = z + shift[2];
    const int64_t wx = xs / L, wy = ys / W, wz = zs / H;
    const int64_t xi = xs - wx * L, yi = ys - wy * W, zi = zs - wz * H;
    keys[i].win = ((b * nWx + wx) * nWy + wy) * nWz + wz;
    keys[i].inner = axis == 0 ? (xi * W + yi) * H + zi : (yi * L + xi) * H + zi;
    keys[i].idx = i;
    cnt[keys[i].win] += 1;
  }
  qsort(keys, (size_t)n, sizeof(ref_key), ref_key_cmp);
  if (perm)
    for (int32_t i = 0; i < n; ++i) perm[i] = keys[i].idx;

  int64_t start = 0, setoff = 0;
  int rc = REF_OK;
  for (int64_t w = 0; w < num_windows; ++w) {
    const int64_t N = cnt[w];
    const int64_t S = N > 0 ? dsvt_ref_num_sets(N, set_size) : 0; /* Eq. 2 */
    if (win_count) win_count[w] = (int32_t)N;
    if (win_start) win_start[w] = (int32_t)start;
    if (win_setoff) win_setoff[w] = (int32_t)setoff;
    if (N > 0) {
      if (setoff + S > cap_sets) {
        rc = REF_ERR_CAPACITY;
      } else {
        for (int64_t j = 0; j < S; ++j)
          for (int64_t k = 0; k < set_size; ++k) {
            const int64_t q = ((j * set_size + k) * N) / (S * set_size); /* Eq. 3 */
            set_table[(setoff + j) * set_size + k] = keys[start + q].idx; /* Eq. 4: rank -> voxel */
          }
      }
    }
    start += N;
    setoff += S;
  }
  if (win_start) win_start[num_windows] = (int32_t)start;
  if (win_setoff) win_setoff[num_windows] = (int32_t)setoff;
  *num_sets = (int32_t)setoff;
  free(keys);
  free(cnt);
  return rc;
}

int dsvt_ref_partition(const int32_t* coords, int32_t n, int32_t batch, const int32_t* grid, const int32_t* window,
                       int32_t set_size, int32_t axis, int32_t* set_table, int32_t cap_sets, int32_t* num_sets,
                       int32_t* perm, int32_t* win_start, int32_t* win_count, int32_t* win_setoff) {
  const int32_t no_shift[3] = {0, 0, 0};
  return dsvt_ref_partition_shifted(coords, n, batch, grid, window, no_shift, set_size, axis, set_table, cap_sets,
                                    num_sets, perm, win_start, win_count, win_setoff);
}

/* ------------------------------------------------------------------ */
/* Masked-duplicate multi-head self attention over the sets           */
/* (Eq. 4 gather; text after Eq. 3: duplicated voxels are masked;     */
/*  Eq. 5 MHSA).                                                       */
/* ------------------------------------------------------------------ */

/* y[o] = sum_c W[o][c] * x[c] + b[o];  W is [out][in] row-major. */
static void ref_linear(const double* W, const double* b, const double* x, int out, int in, double* y) {
  for (int o = 0; o < out; ++o) {
    double acc = b ? b[o] : 0.0;
    for (int c = 0; c < in; ++c) acc += W[(size_t)o * in + c] * x[c];
    y[o] = acc;
  }
}

/*
 * Relative position bias, the mechanism of the Swin transformer that the text after Eq. 5 points to
 * for PE(.): a learned scalar per head and per coordinate offset between query and key, added to
 * the scaled logit.  Voxels of one set lie in one window of extent (L, W, H), so an offset component
 * lies in [-(L-1), L-1] etc.; the table holds (2L-1)(2W-1)(2H-1) entries per head and the entry for
 * offset (dx, dy, dz) = coords[query] - coords[key] sits at
 *   ((dx + L-1) * (2W-1) + (dy + W-1)) * (2H-1) + (dz + H-1).
 */
typedef struct {
  const double* table;   /* [heads][(2L-1)(2W-1)(2H-1)] */
  const int32_t* coords; /* [n][4] = (b, x, y, z) */
  int32_t ext[3];        /* L, W, H */
} ref_rel_bias;

static size_t ref_rel_bias_len(const ref_rel_bias* rb) {
  return (size_t)(2 * rb->ext[0] - 1) * (size_t)(2 * rb->ext[1] - 1) * (size_t)(2 * rb->ext[2] - 1);
}

static size_t ref_rel_bias_index(const ref_rel_bias* rb, int32_t query, int32_t key) {
  const int32_t* cq = rb->coords + (size_t)query * 4;
  const int32_t* ck = rb->coords + (size_t)key * 4;
  const int dx = cq[1] - ck[1], dy = cq[2] - ck[2], dz = cq[3] - ck[3];
  const int L = rb->ext[0], W = rb->ext[1], H = rb->ext[2];
  return ((size_t)(dx + L - 1) * (size_t)(2 * W - 1) + (size_t)(dy + W - 1)) * (size_t)(2 * H - 1) + (size_t)(dz + H - 1);
}

/* 1 iff every pair of members of every table row has an offset the table covers */
static int ref_rel_bias_covers(const ref_rel_bias* rb, const int32_t* set_table, int32_t num_sets, int32_t tau) {
  for (int32_t s = 0; s < num_sets; ++s) {
    const int32_t* rows = set_table + (size_t)s * tau;
    int32_t lo[3], hi[3];
    for (int a = 0; a < 3; ++a) lo[a] = hi[a] = rb->coords[(size_t)rows[0] * 4 + 1 + a];
    for (int k = 1; k < tau; ++k)
      for (int a = 0; a < 3; ++a) {
        const int32_t v = rb->coords[(size_t)rows[k] * 4 + 1 + a];
        if (v < lo[a]) lo[a] = v;
        if (v > hi[a]) hi[a] = v;
      }
    for (int a = 0; a < 3; ++a)
      if (hi[a] - lo[a] > rb->ext[a] - 1) return 0;
  }
  return 1;
}

/*
 * One set: rows[tau] voxel indices.  Slot k is a masked key iff k > 0 and
 * rows[k] == rows[k-1].  Z[tau][C] receives the projected attention output of
 * every slot; keep[k] says whether slot k is a non-duplicate.
 */
static void ref_attend_one_set(const double* feats, const double* pe, int C, const int32_t* rows, int tau,
                               const double* W_qkv, const double* b_qkv, const double* W_o, const double* b_o,
                               int heads, const ref_rel_bias* rb, double* Z, int* keep, double* work) {
  const int d = C / heads;
  double* Q = work;                       /* [tau][C] */
  double* K = Q + (size_t)tau * C;        /* [tau][C] */
  double* V = K + (size_t)tau * C;        /* [tau][C] */
  double* Y = V + (size_t)tau * C;        /* [tau][C] */
  double* xin = Y + (size_t)tau * C;      /* [C] */
  double* logit = xin + C;                /* [tau] */
  for (int k = 0; k < tau; ++k) {
    keep[k] = !(k > 0 && rows[k] == rows[k - 1]);
    const double* f = feats + (size_t)rows[k] * C; /* Eq. 4: INDEX */
    /* optional positional term: added to the input of the Q and K projections only */
    for (int c = 0; c < C; ++c) xin[c] = f[c] + (pe ? pe[(size_t)rows[k] * C + c] : 0.0);
    ref_linear(W_qkv, b_qkv, xin, C, C, Q + (size_t)k * C);
    ref_linear(W_qkv + (size_t)C * C, b_qkv ? b_qkv + C : NULL, xin, C, C, K + (size_t)k * C);
    ref_linear(W_qkv + (size_t)2 * C * C, b_qkv ? b_qkv + 2 * C : NULL, f, C, C, V + (size_t)k * C);
  }
  const double scale = 1.0 / sqrt((double)d);
  for (int h = 0; h < heads; ++h) {
    for (int a = 0; a < tau; ++a) {
      double mx = -INFINITY;
      for (int b = 0; b < tau; ++b) {
        if (!keep[b]) continue;
        double s = 0.0;
        for (int c = 0; c < d; ++c) s += Q[(size_t)a * C + h * d + c] * K[(size_t)b * C + h * d + c];
        logit[b] = s * scale;
        if (rb) logit[b] += rb->table[(size_t)h * ref_rel_bias_len(rb) + ref_rel_bias_index(rb, rows[a], rows[b])];
        if (logit[b] > mx) mx = logit[b];
      }
      double den = 0.0;
      for (int b = 0; b < tau; ++b)
        if (keep[b]) { logit[b] = exp(logit[b] - mx); den += logit[b]; }
      for (int c = 0; c < d; ++c) {
        double acc = 0.0;
        for (int b = 0; b < tau; ++b)
          if (keep[b]) acc += logit[b] * V[(size_t)b * C + h * d + c];
        Y[(size_t)a * C + h * d + c] = acc / den;
      }
    }
  }
  for (int k = 0; k < tau; ++k) ref_linear(W_o, b_o, Y + (size_t)k * C, C, C, Z + (size_t)k * C);
}

static size_t ref_attend_work_doubles(int tau, int C) { return (size_t)4 * tau * C + C + tau; }

/*
 * out[v] = Z of the set slot holding v, for every non-duplicate slot of every
 * table row.  Rows of `out` for voxels in no table row are left untouched.
 * `covered` (optional, int32[n]) is set to 1 for written voxels.
 */
int dsvt_ref_set_attention_rpb(const double* feats, int32_t n, int32_t C, const int32_t* set_table,
                               int32_t num_sets, int32_t set_size, const double* W_qkv, const double* b_qkv,
                               const double* W_o, const double* b_o, int32_t heads, const double* pe,
                               const double* rpb, const int32_t* coords, const int32_t* rpb_extent, double* out,
                               int32_t* covered) {
  if (n < 0 || C < 1 || heads < 1 || C % heads != 0 || set_size < 1 || num_sets < 0) return REF_ERR_ARG;
  for (int64_t i = 0; i < (int64_t)num_sets * set_size; ++i)
    if (set_table[i] < 0 || set_table[i] >= n) return REF_ERR_BAD_INPUT;
  ref_rel_bias rbv, *rb = NULL;
  if (rpb) {
    if (!coords || !rpb_extent || rpb_extent[0] < 1 || rpb_extent[1] < 1 || rpb_extent[2] < 1) return REF_ERR_ARG;
    rbv.table = rpb; rbv.coords = coords;
    rbv.ext[0] = rpb_extent[0]; rbv.ext[1] = rpb_extent[1]; rbv.ext[2] = rpb_extent[2];
    if (!ref_rel_bias_covers(&rbv, set_table, num_sets, set_size)) return REF_ERR_BAD_INPUT;
    rb = &rbv;
  }
  int s;
#pragma omp parallel for schedule(dynamic, 4) num_threads(g_threads)
  for (s = 0; s < num_sets; ++s) {
    const int tau = set_size;
    double* work = (double*)malloc(sizeof(double) * (ref_attend_work_doubles(tau, C) + (size_t)tau * C));
    int* keep = (int*)malloc(sizeof(int) * (size_t)tau);
    double* Z = work + ref_attend_work_doubles(tau, C);
    const int32_t* rows = set_table + (size_t)s * tau;
    ref_attend_one_set(feats, pe, C, rows, tau, W_qkv, b_qkv, W_o, b_o, heads, rb, Z, keep, work);
    for (int k = 0; k < tau; ++k)
      if (keep[k]) {
        memcpy(out + (size_t)rows[k] * C, Z + (size_t)k * C, sizeof(double) * (size_t)C);
        if (covered) covered[rows[k]] = 1;
      }
    free(work);
    free(keep);
  }
  return REF_OK;
}

int dsvt_ref_set_attention(const double* feats, int32_t n, int32_t C, const int32_t* set_table, int32_t num_sets,
                           int32_t set_size, const double* W_qkv, const double* b_qkv, const double* W_o,
                           const double* b_o, int32_t heads, const double* pe, double* out, int32_t* covered) {
  return dsvt_ref_set_attention_rpb(feats, n, C, set_table, num_sets, set_size, W_qkv, b_qkv, W_o, b_o, heads, pe,
                                    NULL, NULL, NULL, out, covered);
}

/* ------------------------------------------------------------------ */
/* Layer and block (Eq. 5; Appendix B.1.1)                             */
/* ------------------------------------------------------------------ */
typedef struct {
  int32_t C, heads, hidden, set_size;
  double ln_eps;
  const double *W_qkv, *b_qkv; /* [3C][C], [3C] */
  const double *W_o, *b_o;     /* [C][C], [C] */
  const double *W_1, *b_1;     /* [hidden][C], [hidden]; hidden == 0: no MLP */
  const double *W_2, *b_2;     /* [C][hidden], [C] */
  const double *ln1_g, *ln1_b; /* NULL gain: no LayerNorm after the attention */
  const double *ln2_g, *ln2_b; /* NULL gain: no LayerNorm after the MLP */
  const double* pe;            /* [n][C] or NULL */
  const double* rpb;           /* relative position bias [heads][(2L-1)(2W-1)(2H-1)] or NULL */
  const int32_t* coords;       /* [n][4], read when rpb is given */
  int32_t rpb_extent[3];       /* L, W, H */
} dsvt_ref_layer_params;

/* LayerNorm over C channels, biased variance. */
static void ref_layernorm(double* v, int C, const double* g, const double* b, double eps) {
  double mean = 0.0;
  for (int c = 0; c < C; ++c) mean += v[c];
  mean /= C;
  double var = 0.0;
  for (int c = 0; c < C; ++c) var += (v[c] - mean) * (v[c] - mean);
  var /= C;
  const double inv = 1.0 / sqrt(var + eps);
  for (int c = 0; c < C; ++c) v[c] = (v[c] - mean) * inv * g[c] + (b ? b[c] : 0.0);
}

static double ref_gelu(double x) { return 0.5 * x * (1.0 + erf(x / sqrt(2.0))); }

/*
 * x1 = LN1(x + MHSA(x));  x2 = LN2(x1 + W_2 gelu(W_1 x1 + b_1) + b_2).
 * Rows of voxels that appear in no table row are copied from x unchanged.
 */
int dsvt_ref_layer(const double* x, int32_t n, const int32_t* set_table, int32_t num_sets,
                   const dsvt_ref_layer_params* p, double* y) {
  if (!p || p->C < 1) return REF_ERR_ARG;
  const int C = p->C, Hd = p->hidden;
  double* Z = (double*)calloc((size_t)(n > 0 ? n : 1) * C, sizeof(double));
  int32_t* covered = (int32_t*)calloc((size_t)(n > 0 ? n : 1), sizeof(int32_t));
  int rc = dsvt_ref_set_attention_rpb(x, n, C, set_table, num_sets, p->set_size, p->W_qkv, p->b_qkv, p->W_o, p->b_o,
                                      p->heads, p->pe, p->rpb, p->coords, p->rpb_extent, Z, covered);
  if (rc != REF_OK) { free(Z); free(covered); return rc; }
  int i;
#pragma omp parallel for schedule(static) num_threads(g_threads)
  for (i = 0; i < n; ++i) {
    double* yi = y + (size_t)i * C;
    const double* xi = x + (size_t)i * C;
    if (!covered[i]) { memmove(yi, xi, sizeof(double) * (size_t)C); continue; }
    double* t = (double*)malloc(sizeof(double) * (size_t)(C + Hd + C));
    double* hbuf = t + C;
    double* m = hbuf + Hd;
    for (int c = 0; c < C; ++c) t[c] = xi[c] + Z[(size_t)i * C + c]; /* residual after the attention module */
    if (p->ln1_g) ref_layernorm(t, C, p->ln1_g, p->ln1_b, p->ln_eps);
    if (Hd > 0) {
      ref_linear(p->W_1, p->b_1, t, Hd, C, hbuf);
      for (int o = 0; o < Hd; ++o) hbuf[o] = ref_gelu(hbuf[o]);
      ref_linear(p->W_2, p->b_2, hbuf, C, Hd, m);
      for (int c = 0; c < C; ++c) t[c] += m[c]; /* residual after the MLP */
      if (p->ln2_g) ref_layernorm(t, C, p->ln2_g, p->ln2_b, p->ln_eps);
    }
    memcpy(yi, t, sizeof(double) * (size_t)C);
    free(t);
  }
  free(Z);
  free(covered);
  return REF_OK;
}

/* Block = layer with the X-axis table, then layer with the Y-axis table (Eq. 5). */
int dsvt_ref_block(const double* x, int32_t n, const int32_t* table_axis0, int32_t num_sets0,
                   const int32_t* table_axis1, int32_t num_sets1, const dsvt_ref_layer_params* layers, double* y) {
  double* mid = (double*)malloc(sizeof(double) * (size_t)(n > 0 ? n : 1) * layers[0].C);
  int rc = dsvt_ref_layer(x, n, table_axis0, num_sets0, &layers[0], mid);
  if (rc == REF_OK) rc = dsvt_ref_layer(mid, n, table_axis1, num_sets1, &layers[1], y);
  free(mid);
  return rc;
}

/* ------------------------------------------------------------------ */
/* Attention-style 3D pooling (Eq. 6, Eq. 7)                           */
/* ------------------------------------------------------------------ */
typedef struct {
  int64_t key;
  int32_t idx;
} ref_rkey;

static int ref_rkey_cmp(const void* a, const void* b) {
  const ref_rkey* p = (const ref_rkey*)a;
  const ref_rkey* q = (const ref_rkey*)b;
  if (p->key != q->key) return p->key < q->key ? -1 : 1;
  if (p->idx != q->idx) return p->idx < q->idx ? -1 : 1;
  return 0;
}

/*
 * Region of voxel (b,x,y,z): (b, x/l, y/w, z/h); slot inside the region:
 * ((x%l)*w + y%w)*h + z%h.  Each non-empty region becomes one output voxel,
 * in ascending order of ((b*GX + X)*GY + Y)*GZ + Z.
 * The region is padded to l*w*h dense slots with zero rows (Eq. 6 text).
 * mask_empty == 0: max-pool and keys/values run over all dense slots;
 * mask_empty == 1: over the non-empty slots only.
 * P~ = W_o * MHA(q = W_q P + b_q; k_s = W_k (p~_s + e_s) + b_k; v_s likewise) + b_o,
 * e_s = slot_pe[s] or 0.
 */
int dsvt_ref_pool(const int32_t* coords, const double* feats, int32_t n, int32_t C, int32_t batch, const int32_t* grid,
                  const int32_t* pool, const double* W_q, const double* W_k, const double* W_v, const double* W_o,
                  const double* b_q, const double* b_k, const double* b_v, const double* b_o, const double* slot_pe,
                  int32_t heads, int32_t mask_empty, int32_t* out_coords, double* out_feats, int32_t cap_m,
                  int32_t* num_out, int32_t* region_of, int32_t* slot_of) {
  if (n < 0 || C < 1 || heads < 1 || C % heads != 0 || batch < 1) return REF_ERR_ARG;
  for (int a = 0; a < 3; ++a)
    if (grid[a] < 1 || pool[a] < 1) return REF_ERR_ARG;
  const int64_t l = pool[0], w = pool[1], h = pool[2];
  const int64_t GX = ceil_div64(grid[0], l), GY = ceil_div64(grid[1], w), GZ = ceil_div64(grid[2], h);
  const int nslots = (int)(l * w * h);
  ref_rkey* rk = (ref_rkey*)malloc(sizeof(ref_rkey) * (size_t)(n > 0 ? n : 1));
  int32_t* slot = (int32_t*)malloc(sizeof(int32_t) * (size_t)(n > 0 ? n : 1));
  for (int32_t i = 0; i < n; ++i) {
    const int64_t b = coords[4 * i], x = coords[4 * i + 1], y = coords[4 * i + 2], z = coords[4 * i + 3];
    if (b < 0 || b >= batch || x < 0 || x >= grid[0] || y < 0 || y >= grid[1] || z < 0 || z >= grid[2]) {
      free(rk); free(slot);
      return REF_ERR_BAD_INPUT;
    }
    rk[i].key = ((b * GX + x / l) * GY + y / w) * GZ + z / h;
    rk[i].idx = i;
    slot[i] = (int32_t)(((x % l) * w + (y % w)) * h + (z % h));
    if (slot_of) slot_of[i] = slot[i];
  }
  qsort(rk, (size_t)n, sizeof(ref_rkey), ref_rkey_cmp);
  /* region boundaries */
  int32_t* rstart = (int32_t*)malloc(sizeof(int32_t) * (size_t)(n + 1));
  int32_t m = 0;
  for (int32_t i = 0; i < n; ++i)
    if (i == 0 || rk[i].key != rk[i - 1].key) rstart[m++] = i;
  rstart[m] = n;
  *num_out = m;
  if (m > cap_m) { free(rk); free(slot); free(rstart); return REF_ERR_CAPACITY; }
  int bad = 0;
  const int d = C / heads;
  const double scale = 1.0 / sqrt((double)d);
  int r;
#pragma omp parallel for schedule(dynamic, 16) num_threads(g_threads)
  for (r = 0; r < m; ++r) {
    const int64_t key = rk[rstart[r]].key;
    out_coords[4 * r + 3] = (int32_t)(key % GZ);
    out_coords[4 * r + 2] = (int32_t)((key / GZ) % GY);
    out_coords[4 * r + 1] = (int32_t)((key / (GZ * GY)) % GX);
    out_coords[4 * r + 0] = (int32_t)(key / (GZ * GY * GX));
    double* dense = (double*)calloc((size_t)nslots * C, sizeof(double)); /* zero padding */
    int* occ = (int*)calloc((size_t)nslots, sizeof(int));
    double* buf = (double*)malloc(sizeof(double) * ((size_t)2 * nslots * C + 5 * (size_t)C + nslots));
    double* Kp = buf;
    double* Vp = Kp + (size_t)nslots * C;
    double* P = Vp + (size_t)nslots * C;
    double* q = P + C;
    double* att = q + C;
    double* tmp = att + C;
    double* o = tmp + C;
    double* logit = o + C;
    for (int32_t i = rstart[r]; i < rstart[r + 1]; ++i) {
      const int32_t v = rk[i].idx;
      if (region_of) region_of[v] = r;
      if (occ[slot[v]]) {
#pragma omp atomic write
        bad = 1;
      }
      occ[slot[v]] = 1;
      memcpy(dense + (size_t)slot[v] * C, feats + (size_t)v * C, sizeof(double) * (size_t)C);
    }
    /* Eq. 6: max over the (padded) slots, channel by channel */
    for (int c = 0; c < C; ++c) {
      double mx = -INFINITY;
      for (int s = 0; s < nslots; ++s)
        if (!mask_empty || occ[s])
          if (dense[(size_t)s * C + c] > mx) mx = dense[(size_t)s * C + c];
      P[c] = mx;
    }
    /* Eq. 7: query from the pooled feature, keys/values from the padded slots */
    ref_linear(W_q, b_q, P, C, C, q);
    for (int s = 0; s < nslots; ++s) {
      for (int c = 0; c < C; ++c) tmp[c] = dense[(size_t)s * C + c] + (slot_pe ? slot_pe[(size_t)s * C + c] : 0.0);
      ref_linear(W_k, b_k, tmp, C, C, Kp + (size_t)s * C);
      ref_linear(W_v, b_v, tmp, C, C, Vp + (size_t)s * C);
    }
    for (int hh = 0; hh < heads; ++hh) {
      double mx = -INFINITY;
      for (int s = 0; s < nslots; ++s) {
        if (mask_empty && !occ[s]) continue;
        double acc = 0.0;
        for (int c = 0; c < d; ++c) acc += q[hh * d + c] * Kp[(size_t)s * C + hh * d + c];
        logit[s] = acc * scale;
        if (logit[s] > mx) mx = logit[s];
      }
      double den = 0.0;
      for (int s = 0; s < nslots; ++s)
        if (!mask_empty || occ[s]) { logit[s] = exp(logit[s] - mx); den += logit[s]; }
      for (int c = 0; c < d; ++c) {
        double acc = 0.0;
        for (int s = 0; s < nslots; ++s)
          if (!mask_empty || occ[s]) acc += logit[s] * Vp[(size_t)s * C + hh * d + c];
        att[hh * d + c] = acc / den;
      }
    }
    ref_linear(W_o, b_o, att, C, C, o);
    memcpy(out_feats + (size_t)r * C, o, sizeof(double) * (size_t)C);
    free(dense);
    free(occ);
    free(buf);
  }
  free(rk);
  free(slot);
  free(rstart);
  return bad ? REF_ERR_BAD_INPUT : REF_OK;
}

/* ------------------------------------------------------------------ */
/* BEV projection (Sec. 3.1: the backbone's voxel features are         */
/* projected to a bird's-eye-view feature map)                         */
/* ------------------------------------------------------------------ */
/*
 * Dense map of the grid's (x, y) plane; the z cells of a column are stacked into channels:
 * channel c*Z + z of cell (b, y, x) = feats[i][c] of the voxel i at (b, x, y, z); cells without a voxel are 0.
 * channels_last == 0: out[b][c*Z + z][y][x]  (the image's rows run along y, its columns along x);
 * channels_last == 1: out[b][y][x][c*Z + z].
 * Two voxels in one cell are an input error.
 */
int dsvt_ref_bev_scatter(const int32_t* coords, const double* feats, int32_t n, int32_t C, int32_t batch,
                         const int32_t* grid, int32_t channels_last, double* out) {
  if (n < 0 || C < 1 || batch < 1 || grid[0] < 1 || grid[1] < 1 || grid[2] < 1) return REF_ERR_ARG;
  const int64_t X = grid[0], Y = grid[1], Z = grid[2], CH = (int64_t)C * Z;
  const int64_t total = (int64_t)batch * CH * Y * X;
  unsigned char* seen = (unsigned char*)calloc((size_t)((int64_t)batch * X * Y * Z), 1);
  for (int64_t i = 0; i < total; ++i) out[i] = 0.0;
  for (int32_t i = 0; i < n; ++i) {
    const int64_t b = coords[4 * (size_t)i], x = coords[4 * (size_t)i + 1], y = coords[4 * (size_t)i + 2],
                  z = coords[4 * (size_t)i + 3];
    if (b < 0 || b >= batch || x < 0 || x >= X || y < 0 || y >= Y || z < 0 || z >= Z) { free(seen); return REF_ERR_BAD_INPUT; }
    const int64_t cell = ((b * X + x) * Y + y) * Z + z;
    if (seen[cell]) { free(seen); return REF_ERR_BAD_INPUT; }
    seen[cell] = 1;
    for (int64_t c = 0; c < C; ++c) {
      const int64_t ch = c * Z + z;
      const int64_t o = channels_last ? ((b * Y + y) * X + x) * CH + ch : ((b * CH + ch) * Y + y) * X + x;
      out[o] = feats[(size_t)i * C + c];
    }
  }
  free(seen);
  return REF_OK;
}
