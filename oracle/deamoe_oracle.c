/*
 * DeaMoE layer oracle -- TEST INFRASTRUCTURE, not product code.
 *
 * A plain, slow, fp64 CPU statement of what one DeaMoE layer (and the standard
 * MoE layer it is compared with) computes, written from the paper's definitions:
 *
 *   Eq. (1)  standard expert   MoE_i(x) = W_down^T ( SiLU(W_gate x) * (W_up x) )
 *   Eq. (2)  router            S(x) = TopK(W_r x, k_expert)
 *   Eq. (3)  layer output      sum_{i in S(x)} p_i(x) Expert_i(x)
 *   Eq. (4)  DeaMoE expert i of department j (Section 3.1):
 *              g^ = SiLU(A_g^i sigma(W_g^j x)),  u^ = A_u^i sigma(W_u^j x),
 *              DeaMoE_i(x) = (W_d^j)^T sigma((A_d^i)^T (g^ * u^))
 *   Section 3.2  department token sets X^j and per-expert token lists.
 *
 * The two-stage schedule of Section 3.2 re-orders work but reaches exactly the
 * result of evaluating Eq. (4) per selected expert and summing with Eq. (3), so
 * the VALUES here are that plain definition, token by token and expert by
 * expert, with no bucketing; the SETS and LISTS of Section 3.2 are produced by a
 * separate plain routine.
 *
 * Readings taken where the paper is silent:
 *   - private matrices are [priv, ffn]; the paper's own case is priv == ffn;
 *     priv == 0 means A_g = A_u = A_d = identity (nothing stored);
 *   - ties in TopK go to the lowest expert index; the order of S(x) is
 *     (logit descending, index ascending);
 *   - p = route_scale * softmax over the selected logits (norm_topk = 1) or
 *     over all n logits without renormalisation (norm_topk = 0); norm_topk = 2
 *     is a variant the paper does not have (Section 3.1 only says "softmax
 *     normalization and scaling"): p_i = route_scale * s_i / sum of s over the
 *     selection, s = 1 / (1 + exp(-logit)), the selection still by raw logit;
 *   - k_dept > 0 selects group-limited routing: department score = the largest
 *     logit in the department, the k_dept best departments (ties to the lowest
 *     department index) survive, TopK runs over their experts only;
 *   - department of expert i is i div experts_per_dept;
 *   - an optional always-on shared expert is Eq. (1) with weight 1;
 *   - strict department coverage (the variant Section 3.3 evaluates and rejects): while the
 *     selection spans fewer than min(k_dept, k) departments, the lowest-ranked selected expert
 *     whose department holds another selected expert is replaced, in place, by the expert with
 *     the largest logit (ties: lowest index) among the departments not yet covered;
 *   - sigma = RMSNorm (one of the operators of Section 3.4 / Table 4) acts on the whole
 *     length-f vector: v / sqrt(mean(v^2) + 1e-6), no learned gain;
 *   - a department slice (dept_begin, dept_end) evaluates Eq. (3) over the selected experts of
 *     those departments only; the slices of a partition add up to the layer.
 *
 * Only tests, the smoke check and the benchmark's cpu_baseline leg may call
 * this file.  It shares no code with the CUDA library.
 *
 * All loops are the textbook ones.  OpenMP only splits independent output
 * elements across threads; each element is still one sequential fp64 sum in
 * index order, so results do not depend on the thread count.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { ORACLE_F32 = 0, ORACLE_BF16 = 1 };
enum { ORACLE_SIGMA_NONE = 0, ORACLE_SIGMA_SILU = 1, ORACLE_SIGMA_GELU = 2, ORACLE_SIGMA_RMSNORM = 3 };
#define ORACLE_RMS_EPS 1e-6

typedef struct {
  int32_t hidden;           /* h */
  int32_t n_dept;           /* m */
  int32_t experts_per_dept; /* g, n = m*g */
  int32_t ffn;              /* f */
  int32_t priv;             /* r, 0 = identity private transforms */
  int32_t top_k;            /* k_expert */
  int32_t k_dept;           /* 0 = no group limit */
  int32_t n_shared;         /* 0 or 1 */
  int32_t shared_ffn;
  int32_t sigma;
  int32_t norm_topk;
  int32_t weight_dtype;
  int32_t act_dtype;
  int32_t residual;         /* 1: out = x + layer(x) */
  int32_t strict_dept;      /* 1: strict department coverage (Section 3.3, last paragraph) */
  double route_scale;
  int32_t dept_begin, dept_end; /* 0, 0: the whole layer; else only the experts of departments
                                   [dept_begin, dept_end) contribute to oracle_deamoe_forward: the
                                   partial sum of one slice of a department-sharded layer (Eq. (3)
                                   is a sum over experts, Section 3.1's departments are independent) */
} oracle_config_t;

/* Pointer tables: one pointer per department / per expert, so a caller may
 * leave entries it knows to be unused as NULL (the oracle reports an error if
 * it needs one of them). */
typedef struct {
  const float *router;             /* [n, h] fp32 */
  const void *const *dept_gate;    /* m x [f, h] */
  const void *const *dept_up;
  const void *const *dept_down;    /* [f, h], applied transposed */
  const void *const *priv_gate;    /* n x [r, f]; table may be NULL iff priv == 0 */
  const void *const *priv_up;
  const void *const *priv_down;    /* [r, f], applied transposed */
  const void *shared_gate;         /* [shared_ffn, h] */
  const void *shared_up;
  const void *shared_down;
} oracle_weights_t;

static int g_threads = 1;

int oracle_set_threads(int t) {
  if (t < 1) t = 1;
  g_threads = t;
#ifdef _OPENMP
  omp_set_num_threads(t);
#endif
  return g_threads;
}

int oracle_get_threads(void) {
#ifdef _OPENMP
  return g_threads;
#else
  return 1;
#endif
}

/* exact widening of one stored number to fp64 */
static inline double ld(const void *p, int dtype, size_t i) {
  if (dtype == ORACLE_F32) return (double)((const float *)p)[i];
  uint32_t bits = ((uint32_t)((const uint16_t *)p)[i]) << 16;
  float v;
  memcpy(&v, &bits, 4);
  return (double)v;
}

static inline double silu(double v) { return v / (1.0 + exp(-v)); }

static inline double sigma_fn(int kind, double v) {
  switch (kind) {
    case ORACLE_SIGMA_SILU: return silu(v);
    case ORACLE_SIGMA_GELU: return 0.5 * v * (1.0 + erf(v * 0.70710678118654752440));
    default: return v;
  }
}

/* sigma of Section 3.1 / 3.4 on a whole vector: element-wise for SiLU / GeLU / none,
 * root-mean-square normalisation over the vector for RMSNorm */
static void sigma_vec(int kind, double *v, int n) {
  if (kind == ORACLE_SIGMA_RMSNORM) {
    double ss = 0.0;
    for (int q = 0; q < n; ++q) ss += v[q] * v[q];
    const double d = sqrt(ss / (double)n + ORACLE_RMS_EPS);
    for (int q = 0; q < n; ++q) v[q] = v[q] / d;
    return;
  }
  for (int q = 0; q < n; ++q) v[q] = sigma_fn(kind, v[q]);
}

/* y[r] = sum_c W[r, c] x[c],  W is [rows, cols] row-major */
static void matvec(const void *W, int dtype, int rows, int cols, const double *x, double *y) {
#pragma omp parallel for schedule(static)
  for (int r = 0; r < rows; ++r) {
    double s = 0.0;
    for (int c = 0; c < cols; ++c) s += ld(W, dtype, (size_t)r * cols + c) * x[c];
    y[r] = s;
  }
}

/* y[c] = sum_r W[r, c] x[r]  (W^T x),  W is [rows, cols] row-major */
static void matvec_t(const void *W, int dtype, int rows, int cols, const double *x, double *y) {
#pragma omp parallel for schedule(static)
  for (int c = 0; c < cols; ++c) {
    double s = 0.0;
    for (int r = 0; r < rows; ++r) s += ld(W, dtype, (size_t)r * cols + c) * x[r];
    y[c] = s;
  }
}

/* Eq. (1): out[h] = Wd^T ( SiLU(Wg x) * (Wu x) ), all three [f, h]. */
int oracle_swiglu(const void *Wg, const void *Wu, const void *Wd, int dtype, int h, int f,
                  const double *x, double *out) {
  if (!Wg || !Wu || !Wd) return 2;
  double *a = (double *)malloc(sizeof(double) * (size_t)f * 2);
  if (!a) return 3;
  double *b = a + f;
  matvec(Wg, dtype, f, h, x, a);
  matvec(Wu, dtype, f, h, x, b);
  for (int q = 0; q < f; ++q) a[q] = silu(a[q]) * b[q];
  matvec_t(Wd, dtype, f, h, a, out);
  free(a);
  return 0;
}

/* Eq. (4): one DeaMoE expert on one token.  Optional taps return the
 * intermediates of Section 3.2: G = sigma(W_g x), U = sigma(W_u x) (length f),
 * Y (length r, or f when priv == 0), Z (length f). */
int oracle_deamoe_expert(const oracle_config_t *c, const void *Wg, const void *Wu, const void *Wd,
                         const void *Ag, const void *Au, const void *Ad, const double *x,
                         double *out, double *tapG, double *tapU, double *tapY, double *tapZ) {
  const int h = c->hidden, f = c->ffn, r = c->priv > 0 ? c->priv : c->ffn;
  const int dt = c->weight_dtype;
  if (!Wg || !Wu || !Wd) return 2;
  if (c->priv > 0 && (!Ag || !Au || !Ad)) return 2;
  double *G = (double *)malloc(sizeof(double) * ((size_t)3 * f + 3 * (size_t)r));
  if (!G) return 3;
  double *U = G + f, *Z = U + f, *yg = Z + f, *yu = yg + r, *Y = yu + r;
  matvec(Wg, dt, f, h, x, G);
  matvec(Wu, dt, f, h, x, U);
  sigma_vec(c->sigma, G, f);
  sigma_vec(c->sigma, U, f);
  if (c->priv > 0) {
    matvec(Ag, dt, r, f, G, yg);
    matvec(Au, dt, r, f, U, yu);
  } else { /* identity private transforms */
    memcpy(yg, G, sizeof(double) * f);
    memcpy(yu, U, sizeof(double) * f);
  }
  for (int q = 0; q < r; ++q) Y[q] = silu(yg[q]) * yu[q];
  if (c->priv > 0) {
    matvec_t(Ad, dt, r, f, Y, Z);
  } else {
    memcpy(Z, Y, sizeof(double) * f);
  }
  sigma_vec(c->sigma, Z, f);
  matvec_t(Wd, dt, f, h, Z, out);
  if (tapG) memcpy(tapG, G, sizeof(double) * f);
  if (tapU) memcpy(tapU, U, sizeof(double) * f);
  if (tapY) memcpy(tapY, Y, sizeof(double) * r);
  if (tapZ) memcpy(tapZ, Z, sizeof(double) * f);
  free(G);
  return 0;
}

/* ---- routing: Eq. (2) and the gate weights of Eq. (3) ---- */

typedef struct { double v; int32_t i; } keyed_t;

static int cmp_desc_then_index(const void *a, const void *b) {
  const keyed_t *x = (const keyed_t *)a, *y = (const keyed_t *)b;
  if (x->v > y->v) return -1;
  if (x->v < y->v) return 1;
  return (x->i > y->i) - (x->i < y->i);
}

/*
 * tokens [B, h] in act_dtype.  Outputs (any may be NULL except topk_idx/topk_w):
 *   topk_idx [B, k]   selected experts in (logit desc, index asc) order
 *   topk_w   [B, k]   gate weights p (fp64)
 *   logits   [B, n]   fp64 router logits
 *   gap      [B]      how far the token's selection and its order are from a tie: the
 *                     smallest margin of any comparison that decided them, i.e. the
 *                     minimum of the three entries of gap_parts
 *   gap_parts [B, 3]  [0] smallest difference between neighbours among the first
 *                         min(k+1, candidates) sorted candidate logits;
 *                     [1] group limit: score of the k_dept-th best department minus the
 *                         score of the first department left out (INFINITY without a cut);
 *                     [2] strict coverage: over all replacements, the newcomer's logit minus
 *                         the next-best logit among the experts of the departments not yet
 *                         covered (INFINITY if nothing was replaced or nothing else competed)
 * The gaps are diagnostics for the tests (an fp32 router may legitimately decide a
 * comparison the other way when its margin is at rounding level); they change no result.
 */
int oracle_route(const oracle_config_t *c, const float *router, const void *tokens, int B,
                 int32_t *topk_idx, double *topk_w, double *logits, double *gap, double *gap_parts) {
  const int h = c->hidden, g = c->experts_per_dept, m = c->n_dept, n = m * g, k = c->top_k;
  if (!router || !tokens || !topk_idx || !topk_w || k < 1 || k > n) return 1;
  double *x = (double *)malloc(sizeof(double) * ((size_t)h + n));
  keyed_t *key = (keyed_t *)malloc(sizeof(keyed_t) * ((size_t)n + m));
  char *alive = (char *)malloc((size_t)m);
  if (!x || !key || !alive) { free(x); free(key); free(alive); return 3; }
  double *l = x + h;
  keyed_t *dkey = key + n;
  int rc = 0;
  for (int t = 0; t < B && rc == 0; ++t) {
    for (int q = 0; q < h; ++q) x[q] = ld(tokens, c->act_dtype, (size_t)t * h + q);
    matvec(router, ORACLE_F32, n, h, x, l);
    if (logits) memcpy(logits + (size_t)t * n, l, sizeof(double) * n);
    double gap_sel = INFINITY, gap_dept = INFINITY, gap_strict = INFINITY;
    /* group limit: keep the k_dept departments with the largest best logit */
    memset(alive, 1, (size_t)m);
    if (c->k_dept > 0 && c->k_dept < m) {
      for (int j = 0; j < m; ++j) {
        double best = l[(size_t)j * g];
        for (int e = 1; e < g; ++e) if (l[(size_t)j * g + e] > best) best = l[(size_t)j * g + e];
        dkey[j].v = best; dkey[j].i = j;
      }
      qsort(dkey, (size_t)m, sizeof(keyed_t), cmp_desc_then_index);
      memset(alive, 0, (size_t)m);
      for (int q = 0; q < c->k_dept; ++q) alive[dkey[q].i] = 1;
      gap_dept = dkey[c->k_dept - 1].v - dkey[c->k_dept].v;
    }
    int cand = 0;
    for (int i = 0; i < n; ++i)
      if (alive[i / g]) { key[cand].v = l[i]; key[cand].i = i; ++cand; }
    if (cand < k) { rc = 1; break; }
    qsort(key, (size_t)cand, sizeof(keyed_t), cmp_desc_then_index);
    { /* smallest difference between neighbours of the sorted order, up to the first expert left out */
      int upto = (k + 1 < cand) ? k + 1 : cand;
      for (int q = 1; q < upto; ++q) {
        double d = key[q - 1].v - key[q].v;
        if (d < gap_sel) gap_sel = d;
      }
    }
    /* strict department coverage: swap duplicates out until min(k_dept, k) departments are covered */
    if (c->strict_dept && c->k_dept > 0) {
      const int target = (c->k_dept < k ? c->k_dept : k) < m ? (c->k_dept < k ? c->k_dept : k) : m;
      for (;;) {
        int covered = 0;
        for (int j = 0; j < m; ++j) {
          int hit = 0;
          for (int q = 0; q < k; ++q) if (key[q].i / g == j) hit = 1;
          covered += hit;
        }
        if (covered >= target) break;
        int victim = -1;
        for (int q = 0; q < k; ++q) {
          int same = 0;
          for (int q2 = 0; q2 < k; ++q2) if (q2 != q && key[q2].i / g == key[q].i / g) same = 1;
          if (same) victim = q; /* the last such q is the lowest-ranked one */
        }
        if (victim < 0) break;
        int best = -1;
        double runner_up = -INFINITY; /* diagnostic only: the largest logit the newcomer beat */
        for (int i = 0; i < n; ++i) {
          int used = 0;
          for (int q = 0; q < k; ++q) if (key[q].i / g == i / g) used = 1;
          if (used) continue;
          if (best < 0 || l[i] > l[best]) { /* ascending i: ties keep the lowest index */
            if (best >= 0 && l[best] > runner_up) runner_up = l[best];
            best = i;
          } else if (l[i] > runner_up) {
            runner_up = l[i];
          }
        }
        if (best < 0) break;
        if (l[best] - runner_up < gap_strict) gap_strict = l[best] - runner_up;
        key[victim].i = best;
        key[victim].v = l[best];
      }
    }
    for (int q = 0; q < k; ++q) topk_idx[(size_t)t * k + q] = key[q].i;
    if (gap_parts) {
      gap_parts[(size_t)t * 3 + 0] = gap_sel;
      gap_parts[(size_t)t * 3 + 1] = gap_dept;
      gap_parts[(size_t)t * 3 + 2] = gap_strict;
    }
    if (gap) {
      double gmin = gap_sel;
      if (gap_dept < gmin) gmin = gap_dept;
      if (gap_strict < gmin) gmin = gap_strict;
      gap[t] = gmin;
    }
    if (c->norm_topk == 2) { /* sigmoid scores, normalised over the selection */
      double den = 0.0;
      for (int q = 0; q < k; ++q) den += 1.0 / (1.0 + exp(-key[q].v));
      for (int q = 0; q < k; ++q)
        topk_w[(size_t)t * k + q] = c->route_scale * (1.0 / (1.0 + exp(-key[q].v))) / den;
      continue;
    }
    /* softmax (max-subtracted) over the selection, or over all n logits */
    double mx = key[0].v, den = 0.0;
    if (c->norm_topk) {
      for (int q = 0; q < k; ++q) den += exp(key[q].v - mx);
    } else {
      mx = l[0];
      for (int i = 1; i < n; ++i) if (l[i] > mx) mx = l[i];
      for (int i = 0; i < n; ++i) den += exp(l[i] - mx);
    }
    for (int q = 0; q < k; ++q)
      topk_w[(size_t)t * k + q] = c->route_scale * exp(key[q].v - mx) / den;
  }
  free(x); free(key); free(alive);
  return rc;
}

/*
 * Section 3.2 sets and lists from the selection topk_idx [B, k]:
 *   dept_mask  [ceil(m/64)] bit j set iff department j received a token
 *   dept_off   [m+1], dept_tok[dept_off[j] .. dept_off[j+1])  = X^j, the distinct
 *              tokens that selected any expert of department j, ascending
 *   expert_off [n+1], expert_tok likewise per expert
 * dept_tok must hold B*min(k, m) entries, expert_tok B*k.
 */
int oracle_bucket(const oracle_config_t *c, const int32_t *topk_idx, int B, uint64_t *dept_mask,
                  int32_t *dept_off, int32_t *dept_tok, int32_t *expert_off, int32_t *expert_tok) {
  const int g = c->experts_per_dept, m = c->n_dept, n = m * g, k = c->top_k;
  if (!topk_idx || !dept_mask || !dept_off || !dept_tok || !expert_off || !expert_tok) return 1;
  for (int w = 0; w < (m + 63) / 64; ++w) dept_mask[w] = 0;
  int pos = 0;
  for (int j = 0; j < m; ++j) {
    dept_off[j] = pos;
    for (int t = 0; t < B; ++t) {
      int hit = 0;
      for (int q = 0; q < k; ++q)
        if (topk_idx[(size_t)t * k + q] / g == j) hit = 1;
      if (hit) dept_tok[pos++] = t;
    }
    if (pos > dept_off[j]) dept_mask[j / 64] |= (uint64_t)1 << (j % 64);
  }
  dept_off[m] = pos;
  pos = 0;
  for (int i = 0; i < n; ++i) {
    expert_off[i] = pos;
    for (int t = 0; t < B; ++t)
      for (int q = 0; q < k; ++q)
        if (topk_idx[(size_t)t * k + q] == i) { expert_tok[pos++] = t; break; }
  }
  expert_off[n] = pos;
  return 0;
}

/* ---- whole layers ---- */

static int shared_and_residual(const oracle_config_t *c, const oracle_weights_t *w, const void *tokens,
                               int t, const double *x, double *o, double *tmp) {
  const int h = c->hidden;
  (void)tokens; (void)t;
  if (c->n_shared) {
    int rc = oracle_swiglu(w->shared_gate, w->shared_up, w->shared_down, c->weight_dtype, h,
                           c->shared_ffn, x, tmp);
    if (rc) return rc;
    for (int q = 0; q < h; ++q) o[q] += tmp[q];
  }
  if (c->residual)
    for (int q = 0; q < h; ++q) o[q] += x[q];
  return 0;
}

/*
 * DeaMoE layer: route (Eq. 2), evaluate Eq. (4) for every selected expert of
 * every token, combine with Eq. (3), add the shared expert / residual if
 * configured.  out is [B, h] fp64.  Only the rows listed in `rows`
 * (n_rows entries, NULL = all B tokens) are evaluated; the others are left
 * untouched.  Routing always covers all B tokens.
 */
int oracle_deamoe_forward(const oracle_config_t *c, const oracle_weights_t *w, const void *tokens,
                          int B, const int32_t *rows, int n_rows, double *out, int32_t *topk_idx,
                          double *topk_w) {
  const int h = c->hidden, g = c->experts_per_dept, k = c->top_k;
  int32_t *idx = topk_idx ? topk_idx : (int32_t *)malloc(sizeof(int32_t) * (size_t)B * k);
  double *p = topk_w ? topk_w : (double *)malloc(sizeof(double) * (size_t)B * k);
  double *x = (double *)malloc(sizeof(double) * (size_t)h * 2);
  int rc = (!idx || !p || !x) ? 3 : oracle_route(c, w->router, tokens, B, idx, p, NULL, NULL, NULL);
  double *e = x ? x + h : NULL;
  const int count = rows ? n_rows : B;
  for (int s = 0; s < count && rc == 0; ++s) {
    const int t = rows ? rows[s] : s;
    if (t < 0 || t >= B) { rc = 1; break; }
    double *o = out + (size_t)t * h;
    for (int q = 0; q < h; ++q) { x[q] = ld(tokens, c->act_dtype, (size_t)t * h + q); o[q] = 0.0; }
    for (int q = 0; q < k && rc == 0; ++q) {
      const int i = idx[(size_t)t * k + q], j = i / g;
      if (c->dept_end > 0 && (j < c->dept_begin || j >= c->dept_end)) continue; /* another slice's expert */
      rc = oracle_deamoe_expert(c, w->dept_gate[j], w->dept_up[j], w->dept_down[j],
                                c->priv > 0 ? w->priv_gate[i] : NULL,
                                c->priv > 0 ? w->priv_up[i] : NULL,
                                c->priv > 0 ? w->priv_down[i] : NULL, x, e, NULL, NULL, NULL, NULL);
      if (rc) break;
      const double pi = p[(size_t)t * k + q];
      for (int u = 0; u < h; ++u) o[u] += pi * e[u];
    }
    if (rc == 0) rc = shared_and_residual(c, w, tokens, t, x, o, e);
  }
  if (!topk_idx) free(idx);
  if (!topk_w) free(p);
  free(x);
  return rc;
}

/*
 * Standard MoE layer, Eq. (1)-(3): n = m*g independent experts.  The tables
 * dept_gate/dept_up/dept_down of `w` are read as n per-EXPERT pointers here;
 * the private tables are ignored.
 */
int oracle_vanilla_forward(const oracle_config_t *c, const oracle_weights_t *w, const void *tokens,
                           int B, const int32_t *rows, int n_rows, double *out, int32_t *topk_idx,
                           double *topk_w) {
  const int h = c->hidden, k = c->top_k;
  int32_t *idx = topk_idx ? topk_idx : (int32_t *)malloc(sizeof(int32_t) * (size_t)B * k);
  double *p = topk_w ? topk_w : (double *)malloc(sizeof(double) * (size_t)B * k);
  double *x = (double *)malloc(sizeof(double) * (size_t)h * 2);
  int rc = (!idx || !p || !x) ? 3 : oracle_route(c, w->router, tokens, B, idx, p, NULL, NULL, NULL);
  double *e = x ? x + h : NULL;
  const int count = rows ? n_rows : B;
  for (int s = 0; s < count && rc == 0; ++s) {
    const int t = rows ? rows[s] : s;
    if (t < 0 || t >= B) { rc = 1; break; }
    double *o = out + (size_t)t * h;
    for (int q = 0; q < h; ++q) { x[q] = ld(tokens, c->act_dtype, (size_t)t * h + q); o[q] = 0.0; }
    for (int q = 0; q < k && rc == 0; ++q) {
      const int i = idx[(size_t)t * k + q];
      rc = oracle_swiglu(w->dept_gate[i], w->dept_up[i], w->dept_down[i], c->weight_dtype, h,
                         c->ffn, x, e);
      if (rc) break;
      const double pi = p[(size_t)t * k + q];
      for (int u = 0; u < h; ++u) o[u] += pi * e[u];
    }
    if (rc == 0) rc = shared_and_residual(c, w, tokens, t, x, o, e);
  }
  if (!topk_idx) free(idx);
  if (!topk_w) free(p);
  free(x);
  return rc;
}
