/*
 * ckv_oracle.c -- TEST INFRASTRUCTURE, not the product.
 *
 * A plain, slow, fp64 CPU statement of the end-of-prefill KV retention pass of
 * CompilerKV (arxiv 2602.08686).  It exists so that the CUDA library can be
 * checked against something written directly from the paper.  It shares no code
 * with the CUDA path, and only the tests, the smoke check and the benchmark's
 * cpu-baseline leg may call it.
 *
 * Notation (the build's, not the paper's):  L = prompt length (paper: T),
 * W = observation-window size |Omega|, n = L - W = prefix length, H = query
 * heads, Hkv = KV heads, G = H / Hkv, d = head_dim, B = kept rows per KV head on
 * average (window included).  A "unit" is one (sequence, layer) pair.
 *
 * Steps, in the paper's order:
 *   O1  logits     s[h,i,t] = q[h,i].k[g,t] / sqrt(d), g = h / G        (Sec. 3)
 *   O2  softmax    over the keys a window row can see (causal)          (Sec. 3)
 *   O3  column sum c_h[t] = sum_{i in Omega} A[h,i,t]           (Eq. 4, Alg. 1 (A))
 *   O4  scale      alpha_h[t] = (L / W) c_h[t]                          (Eq. 4)
 *   O5  1-D pooling of alpha_h over the prefix (argument; size 1 = the paper)
 *   O5b value-norm ratio (optional) rho_g[t] = |v_g[t]|_2 / (mean_k |v_g[k]|_2 + eps),
 *       u_h[t] = pooled_h[t] * rho_g[t]                    (Eq. 4, Alg. 1 (B))
 *   O6  head table u_g[t] = max_{h in group g} W_head[h] * u_h[t]       (Eq. 6)
 *   O7  risk coordinate: entropy of the normalised window mass, bucket,
 *       threshold tau = table[bucket]                    (Eq. 7 left, Alg. 1 (A),(D));
 *       with gate_layers set the table is the paper's T_gate[l, b_ent, b_ppl, B_l]
 *       (Sec. 4.3), the perplexity bin and the layer / budget rows supplied per unit
 *   O8  candidate counts under tau (Eq. 8's candidate set) -> per-head budgets
 *       clamped so that they sum to the total budget
 *   O9  Top-k per KV head, ties to the lowest index, window always kept (Eq. 8)
 *   O10 gather of the kept K/V rows                               (Sec. 3, Alg. 1 (D))
 * With shared_elastic set, O6-O9 take the paper's own form instead: the weighted max of
 * Eq. 6 runs over all H heads of the unit, the retained set is Eq. 8's (all candidates if
 * they fit the budget, else the Top-B of them) and every KV head keeps that one set.
 * With global_alpha set, O4 and O7 take the paper's form: the attention is averaged over all
 * layers and heads of the prompt before the window sum (Alg. 1 (A)), so one alpha and one risk
 * coordinate serve all of the prompt's units (units_per_prompt consecutive units each).
 *
 * Pins (tests/test_oracle_*.py): the mass identity sum_t c_h[t] = W (text after
 * Eq. 4), closed-form attention on constant / single-spike inputs, torch's fp64
 * softmax and pooling routines on special cases, Shannon entropy of uniform and
 * one-hot distributions, hand-computed norms, the mean identity and scale
 * invariance of O5b, brute-force rational water-filling for O8, brute-force
 * sorting for O9, direct indexing for O10, FullKV reproduction, and the
 * identity |p - p~|_1 = 2m of Eq. A2, a hand-built gate table with one distinct
 * value per cell, and numpy's linear interpolation for the depth mapping.
 * Parity unpinned by the paper itself (the paper has no such step; pinned only
 * by the invariants above): the O8 redistribution rule, the bucket edges of O7,
 * and the edge rule of the O5 pooling.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define OR_BF16 0
#define OR_F32 1
#define OR_POOL_NONE 0
#define OR_POOL_MAX 1
#define OR_POOL_AVG 2

typedef struct {
  int32_t n_units, n_q_heads, n_kv_heads, head_dim, seq_len, window;
  int32_t dtype; /* OR_BF16: uint16 bit patterns; OR_F32: float */
} or_shape;

typedef struct {
  int32_t pool_kind, pool_size;
  int32_t budget_per_head; /* B */
  int32_t floor_per_head;  /* f: minimum prefix rows per KV head */
  int32_t n_buckets;
  int32_t bucket_override; /* -1: bucket from the entropy */
  int32_t head_w_per_unit; /* 0: one [H] row shared by all units; 1: [Nu,H] */
  int32_t sens_per_unit;   /* 0: one [n_buckets] row; 1: [Nu,n_buckets] */
  int32_t value_norm;      /* 1: multiply the pooled window mass by the value-norm ratio (O5b) */
  float value_norm_eps;    /* the eps of Alg. 1 (B) */
  int32_t shared_elastic;  /* 1: one elastic set per unit (Eq. 6 over all heads, Eq. 8), shared by its KV heads */
  int32_t global_alpha;    /* 1: alpha from the mean attention over all layers and heads of the prompt */
  int32_t units_per_prompt; /* layers of one prompt: units [s N, (s + 1) N) belong to prompt s (global_alpha) */
  /* The threshold table as the paper indexes it (Sec. 4.3, Alg. 1 (D)): tau = T_gate[l, b_ent, b_ppl, B_l].
   * gate_layers > 0 switches it on: the table argument is then [gate_layers][n_buckets][ppl_bins][budget_levels]
   * (n_buckets entropy bins) and gate_coords [Nu,3] holds, per unit, the layer row l, the perplexity bin b_ppl
   * (computed by the caller from the language model's logits, Eq. 7 right) and the index of the budget level. */
  int32_t gate_layers, ppl_bins, budget_levels;
  const int32_t *gate_coords;
} or_params;

/* exact widening of an input element to double */
static double widen(const void *base, int dtype, int64_t idx) {
  if (dtype == OR_F32) return (double)((const float *)base)[idx];
  uint32_t bits = ((uint32_t)((const uint16_t *)base)[idx]) << 16;
  float f;
  memcpy(&f, &bits, 4);
  return (double)f;
}

/* ------------------------------------------------------------------ O1 + O2
 * One window row of the causal attention matrix: row i of the window sits at
 * absolute position n + i and sees keys t <= n + i.  A[t] = 0 for hidden keys. */
static void attention_row(const or_shape *s, const void *q, const void *k, int u, int h, int i,
                          double *A /* [L] */) {
  const int L = s->seq_len, W = s->window, d = s->head_dim, H = s->n_q_heads, Hkv = s->n_kv_heads;
  const int G = H / Hkv, g = h / G, n = L - W;
  const int last = n + i; /* last visible key */
  const int64_t qoff = (((int64_t)u * H + h) * W + i) * d;
  const int64_t koff = ((int64_t)u * Hkv + g) * (int64_t)L * d;
  const double inv_sqrt_d = 1.0 / sqrt((double)d);
  double m = -INFINITY;
  for (int t = 0; t <= last; ++t) {
    double acc = 0.0;
    for (int c = 0; c < d; ++c) acc += widen(q, s->dtype, qoff + c) * widen(k, s->dtype, koff + (int64_t)t * d + c);
    A[t] = acc * inv_sqrt_d;
    if (A[t] > m) m = A[t];
  }
  double l = 0.0;
  for (int t = 0; t <= last; ++t) {
    A[t] = exp(A[t] - m);
    l += A[t];
  }
  for (int t = 0; t <= last; ++t) A[t] /= l;
  for (int t = last + 1; t < L; ++t) A[t] = 0.0;
}

/* The W x L block of attention rows of every (unit, head): A [Nu,H,W,L]. */
int oracle_window_attention(const or_shape *s, const void *q, const void *k, double *A) {
  const int L = s->seq_len, W = s->window, H = s->n_q_heads;
  if (s->n_q_heads % s->n_kv_heads || W > L || W < 1) return 1;
#pragma omp parallel for collapse(2) schedule(dynamic)
  for (int u = 0; u < s->n_units; ++u)
    for (int h = 0; h < H; ++h)
      for (int i = 0; i < W; ++i) attention_row(s, q, k, u, h, i, A + ((((int64_t)u * H + h) * W + i) * (int64_t)L));
  return 0;
}

/* ------------------------------------------------------------------ O3
 * c_h[t] = sum over the window rows of A[h,i,t]; csum [Nu,H,L]. */
int oracle_colsum(const or_shape *s, const void *q, const void *k, double *csum) {
  const int L = s->seq_len, W = s->window, H = s->n_q_heads;
  if (s->n_q_heads % s->n_kv_heads || W > L || W < 1) return 1;
  int err = 0;
#pragma omp parallel for collapse(2) schedule(dynamic)
  for (int u = 0; u < s->n_units; ++u)
    for (int h = 0; h < H; ++h) {
      double *row = (double *)malloc(sizeof(double) * (size_t)L);
      double *c = csum + ((int64_t)u * H + h) * (int64_t)L;
      if (!row) {
        err = 2;
        continue;
      }
      for (int t = 0; t < L; ++t) c[t] = 0.0;
      for (int i = 0; i < W; ++i) {
        attention_row(s, q, k, u, h, i, row);
        for (int t = 0; t < L; ++t) c[t] += row[t];
      }
      free(row);
    }
  return err;
}

/* ------------------------------------------------------------------ O5
 * Centred stride-1 pooling of x[0..n) with an odd kernel: MAX ignores
 * positions outside the array (padding with -inf); AVG treats them as zeros
 * and always divides by the kernel size.  Size 1 / NONE is the identity. */
int oracle_pool1d(int kind, int size, int n, const double *x, double *out) {
  if (kind == OR_POOL_NONE || size == 1) {
    for (int t = 0; t < n; ++t) out[t] = x[t];
    return 0;
  }
  if (size < 1 || (size & 1) == 0) return 1;
  const int r = size / 2;
  for (int t = 0; t < n; ++t) {
    if (kind == OR_POOL_MAX) {
      double m = -INFINITY;
      for (int j = t - r; j <= t + r; ++j)
        if (j >= 0 && j < n && x[j] > m) m = x[j];
      out[t] = m;
    } else if (kind == OR_POOL_AVG) {
      double a = 0.0;
      for (int j = t - r; j <= t + r; ++j)
        if (j >= 0 && j < n) a += x[j];
      out[t] = a / (double)size;
    } else
      return 1;
  }
  return 0;
}

/* ------------------------------------------------------------------ O5b (Eq. 4's rho, Alg. 1 (B))
 * r[t] = |v[u,g,t,:]|_2 over all L tokens, mu = mean_t r[t], rho[u,g,t] = r[t] / (mu + eps).
 * Under GQA the values belong to the KV head, so the ratio is shared by the group's query heads. */
int oracle_vnorm(const or_shape *s, const void *v, double eps, double *rho) {
  const int L = s->seq_len, Hkv = s->n_kv_heads, Nu = s->n_units, d = s->head_dim;
  for (int u = 0; u < Nu; ++u)
    for (int g = 0; g < Hkv; ++g) {
      double *r = rho + ((int64_t)u * Hkv + g) * (int64_t)L;
      double total = 0.0;
      for (int t = 0; t < L; ++t) {
        double ss = 0.0;
        for (int j = 0; j < d; ++j) {
          const double x = widen(v, s->dtype, (((int64_t)u * Hkv + g) * L + t) * d + j);
          ss += x * x;
        }
        r[t] = sqrt(ss);
        total += r[t];
      }
      const double mu = total / (double)L;
      for (int t = 0; t < L; ++t) r[t] = r[t] / (mu + eps);
    }
  return 0;
}

/* ------------------------------------------------------------------ O4-O6 (+ the mass for O7)
 * scores  [Nu,Hkv,n] : u_g[t] = max_{h in g} head_w[h] * (pool((L/W) c_h)[t] * rho_g[t])
 * colmass [Nu,L]     : sum_h c_h[t]   (all heads of the unit, window columns included)
 * csum    [Nu,H,L]   : c_h[t] (optional)
 * rho     [Nu,Hkv,L] : value-norm ratios of O5b, or NULL for rho = 1 (the paper's "u = alpha" ablation) */
int oracle_score(const or_shape *s, const or_params *p, const void *q, const void *k, const float *head_w,
                 const double *rho_or_null, double *scores, double *colmass, double *csum_or_null) {
  const int L = s->seq_len, W = s->window, H = s->n_q_heads, Hkv = s->n_kv_heads, Nu = s->n_units;
  if (H % Hkv || W > L || W < 1) return 1;
  const int G = H / Hkv, n = L - W;
  double *csum = csum_or_null ? csum_or_null : (double *)malloc(sizeof(double) * (size_t)Nu * H * L);
  if (!csum) return 2;
  int rc = oracle_colsum(s, q, k, csum);
  if (rc) goto done;
  for (int u = 0; u < Nu; ++u)
    for (int t = 0; t < L; ++t) {
      double m = 0.0;
      for (int h = 0; h < H; ++h) m += csum[((int64_t)u * H + h) * L + t];
      colmass[(int64_t)u * L + t] = m;
    }
  if (p->global_alpha) {
    /* Alg. 1 (A): A-bar = mean over layers and heads of the prompt; its window column sums are the mean of the
     * units' column masses over N H.  Every unit of the prompt then carries the prompt's mean mass. */
    const int N = p->units_per_prompt;
    if (N < 1 || Nu % N) {
      rc = 3;
      goto done;
    }
    for (int s0 = 0; s0 < Nu; s0 += N)
      for (int t = 0; t < L; ++t) {
        double m = 0.0;
        for (int u = s0; u < s0 + N; ++u) m += colmass[(int64_t)u * L + t];
        for (int u = s0; u < s0 + N; ++u) colmass[(int64_t)u * L + t] = m / (double)N;
      }
  }
#pragma omp parallel for schedule(dynamic)
  for (int u = 0; u < Nu; ++u) {
    double *alpha = (double *)malloc(sizeof(double) * (size_t)(n > 0 ? n : 1));
    double *pooled = (double *)malloc(sizeof(double) * (size_t)(n > 0 ? n : 1));
    for (int g = 0; g < Hkv; ++g) {
      double *out = scores + ((int64_t)u * Hkv + g) * (int64_t)n;
      for (int t = 0; t < n; ++t) out[t] = -INFINITY;
      for (int h = g * G; h < (g + 1) * G; ++h) {
        const double w = (double)head_w[p->head_w_per_unit ? (int64_t)u * H + h : h];
        const double *c = csum + ((int64_t)u * H + h) * (int64_t)L;
        for (int t = 0; t < n; ++t)   /* Eq. 4's alpha: this head's window mass, or the prompt-wide mean per head */
          alpha[t] = ((double)L / (double)W) * (p->global_alpha ? colmass[(int64_t)u * L + t] / (double)H : c[t]);
        oracle_pool1d(p->pool_kind, p->pool_size, n, alpha, pooled);
        for (int t = 0; t < n; ++t) {
          const double ratio = rho_or_null ? rho_or_null[((int64_t)u * Hkv + g) * (int64_t)L + t] : 1.0;
          const double v = w * (pooled[t] * ratio);
          if (v > out[t]) out[t] = v;
        }
      }
    }
    if (p->shared_elastic) {
      /* Eq. 6 over all H heads of the unit: the max of the groups' maxima; every KV head carries it */
      for (int t = 0; t < n; ++t) {
        double m = -INFINITY;
        for (int g = 0; g < Hkv; ++g) {
          const double x = scores[((int64_t)u * Hkv + g) * (int64_t)n + t];
          if (x > m) m = x;
        }
        for (int g = 0; g < Hkv; ++g) scores[((int64_t)u * Hkv + g) * (int64_t)n + t] = m;
      }
    }
    free(alpha);
    free(pooled);
  }
done:
  if (!csum_or_null) free(csum);
  return rc;
}

/* ------------------------------------------------------------------ O7
 * p[t] = colmass[t] / (W H) is a distribution over the L keys (each of the W H
 * softmax rows sums to one).  ent = -sum p ln p, hn = ent / ln L in [0,1],
 * bucket = min(nb - 1, floor(hn nb)). */
static void risk_bucket(const double *colmass, int L, int W, int H, int nb, double *ent_out, int *bucket_out) {
  double ent = 0.0;
  for (int t = 0; t < L; ++t) {
    const double pt = colmass[t] / ((double)W * (double)H);
    if (pt > 0.0) ent -= pt * log(pt);
  }
  double hn = (L > 1) ? ent / log((double)L) : 0.0;
  int b = (int)floor(hn * (double)nb);
  if (b > nb - 1) b = nb - 1;
  if (b < 0) b = 0;
  *ent_out = ent;
  *bucket_out = b;
}

/* ------------------------------------------------------------------ O8
 * Split P prefix rows over Hkv heads in proportion to demands dem[g] >= 1,
 * every share held inside [f, n]:  x_g = clamp(lambda dem_g, f, n) with lambda
 * the water level at which the shares sum to P (unique shares because the sum
 * is continuous and non-decreasing in lambda).  All comparisons are between
 * integers.  The real shares of the unclamped heads are then rounded down and
 * the left-over rows go, one each, to the largest fractional parts, ties to the
 * lowest head index.  Requires f Hkv <= P <= n Hkv.  Returns 0 on success. */
int oracle_allocate(int Hkv, int64_t n, int64_t f, int64_t P, const int64_t *dem, int64_t *e) {
  if (Hkv < 1 || f < 0 || f > n || P < f * Hkv || P > n * Hkv) return 1;
  for (int g = 0; g < Hkv; ++g)
    if (dem[g] < 1) return 1;
  /* lambda = num/den runs over the break points f/dem_g and n/dem_g; at each
   * candidate level classify every head and test whether the level that makes
   * the unclamped heads absorb the rest lies in the same linear piece. */
  for (int cand = 0; cand < 2 * Hkv + 1; ++cand) {
    /* the piece just above break point `cand` (cand == 2 Hkv: the piece below all of them) */
    int64_t bn, bd; /* break point = bn / bd */
    if (cand == 2 * Hkv) {
      bn = 0;
      bd = 1;
    } else {
      bn = (cand < Hkv) ? f : n;
      bd = dem[cand % Hkv];
    }
    /* classify at a level infinitesimally above bn/bd:
       low  (share f): lambda dem_g <= f  <=> bn dem_g <  f bd   (strict: at equality the head is leaving the clamp)
       high (share n): lambda dem_g >= n  <=> bn dem_g >= n bd
       else free. */
    int64_t R = P, D = 0;
    int state[64];
    if (Hkv > 64) return 1;
    for (int g = 0; g < Hkv; ++g) {
      if (bn * dem[g] >= n * bd) {
        state[g] = 2;
        R -= n;
      } else if (bn * dem[g] < f * bd) {
        state[g] = 0;
        R -= f;
      } else {
        state[g] = 1;
        D += dem[g];
      }
    }
    int ok = 1;
    if (D == 0) {
      ok = (R == 0);
    } else {
      /* lambda* = R / D must keep every free head inside [f, n], every low head
         at or below f and every high head at or above n */
      if (R < 0) ok = 0;
      for (int g = 0; g < Hkv && ok; ++g) {
        const int64_t lhs = R * dem[g];
        if (state[g] == 1 && (lhs < f * D || lhs > n * D)) ok = 0;
        if (state[g] == 0 && lhs > f * D) ok = 0;
        if (state[g] == 2 && lhs < n * D) ok = 0;
      }
    }
    if (!ok) continue;
    int64_t given = 0;
    int64_t rem[64];
    for (int g = 0; g < Hkv; ++g) {
      if (state[g] == 0) {
        e[g] = f;
        rem[g] = -1;
      } else if (state[g] == 2) {
        e[g] = n;
        rem[g] = -1;
      } else {
        e[g] = (R * dem[g]) / D;
        rem[g] = (R * dem[g]) % D;
        given += e[g];
      }
    }
    /* hand the left-over rows out: the free heads in the order (larger fractional part first, lower head index
       first among equal parts) each take one row until none is left */
    int64_t left = (D > 0) ? R - given : 0;
    int order[64], n_free = 0;
    for (int g = 0; g < Hkv; ++g) {
      if (rem[g] < 0) continue;
      int at = n_free++;
      while (at > 0 && rem[order[at - 1]] < rem[g]) { /* strictly smaller parts move back: equal parts keep head order */
        order[at] = order[at - 1];
        --at;
      }
      order[at] = g;
    }
    if (left > n_free) return 3; /* cannot happen: the fractional parts sum to `left` and each is below one */
    for (int r = 0; r < left; ++r) {
      if (rem[order[r]] == 0) return 3;
      e[order[r]] += 1;
    }
    return 0;
  }
  return 2;
}

/* budgets [Nu,Hkv], offsets [Nu,Hkv+1], bucket [Nu], entropy [Nu], tau [Nu], counts [Nu,Hkv] (optional) */
int oracle_budget(const or_shape *s, const or_params *p, const double *scores, const double *colmass,
                  const float *sens, int32_t *budgets, int32_t *offsets, int32_t *bucket, double *entropy,
                  double *tau_out, int32_t *counts_or_null) {
  const int L = s->seq_len, W = s->window, H = s->n_q_heads, Hkv = s->n_kv_heads, Nu = s->n_units;
  const int n = L - W, B = p->budget_per_head, f = p->floor_per_head;
  if (p->n_buckets < 1 || Hkv > 64) return 1;
  if (B < L && (B < W || f > B - W || f < 0)) return 1;
  for (int u = 0; u < Nu; ++u) {
    double ent;
    int b;
    risk_bucket(colmass + (int64_t)u * L, L, W, H, p->n_buckets, &ent, &b);
    if (p->bucket_override >= 0) b = p->bucket_override < p->n_buckets ? p->bucket_override : p->n_buckets - 1;
    double tau;
    if (p->gate_layers > 0) { /* Alg. 1 (D): tau = T_gate[l, b_ent, b_ppl, B_l], row-major */
      if (!p->gate_coords || p->ppl_bins < 1 || p->budget_levels < 1) return 1;
      const int32_t *c = p->gate_coords + (int64_t)u * 3;
      const int l = c[0], bp = c[1], bb = c[2];
      if (l < 0 || l >= p->gate_layers || bp < 0 || bp >= p->ppl_bins || bb < 0 || bb >= p->budget_levels) return 1;
      tau = (double)sens[(((int64_t)l * p->n_buckets + b) * p->ppl_bins + bp) * p->budget_levels + bb];
    } else {
      tau = (double)sens[(p->sens_per_unit ? (int64_t)u * p->n_buckets : 0) + b];
    }
    bucket[u] = b;
    entropy[u] = ent;
    if (tau_out) tau_out[u] = tau;
    int64_t dem[64], e[64];
    for (int g = 0; g < Hkv; ++g) {
      const double *sc = scores + ((int64_t)u * Hkv + g) * (int64_t)n;
      int64_t c = 0;
      for (int t = 0; t < n; ++t) c += (sc[t] >= tau);
      if (counts_or_null) counts_or_null[(int64_t)u * Hkv + g] = (int32_t)c;
      int64_t lo = f > 1 ? f : 1;
      dem[g] = c < lo ? lo : (c > n ? n : c);
    }
    if (B >= L) {
      for (int g = 0; g < Hkv; ++g) e[g] = n; /* FullKV: the whole prefix, then the window */
    } else if (p->shared_elastic) {
      /* Eq. 8: all candidates when they fit the budget, else the Top-B of them (B counts the window here);
       * the floor argument still bounds the prefix part from below.  The heads' scores are identical. */
      const double *sc = scores + (int64_t)u * Hkv * (int64_t)n;
      int64_t c = 0;
      for (int t = 0; t < n; ++t) c += (sc[t] >= tau);
      int64_t keep = c < (int64_t)(B - W) ? c : (int64_t)(B - W);
      if (keep < f) keep = f;
      if (keep > n) keep = n;
      for (int g = 0; g < Hkv; ++g) e[g] = keep;
    } else {
      int rc = oracle_allocate(Hkv, n, f, (int64_t)Hkv * (B - W), dem, e);
      if (rc) return 10 + rc;
    }
    int32_t off = 0;
    for (int g = 0; g < Hkv; ++g) {
      budgets[(int64_t)u * Hkv + g] = (int32_t)(e[g] + W);
      offsets[(int64_t)u * (Hkv + 1) + g] = off;
      off += (int32_t)(e[g] + W);
    }
    offsets[(int64_t)u * (Hkv + 1) + Hkv] = off;
  }
  return 0;
}

/* ------------------------------------------------------------------ O9 */
typedef struct {
  double score;
  int32_t idx;
} or_item;

static int by_score_desc_then_index(const void *a, const void *b) {
  const or_item *x = (const or_item *)a, *y = (const or_item *)b;
  if (x->score > y->score) return -1;
  if (x->score < y->score) return 1;
  return (x->idx > y->idx) - (x->idx < y->idx);
}
static int by_index(const void *a, const void *b) {
  const or_item *x = (const or_item *)a, *y = (const or_item *)b;
  return (x->idx > y->idx) - (x->idx < y->idx);
}

/* indices [Nu, unit_rows]: unit u starts at u * unit_rows (unit_rows = Hkv min(B, L), which the
 * heads' budgets fill exactly unless the selection is elastic), head g at offsets[u,g]: the
 * budgets[g] - W best prefix positions in ascending order, then n .. L-1. */
int oracle_select(const or_shape *s, const double *scores, const int32_t *budgets, const int32_t *offsets,
                  int64_t unit_rows, int32_t *indices) {
  const int L = s->seq_len, W = s->window, Hkv = s->n_kv_heads, Nu = s->n_units, n = L - W;
  int err = 0;
#pragma omp parallel for collapse(2) schedule(dynamic)
  for (int u = 0; u < Nu; ++u)
    for (int g = 0; g < Hkv; ++g) {
      const int e = budgets[(int64_t)u * Hkv + g] - W;
      int32_t *out = indices + (int64_t)u * unit_rows + offsets[(int64_t)u * (Hkv + 1) + g];
      if (e < 0 || e > n) {
        err = 1;
        continue;
      }
      or_item *it = (or_item *)malloc(sizeof(or_item) * (size_t)(n > 0 ? n : 1));
      const double *sc = scores + ((int64_t)u * Hkv + g) * (int64_t)n;
      for (int t = 0; t < n; ++t) {
        it[t].score = sc[t];
        it[t].idx = t;
      }
      qsort(it, (size_t)n, sizeof(or_item), by_score_desc_then_index);
      qsort(it, (size_t)e, sizeof(or_item), by_index);
      for (int j = 0; j < e; ++j) out[j] = it[j].idx;
      for (int i = 0; i < W; ++i) out[e + i] = n + i;
      free(it);
    }
  return err;
}

/* ------------------------------------------------------------------ O10 */
int oracle_gather(const or_shape *s, const void *k, const void *v, const int32_t *indices, const int32_t *budgets,
                  const int32_t *offsets, int64_t unit_rows, void *k_out, void *v_out) {
  const int L = s->seq_len, d = s->head_dim, Hkv = s->n_kv_heads, Nu = s->n_units;
  const size_t esz = s->dtype == OR_F32 ? 4 : 2, row = esz * (size_t)d;
  for (int u = 0; u < Nu; ++u) {
    for (int g = 0; g < Hkv; ++g) {
      const int64_t o = (int64_t)u * unit_rows + offsets[(int64_t)u * (Hkv + 1) + g];
      for (int j = 0; j < budgets[(int64_t)u * Hkv + g]; ++j) {
        const int32_t t = indices[o + j];
        if (t < 0 || t >= L) return 1;
        const size_t src = (((size_t)u * Hkv + g) * (size_t)L + (size_t)t) * row;
        memcpy((char *)k_out + (size_t)(o + j) * row, (const char *)k + src, row);
        memcpy((char *)v_out + (size_t)(o + j) * row, (const char *)v + src, row);
      }
    }
  }
  return 0;
}

/* ------------------------------------------------------------------ whole pass
 * Outputs are sized for B' = min(B, L) rows per KV head:
 * k_out, v_out [Nu, Hkv B', d]; indices [Nu, Hkv B']; budgets [Nu,Hkv];
 * offsets [Nu,Hkv+1]; scores [Nu,Hkv,n] (fp64, optional). */
int oracle_compress(const or_shape *s, const or_params *p, const void *q, const void *k, const void *v,
                    const float *head_w, const float *sens, void *k_out, void *v_out, int32_t *indices,
                    int32_t *budgets, int32_t *offsets, int32_t *bucket, double *entropy, double *scores_or_null) {
  const int L = s->seq_len, W = s->window, Hkv = s->n_kv_heads, Nu = s->n_units, n = L - W;
  double *scores = scores_or_null ? scores_or_null : (double *)malloc(sizeof(double) * (size_t)Nu * Hkv * (n > 0 ? n : 1));
  double *colmass = (double *)malloc(sizeof(double) * (size_t)Nu * L);
  double *rho = p->value_norm ? (double *)malloc(sizeof(double) * (size_t)Nu * Hkv * L) : NULL;
  int rc = 2;
  if (scores && colmass && (rho || !p->value_norm)) {
    rc = rho ? oracle_vnorm(s, v, (double)p->value_norm_eps, rho) : 0;
    if (!rc) rc = oracle_score(s, p, q, k, head_w, rho, scores, colmass, NULL);
    if (!rc) rc = oracle_budget(s, p, scores, colmass, sens, budgets, offsets, bucket, entropy, NULL, NULL);
    const int64_t unit_rows = (int64_t)Hkv * (p->budget_per_head < L ? p->budget_per_head : L);
    if (!rc) rc = oracle_select(s, scores, budgets, offsets, unit_rows, indices);
    if (!rc) rc = oracle_gather(s, k, v, indices, budgets, offsets, unit_rows, k_out, v_out);
  }
  if (!scores_or_null) free(scores);
  free(colmass);
  free(rho);
  return rc;
}

/* ------------------------------------------------------------------ decode-side check (Prop. 4.1)
 * Softmax attention of n_dec decode queries per query head over a K/V array.  A decode query comes after the
 * prompt and sees every row.  compressed == 0: the rows are all L tokens of k, v [Nu,Hkv,L,d].  compressed == 1:
 * k, v are the gathered k_out, v_out [Nu, unit_rows, d] and head g of unit u owns budgets[u,g] rows from row
 * offsets[u,g].  out[u,h,j,:] = sum_t p_t v_t with p = softmax(q.k_t / sqrt d);  lse[u,h,j] = ln sum_t exp(q.k_t / sqrt d).
 * The mass a restriction to a subset S keeps is sum_{t in S} p_t = exp(lse_S - lse_all). */
int oracle_attend(const or_shape *s, const void *q_dec, int n_dec, const void *k, const void *v, int compressed,
                  const int32_t *budgets, const int32_t *offsets, int64_t unit_rows, double *out, double *lse) {
  const int L = s->seq_len, H = s->n_q_heads, Hkv = s->n_kv_heads, G = H / Hkv, d = s->head_dim;
#pragma omp parallel for collapse(2) schedule(dynamic)
  for (int u = 0; u < s->n_units; ++u)
    for (int h = 0; h < H; ++h) {
      const int g = h / G;
      const int64_t rows = compressed ? budgets[(int64_t)u * Hkv + g] : L;
      const int64_t base = compressed ? (int64_t)u * unit_rows + offsets[(int64_t)u * (Hkv + 1) + g]
                                      : ((int64_t)u * Hkv + g) * (int64_t)L;
      double *x = (double *)malloc(sizeof(double) * (size_t)(rows > 0 ? rows : 1));
      for (int j = 0; j < n_dec; ++j) {
        const int64_t qo = (((int64_t)u * H + h) * n_dec + j) * d;
        double mx = -INFINITY;
        for (int64_t t = 0; t < rows; ++t) {
          double dot = 0.0;
          for (int c = 0; c < d; ++c) dot += widen(q_dec, s->dtype, qo + c) * widen(k, s->dtype, (base + t) * d + c);
          x[t] = dot / sqrt((double)d);
          if (x[t] > mx) mx = x[t];
        }
        double z = 0.0;
        for (int64_t t = 0; t < rows; ++t) z += exp(x[t] - mx);
        double *o = out + qo;
        for (int c = 0; c < d; ++c) o[c] = 0.0;
        for (int64_t t = 0; t < rows; ++t) {
          const double p = exp(x[t] - mx) / z;
          for (int c = 0; c < d; ++c) o[c] += p * widen(v, s->dtype, (base + t) * d + c);
        }
        lse[((int64_t)u * H + h) * n_dec + j] = mx + log(z);
      }
      free(x);
    }
  return 0;
}

/* ------------------------------------------------------------------ diagnostic (Prop. 4.1)
 * kept[u,h,i] = sum_{t in S_g} A[h,i,t]: attention mass of window row i that
 * survives the selection; the discarded mass is m = 1 - kept. */
int oracle_kept_mass(const or_shape *s, const void *q, const void *k, const int32_t *indices, const int32_t *budgets,
                     const int32_t *offsets, int64_t unit_rows, double *kept) {
  const int L = s->seq_len, W = s->window, H = s->n_q_heads, Hkv = s->n_kv_heads, G = H / Hkv;
#pragma omp parallel for collapse(2) schedule(dynamic)
  for (int u = 0; u < s->n_units; ++u)
    for (int h = 0; h < H; ++h) {
      const int g = h / G;
      double *row = (double *)malloc(sizeof(double) * (size_t)L);
      const int32_t *idx = indices + (int64_t)u * unit_rows + offsets[(int64_t)u * (Hkv + 1) + g];
      for (int i = 0; i < W; ++i) {
        attention_row(s, q, k, u, h, i, row);
        double a = 0.0;
        for (int j = 0; j < budgets[(int64_t)u * Hkv + g]; ++j) a += row[idx[j]];
        kept[((int64_t)u * H + h) * W + i] = a;
      }
      free(row);
    }
  return 0;
}

/* ------------------------------------------------------------------ depth mapping of a compiled table
 * A table compiled for n_src layers is reused on a model of n_dst layers by relative depth (the appendix on
 * cross-architecture use: "monotonic depth mapping, e.g. relative-depth interpolation"): target layer l sits
 * at relative depth r = l / (n_dst - 1), i.e. at position x = r (n_src - 1) of the source's layer axis, and
 * takes the linear interpolation of the two source rows around x.  First and last layers map onto first and
 * last; n_dst == n_src is the identity.  src [n_src,row], dst [n_dst,row], fp32 tables, arithmetic in double. */
int oracle_depth_map(const float *src, int n_src, int n_dst, int64_t row, float *dst) {
  if (n_src < 1 || n_dst < 1 || row < 1) return 1;
  for (int l = 0; l < n_dst; ++l) {
    const double x = (n_dst > 1) ? (double)l * (double)(n_src - 1) / (double)(n_dst - 1) : 0.0;
    int lo = (int)floor(x);
    if (lo > n_src - 1) lo = n_src - 1;
    const int hi = lo + 1 < n_src ? lo + 1 : n_src - 1;
    const double w = x - (double)lo;
    for (int64_t c = 0; c < row; ++c)
      dst[(int64_t)l * row + c] = (float)((1.0 - w) * (double)src[(int64_t)lo * row + c] + w * (double)src[(int64_t)hi * row + c]);
  }
  return 0;
}

int oracle_num_threads(void) {
  int nt = 1;
#ifdef _OPENMP
#pragma omp parallel
  {
#pragma omp single
    nt = omp_get_num_threads();
  }
#endif
  return nt;
}
