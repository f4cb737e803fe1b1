/*
 * MixKV prefill KV-cache compression -- plain CPU oracle.
 *
 * THIS FILE IS TEST INFRASTRUCTURE.  It exists so that the CUDA library can be
 * checked against something written straight from the paper.  Only the test
 * suite, the smoke check and the benchmark's cpu_baseline leg may call it; the
 * product never does, and it shares no code, header, table or helper with the
 * CUDA path (it has its own parameter struct and its own bf16 widening).
 *
 * Everything is computed the slow, obvious way: bf16 inputs are widened exactly
 * to double, all sums are double, every step is a plain loop in the order the
 * paper gives it (Sec. 3.2, Sec. 3.3, Eq. 2-5, Algorithm 1).  Scores are rounded
 * to float only when they are handed back; the top-B decision is then taken on
 * those float scores (the precision the library itself selects in).
 *
 * Parity pins (checked by the CPU tests): softmax rows sum to 1, zero queries give
 * the closed-form harmonic score, the attention mass of a head sums to G, Eq. 4
 * against the brute-force off-diagonal mean of the cosine matrix, the diversity
 * score against the brute-force mean cosine, the normalisation invariants of
 * Sec. 3.2 / 3.3, the r = 0 / r = 1 limits of Eq. 5, budget >= L keeping every
 * row, brute-force sorting for the top-B, and equality with an independently
 * written plain SnapKV selector when the mix degenerates to pure importance.
 * Parity unpinned: the head-adaptive ("AdaKV-style") budget split -- the paper
 * gives it one sentence and no formula; the rule implemented here is this
 * build's reading and is pinned only by its own invariants (budgets sum to the
 * total, floor = 1 reduces to fixed budgets, brute force on tiny inputs).
 *
 * Layouts (row-major):
 *   K, V   [H, Ltot, d]        bf16 bit patterns, sequences concatenated along Ltot
 *   Q      [batch, H*G, W, d]  last W queries of each sequence; query head q
 *                              belongs to KV head q / G
 *   cu     [batch + 1]         sequence offsets into Ltot
 *   scores [H, Ptot]           Ptot = Ltot - batch*W; sequence b's prefix starts at
 *                              cu[b] - b*W and has P_b = L_b - W entries
 *   rbar   [batch, H]
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef struct {
  int32_t kv_heads;      /* H */
  int32_t gqa_ratio;     /* G */
  int32_t head_dim;      /* d */
  int32_t window;        /* W, observation window (Sec. 3.2, default 32) */
  int32_t pool_kernel;   /* odd, 1 = no pooling */
  int32_t pool_mode;     /* 0 = average (zero padded), 1 = max */
  int32_t use_vnorm;     /* intrinsic term of Eq. 2: 1 = VNorm (the default), 2 = KNorm (minus the
                            key norm, Sec. 3.2), 0 = none */
  int32_t mix_mode;      /* 0 Eq. 5, 1 importance only, 2 diversity only, 3 plain sum */
  int32_t budget_mode;   /* 0 fixed B per head, 1 head-adaptive under a total of B*H */
  int32_t budget;        /* B: rows kept per head INCLUDING the W window rows */
  double ada_floor;      /* adaptive: fraction of (B - W) guaranteed to each head */
  double eps;            /* the epsilon of Sec. 3.2 / 3.3 */
  double softmax_scale;  /* 0 => 1/sqrt(d) */
} oracle_params;

int mixkv_oracle_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

void mixkv_oracle_set_threads(int n) {
#ifdef _OPENMP
  if (n > 0) omp_set_num_threads(n);
#else
  (void)n;
#endif
}

static double widen(uint16_t bits) {
  union { uint32_t u; float f; } x;
  x.u = ((uint32_t)bits) << 16;
  return (double)x.f;
}

/* ------------------------------------------------------------------ Sec. 3.2
 * Extrinsic importance: attention of the W window queries of the G query heads
 * of one KV head to every key, averaged over the window and summed over the
 * group.  Query row j (0-based inside the window) sits at sequence position
 * P + j, so it sees keys 0 .. P + j (causal).  The softmax runs over all the
 * keys the row may see.  s_ex_raw has L entries (the window columns are kept so
 * that the total mass G can be checked); row_sums (optional) has G*W entries. */
void mixkv_oracle_window_attention(const uint16_t* Kh, const uint16_t* Qg, int G, int W, int L,
                                   int d, double scale, double* s_ex_raw, double* row_sums) {
  const int P = L - W;
  const int rows = G * W;
  double* A = (double*)malloc((size_t)rows * (size_t)L * sizeof(double));
#pragma omp parallel for schedule(static)
  for (int r = 0; r < rows; ++r) {
    const int j = r % W;
    const int allowed = P + j + 1; /* keys 0 .. P+j */
    const uint16_t* q = Qg + (size_t)r * d;
    double* a = A + (size_t)r * L;
    double m = -INFINITY;
    for (int i = 0; i < allowed; ++i) {
      const uint16_t* k = Kh + (size_t)i * d;
      double dot = 0.0;
      for (int c = 0; c < d; ++c) dot += widen(q[c]) * widen(k[c]);
      a[i] = dot * scale;
      if (a[i] > m) m = a[i];
    }
    double Z = 0.0;
    for (int i = 0; i < allowed; ++i) {
      a[i] = exp(a[i] - m);
      Z += a[i];
    }
    double rs = 0.0;
    for (int i = 0; i < allowed; ++i) {
      a[i] /= Z;
      rs += a[i];
    }
    for (int i = allowed; i < L; ++i) a[i] = 0.0;
    if (row_sums) row_sums[r] = rs;
  }
#pragma omp parallel for schedule(static)
  for (int i = 0; i < L; ++i) {
    double acc = 0.0;
    for (int g = 0; g < G; ++g) {
      double mean_w = 0.0;
      for (int j = 0; j < W; ++j) mean_w += A[((size_t)g * W + j) * L + i];
      acc += mean_w / (double)W; /* window mean (Sec. 3.2), then the GQA sum */
    }
    s_ex_raw[i] = acc;
  }
  free(A);
}

/* 1-D pooling over n entries, stride 1, half-width k/2.  Average pooling pads with
 * zeros and always divides by k; max pooling looks at in-range neighbours only. */
void mixkv_oracle_pool(const double* in, int n, int k, int mode, double* out) {
  const int half = k / 2;
  for (int i = 0; i < n; ++i) {
    if (mode == 0) {
      double s = 0.0;
      for (int t = -half; t <= half; ++t) {
        const int p = i + t;
        if (p >= 0 && p < n) s += in[p];
      }
      out[i] = s / (double)k;
    } else {
      double m = -INFINITY;
      for (int t = -half; t <= half; ++t) {
        const int p = i + t;
        if (p >= 0 && p < n && in[p] > m) m = in[p];
      }
      out[i] = m;
    }
  }
}

/* VNorm (Sec. 3.2): the l2 norm of each value row. */
void mixkv_oracle_row_norms(const uint16_t* X, int n, int d, double* out) {
  for (int i = 0; i < n; ++i) {
    double s = 0.0;
    for (int c = 0; c < d; ++c) {
      const double v = widen(X[(size_t)i * d + c]);
      s += v * v;
    }
    out[i] = sqrt(s);
  }
}

/* Sec. 3.2 "Diversity Metrics" and Sec. 3.3 Eq. 3-4, over all L keys of one head:
 * unit keys, their mean, the diversity score -cos(key, mean key) and the
 * off-diagonal mean similarity in closed form.  A zero key normalises to zero. */
void mixkv_oracle_key_geometry(const uint16_t* Kh, int L, int d, double* s_div, double* rbar,
                               double* kbar_out) {
  double* khat = (double*)malloc((size_t)L * d * sizeof(double));
  double* kbar = (double*)calloc((size_t)d, sizeof(double));
  for (int i = 0; i < L; ++i) {
    double s = 0.0;
    for (int c = 0; c < d; ++c) {
      const double v = widen(Kh[(size_t)i * d + c]);
      s += v * v;
    }
    double nrm = sqrt(s);
    if (nrm < 1e-12) nrm = 1e-12;
    for (int c = 0; c < d; ++c) khat[(size_t)i * d + c] = widen(Kh[(size_t)i * d + c]) / nrm;
  }
  for (int i = 0; i < L; ++i)
    for (int c = 0; c < d; ++c) kbar[c] += khat[(size_t)i * d + c];
  for (int c = 0; c < d; ++c) kbar[c] /= (double)L;
  double nk2 = 0.0;
  for (int c = 0; c < d; ++c) nk2 += kbar[c] * kbar[c];
  const double T = (double)L;
  *rbar = (T * T * nk2 - T) / (T * (T - 1.0)); /* Eq. 4 */
  for (int i = 0; i < L; ++i) {
    double dot = 0.0;
    for (int c = 0; c < d; ++c) dot += khat[(size_t)i * d + c] * kbar[c];
    s_div[i] = -dot;
  }
  if (kbar_out) memcpy(kbar_out, kbar, (size_t)d * sizeof(double));
  free(khat);
  free(kbar);
}

static void min_max_mean(const double* x, int n, double* mn, double* mx, double* mean) {
  double lo = INFINITY, hi = -INFINITY, s = 0.0;
  for (int i = 0; i < n; ++i) {
    if (x[i] < lo) lo = x[i];
    if (x[i] > hi) hi = x[i];
    s += x[i];
  }
  *mn = lo;
  *mx = hi;
  *mean = s / (double)n;
}

/* Eq. 2 and Eq. 5 over the P candidate positions of one head.
 *   s_in_norm   = (n - min n) / (max n - min n + eps)
 *   s_in_scaled = s_in_norm * mean(s_ex) / (mean(s_in_norm) + eps)
 *   s_imp       = s_ex + s_in_scaled                       (Eq. 2; s_ex if VNorm is off)
 *   s_div_norm  = (s_div - min) / (max - min + eps)
 *   s_div_scaled= s_div_norm * mean(s_imp) / (mean(s_div_norm) + eps)
 *   s_comp      = (1 - r) s_imp + r s_div_scaled           (Eq. 5)
 * vnorm may be NULL when use_vnorm is 0.  Optional outputs may be NULL. */
void mixkv_oracle_mix(const double* s_ex, const double* vnorm, const double* s_div, int P,
                      double rbar, int use_vnorm, int mix_mode, double eps, double* s_comp,
                      double* s_imp_out, double* s_div_scaled_out, double* s_in_scaled_out) {
  double* s_imp = (double*)malloc((size_t)P * sizeof(double));
  double* tmp = (double*)malloc((size_t)P * sizeof(double));
  double mn, mx, mean;
  if (use_vnorm) {
    min_max_mean(vnorm, P, &mn, &mx, &mean);
    for (int i = 0; i < P; ++i) tmp[i] = (vnorm[i] - mn) / (mx - mn + eps);
    double mean_in = 0.0, mean_ex = 0.0;
    for (int i = 0; i < P; ++i) {
      mean_in += tmp[i];
      mean_ex += s_ex[i];
    }
    mean_in /= (double)P;
    mean_ex /= (double)P;
    for (int i = 0; i < P; ++i) {
      const double s_in_scaled = tmp[i] * (mean_ex / (mean_in + eps));
      if (s_in_scaled_out) s_in_scaled_out[i] = s_in_scaled;
      s_imp[i] = s_ex[i] + s_in_scaled;
    }
  } else {
    for (int i = 0; i < P; ++i) {
      s_imp[i] = s_ex[i];
      if (s_in_scaled_out) s_in_scaled_out[i] = 0.0;
    }
  }
  min_max_mean(s_div, P, &mn, &mx, &mean);
  double mean_imp = 0.0, mean_dn = 0.0;
  for (int i = 0; i < P; ++i) {
    tmp[i] = (s_div[i] - mn) / (mx - mn + eps);
    mean_dn += tmp[i];
    mean_imp += s_imp[i];
  }
  mean_dn /= (double)P;
  mean_imp /= (double)P;
  for (int i = 0; i < P; ++i) {
    const double s_div_scaled = tmp[i] * (mean_imp / (mean_dn + eps));
    if (s_div_scaled_out) s_div_scaled_out[i] = s_div_scaled;
    double c;
    switch (mix_mode) {
      case 0: c = (1.0 - rbar) * s_imp[i] + rbar * s_div_scaled; break; /* Eq. 5 */
      case 1: c = s_imp[i]; break;                                      /* importance only */
      case 2: c = s_div[i]; break;                                      /* diversity only */
      default: c = s_imp[i] + s_div_scaled; break;                      /* plain sum */
    }
    s_comp[i] = c;
    if (s_imp_out) s_imp_out[i] = s_imp[i];
  }
  free(s_imp);
  free(tmp);
}

static int check_params(const oracle_params* p, const int32_t* cu, int batch) {
  if (!p || !cu || batch < 1) return -1;
  if (p->kv_heads < 1 || p->gqa_ratio < 1 || p->head_dim < 1 || p->window < 1) return -1;
  if (p->pool_kernel < 1 || (p->pool_kernel % 2) == 0) return -1;
  for (int b = 0; b < batch; ++b) {
    const int L = cu[b + 1] - cu[b];
    if (L < p->window + 1 || L < 2) return -1;
  }
  return 0;
}

/* Score every candidate key of one layer (Algorithm 1, step 1 and the mixing half of
 * step 2).  Outputs are float; any of s_ex (pooled), s_ex_raw, s_div, rbar may be NULL.
 * rbar_in (optional, [batch, H]) replaces the per-sample redundancy (the offline
 * head-weight variant of Sec. 4.3). */
int mixkv_oracle_scores(const uint16_t* K, const uint16_t* V, const uint16_t* Q, const int32_t* cu,
                        int batch, const oracle_params* p, float* s_comp, float* s_ex,
                        float* s_ex_raw, float* s_div, float* rbar, const float* rbar_in) {
  if (check_params(p, cu, batch) != 0) return -1;
  const int H = p->kv_heads, G = p->gqa_ratio, d = p->head_dim, W = p->window;
  const int64_t Ltot = cu[batch];
  const int64_t Ptot = Ltot - (int64_t)batch * W;
  const double scale = p->softmax_scale > 0.0 ? p->softmax_scale : 1.0 / sqrt((double)d);
  for (int b = 0; b < batch; ++b) {
    const int L = cu[b + 1] - cu[b];
    const int P = L - W;
    const int64_t poff = (int64_t)cu[b] - (int64_t)b * W;
    for (int h = 0; h < H; ++h) {
      const uint16_t* Kh = K + ((size_t)h * Ltot + cu[b]) * d;
      const uint16_t* Vh = V ? V + ((size_t)h * Ltot + cu[b]) * d : NULL;
      const uint16_t* Qg = Q + (((size_t)b * H + h) * G) * (size_t)W * d;
      double* ex_raw = (double*)malloc((size_t)L * sizeof(double));
      double* ex = (double*)malloc((size_t)P * sizeof(double));
      double* dv = (double*)malloc((size_t)L * sizeof(double));
      double* vn = (double*)malloc((size_t)P * sizeof(double));
      double* comp = (double*)malloc((size_t)P * sizeof(double));
      double r;
      mixkv_oracle_window_attention(Kh, Qg, G, W, L, d, scale, ex_raw, NULL);
      mixkv_oracle_pool(ex_raw, P, p->pool_kernel, p->pool_mode, ex); /* prefix only */
      mixkv_oracle_key_geometry(Kh, L, d, dv, &r, NULL);               /* all L keys */
      if (p->use_vnorm == 1) mixkv_oracle_row_norms(Vh, P, d, vn);       /* VNorm (default) */
      if (p->use_vnorm == 2) {                                           /* KNorm: minus the key norm */
        mixkv_oracle_row_norms(Kh, P, d, vn);
        for (int i = 0; i < P; ++i) vn[i] = -vn[i];
      }
      const double r_mix = rbar_in ? (double)rbar_in[(size_t)b * H + h] : r;
      mixkv_oracle_mix(ex, p->use_vnorm ? vn : NULL, dv, P, r_mix, p->use_vnorm, p->mix_mode,
                       p->eps, comp, NULL, NULL, NULL);
      float* o = s_comp + (size_t)h * Ptot + poff;
      for (int i = 0; i < P; ++i) o[i] = (float)comp[i];
      if (s_ex)
        for (int i = 0; i < P; ++i) s_ex[(size_t)h * Ptot + poff + i] = (float)ex[i];
      if (s_ex_raw)
        for (int i = 0; i < P; ++i) s_ex_raw[(size_t)h * Ptot + poff + i] = (float)ex_raw[i];
      if (s_div)
        for (int i = 0; i < P; ++i) s_div[(size_t)h * Ptot + poff + i] = (float)dv[i];
      if (rbar) rbar[(size_t)b * H + h] = (float)r;
      free(ex_raw); free(ex); free(dv); free(vn); free(comp);
    }
  }
  return 0;
}

/* ------------------------------------------------------------------ selection */
typedef struct { float s; int64_t pos; } scored;

static int by_score_then_pos(const void* a, const void* b) {
  const scored* x = (const scored*)a;
  const scored* y = (const scored*)b;
  if (x->s > y->s) return -1;
  if (x->s < y->s) return 1;
  return (x->pos > y->pos) - (x->pos < y->pos);
}

static int by_pos(const void* a, const void* b) {
  const scored* x = (const scored*)a;
  const scored* y = (const scored*)b;
  return (x->pos > y->pos) - (x->pos < y->pos);
}

/* TopB of Sec. 3.1: the b highest scores among n, ties to the lower position,
 * returned in ascending position order. */
void mixkv_oracle_topb(const float* s, int n, int b, int32_t* idx) {
  scored* t = (scored*)malloc((size_t)n * sizeof(scored));
  for (int i = 0; i < n; ++i) { t[i].s = s[i]; t[i].pos = i; }
  qsort(t, (size_t)n, sizeof(scored), by_score_then_pos);
  qsort(t, (size_t)b, sizeof(scored), by_pos);
  for (int i = 0; i < b; ++i) idx[i] = (int32_t)t[i].pos;
  free(t);
}

/* Budgets of one sequence (Algorithm 1: B' = B - W candidates kept per head).
 * Fixed: every head gets min(B - W, P).  Adaptive (the reading taken here of the
 * one-sentence AdaKV description): each head is guaranteed f = floor(floor_frac *
 * (B - W)); the remaining H * (B - W - f) slots go to the globally highest scores
 * of the H heads together (ties to the lower (head, position)); head h gets
 * min(f + its share, P). */
void mixkv_oracle_budgets(const float* scores, int64_t head_stride, int H, int P, int W, int B,
                          int budget_mode, double ada_floor, int32_t* b_h) {
  const int Bp = B - W;
  if (budget_mode == 0) {
    for (int h = 0; h < H; ++h) b_h[h] = Bp < P ? Bp : P;
    return;
  }
  int f = (int)floor(ada_floor * (double)Bp);
  if (f > Bp) f = Bp;
  if (f < 0) f = 0;
  int64_t N = (int64_t)H * (Bp - f);
  const int64_t total = (int64_t)H * P;
  if (N > total) N = total;
  scored* t = (scored*)malloc((size_t)total * sizeof(scored));
  for (int h = 0; h < H; ++h)
    for (int i = 0; i < P; ++i) {
      t[(size_t)h * P + i].s = scores[(size_t)h * head_stride + i];
      t[(size_t)h * P + i].pos = (int64_t)h * P + i;
    }
  qsort(t, (size_t)total, sizeof(scored), by_score_then_pos);
  for (int h = 0; h < H; ++h) b_h[h] = f;
  for (int64_t n = 0; n < N; ++n) b_h[t[n].pos / P] += 1;
  for (int h = 0; h < H; ++h)
    if (b_h[h] > P) b_h[h] = P;
  free(t);
}

/* Select on given scores [H, Ptot].  counts [batch*H]; idx is packed in (b, h) order,
 * idx_offsets [batch*H + 1] is the exclusive prefix sum of counts. */
int mixkv_oracle_select(const float* scores, const int32_t* cu, int batch, const oracle_params* p,
                        int32_t* idx, int32_t* counts, int32_t* idx_offsets) {
  if (check_params(p, cu, batch) != 0 || p->budget <= p->window) return -1;
  const int H = p->kv_heads, W = p->window;
  const int64_t Ptot = (int64_t)cu[batch] - (int64_t)batch * W;
  int32_t off = 0;
  for (int b = 0; b < batch; ++b) {
    const int P = cu[b + 1] - cu[b] - W;
    const int64_t poff = (int64_t)cu[b] - (int64_t)b * W;
    int32_t* bh = counts + (size_t)b * H;
    mixkv_oracle_budgets(scores + poff, Ptot, H, P, W, p->budget, p->budget_mode, p->ada_floor, bh);
    for (int h = 0; h < H; ++h) {
      idx_offsets[(size_t)b * H + h] = off;
      mixkv_oracle_topb(scores + (size_t)h * Ptot + poff, P, bh[h], idx + off);
      off += bh[h];
    }
  }
  idx_offsets[(size_t)batch * H] = off;
  return 0;
}

/* Gather (Algorithm 1, last step): for every (b, h) the selected prefix rows in
 * ascending position order, then the W window rows.  Output rows are packed in
 * (b, h) order; out_row_offsets [batch*H + 1]. */
void mixkv_oracle_gather(const uint16_t* X, const int32_t* cu, int batch, int H, int d, int W,
                         const int32_t* idx, const int32_t* idx_offsets, uint16_t* X_out,
                         int32_t* out_row_offsets) {
  const int64_t Ltot = cu[batch];
  int64_t row = 0;
  for (int b = 0; b < batch; ++b) {
    const int L = cu[b + 1] - cu[b];
    const int P = L - W;
    for (int h = 0; h < H; ++h) {
      const int bh = b * H + h;
      const uint16_t* Xh = X + ((size_t)h * Ltot + cu[b]) * d;
      if (out_row_offsets) out_row_offsets[bh] = (int32_t)row;
      for (int32_t n = idx_offsets[bh]; n < idx_offsets[bh + 1]; ++n, ++row)
        memcpy(X_out + (size_t)row * d, Xh + (size_t)idx[n] * d, (size_t)d * sizeof(uint16_t));
      for (int j = 0; j < W; ++j, ++row)
        memcpy(X_out + (size_t)row * d, Xh + (size_t)(P + j) * d, (size_t)d * sizeof(uint16_t));
    }
  }
  if (out_row_offsets) out_row_offsets[(size_t)batch * H] = (int32_t)row;
}

/* The whole per-layer step: score, select, gather. */
int mixkv_oracle_compress_layer(const uint16_t* K, const uint16_t* V, const uint16_t* Q,
                                const int32_t* cu, int batch, const oracle_params* p,
                                const float* rbar_in, float* s_comp, uint16_t* K_out,
                                uint16_t* V_out, int32_t* out_row_offsets, int32_t* idx,
                                int32_t* counts, int32_t* idx_offsets) {
  int rc = mixkv_oracle_scores(K, V, Q, cu, batch, p, s_comp, NULL, NULL, NULL, NULL, rbar_in);
  if (rc) return rc;
  rc = mixkv_oracle_select(s_comp, cu, batch, p, idx, counts, idx_offsets);
  if (rc) return rc;
  mixkv_oracle_gather(K, cu, batch, p->kv_heads, p->head_dim, p->window, idx, idx_offsets, K_out,
                      out_row_offsets);
  mixkv_oracle_gather(V, cu, batch, p->kv_heads, p->head_dim, p->window, idx, idx_offsets, V_out,
                      NULL);
  return 0;
}
