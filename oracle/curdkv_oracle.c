/*
 * CurDKV / AdaCurDKV oracle -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.
 *
 * A plain, slow, fp64 CPU statement of the prefill-time KV selection of
 * "Value-Guided KV Compression for LLMs via Approximated CUR Decomposition"
 * (Algorithm 1 and the "Adaptive budget allocation" paragraph of Sec. 3.2).
 * Only tests, the smoke check and the benchmark's cpu-baseline leg may call it.
 * It shares no code with the CUDA path and is never tuned for speed: naive
 * loops in the order the algorithm states them, fp64 throughout, full sorts
 * for every top-k.  The only parallelism is OpenMP across independent
 * (batch, KV head) problems.
 *
 * Pins (see tests/test_oracle_*.py): orthogonal-G closed form, chi-square
 * moments of the sketch, SVD leverage scores on flat-spectrum matrices,
 * sum-to-one / scale / permutation invariants, brute-force top-k, hand-made
 * tie cases, AdaCurDKV special cases (alpha = 1, one head, all mass in one
 * head).  Unpinned: selection on real model activations (the paper prints no
 * worked numeric example) -- "parity unpinned" for that case only.
 *
 * Layout conventions (all host memory):
 *   K, V     : bf16 stored as uint16_t, element (b,h,j,c) at
 *              b*stride_b + h*stride_h + j*stride_n + c   (strides in elements)
 *   G        : fp32 [d][r] row-major (g_per_head = 0) or [H][d][r]
 *   seqlens  : int32 [B] or NULL (every sequence has n_max rows)
 *   scores   : fp64 [B][H][n_max]; entries j >= n_b are written as 0
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

static double bf16_to_f64(uint16_t x) {
  uint32_t u = ((uint32_t)x) << 16;
  float f;
  memcpy(&f, &u, sizeof f);
  return (double)f;
}

static int clampi(int x, int lo, int hi) { return x < lo ? lo : (x > hi ? hi : x); }

static int seq_len(const int32_t *seqlens, int b, int n_max) {
  return seqlens ? clampi(seqlens[b], 0, n_max) : n_max;
}

/* ------------------------------------------------------------------------
 * Algorithm 1, scoring steps: sketch, squared row norms, product, normalise.
 *   score_mode 0: l = lK * lV (paper default)   1: l = lK   2: l = lV
 *   use_projection 0: rows are used as they are (ablation of App. C.3)
 * Optional outputs lK, lV (fp64 [B][H][n_max]) may be NULL.
 * ---------------------------------------------------------------------- */
static void row_score(const uint16_t *row, int d, const float *G, int r, int use_projection,
                      double *out) {
  double acc = 0.0;
  if (use_projection) {
    for (int c = 0; c < r; ++c) {          /* y_c = sum_t a_t G[t][c] */
      double y = 0.0;
      for (int t = 0; t < d; ++t) y += bf16_to_f64(row[t]) * (double)G[(size_t)t * r + c];
      acc += y * y;                        /* l_j = ||a_j G||_2^2 */
    }
  } else {
    for (int t = 0; t < d; ++t) {
      double a = bf16_to_f64(row[t]);
      acc += a * a;
    }
  }
  *out = acc;
}

void oracle_score(const uint16_t *K, const uint16_t *V, int B, int H, int n_max, int d,
                  int64_t ksb, int64_t ksh, int64_t ksn, int64_t vsb, int64_t vsh, int64_t vsn,
                  const int32_t *seqlens, const float *G, int r, int g_per_head, int score_mode,
                  int use_projection, double *scores, double *head_sums, double *lK_out,
                  double *lV_out) {
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
  for (int b = 0; b < B; ++b) {
    for (int h = 0; h < H; ++h) {
      const int n = seq_len(seqlens, b, n_max);
      const float *Gh = g_per_head ? G + (size_t)h * d * r : G;
      double *sc = scores + ((size_t)b * H + h) * n_max;
      double *lKo = lK_out ? lK_out + ((size_t)b * H + h) * n_max : NULL;
      double *lVo = lV_out ? lV_out + ((size_t)b * H + h) * n_max : NULL;
      double S = 0.0;
      for (int j = 0; j < n; ++j) {
        double lK, lV, l;
        row_score(K + b * ksb + h * ksh + j * ksn, d, Gh, r, use_projection, &lK);
        row_score(V + b * vsb + h * vsh + j * vsn, d, Gh, r, use_projection, &lV);
        l = score_mode == 1 ? lK : (score_mode == 2 ? lV : lK * lV);
        sc[j] = l;
        if (lKo) lKo[j] = lK;
        if (lVo) lVo[j] = lV;
        S += l;                            /* over all n tokens, forced ones included */
      }
      for (int j = 0; j < n; ++j) sc[j] = S > 0.0 ? sc[j] / S : 0.0;
      for (int j = n; j < n_max; ++j) {
        sc[j] = 0.0;
        if (lKo) lKo[j] = 0.0;
        if (lVo) lVo[j] = 0.0;
      }
      head_sums[(size_t)b * H + h] = S;
    }
  }
}

/* ------------------------------------------------------------------------
 * Forced-keep set (the sink step of Algorithm 1, extended by the recent window):
 *   F = {0..s-1}  U  {n-w..n-1}, clipped to the sequence.  If the budget
 * cannot hold all of F, the window's most recent tokens come first, then the
 * sinks in index order.  flag[j] = 1 for forced tokens; returns |F| kept.
 * ---------------------------------------------------------------------- */
static int forced_set(int n, int s, int w, int k_eff, uint8_t *flag) {
  int cnt = 0;
  memset(flag, 0, (size_t)n);
  for (int j = n - 1; j >= 0 && j >= n - w && cnt < k_eff; --j) { flag[j] = 1; ++cnt; }
  for (int j = 0; j < s && j < n && cnt < k_eff; ++j)
    if (!flag[j]) { flag[j] = 1; ++cnt; }
  return cnt;
}

typedef struct { double score; int32_t head; int32_t idx; } cand_t;

/* score descending, then head ascending, then token index ascending */
static int cand_cmp(const void *pa, const void *pb) {
  const cand_t *a = (const cand_t *)pa, *b = (const cand_t *)pb;
  if (a->score > b->score) return -1;
  if (a->score < b->score) return 1;
  if (a->head != b->head) return a->head < b->head ? -1 : 1;
  if (a->idx != b->idx) return a->idx < b->idx ? -1 : 1;
  return 0;
}

/* NaN scores rank as 0 so that every output stays a valid index set. */
static double key_of(double s) { return (s == s && s > 0.0) ? s : 0.0; }

/* ------------------------------------------------------------------------
 * Algorithm 1, selection steps (sinks, top-k, union), fixed budget per head.
 *   budget        k: rows kept per head, forced tokens included
 *   head_budgets  NULL, or int32 [B][H] caller-fixed k per head (<= budget)
 *   idx           int32 [B][H][budget], ascending token index, tail = -1
 *   counts        int32 [B][H] = min(k, n_b)
 * ---------------------------------------------------------------------- */
void oracle_select_fixed(const double *scores, int B, int H, int n_max, const int32_t *seqlens,
                         int budget, const int32_t *head_budgets, int num_sink, int window,
                         int32_t *idx, int32_t *counts) {
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
  for (int b = 0; b < B; ++b) {
    for (int h = 0; h < H; ++h) {
      const int n = seq_len(seqlens, b, n_max);
      const double *sc = scores + ((size_t)b * H + h) * n_max;
      int32_t *out = idx + ((size_t)b * H + h) * budget;
      int k = head_budgets ? clampi(head_budgets[(size_t)b * H + h], 0, budget) : budget;
      int k_eff = k < n ? k : n;
      uint8_t *keep = (uint8_t *)malloc((size_t)n + 1);
      cand_t *cand = (cand_t *)malloc(((size_t)n + 1) * sizeof(cand_t));
      int f = forced_set(n, num_sink, window, k_eff, keep);
      int nc = 0;
      for (int j = 0; j < n; ++j)
        if (!keep[j]) { cand[nc].score = key_of(sc[j]); cand[nc].head = 0; cand[nc].idx = j; ++nc; }
      qsort(cand, (size_t)nc, sizeof(cand_t), cand_cmp);       /* TopK(l[s:], k - s) */
      for (int t = 0; t < k_eff - f; ++t) keep[cand[t].idx] = 1; /* S = S_forced U S_top */
      int c = 0;
      for (int j = 0; j < n; ++j) if (keep[j]) out[c++] = j;
      for (int t = c; t < budget; ++t) out[t] = -1;
      counts[(size_t)b * H + h] = c;
      free(keep);
      free(cand);
    }
  }
}

/* ------------------------------------------------------------------------
 * AdaCurDKV (Sec. 3.2, "Adaptive budget allocation"): one top-k over the
 * scores of all heads of a (layer, batch element), with a safeguard fraction
 * alpha of the nominal per-head budget k kept in every head.
 *   m = floor(alpha * k); every head first protects its forced tokens and its
 *   best tokens (score desc, index asc) up to p = min(max(m,|F|), k_eff);
 *   the pooled remainder H*k_eff - H*p goes to the globally best unprotected
 *   (score desc, head asc, index asc).
 * Outputs: packed idx (per head ascending), counts [B][H],
 *          offsets [B*H+1] exclusive prefix sums of counts.
 * ---------------------------------------------------------------------- */
void oracle_select_adaptive(const double *scores, int B, int H, int n_max,
                            const int32_t *seqlens, int budget, int num_sink, int window,
                            double alpha, int32_t *idx, int32_t *counts, int32_t *offsets) {
  const int m = (int)floor(alpha * (double)budget);
  /* selection is independent per batch element; flags kept for the final packing */
  uint8_t *keep_all = (uint8_t *)calloc((size_t)B * H * (n_max > 0 ? n_max : 1), 1);
#pragma omp parallel for schedule(dynamic, 1)
  for (int b = 0; b < B; ++b) {
    const int n = seq_len(seqlens, b, n_max);
    const int k_eff = budget < n ? budget : n;
    uint8_t *forced = (uint8_t *)malloc((size_t)n + 1);
    cand_t *cand = (cand_t *)malloc(((size_t)n + 1) * sizeof(cand_t));
    cand_t *pool = (cand_t *)malloc(((size_t)H * n + 1) * sizeof(cand_t));
    int f = forced_set(n, num_sink, window, k_eff, forced);
    int p = m > f ? m : f;
    if (p > k_eff) p = k_eff;
    size_t np = 0;
    for (int h = 0; h < H; ++h) {
      const double *sc = scores + ((size_t)b * H + h) * n_max;
      uint8_t *keep = keep_all + ((size_t)b * H + h) * n_max;
      int nc = 0;
      for (int j = 0; j < n; ++j) {
        keep[j] = forced[j];
        if (!forced[j]) { cand[nc].score = key_of(sc[j]); cand[nc].head = h; cand[nc].idx = j; ++nc; }
      }
      qsort(cand, (size_t)nc, sizeof(cand_t), cand_cmp);
      for (int t = 0; t < nc; ++t) {
        if (t < p - f) keep[cand[t].idx] = 1;       /* safeguard share of head h */
        else pool[np++] = cand[t];                  /* competes layer-wide */
      }
    }
    qsort(pool, np, sizeof(cand_t), cand_cmp);
    size_t remainder = (size_t)H * (size_t)(k_eff - p);
    for (size_t t = 0; t < remainder && t < np; ++t)
      keep_all[((size_t)b * H + pool[t].head) * n_max + pool[t].idx] = 1;
    free(forced);
    free(cand);
    free(pool);
  }
  int32_t off = 0;
  for (int b = 0; b < B; ++b) {
    const int n = seq_len(seqlens, b, n_max);
    for (int h = 0; h < H; ++h) {
      const uint8_t *keep = keep_all + ((size_t)b * H + h) * n_max;
      int c = 0;
      offsets[(size_t)b * H + h] = off;
      for (int j = 0; j < n; ++j) if (keep[j]) idx[off + c++] = j;
      counts[(size_t)b * H + h] = c;
      off += c;
    }
  }
  offsets[(size_t)B * H] = off;
  free(keep_all);
}

/* ------------------------------------------------------------------------
 * Algorithm 1, gather step: K'_i = K_i[S_i], V'_i = V_i[S_i] -- byte copies of the
 * original (unprojected) rows.  out_stride_h > 0: row t of head (b,h) goes to
 * ((b*H+h)*out_stride_h + t) * d (idx row stride idx_stride); out_stride_h = 0:
 * packed, head (b,h) starts at row offsets[b*H+h] in both idx and the output.
 * ---------------------------------------------------------------------- */
void oracle_compact(const uint16_t *K, const uint16_t *V, int B, int H, int d, int64_t ksb,
                    int64_t ksh, int64_t ksn, int64_t vsb, int64_t vsh, int64_t vsn,
                    const int32_t *idx, int64_t idx_stride, const int32_t *counts,
                    const int32_t *offsets, uint16_t *K_out, uint16_t *V_out,
                    int64_t out_stride_h) {
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
  for (int b = 0; b < B; ++b) {
    for (int h = 0; h < H; ++h) {
      const size_t bh = (size_t)b * H + h;
      const int32_t *ix = out_stride_h > 0 ? idx + bh * idx_stride : idx + offsets[bh];
      const size_t row0 = out_stride_h > 0 ? bh * (size_t)out_stride_h : (size_t)offsets[bh];
      for (int t = 0; t < counts[bh]; ++t) {
        const int j = ix[t];
        memcpy(K_out + (row0 + t) * d, K + b * ksb + h * ksh + j * ksn, (size_t)d * 2);
        memcpy(V_out + (row0 + t) * d, V + b * vsb + h * vsh + j * vsn, (size_t)d * 2);
      }
    }
  }
}

/* GQA (Sec. 3.2): the Hq/Hkv query heads of a group share their KV head's selection. */
int oracle_kv_head_of_query(int q_head, int q_heads, int kv_heads) {
  return q_head / (q_heads / kv_heads);
}

int oracle_num_threads(void) {
#ifdef _OPENMP
  extern int omp_get_max_threads(void);
  return omp_get_max_threads();
#else
  return 1;
#endif
}
