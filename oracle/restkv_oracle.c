/*
 * ReST-KV eviction scoring -- CPU oracle (TEST INFRASTRUCTURE, not the product).
 *
 * A plain, slow, fp64 restatement of what the paper defines, written so a reader can
 * check it against the paper by eye.  Only tests, the smoke check and the CPU-baseline
 * leg of the benchmark may call it.  It shares no code with the CUDA library.
 *
 * Inputs are float arrays holding values that are exactly representable in the dtype
 * under test (bf16- or fp32-rounded); every operation below widens to double first.
 *
 * Tensor layouts (all contiguous, row-major):
 *   Q  [batch, Hq,  w,    d]   window queries, oldest query first
 *   K  [batch, Hkv, n_kv, d]   n_kv = n + causal_tail
 *   V  [batch, Hkv, n_kv, d]
 * Query head hq belongs to KV head hq / (Hq / Hkv).
 *
 * Steps and where the paper defines them:
 *   logits, softmax, output        Eq. 3   (Section 3.1)
 *   reconstruction indicator       Eq. 7   (Section 3.2), W_O the identity unless one is given (Eq. 4)
 *   EMA temporal smoothing         Eq. 8-9 (Section 3.3), recursion as written
 *   adaptive window parameters     Eq. 10-12
 *   box pooling (final indicator)  Eq. 13
 *   top-B and gather               Eq. 14
 *   ablation variants              Appendix G.1 (indicators: attention weight alone, attention weight times
 *                                  the value's norm), Appendix G.2 (temporal: none, mean, inverted EMA;
 *                                  spatial: max instead of mean over the box)
 *
 * Pins (tests that do not depend on this file's own arithmetic): brute-force token
 * deletion (Eq. 6) in NumPy, the renormalisation relation of Appendix A, uniform-logit
 * and two-token closed forms, EMA closed-form weights, pooling identities, a library
 * stable sort for the selection, library softmax attention for decode; for the variants:
 * library softmax and norms, closed-form temporal weights, time reversal, a library maximum filter.
 * Readings with no independent pin ("parity unpinned"): mean over the query heads of a
 * GQA group (the paper is silent), and how a fixed kernel width combines with the
 * adaptive width (box of width W_s + base_width - 1).
 */
#include <math.h>
#include <stdlib.h>
#include <string.h>
#include <stdint.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORACLE_OK 0
#define ORACLE_BAD_ARG 1
#define ORACLE_NO_MEM 2

typedef struct { double score; int index; } scored_t;

/* descending score, ascending index on equal scores: a total order, so qsort is as good
 * as a stable sort */
static int cmp_desc_score_asc_index(const void* a, const void* b) {
  const scored_t* x = (const scored_t*)a;
  const scored_t* y = (const scored_t*)b;
  if (x->score > y->score) return -1;
  if (x->score < y->score) return 1;
  return (x->index > y->index) - (x->index < y->index);
}
static int cmp_int_asc(const void* a, const void* b) {
  int x = *(const int*)a, y = *(const int*)b;
  return (x > y) - (x < y);
}

int restkv_oracle_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}
void restkv_oracle_set_threads(int t) {
#ifdef _OPENMP
  if (t > 0) omp_set_num_threads(t);
#else
  (void)t;
#endif
}

/* Top-`count` indices of x[0:n] (largest first, lower index wins ties), written in
 * ascending index order.  Eq. 14's argmax_B. */
static int top_indices(const double* x, int n, int count, int* out) {
  scored_t* s = (scored_t*)malloc((size_t)n * sizeof(scored_t));
  if (!s) return ORACLE_NO_MEM;
  for (int j = 0; j < n; ++j) { s[j].score = x[j]; s[j].index = j; }
  qsort(s, (size_t)n, sizeof(scored_t), cmp_desc_score_asc_index);
  for (int r = 0; r < count; ++r) out[r] = s[r].index;
  qsort(out, (size_t)count, sizeof(int), cmp_int_asc);
  free(s);
  return ORACLE_OK;
}

/*
 * Scores for every (batch, KV head).
 *
 *  causal_tail  0: K,V hold the n scored prefix rows only, every query sees every row.
 *               w: K,V hold n + w rows; trailing row n+j' is window token j' itself and
 *                  query i sees it only if j' <= i.  Trailing rows get score +inf (Omega).
 *  scale        softmax scale (1/sqrt(d_k) in Eq. 3)
 *  ema_decay    1 - alpha of Eq. 9
 *  pool_mode    0 fixed (width, shift given), 1 adaptive (Eq. 10-12)
 *  width/shift  fixed mode: odd W >= 1 and gamma
 *  beta         Eq. 11-12 scaling factor
 *  base_width   adaptive mode: odd fixed kernel k; box width = W_s + k - 1
 *  budget       adaptive mode: B of Eq. 10
 *  literal_gamma  adaptive mode: 1 = Eq. 12 exactly as printed, 0 = truncate toward zero
 *  group_mode   0 = mean over the G query heads of a KV head, 1 = max over them
 *  indicator_mode  0 = Eq. 7;  1 = the attention weight A[j] alone;  2 = A[j] * ||v_j||_2   (Appendix G.1)
 *  temporal_mode   0 = EMA of Eq. 8-9;  1 = mean over the w queries;  2 = the EMA recursion run from the newest
 *                  query to the oldest ("Inv-EMA": the oldest query weighs most);  3 = none: the newest query's
 *                  indicator alone   (Appendix G.2)
 *  spatial_mode    0 = box mean of Eq. 13;  1 = maximum over the same box, taps outside the scored rows count
 *                  as 0 as they do in the mean   (Appendix G.2)
 *  W_O, d_model    the output projection of Eq. 4 as [Hq, d, d_model] (query head hq owns rows hq*d .. hq*d+d-1 of
 *                  the model's W_O); Eq. 7 then measures || (z_t - v_j) W_O^(hq) ||_2.  NULL: identity.
 *
 * Optional outputs (NULL to skip):
 *  A_out     [batch, Hq, w, n_kv]  attention weights (Eq. 3)
 *  O_out     [batch, Hq, w, d]     window outputs
 *  I_raw     [batch, Hq, w, n]     Eq. 7 per query
 *  I_hat     [batch, Hkv, n]       after EMA and group reduction
 *  pool_out  [batch, Hkv, 2]       (W, gamma) used
 *  D_out     [batch, Hkv, 2]       (D_front, D_rear), adaptive mode only
 * Required: scores [batch, Hkv, n_kv].
 */
int restkv_oracle_score_variant(const float* Q, const float* K, const float* V,
                        int batch, int Hq, int Hkv, int d, int n_kv, int w, int causal_tail,
                        double scale, double ema_decay,
                        int pool_mode, int width, int shift, double beta, int base_width,
                        int budget, int literal_gamma, int group_mode,
                        int indicator_mode, int temporal_mode, int spatial_mode,
                        const float* W_O, int d_model,
                        double* A_out, double* O_out, double* I_raw, double* I_hat,
                        int* pool_out, double* D_out, double* scores) {
  if (!Q || !K || !V || !scores) return ORACLE_BAD_ARG;
  if (W_O && d_model < 1) return ORACLE_BAD_ARG;
  if (indicator_mode < 0 || indicator_mode > 2 || temporal_mode < 0 || temporal_mode > 3) return ORACLE_BAD_ARG;
  if (spatial_mode < 0 || spatial_mode > 1) return ORACLE_BAD_ARG;
  if (batch < 1 || Hq < 1 || Hkv < 1 || d < 1 || w < 1 || n_kv < 1) return ORACLE_BAD_ARG;
  if (Hq % Hkv != 0) return ORACLE_BAD_ARG;
  if (causal_tail != 0 && causal_tail != w) return ORACLE_BAD_ARG;
  const int n = n_kv - causal_tail; /* scored prefix rows */
  if (n < 1) return ORACLE_BAD_ARG;
  if (pool_mode == 0 && (width < 1 || width % 2 == 0)) return ORACLE_BAD_ARG;
  if (pool_mode == 1 && (base_width < 1 || base_width % 2 == 0 || !(beta > 0.0))) return ORACLE_BAD_ARG;
  if (pool_mode != 0 && pool_mode != 1) return ORACLE_BAD_ARG;
  const int G = Hq / Hkv;
  const double alpha = 1.0 - ema_decay;
  int status = ORACLE_OK;

  for (int b = 0; b < batch; ++b) {
    for (int h = 0; h < Hkv; ++h) {
      const float* Kh = K + ((size_t)b * Hkv + h) * (size_t)n_kv * d;
      const float* Vh = V + ((size_t)b * Hkv + h) * (size_t)n_kv * d;
      /* I for this KV head: [G, w, n] */
      double* Ih = (double*)malloc((size_t)G * w * n * sizeof(double));
      double* ihat = (double*)malloc((size_t)n * sizeof(double));
      if (!Ih || !ihat) { free(Ih); free(ihat); return ORACLE_NO_MEM; }

      /* ---- Eq. 3 and Eq. 7, one query row at a time ---- */
#pragma omp parallel for schedule(dynamic, 1)
      for (int gi = 0; gi < G * w; ++gi) {
        const int g = gi / w, i = gi % w;
        const int hq = h * G + g;
        const float* q = Q + (((size_t)b * Hq + hq) * w + i) * d;
        double* a = (double*)malloc((size_t)n_kv * sizeof(double));
        double* o = (double*)malloc((size_t)d * sizeof(double));
        if (!a || !o) { free(a); free(o);
#pragma omp atomic write
          status = ORACLE_NO_MEM;
          continue; }
        /* rows this query sees: the n prefix rows, plus trailing rows j' <= i */
        const int visible = (causal_tail == 0) ? n_kv : n + i + 1;
        double mx = -INFINITY;
        for (int j = 0; j < visible; ++j) {
          double s = 0.0;
          for (int k = 0; k < d; ++k) s += (double)q[k] * (double)Kh[(size_t)j * d + k];
          a[j] = s * scale;
          if (a[j] > mx) mx = a[j];
        }
        double sum = 0.0;
        for (int j = 0; j < visible; ++j) { a[j] = exp(a[j] - mx); sum += a[j]; }
        for (int j = 0; j < visible; ++j) a[j] /= sum;         /* A_t, Eq. 3 */
        for (int j = visible; j < n_kv; ++j) a[j] = 0.0;       /* masked */
        for (int k = 0; k < d; ++k) o[k] = 0.0;
        for (int j = 0; j < visible; ++j)
          for (int k = 0; k < d; ++k) o[k] += a[j] * (double)Vh[(size_t)j * d + k]; /* z_t = A_t V */
        /* Eq. 7: I[j] = A[j] / (1 - A[j]) * || (z_t - v_j) W_O ||_2, W_O the head's d x d_model slice
         * (Eq. 4) or the identity */
        for (int j = 0; j < n && indicator_mode == 0; ++j) {
          double ss = 0.0;
          if (W_O) {
            const float* Wh = W_O + (size_t)hq * d * d_model;
            for (int mcol = 0; mcol < d_model; ++mcol) {
              double y = 0.0;
              for (int k = 0; k < d; ++k)
                y += (o[k] - (double)Vh[(size_t)j * d + k]) * (double)Wh[(size_t)k * d_model + mcol];
              ss += y * y;
            }
          } else {
            for (int k = 0; k < d; ++k) {
              double df = o[k] - (double)Vh[(size_t)j * d + k];
              ss += df * df;
            }
          }
          double one_minus = 1.0 - a[j];
          /* a single visible row has A = 1 and nothing to redistribute to: define I = 0 */
          Ih[((size_t)g * w + i) * n + j] = (visible == 1) ? 0.0 : a[j] / one_minus * sqrt(ss);
        }
        /* Appendix G.1: the attention weight alone, or weighted by the norm of the value */
        for (int j = 0; j < n && indicator_mode != 0; ++j) {
          double vv = 0.0;
          for (int k = 0; k < d; ++k) vv += (double)Vh[(size_t)j * d + k] * (double)Vh[(size_t)j * d + k];
          Ih[((size_t)g * w + i) * n + j] = (indicator_mode == 1) ? a[j] : a[j] * sqrt(vv);
        }
        if (A_out) memcpy(A_out + (((size_t)b * Hq + hq) * w + i) * n_kv, a, (size_t)n_kv * sizeof(double));
        if (O_out) memcpy(O_out + (((size_t)b * Hq + hq) * w + i) * d, o, (size_t)d * sizeof(double));
        if (I_raw) memcpy(I_raw + (((size_t)b * Hq + hq) * w + i) * n, Ih + ((size_t)g * w + i) * n,
                          (size_t)n * sizeof(double));
        free(a); free(o);
      }
      if (status != ORACLE_OK) { free(Ih); free(ihat); return status; }

      /* ---- Eq. 8-9: EMA over the w window queries, oldest first, by the recursion;
       *      then the reduction over the G query heads of this KV head ---- */
#pragma omp parallel for schedule(static)
      for (int j = 0; j < n; ++j) {
        double red = 0.0;
        for (int g = 0; g < G; ++g) {
          const double* col = Ih + (size_t)g * w * n + j;              /* col[i * n] = I of query i */
          double ema;
          if (temporal_mode == 0) {
            ema = col[0];                                               /* t1 == t2 */
            for (int i = 1; i < w; ++i) ema = alpha * col[(size_t)i * n] + (1.0 - alpha) * ema;
          } else if (temporal_mode == 1) {                              /* Appendix G.2: mean */
            ema = 0.0;
            for (int i = 0; i < w; ++i) ema += col[(size_t)i * n];
            ema /= (double)w;
          } else if (temporal_mode == 2) {                              /* Appendix G.2: EMA in reversed time */
            ema = col[(size_t)(w - 1) * n];
            for (int i = w - 2; i >= 0; --i) ema = alpha * col[(size_t)i * n] + (1.0 - alpha) * ema;
          } else {                                                      /* Appendix G.2: no temporal smoothing */
            ema = col[(size_t)(w - 1) * n];
          }
          if (group_mode == 0) red += ema;
          else red = (g == 0 || ema > red) ? ema : red;
        }
        ihat[j] = (group_mode == 0) ? red / (double)G : red;
      }
      if (I_hat) memcpy(I_hat + ((size_t)b * Hkv + h) * n, ihat, (size_t)n * sizeof(double));

      /* ---- Eq. 10-12: adaptive window parameters ---- */
      int W = width, gamma = shift;
      if (pool_mode == 1) {
        int Bp = budget - causal_tail;
        if (Bp > n) Bp = n;
        if (Bp < 1) { free(Ih); free(ihat); return ORACLE_BAD_ARG; }
        const int w_front = w / 2; /* first half of the window queries */
        double sum_front = 0.0, sum_rear = 0.0;
        long cnt_front = 0, cnt_rear = 0;
        int* idx = (int*)malloc((size_t)Bp * sizeof(int));
        if (!idx) { free(Ih); free(ihat); return ORACLE_NO_MEM; }
        for (int g = 0; g < G; ++g)
          for (int i = 0; i < w; ++i) {
            int rc = top_indices(Ih + ((size_t)g * w + i) * n, n, Bp, idx);
            if (rc != ORACLE_OK) { free(idx); free(Ih); free(ihat); return rc; }
            double s = 0.0;
            for (int r = 0; r < Bp; ++r) s += (double)idx[r];
            if (i < w_front) { sum_front += s; cnt_front += Bp; }
            else             { sum_rear  += s; cnt_rear  += Bp; }
          }
        free(idx);
        /* w == 1 leaves the front half empty: no shift signal */
        double D_front = cnt_front ? sum_front / (double)cnt_front : 0.0;
        double D_rear  = cnt_rear  ? sum_rear  / (double)cnt_rear  : 0.0;
        if (!cnt_front) D_front = D_rear;
        double x = (D_front - D_rear) / beta;
        int Ws = 2 * (int)floor(fabs(x)) + 1;                       /* Eq. 11 */
        if (literal_gamma) gamma = (x > 0.0) ? (int)floor(x) : (int)floor(x) + 1; /* Eq. 12 as printed */
        else               gamma = (int)trunc(x);
        W = Ws + base_width - 1;
        if (D_out) { D_out[((size_t)b * Hkv + h) * 2 + 0] = D_front; D_out[((size_t)b * Hkv + h) * 2 + 1] = D_rear; }
      }
      if (pool_out) { pool_out[((size_t)b * Hkv + h) * 2 + 0] = W; pool_out[((size_t)b * Hkv + h) * 2 + 1] = gamma; }

      /* ---- Eq. 13: box mean over [j - floor(W/2) + gamma, j + floor(W/2) + gamma],
       *      taps outside the scored rows contribute 0, divisor is always W;
       *      Eq. 8: the window's own tokens get Omega = +inf ---- */
      double* sc = scores + ((size_t)b * Hkv + h) * n_kv;
      const int half = W / 2;
      for (int j = 0; j < n; ++j) {
        double s = 0.0, mxv = 0.0;
        for (int k = -half + gamma; k <= half + gamma; ++k) {
          long t = (long)j + k;
          if (t >= 0 && t < n) { s += ihat[t]; if (ihat[t] > mxv) mxv = ihat[t]; }
        }
        sc[j] = (spatial_mode == 0) ? s / (double)W : mxv;
      }
      for (int j = n; j < n_kv; ++j) sc[j] = INFINITY;

      free(Ih); free(ihat);
    }
  }
  return status;
}

/* The method itself: Eq. 7, Eq. 8-9 and Eq. 13 as they are printed. */
int restkv_oracle_score(const float* Q, const float* K, const float* V,
                        int batch, int Hq, int Hkv, int d, int n_kv, int w, int causal_tail,
                        double scale, double ema_decay,
                        int pool_mode, int width, int shift, double beta, int base_width,
                        int budget, int literal_gamma, int group_mode,
                        double* A_out, double* O_out, double* I_raw, double* I_hat,
                        int* pool_out, double* D_out, double* scores) {
  return restkv_oracle_score_variant(Q, K, V, batch, Hq, Hkv, d, n_kv, w, causal_tail, scale, ema_decay,
                                     pool_mode, width, shift, beta, base_width, budget, literal_gamma, group_mode,
                                     0, 0, 0, NULL, 0, A_out, O_out, I_raw, I_hat, pool_out, D_out, scores);
}

/* Eq. 14: per row of `scores` [rows, n_kv], the min(budget, n_kv) largest entries
 * (ties: lower index first), indices written ascending into indices[rows, min(budget, n_kv)]. */
int restkv_oracle_select(const double* scores, int rows, int n_kv, int budget, int* indices) {
  if (!scores || !indices || rows < 1 || n_kv < 1 || budget < 1) return ORACLE_BAD_ARG;
  const int keep = budget < n_kv ? budget : n_kv;
  int status = ORACLE_OK;
#pragma omp parallel for schedule(dynamic, 1)
  for (int r = 0; r < rows; ++r) {
    int rc = top_indices(scores + (size_t)r * n_kv, n_kv, keep, indices + (size_t)r * keep);
    if (rc != ORACLE_OK) {
#pragma omp atomic write
      status = rc;
    }
  }
  return status;
}

/* Eq. 14: gather rows.  src [rows, n_kv, row_bytes] -> dst [rows, n_sel, row_bytes];
 * bytes are copied untouched. */
int restkv_oracle_compact(const unsigned char* src, int rows, int n_kv, size_t row_bytes,
                          const int* indices, int n_sel, unsigned char* dst) {
  if (!src || !dst || !indices) return ORACLE_BAD_ARG;
  for (int r = 0; r < rows; ++r)
    for (int s = 0; s < n_sel; ++s) {
      int j = indices[(size_t)r * n_sel + s];
      if (j < 0 || j >= n_kv) return ORACLE_BAD_ARG;
      memcpy(dst + ((size_t)r * n_sel + s) * row_bytes, src + ((size_t)r * n_kv + j) * row_bytes, row_bytes);
    }
  return ORACLE_OK;
}

/* Decode step over a (compacted) cache: Eq. 3 for one new query per query head.
 * q [batch, Hq, d]; Kc, Vc [batch, Hkv, n_rows, d]; out [batch, Hq, d]; lse optional [batch, Hq]
 * (natural-log sum of exp of the scaled logits). */
int restkv_oracle_decode(const float* q, const float* Kc, const float* Vc,
                         int batch, int Hq, int Hkv, int d, int n_rows, double scale,
                         double* out, double* lse) {
  if (!q || !Kc || !Vc || !out || n_rows < 1 || Hq % Hkv != 0) return ORACLE_BAD_ARG;
  const int G = Hq / Hkv;
  int status = ORACLE_OK;
#pragma omp parallel for schedule(dynamic, 1)
  for (int bh = 0; bh < batch * Hq; ++bh) {
    const int b = bh / Hq, hq = bh % Hq, h = hq / G;
    const float* qq = q + (size_t)bh * d;
    const float* Kh = Kc + ((size_t)b * Hkv + h) * (size_t)n_rows * d;
    const float* Vh = Vc + ((size_t)b * Hkv + h) * (size_t)n_rows * d;
    double* a = (double*)malloc((size_t)n_rows * sizeof(double));
    if (!a) {
#pragma omp atomic write
      status = ORACLE_NO_MEM;
      continue;
    }
    double mx = -INFINITY;
    for (int j = 0; j < n_rows; ++j) {
      double s = 0.0;
      for (int k = 0; k < d; ++k) s += (double)qq[k] * (double)Kh[(size_t)j * d + k];
      a[j] = s * scale;
      if (a[j] > mx) mx = a[j];
    }
    double sum = 0.0;
    for (int j = 0; j < n_rows; ++j) { a[j] = exp(a[j] - mx); sum += a[j]; }
    for (int k = 0; k < d; ++k) {
      double acc = 0.0;
      for (int j = 0; j < n_rows; ++j) acc += a[j] / sum * (double)Vh[(size_t)j * d + k];
      out[(size_t)bh * d + k] = acc;
    }
    if (lse) lse[bh] = mx + log(sum);
    free(a);
  }
  return status;
}
