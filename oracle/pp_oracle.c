/*
 * TEST INFRASTRUCTURE -- not part of the product path.
 *
 * Plain CPU fp64 oracle for preference-packed attention (paper Sec. 3.2): one
 * sequence holds a prompt followed by its K responses, and the attention mask
 * lets every response see the prompt and itself, never a sibling response.
 * The paper states that this reproduces the unpacked computation exactly, so
 * the oracle is simply the textbook definition of masked softmax attention and
 * of its gradient, evaluated over an explicit dense mask in double precision.
 *
 * Parity status: every exported function is pinned by tests that do not use
 * this file's arithmetic (unpacked-equivalence brute force, torch fp64
 * autograd, closed forms for Q = 0, finite differences, mask popcounts).
 *
 * No blocking, no online softmax, no fusion: for every query the full score
 * row over its sequence is formed, masked, normalised and used.  OpenMP only
 * spreads independent (head, query) or (head, key) units over threads.
 *
 * Shares no code with the CUDA library.  Only tests, the smoke check and the
 * benchmark's cpu_baseline leg may load it.
 *
 * Layouts (same as the CUDA library so identical bit patterns can be fed):
 *   q, d_out : uint16 bf16 bits  [T][Hq][D]     k, v : [T][Hkv][D]
 *   O, dQ    : double [T][Hq][D]  dK, dV : double [T][Hkv][D]   LSE : double [Hq][T]
 * Query head h reads KV head h / (Hq / Hkv).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define PPO_OK 0
#define PPO_ERR_ARG (-1)
#define PPO_ERR_MEM (-2)

typedef struct {
  int32_t num_rows;
  const int32_t *row_group_off;   /* [num_rows + 1] */
  const int32_t *grp_prompt_len;  /* [G] */
  const int32_t *grp_resp_off;    /* [G + 1] */
  const int32_t *resp_len;        /* [N] */
} ppo_desc;

static double bf16_to_double(uint16_t b) {
  uint32_t u = ((uint32_t)b) << 16;
  float f;
  memcpy(&f, &u, sizeof f);
  return (double)f;
}

/* Token -> (row, group, segment) ids.  segment 0 = prompt, k >= 1 = k-th response.
 * Returns the token count, or a negative error.  Arrays may be NULL to only count. */
long ppo_token_ids(const ppo_desc *d, int32_t *tok_row, int32_t *tok_grp, int32_t *tok_seg) {
  if (!d || d->num_rows < 0 || !d->row_group_off || !d->grp_prompt_len || !d->grp_resp_off ||
      !d->resp_len)
    return PPO_ERR_ARG;
  long t = 0;
  for (int r = 0; r < d->num_rows; ++r) {
    if (d->row_group_off[r + 1] < d->row_group_off[r]) return PPO_ERR_ARG;
    for (int g = d->row_group_off[r]; g < d->row_group_off[r + 1]; ++g) {
      int p = d->grp_prompt_len[g];
      if (p < 1 || d->grp_resp_off[g + 1] < d->grp_resp_off[g]) return PPO_ERR_ARG;
      for (int x = 0; x < p; ++x, ++t) {
        if (tok_row) tok_row[t] = r;
        if (tok_grp) tok_grp[t] = g;
        if (tok_seg) tok_seg[t] = 0;
      }
      int kk = 0;
      for (int s = d->grp_resp_off[g]; s < d->grp_resp_off[g + 1]; ++s) {
        ++kk;
        if (d->resp_len[s] < 1) return PPO_ERR_ARG;
        for (int x = 0; x < d->resp_len[s]; ++x, ++t) {
          if (tok_row) tok_row[t] = r;
          if (tok_grp) tok_grp[t] = g;
          if (tok_seg) tok_seg[t] = kk;
        }
      }
    }
  }
  return t;
}

/* The mask, Sec. 3.2: causal; same group; the key is a prompt token or lies in the
 * query's own response. */
static int visible(const int32_t *grp, const int32_t *seg, long i, long j) {
  return j <= i && grp[i] == grp[j] && (seg[j] == 0 || seg[j] == seg[i]);
}

/* Dense L x L mask of one row (row-major, mask[i*L + j], i = query, j = key, both
 * relative to the row start). */
int ppo_dense_mask(const ppo_desc *d, int row, uint8_t *mask) {
  long T = ppo_token_ids(d, NULL, NULL, NULL);
  if (T < 0 || row < 0 || row >= d->num_rows || !mask) return PPO_ERR_ARG;
  int32_t *tr = malloc(sizeof(int32_t) * (size_t)(T + 1));
  int32_t *tg = malloc(sizeof(int32_t) * (size_t)(T + 1));
  int32_t *ts = malloc(sizeof(int32_t) * (size_t)(T + 1));
  if (!tr || !tg || !ts) { free(tr); free(tg); free(ts); return PPO_ERR_MEM; }
  ppo_token_ids(d, tr, tg, ts);
  long lo = 0;
  while (lo < T && tr[lo] != row) ++lo;
  long hi = lo;
  while (hi < T && tr[hi] == row) ++hi;
  long L = hi - lo;
  for (long i = 0; i < L; ++i)
    for (long j = 0; j < L; ++j) mask[i * L + j] = (uint8_t)visible(tg, ts, lo + i, lo + j);
  free(tr); free(tg); free(ts);
  return PPO_OK;
}

typedef struct {
  long T;
  int Hq, Hkv, D;
  int32_t *tok_row, *tok_grp, *tok_seg;
  long *row_lo, *row_hi; /* per token: its row's token range */
  double *q, *k, *v, *dout;
} ppo_ctx;

static void ctx_free(ppo_ctx *c) {
  free(c->tok_row); free(c->tok_grp); free(c->tok_seg); free(c->row_lo); free(c->row_hi);
  free(c->q); free(c->k); free(c->v); free(c->dout);
}

static double *widen(const uint16_t *src, size_t n) {
  if (!src) return NULL;
  double *dst = malloc(sizeof(double) * (n ? n : 1));
  if (!dst) return NULL;
  for (size_t i = 0; i < n; ++i) dst[i] = bf16_to_double(src[i]);
  return dst;
}

static int ctx_init(ppo_ctx *c, const ppo_desc *d, int Hq, int Hkv, int D, const uint16_t *q,
                    const uint16_t *k, const uint16_t *v, const uint16_t *dout) {
  memset(c, 0, sizeof *c);
  if (Hq < 1 || Hkv < 1 || D < 1 || Hq % Hkv != 0 || !q || !k || !v) return PPO_ERR_ARG;
  long T = ppo_token_ids(d, NULL, NULL, NULL);
  if (T < 0) return (int)T;
  c->T = T; c->Hq = Hq; c->Hkv = Hkv; c->D = D;
  size_t n = (size_t)T + 1;
  c->tok_row = malloc(sizeof(int32_t) * n);
  c->tok_grp = malloc(sizeof(int32_t) * n);
  c->tok_seg = malloc(sizeof(int32_t) * n);
  c->row_lo = malloc(sizeof(long) * n);
  c->row_hi = malloc(sizeof(long) * n);
  c->q = widen(q, (size_t)T * Hq * D);
  c->k = widen(k, (size_t)T * Hkv * D);
  c->v = widen(v, (size_t)T * Hkv * D);
  c->dout = widen(dout, (size_t)T * Hq * D);
  if (!c->tok_row || !c->tok_grp || !c->tok_seg || !c->row_lo || !c->row_hi || !c->q || !c->k ||
      !c->v || (dout && !c->dout)) {
    ctx_free(c);
    return PPO_ERR_MEM;
  }
  ppo_token_ids(d, c->tok_row, c->tok_grp, c->tok_seg);
  long lo = 0;
  while (lo < T) {
    long hi = lo;
    while (hi < T && c->tok_row[hi] == c->tok_row[lo]) ++hi;
    for (long i = lo; i < hi; ++i) { c->row_lo[i] = lo; c->row_hi[i] = hi; }
    lo = hi;
  }
  return PPO_OK;
}

static double dotd(const double *a, const double *b, int D) {
  double s = 0.0;
#pragma omp simd reduction(+ : s)
  for (int x = 0; x < D; ++x) s += a[x] * b[x];
  return s;
}

/* Scores of query i (head h) against every key of its row: s[j - lo] = scale * q.k where
 * the mask allows, -inf elsewhere.  Returns the row maximum. */
static double score_row(const ppo_ctx *c, double scale, long i, int h, double *s) {
  int kvh = h / (c->Hq / c->Hkv);
  long lo = c->row_lo[i], hi = c->row_hi[i];
  const double *qi = c->q + ((size_t)i * c->Hq + h) * c->D;
  double m = -INFINITY;
  for (long j = lo; j < hi; ++j) {
    if (visible(c->tok_grp, c->tok_seg, i, j)) {
      double x = scale * dotd(qi, c->k + ((size_t)j * c->Hkv + kvh) * c->D, c->D);
      s[j - lo] = x;
      if (x > m) m = x;
    } else {
      s[j - lo] = -INFINITY;
    }
  }
  return m;
}

static void fwd_core(const ppo_ctx *c, double scale, double *O, double *LSE, long maxL) {
  long T = c->T;
  int Hq = c->Hq, Hkv = c->Hkv, D = c->D;
#pragma omp parallel
  {
    double *s = malloc(sizeof(double) * (size_t)(maxL + 1));
#pragma omp for collapse(2) schedule(dynamic, 16)
    for (int h = 0; h < Hq; ++h) {
      for (long i = 0; i < T; ++i) {
        int kvh = h / (Hq / Hkv);
        long lo = c->row_lo[i], hi = c->row_hi[i];
        double m = score_row(c, scale, i, h, s);
        double l = 0.0;
        for (long j = lo; j < hi; ++j)
          if (s[j - lo] != -INFINITY) l += exp(s[j - lo] - m);
        double lse = m + log(l);
        double *o = O + ((size_t)i * Hq + h) * D;
        for (int x = 0; x < D; ++x) o[x] = 0.0;
        for (long j = lo; j < hi; ++j) {
          if (s[j - lo] == -INFINITY) continue;
          double p = exp(s[j - lo] - lse);
          const double *vj = c->v + ((size_t)j * Hkv + kvh) * D;
#pragma omp simd
          for (int x = 0; x < D; ++x) o[x] += p * vj[x];
        }
        LSE[(size_t)h * T + i] = lse;
      }
    }
    free(s);
  }
}

static long max_row_len(const ppo_ctx *c) {
  long m = 0;
  for (long i = 0; i < c->T; ++i)
    if (c->row_hi[i] - c->row_lo[i] > m) m = c->row_hi[i] - c->row_lo[i];
  return m;
}

static void set_threads(int n) {
#ifdef _OPENMP
  if (n > 0) omp_set_num_threads(n);
#else
  (void)n;
#endif
}

int ppo_max_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

/* Forward: O = softmax(mask(scale Q K^T)) V and LSE = ln sum_j exp(S_ij). */
int ppo_attn_fwd(const ppo_desc *d, int Hq, int Hkv, int D, const uint16_t *q, const uint16_t *k,
                 const uint16_t *v, double scale, double *O, double *LSE, int num_threads) {
  if (!O || !LSE) return PPO_ERR_ARG;
  ppo_ctx c;
  int rc = ctx_init(&c, d, Hq, Hkv, D, q, k, v, NULL);
  if (rc) return rc;
  set_threads(num_threads);
  fwd_core(&c, scale, O, LSE, max_row_len(&c));
  ctx_free(&c);
  return PPO_OK;
}

/* Forward + backward.  With P_ij = exp(S_ij - LSE_i):
 *   Delta_i = sum_d dO_id O_id          dP_ij = dO_i . V_j        dS_ij = P_ij (dP_ij - Delta_i)
 *   dQ_i = scale sum_j dS_ij K_j        dK_j = scale sum_{h,i} dS_ij Q_i     dV_j = sum_{h,i} P_ij dO_i
 * where the sums for dK, dV run over the query heads that read this KV head. */
int ppo_attn_fwd_bwd(const ppo_desc *d, int Hq, int Hkv, int D, const uint16_t *q,
                     const uint16_t *k, const uint16_t *v, const uint16_t *dout, double scale,
                     double *O, double *LSE, double *dQ, double *dK, double *dV, int num_threads) {
  if (!O || !LSE || !dQ || !dK || !dV || !dout) return PPO_ERR_ARG;
  ppo_ctx c;
  int rc = ctx_init(&c, d, Hq, Hkv, D, q, k, v, dout);
  if (rc) return rc;
  set_threads(num_threads);
  long T = c.T, maxL = max_row_len(&c);
  int r = Hq / Hkv;
  fwd_core(&c, scale, O, LSE, maxL);

  double *delta = malloc(sizeof(double) * ((size_t)T * Hq + 1));
  if (!delta) { ctx_free(&c); return PPO_ERR_MEM; }
#pragma omp parallel for collapse(2)
  for (int h = 0; h < Hq; ++h)
    for (long i = 0; i < T; ++i)
      delta[(size_t)h * T + i] =
          dotd(c.dout + ((size_t)i * Hq + h) * D, O + ((size_t)i * Hq + h) * D, D);

  /* dQ: one (head, query) at a time */
#pragma omp parallel
  {
    double *s = malloc(sizeof(double) * (size_t)(maxL + 1));
#pragma omp for collapse(2) schedule(dynamic, 16)
    for (int h = 0; h < Hq; ++h) {
      for (long i = 0; i < T; ++i) {
        int kvh = h / r;
        long lo = c.row_lo[i], hi = c.row_hi[i];
        score_row(&c, scale, i, h, s);
        double lse = LSE[(size_t)h * T + i], dl = delta[(size_t)h * T + i];
        const double *doi = c.dout + ((size_t)i * Hq + h) * D;
        double *dq = dQ + ((size_t)i * Hq + h) * D;
        for (int x = 0; x < D; ++x) dq[x] = 0.0;
        for (long j = lo; j < hi; ++j) {
          if (s[j - lo] == -INFINITY) continue;
          double p = exp(s[j - lo] - lse);
          double dp = dotd(doi, c.v + ((size_t)j * Hkv + kvh) * D, D);
          double ds = p * (dp - dl);
          const double *kj = c.k + ((size_t)j * Hkv + kvh) * D;
#pragma omp simd
          for (int x = 0; x < D; ++x) dq[x] += scale * ds * kj[x];
        }
      }
    }
    free(s);
  }

  /* dK, dV: one (kv head, key) at a time, summing over its query heads and all queries */
#pragma omp parallel for collapse(2) schedule(dynamic, 16)
  for (int kvh = 0; kvh < Hkv; ++kvh) {
    for (long j = 0; j < T; ++j) {
      long hi = c.row_hi[j];
      const double *kj = c.k + ((size_t)j * Hkv + kvh) * D;
      const double *vj = c.v + ((size_t)j * Hkv + kvh) * D;
      double *dk = dK + ((size_t)j * Hkv + kvh) * D;
      double *dv = dV + ((size_t)j * Hkv + kvh) * D;
      for (int x = 0; x < D; ++x) { dk[x] = 0.0; dv[x] = 0.0; }
      for (int h = kvh * r; h < (kvh + 1) * r; ++h) {
        for (long i = c.row_lo[j]; i < hi; ++i) {
          if (!visible(c.tok_grp, c.tok_seg, i, j)) continue;
          const double *qi = c.q + ((size_t)i * Hq + h) * D;
          const double *doi = c.dout + ((size_t)i * Hq + h) * D;
          double p = exp(scale * dotd(qi, kj, D) - LSE[(size_t)h * T + i]);
          double ds = p * (dotd(doi, vj, D) - delta[(size_t)h * T + i]);
#pragma omp simd
          for (int x = 0; x < D; ++x) {
            dv[x] += p * doi[x];
            dk[x] += scale * ds * qi[x];
          }
        }
      }
    }
  }
  free(delta);
  ctx_free(&c);
  return PPO_OK;
}

/* Dense intermediates of one (row, query head) for tiny cases: S (scaled, masked = -inf),
 * P, dP, dS, each L x L row-major with i = query, j = key relative to the row. */
int ppo_dump_intermediates(const ppo_desc *d, int Hq, int Hkv, int D, const uint16_t *q,
                           const uint16_t *k, const uint16_t *v, const uint16_t *dout,
                           double scale, int row, int head, double *S, double *P, double *dP,
                           double *dS) {
  ppo_ctx c;
  int rc = ctx_init(&c, d, Hq, Hkv, D, q, k, v, dout);
  if (rc) return rc;
  if (row < 0 || row >= d->num_rows || head < 0 || head >= Hq || !S || !P || !dP || !dS || !dout) {
    ctx_free(&c);
    return PPO_ERR_ARG;
  }
  long lo = 0;
  while (lo < c.T && c.tok_row[lo] != row) ++lo;
  long hi = c.row_hi[lo], L = hi - lo;
  int kvh = head / (Hq / Hkv);
  for (long i = lo; i < hi; ++i) {
    double *s = S + (i - lo) * L;
    double m = score_row(&c, scale, i, head, s);
    double l = 0.0;
    for (long j = 0; j < L; ++j)
      if (s[j] != -INFINITY) l += exp(s[j] - m);
    double lse = m + log(l), dl = 0.0;
    const double *doi = c.dout + ((size_t)i * Hq + head) * D;
    for (long j = 0; j < L; ++j) {
      double p = s[j] == -INFINITY ? 0.0 : exp(s[j] - lse);
      double dp = dotd(doi, c.v + ((size_t)(lo + j) * Hkv + kvh) * D, D);
      P[(i - lo) * L + j] = p;
      dP[(i - lo) * L + j] = dp;
      dl += p * dp;
    }
    for (long j = 0; j < L; ++j)
      dS[(i - lo) * L + j] = P[(i - lo) * L + j] * (dP[(i - lo) * L + j] - dl);
  }
  ctx_free(&c);
  return PPO_OK;
}
