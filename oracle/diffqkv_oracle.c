/*
 * DiffQKV attention oracle: plain, slow, float64 CPU code.
 *
 * THIS IS TEST INFRASTRUCTURE, NOT THE PRODUCT.  It exists so that the CUDA
 * library can be checked element by element against the plain definition of
 * what the paper's method computes.  It shares no code, header, table or
 * helper with the CUDA path and must never be called from it; only the test
 * suite, the smoke check and the benchmark's CPU-baseline leg use it.
 *
 * What it follows (paper sections, equations, listings):
 *   - Section 2, "Formulation of DiffQKV Attention": q, K, V with separate
 *     head counts n_q, n_k, n_v; scores = softmax over cached positions of
 *     <q_i, K_(j,i)> / sqrt(d_k); o_i = sum_j alpha_(j,i) V_(j,i).
 *   - Section 3.2, Eq. (idx): idx_k = idx_q * n_k / n_q, idx_v = idx_q * n_v / n_q
 *     (read as integer floor; n_k and n_v must divide n_q).
 *   - Appendix "KV Group Sharing" listing: replicated heads are adjacent,
 *     which is the same contiguous grouping as the floor in Eq. (idx).
 *   - Section 3.2: the split kernel produces per-chunk outputs and the combine
 *     kernel assembles them; oracle_combine is the log-sum-exp merge that makes
 *     "assemble" exact.
 *   - Appendix attention listing: augmented Q = W_down(act(W_gate x) * (W_up x))
 *     with x = h W_Q; the activation is read as SiLU (the model's own MLP is
 *     SwiGLU), no biases.
 *
 * Everything is computed in double from the stored (bf16 or fp32) values, which
 * convert to double exactly.  Loops are the definition written out: no
 * blocking, no online softmax, no fusion.  OpenMP is used only to spread
 * independent (sequence, head) or row work over host cores.
 *
 * Pins (tests/test_oracle_pins.py): textbook multi-head attention when
 * n_q = n_k = n_v (library softmax/matmul), K-replication identity from the
 * paper's group-sharing listing, identical keys give the mean of V, a dominant
 * key returns its V row within (len-1)e^-gap, a pure-Python brute force on tiny
 * shapes, split/combine invariance, page-table invariance, prefill row i equals
 * decode at length i+1, and hand-worked tiny cases for the augmented Q.
 * oracle_linear and oracle_rope (the projections and the rotary embedding around the cache update) are pinned
 * by a library matmul, by closed forms and by the relative-position identity; that the rotary embedding uses the
 * rotate-half pairing is a reading (the listing only names the call): "parity unpinned" for that choice.
 * oracle_decode_kup (keys cached at half width, widened by a feed-forward layer before the inner product) is pinned
 * by its reduction to oracle_decode when the layer is the identity, by a numpy restatement on small shapes, and by
 * the identity <q, W k> = <W^T q, k> against oracle_decode on folded queries; that the layer is linear, bias-free
 * and per K head is a reading: "parity unpinned" for that choice.
 * The choice of SiLU as act_fn is a reading of the paper, not pinned by it:
 * for oracle_augq the activation choice is "parity unpinned" (the rest of the
 * chain is pinned by closed forms).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { ORACLE_BF16 = 0, ORACLE_F32 = 1 };

/* Exact widening of a stored element to double. */
static double load_elt(const void *base, int64_t idx, int dtype) {
  if (dtype == ORACLE_F32) {
    return (double)((const float *)base)[idx];
  } else {
    uint32_t bits = ((uint32_t)((const uint16_t *)base)[idx]) << 16;
    float f;
    memcpy(&f, &bits, sizeof f);
    return (double)f;
  }
}

typedef struct {
  const void *k_cache, *v_cache;
  int64_t k_stride_blk, k_stride_head, k_stride_tok; /* in elements */
  int64_t v_stride_blk, v_stride_head, v_stride_tok;
  const int32_t *seqlens;    /* [batch] */
  const int32_t *page_table; /* [batch, max_pages_per_seq] or NULL */
  int32_t page_size, max_pages_per_seq;
} oracle_cache;

/* Element offset of (sequence b, token j, head, channel 0) in a cache pool.
 * Contiguous cache: blk = b, slot = j.  Paged cache: blk = page_table[b][j / page_size],
 * slot = j % page_size.  (The paper defines no page format; this is the
 * library's own layout rule restated.) */
static int64_t cache_row(const oracle_cache *c, int is_v, int b, int64_t j, int head) {
  int64_t blk = b, slot = j;
  if (c->page_table) {
    blk = c->page_table[(int64_t)b * c->max_pages_per_seq + j / c->page_size];
    slot = j % c->page_size;
  }
  if (is_v) return blk * c->v_stride_blk + (int64_t)head * c->v_stride_head + slot * c->v_stride_tok;
  return blk * c->k_stride_blk + (int64_t)head * c->k_stride_head + slot * c->k_stride_tok;
}

int oracle_set_threads(int n) {
#ifdef _OPENMP
  if (n > 0) omp_set_num_threads(n);
  return omp_get_max_threads();
#else
  (void)n;
  return 1;
#endif
}

/* Attention of one query vector q[d_qk] (already double) over tokens [t0, t1) of
 * sequence b, K head hk, V head hv.  Writes the normalised output o[d_v] and
 * lse = m + log(l).  Empty range: o = 0, lse = -inf. */
static void attend_range(const double *q, const oracle_cache *c, int dtype, int b, int hk, int hv,
                         int64_t t0, int64_t t1, int d_qk, int d_v, double scale,
                         double *o, double *lse_out) {
  for (int ch = 0; ch < d_v; ++ch) o[ch] = 0.0;
  if (t1 <= t0) { *lse_out = -INFINITY; return; }
  int64_t n = t1 - t0;
  double *s = (double *)malloc(sizeof(double) * (size_t)n);
  double m = -INFINITY;
  for (int64_t j = t0; j < t1; ++j) {
    int64_t row = cache_row(c, 0, b, j, hk);
    double acc = 0.0;
    for (int ch = 0; ch < d_qk; ++ch) acc += q[ch] * load_elt(c->k_cache, row + ch, dtype);
    acc *= scale;
    s[j - t0] = acc;
    if (acc > m) m = acc;
  }
  double l = 0.0;
  for (int64_t i = 0; i < n; ++i) { s[i] = exp(s[i] - m); l += s[i]; }
  for (int64_t j = t0; j < t1; ++j) {
    int64_t row = cache_row(c, 1, b, j, hv);
    double p = s[j - t0];
    for (int ch = 0; ch < d_v; ++ch) o[ch] += p * load_elt(c->v_cache, row + ch, dtype);
  }
  for (int ch = 0; ch < d_v; ++ch) o[ch] /= l;
  *lse_out = m + log(l);
  free(s);
}

/* Decode: one query token per sequence.
 *   q   [batch, n_q, d_qk] storage dtype, contiguous
 *   out [batch, n_q, d_v] double; lse [batch, n_q] double
 *   pairs: optional list of (b, h) pairs (n_pairs of them); when given only those
 *          rows of out / lse are computed (the others are left untouched).
 * Returns 0, or -1 when n_k or n_v does not divide n_q. */
int oracle_decode(const void *q, const oracle_cache *c, int batch, int n_q, int n_k, int n_v,
                  int d_qk, int d_v, int dtype, double scale, const int32_t *pairs, int n_pairs,
                  double *out, double *lse) {
  if (n_k <= 0 || n_v <= 0 || n_q % n_k || n_q % n_v) return -1;
  int64_t total = pairs ? n_pairs : (int64_t)batch * n_q;
#pragma omp parallel for schedule(dynamic, 1)
  for (int64_t w = 0; w < total; ++w) {
    int b = pairs ? pairs[2 * w] : (int)(w / n_q);
    int h = pairs ? pairs[2 * w + 1] : (int)(w % n_q);
    int hk = (int)(((int64_t)h * n_k) / n_q); /* Eq. (idx), floor */
    int hv = (int)(((int64_t)h * n_v) / n_q);
    double *qd = (double *)malloc(sizeof(double) * (size_t)d_qk);
    for (int ch = 0; ch < d_qk; ++ch) qd[ch] = load_elt(q, ((int64_t)b * n_q + h) * d_qk + ch, dtype);
    attend_range(qd, c, dtype, b, hk, hv, 0, c->seqlens[b], d_qk, d_v, scale,
                 out + ((int64_t)b * n_q + h) * d_v, lse + (int64_t)b * n_q + h);
    free(qd);
  }
  return 0;
}

/* Selective V cache fetching (Section "Selective V Cache Fetching"; Table topkV uses the 100 highest scores):
 * only the V vectors of the `topk` highest attention scores enter the output.  The steps, in the paper's order:
 *   1. scores s_j = scale * <q_h, K[j, hk]> for every cached token j;
 *   2. T = the topk tokens with the highest scores (equal scores: the earlier token first); all tokens if the
 *      sequence has no more than topk;
 *   3. softmax over T only (the paper does not say whether the weights are renormalised over the kept tokens;
 *      read as renormalised, as in the top-k attention it cites), o = sum_{j in T} p_j V[j, hv].
 * out [batch, n_q, d_v], lse [batch, n_q] = log sum_{j in T} exp(s_j); selected (optional) [batch, n_q, topk] int32
 * token ids in descending score order, -1 padded; margin (optional) [batch, n_q] = s_(topk) - s_(topk+1), the gap
 * that decides the selection (+inf when nothing is dropped). */
typedef struct { double s; int32_t j; } scored_token;
static int scored_cmp(const void *a, const void *b) {
  const scored_token *x = (const scored_token *)a, *y = (const scored_token *)b;
  if (x->s > y->s) return -1;
  if (x->s < y->s) return 1;
  return (x->j > y->j) - (x->j < y->j);
}
int oracle_decode_topk(const void *q, const oracle_cache *c, int batch, int n_q, int n_k, int n_v, int d_qk, int d_v,
                       int dtype, double scale, int topk, double *out, double *lse, int32_t *selected, double *margin) {
  if (n_k <= 0 || n_v <= 0 || n_q % n_k || n_q % n_v || topk <= 0) return -1;
#pragma omp parallel for schedule(dynamic, 1)
  for (int64_t w = 0; w < (int64_t)batch * n_q; ++w) {
    int b = (int)(w / n_q), h = (int)(w % n_q);
    int hk = (int)(((int64_t)h * n_k) / n_q);
    int hv = (int)(((int64_t)h * n_v) / n_q);
    int64_t len = c->seqlens[b];
    double *o = out + w * d_v;
    for (int ch = 0; ch < d_v; ++ch) o[ch] = 0.0;
    if (selected) for (int i = 0; i < topk; ++i) selected[w * topk + i] = -1;
    if (margin) margin[w] = INFINITY;
    if (len <= 0) { lse[w] = -INFINITY; continue; }
    scored_token *st = (scored_token *)malloc(sizeof(scored_token) * (size_t)len);
    for (int64_t j = 0; j < len; ++j) {
      int64_t row = cache_row(c, 0, b, j, hk);
      double acc = 0.0;
      for (int ch = 0; ch < d_qk; ++ch)
        acc += load_elt(q, ((int64_t)b * n_q + h) * d_qk + ch, dtype) * load_elt(c->k_cache, row + ch, dtype);
      st[j].s = acc * scale;
      st[j].j = (int32_t)j;
    }
    qsort(st, (size_t)len, sizeof(scored_token), scored_cmp);
    int64_t kept = len < topk ? len : topk;
    if (margin && kept < len) margin[w] = st[kept - 1].s - st[kept].s;
    double m = st[0].s, l = 0.0;
    for (int64_t i = 0; i < kept; ++i) l += exp(st[i].s - m);
    for (int64_t i = 0; i < kept; ++i) {
      double p = exp(st[i].s - m) / l;
      int64_t row = cache_row(c, 1, b, st[i].j, hv);
      for (int ch = 0; ch < d_v; ++ch) o[ch] += p * load_elt(c->v_cache, row + ch, dtype);
      if (selected) selected[w * topk + i] = st[i].j;
    }
    lse[w] = m + log(l);
    free(st);
  }
  return 0;
}

/* Decode with keys cached at a smaller width than the queries (Section 2: when the Q and K head dimensions
 * differ, "Attend" first transforms K to the query width through another feed-forward layer; Observation 2:
 * d_k = d_v / 2 with that trainable layer).  The layer is read as linear, without bias or activation, with one
 * weight matrix per K head (the paper does not print it): W_kup [n_k, d_q, d_k].  In the paper's order, for query
 * head h with K head hk and every cached token j:
 *     k'_j = W_kup[hk] k_j            (width d_k -> d_q)
 *     s_j  = scale * <q_h, k'_j>
 * then softmax over j and the weighted V sum as everywhere else.
 *   q [batch, n_q, d_q]; the K pool holds rows of d_k channels; W_kup, q and the pools share the storage dtype.
 * Returns 0, or -1 when n_k or n_v does not divide n_q. */
int oracle_decode_kup(const void *q, const void *W_kup, const oracle_cache *c, int batch, int n_q, int n_k, int n_v,
                      int d_q, int d_k, int d_v, int dtype, double scale, double *out, double *lse) {
  if (n_k <= 0 || n_v <= 0 || n_q % n_k || n_q % n_v) return -1;
#pragma omp parallel for schedule(dynamic, 1)
  for (int64_t w = 0; w < (int64_t)batch * n_q; ++w) {
    int b = (int)(w / n_q), h = (int)(w % n_q);
    int hk = (int)(((int64_t)h * n_k) / n_q);
    int hv = (int)(((int64_t)h * n_v) / n_q);
    int64_t len = c->seqlens[b];
    double *o = out + w * d_v;
    for (int ch = 0; ch < d_v; ++ch) o[ch] = 0.0;
    if (len <= 0) { lse[w] = -INFINITY; continue; }
    double *s = (double *)malloc(sizeof(double) * (size_t)len);
    double *kw = (double *)malloc(sizeof(double) * (size_t)d_q);
    double m = -INFINITY;
    for (int64_t j = 0; j < len; ++j) {
      int64_t row = cache_row(c, 0, b, j, hk);
      for (int a = 0; a < d_q; ++a) { /* the feed-forward layer on the cached key */
        double acc = 0.0;
        for (int ch = 0; ch < d_k; ++ch)
          acc += load_elt(W_kup, ((int64_t)hk * d_q + a) * d_k + ch, dtype) * load_elt(c->k_cache, row + ch, dtype);
        kw[a] = acc;
      }
      double acc = 0.0;
      for (int a = 0; a < d_q; ++a) acc += load_elt(q, w * d_q + a, dtype) * kw[a];
      s[j] = acc * scale;
      if (s[j] > m) m = s[j];
    }
    double l = 0.0;
    for (int64_t j = 0; j < len; ++j) { s[j] = exp(s[j] - m); l += s[j]; }
    for (int64_t j = 0; j < len; ++j) {
      int64_t row = cache_row(c, 1, b, j, hv);
      for (int ch = 0; ch < d_v; ++ch) o[ch] += s[j] * load_elt(c->v_cache, row + ch, dtype);
    }
    for (int ch = 0; ch < d_v; ++ch) o[ch] /= l;
    lse[w] = m + log(l);
    free(kw);
    free(s);
  }
  return 0;
}

/* Decode restricted to an explicit token range per split: cuts [n_splits + 1]
 * ascending token positions shared by all sequences (clamped to each length).
 * o_partial [batch, n_q, n_splits, d_v], lse_partial [batch, n_q, n_splits]:
 * per-split normalised outputs and log-sum-exps, the objects the combine step merges. */
int oracle_decode_splits(const void *q, const oracle_cache *c, int batch, int n_q, int n_k, int n_v,
                         int d_qk, int d_v, int dtype, double scale, const int64_t *cuts, int n_splits,
                         double *o_partial, double *lse_partial) {
  if (n_k <= 0 || n_v <= 0 || n_q % n_k || n_q % n_v) return -1;
#pragma omp parallel for schedule(dynamic, 1)
  for (int64_t w = 0; w < (int64_t)batch * n_q; ++w) {
    int b = (int)(w / n_q), h = (int)(w % n_q);
    int hk = (int)(((int64_t)h * n_k) / n_q);
    int hv = (int)(((int64_t)h * n_v) / n_q);
    double *qd = (double *)malloc(sizeof(double) * (size_t)d_qk);
    for (int ch = 0; ch < d_qk; ++ch) qd[ch] = load_elt(q, w * d_qk + ch, dtype);
    int64_t len = c->seqlens[b];
    for (int s = 0; s < n_splits; ++s) {
      int64_t t0 = cuts[s] < len ? cuts[s] : len;
      int64_t t1 = cuts[s + 1] < len ? cuts[s + 1] : len;
      attend_range(qd, c, dtype, b, hk, hv, t0, t1, d_qk, d_v, scale,
                   o_partial + (w * n_splits + s) * d_v, lse_partial + w * n_splits + s);
    }
    free(qd);
  }
  return 0;
}

/* Combine (Section 3.2, "combine kernel"): merge per-split normalised outputs.
 *   lse = log sum_s exp(lse_s) over splits with lse_s > -inf,
 *   out = sum_s exp(lse_s - lse) o_s.   All splits empty: out = 0, lse = -inf. */
void oracle_combine(const double *o_partial, const double *lse_partial, int64_t rows /* batch*n_q */,
                    int n_splits, int d_v, double *out, double *lse) {
  for (int64_t r = 0; r < rows; ++r) {
    double m = -INFINITY;
    for (int s = 0; s < n_splits; ++s)
      if (lse_partial[r * n_splits + s] > m) m = lse_partial[r * n_splits + s];
    for (int ch = 0; ch < d_v; ++ch) out[r * d_v + ch] = 0.0;
    if (m == -INFINITY) { lse[r] = -INFINITY; continue; }
    double sum = 0.0;
    for (int s = 0; s < n_splits; ++s) {
      double ls = lse_partial[r * n_splits + s];
      if (ls == -INFINITY) continue;
      sum += exp(ls - m);
    }
    double total = m + log(sum);
    for (int s = 0; s < n_splits; ++s) {
      double ls = lse_partial[r * n_splits + s];
      if (ls == -INFINITY) continue;
      double w = exp(ls - total);
      for (int ch = 0; ch < d_v; ++ch) out[r * d_v + ch] += w * o_partial[(r * n_splits + s) * d_v + ch];
    }
    lse[r] = total;
  }
}

/* Cache append done by prefill (attention listing: past_key_value.update):
 * copy rows k_new [batch, q_len, n_k, d_qk], v_new [batch, q_len, n_v, d_v] into the
 * cache at token positions past_b + i, past_b = seqlens[b] on entry.  Pure byte
 * movement; the cache pointers are written through a non-const alias. */
void oracle_cache_append(const void *k_new, const void *v_new, int q_len, const oracle_cache *c,
                         int batch, int n_k, int n_v, int d_qk, int d_v, int dtype) {
  size_t es = dtype == ORACLE_F32 ? 4 : 2;
  for (int b = 0; b < batch; ++b)
    for (int i = 0; i < q_len; ++i) {
      int64_t j = (int64_t)c->seqlens[b] + i;
      for (int h = 0; h < n_k; ++h)
        memcpy((char *)(uintptr_t)c->k_cache + es * (size_t)cache_row(c, 0, b, j, h),
               (const char *)k_new + es * (size_t)((((int64_t)b * q_len + i) * n_k + h) * d_qk), es * d_qk);
      for (int h = 0; h < n_v; ++h)
        memcpy((char *)(uintptr_t)c->v_cache + es * (size_t)cache_row(c, 1, b, j, h),
               (const char *)v_new + es * (size_t)((((int64_t)b * q_len + i) * n_v + h) * d_v), es * d_v);
    }
}

/* Causal prefill attention over a cache that already holds the new rows.
 *   q [batch, q_len, n_q, d_qk]; query row i of sequence b sits at absolute position
 *   past_b + i and sees tokens 0 .. past_b + i (bottom-right aligned causal mask);
 *   past [batch] = number of tokens that were cached before this call.
 *   rows: optional list of (b, i, h) triples (n_rows of them); out is then
 *   [n_rows, d_v] and lse [n_rows] in list order.  Without a list out is
 *   [batch, q_len, n_q, d_v] and lse [batch, q_len, n_q]. */
int oracle_prefill(const void *q, int q_len, const int32_t *past, const oracle_cache *c, int batch,
                   int n_q, int n_k, int n_v, int d_qk, int d_v, int dtype, double scale,
                   const int32_t *rows, int64_t n_rows, double *out, double *lse) {
  if (n_k <= 0 || n_v <= 0 || n_q % n_k || n_q % n_v) return -1;
  int64_t total = rows ? n_rows : (int64_t)batch * q_len * n_q;
#pragma omp parallel for schedule(dynamic, 4)
  for (int64_t w = 0; w < total; ++w) {
    int b, i, h;
    if (rows) { b = rows[3 * w]; i = rows[3 * w + 1]; h = rows[3 * w + 2]; }
    else { b = (int)(w / ((int64_t)q_len * n_q)); i = (int)((w / n_q) % q_len); h = (int)(w % n_q); }
    int hk = (int)(((int64_t)h * n_k) / n_q);
    int hv = (int)(((int64_t)h * n_v) / n_q);
    double *qd = (double *)malloc(sizeof(double) * (size_t)d_qk);
    int64_t qrow = (((int64_t)b * q_len + i) * n_q + h) * d_qk;
    for (int ch = 0; ch < d_qk; ++ch) qd[ch] = load_elt(q, qrow + ch, dtype);
    attend_range(qd, c, dtype, b, hk, hv, 0, (int64_t)past[b] + i + 1, d_qk, d_v, scale,
                 out + w * d_v, lse + w);
    free(qd);
  }
  return 0;
}

/* Augmented Q (attention listing: q_proj, then q_down_proj(act(q_gate_proj(x)) * q_up_proj(x))).
 * Weights use the nn.Linear layout [out_features, in_features], y = x W^T, no bias:
 *   W_Q [d_q0, d_model], W_gate, W_up [d_aug, d_q0], W_down [d_out, d_aug].
 *   h [T, d_model].  rows: optional list of n_rows token indices; q_out is
 *   [n_rows or T, d_out] double.  No intermediate rounding. */
void oracle_augq(const void *h, const void *W_Q, const void *W_gate, const void *W_up, const void *W_down,
                 int64_t T, int d_model, int d_q0, int d_aug, int d_out, int dtype,
                 const int64_t *rows, int64_t n_rows, double *q_out) {
  int64_t total = rows ? n_rows : T;
#pragma omp parallel for schedule(dynamic, 1)
  for (int64_t w = 0; w < total; ++w) {
    int64_t t = rows ? rows[w] : w;
    double *x = (double *)malloc(sizeof(double) * (size_t)d_q0);
    double *a = (double *)malloc(sizeof(double) * (size_t)d_aug);
    for (int o = 0; o < d_q0; ++o) {
      double acc = 0.0;
      for (int i = 0; i < d_model; ++i)
        acc += load_elt(h, t * d_model + i, dtype) * load_elt(W_Q, (int64_t)o * d_model + i, dtype);
      x[o] = acc;
    }
    for (int o = 0; o < d_aug; ++o) {
      double g = 0.0, u = 0.0;
      for (int i = 0; i < d_q0; ++i) {
        g += x[i] * load_elt(W_gate, (int64_t)o * d_q0 + i, dtype);
        u += x[i] * load_elt(W_up, (int64_t)o * d_q0 + i, dtype);
      }
      double silu = g / (1.0 + exp(-g));
      a[o] = silu * u;
    }
    for (int o = 0; o < d_out; ++o) {
      double acc = 0.0;
      for (int i = 0; i < d_aug; ++i) acc += a[i] * load_elt(W_down, (int64_t)o * d_aug + i, dtype);
      q_out[w * d_out + o] = acc;
    }
    free(x);
    free(a);
  }
}

/* Plain projection (attention listing: k_proj, v_proj, q_proj): y = x W^T with W in the nn.Linear layout
 * [out_features, in_features], no bias.  x [T, d_in] in the storage dtype, y [T, d_out] double. */
void oracle_linear(const void *x, const void *W, int64_t T, int d_in, int d_out, int dtype, double *y) {
#pragma omp parallel for schedule(static)
  for (int64_t t = 0; t < T; ++t)
    for (int o = 0; o < d_out; ++o) {
      double acc = 0.0;
      for (int i = 0; i < d_in; ++i) acc += load_elt(x, t * d_in + i, dtype) * load_elt(W, (int64_t)o * d_in + i, dtype);
      y[t * d_out + o] = acc;
    }
}

/* Rotary position embedding of the attention listing (apply_rotary_pos_emb(q, k, cos, sin)), read as the
 * rotate-half convention of the model family the listing derives from: within a head of width d, channel i < d/2
 * pairs with channel i + d/2,
 *     y_i       = x_i cos_i - x_{i+d/2} sin_i
 *     y_{i+d/2} = x_{i+d/2} cos_i + x_i sin_i,
 * with the angle of pair i at position pos being pos * theta^(-2 i / d) (the paper's model table gives
 * theta = 50 000 and 500 000).  x is [T, n_heads, d] double, rotated in place; pos is [T]. */
void oracle_rope(double *x, const int64_t *pos, int64_t T, int n_heads, int d, double theta) {
  int half = d / 2;
#pragma omp parallel for schedule(static)
  for (int64_t t = 0; t < T; ++t)
    for (int h = 0; h < n_heads; ++h) {
      double *v = x + (t * n_heads + h) * d;
      for (int i = 0; i < half; ++i) {
        double ang = (double)pos[t] * pow(theta, -2.0 * i / d);
        double c = cos(ang), s = sin(ang);
        double a = v[i], b = v[i + half];
        v[i] = a * c - b * s;
        v[i + half] = b * c + a * s;
      }
    }
}

/* KV-cache cost model, Eq. (cache_0) with alpha = element size, beta = 0:
 * bytes moved to stream the cache once for the given lengths. */
double oracle_kv_bytes(const int32_t *seqlens, int batch, int n_k, int n_v, int d_qk, int d_v, int elt_bytes) {
  double tokens = 0.0;
  for (int b = 0; b < batch; ++b) tokens += seqlens[b];
  return tokens * ((double)n_k * d_qk + (double)n_v * d_v) * elt_bytes;
}
