/*
 * CPU oracle for lookahead importance scoring, pooling, top-C selection, K/V
 * compaction and the SpecPC keep set.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the plain, slow, fp64 statement of
 * what the method computes; tests and the benchmark's cpu baseline call it, the
 * product (the CUDA library) never does and shares no code with it.
 *
 * Every function writes out the definition it cites with no tiling, no online
 * softmax and no reordering beyond the loops of the definition itself.  bf16
 * inputs are widened exactly to double; all arithmetic is double.
 *
 * Parity status: every function below is pinned by the CPU test-suite (brute
 * force on tiny inputs, closed forms, library special cases, invariants).
 * Pooling with an EVEN width has no centre and the paper does not say where
 * the window sits; the window used, [j - k/2, j + k/2 - 1], is pinned to the
 * first n outputs of the library pooling routine with padding k/2.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

static double bf16_to_double(uint16_t b) {
  uint32_t u = ((uint32_t)b) << 16;
  float f;
  memcpy(&f, &u, sizeof f);
  return (double)f;
}

int oracle_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

/*
 * Importance scores (Eq. 1; Algorithm 1 lines 8-9; Algorithm 2 lines 4-7).
 *
 * For every sequence s (keys cu[s] .. cu[s+1]-1), layer l and KV head h, and for
 * every query head g of the GQA group of h and every query row r (window rows
 * first, in prompt order, then lookahead rows):
 *     S[j] = scale * <q[s,l,g,r,:], k[l,h,cu[s]+j,:]>
 *     p[j] = exp(S[j] - max S) / sum_j exp(S[j] - max S)          (row softmax)
 *     mode 0:  score[j] += w[r] * p[j]      (sum; dividing by the number of rows gives Eq. 1's mean)
 *     mode 1:  score[j]  = max(score[j], w[r] * p[j])             (Algorithm 1 line 9, MaxReduce)
 * causal_window != 0 masks, for window row r, the keys after that row's own
 * prompt position n - n_window + r.
 *
 * q      [n_seq, L, Hq, R, d] bf16 bits, contiguous
 * k      bf16 bits, element (l, h, t, c) at l*ks_layer + h*ks_head + t*ks_token + c
 * scores [L, Hkv, T] double
 */
int oracle_spec_score(const uint16_t* q, const uint16_t* k, int64_t ks_layer, int64_t ks_head,
                      int64_t ks_token, int n_seq, const int32_t* cu, int L, int Hq, int Hkv, int d,
                      int n_lookahead, int n_window, double scale, const double* row_weight, int mode,
                      int causal_window, int64_t T, double* scores) {
  if (n_seq < 1 || L < 1 || Hkv < 1 || Hq % Hkv != 0 || d < 1) return -1;
  const int R = n_lookahead + n_window;
  const int G = Hq / Hkv;
  if (R < 1) return -1;
  const int64_t n_units = (int64_t)n_seq * L * Hkv;
  int fail = 0;
#pragma omp parallel for schedule(dynamic, 1)
  for (int64_t u = 0; u < n_units; ++u) {
    const int s = (int)(u / ((int64_t)L * Hkv));
    const int l = (int)((u / Hkv) % L);
    const int h = (int)(u % Hkv);
    const int64_t b = cu[s];
    const int n = cu[s + 1] - cu[s];
    if (n <= 0) continue;
    double* out = scores + ((int64_t)l * Hkv + h) * T + b;
    double* S = (double*)malloc(sizeof(double) * (size_t)n);
    double* qrow = (double*)malloc(sizeof(double) * (size_t)d);
    if (!S || !qrow) { fail = 1; free(S); free(qrow); continue; }
    for (int j = 0; j < n; ++j) out[j] = 0.0;
    for (int gi = 0; gi < G; ++gi) {
      const int g = h * G + gi;
      for (int r = 0; r < R; ++r) {
        const uint16_t* qp = q + ((((int64_t)s * L + l) * Hq + g) * R + r) * d;
        for (int c = 0; c < d; ++c) qrow[c] = bf16_to_double(qp[c]);
        int n_vis = n; /* number of visible keys for this row */
        if (causal_window && r < n_window) {
          int last = n - n_window + r; /* this row's own prompt position */
          if (last < 0) last = 0;
          n_vis = last + 1;
          if (n_vis > n) n_vis = n;
        }
        double m = -INFINITY;
        for (int j = 0; j < n_vis; ++j) {
          const uint16_t* kp = k + (int64_t)l * ks_layer + (int64_t)h * ks_head + (b + j) * ks_token;
          double acc = 0.0;
          for (int c = 0; c < d; ++c) acc += qrow[c] * bf16_to_double(kp[c]);
          S[j] = scale * acc;
          if (S[j] > m) m = S[j];
        }
        double Z = 0.0;
        for (int j = 0; j < n_vis; ++j) Z += exp(S[j] - m);
        const double w = row_weight ? row_weight[r] : 1.0;
        for (int j = 0; j < n_vis; ++j) {
          const double p = w * (exp(S[j] - m) / Z);
          if (mode == 0) out[j] += p;
          else if (p > out[j]) out[j] = p;
        }
      }
    }
    free(S);
    free(qrow);
  }
  return fail ? -2 : 0;
}

/*
 * 1-D pooling, stride 1, same length (Algorithm 1 line 10; hyper-parameter table:
 * SpecKV pools with Max, k = 7).  The window of position j is
 * [j - floor(k/2), j - floor(k/2) + k - 1] clipped to [0, n).
 *   pool 0: maximum over the clipped window.
 *   pool 1: sum over the clipped window divided by k (zero padding).
 */
int oracle_pool(const double* s, int n, int pool, int k, double* out) {
  if (k < 1) return -1;
  const int left = k / 2;
  for (int j = 0; j < n; ++j) {
    int lo = j - left, hi = j - left + k - 1;
    if (lo < 0) lo = 0;
    if (hi > n - 1) hi = n - 1;
    if (pool == 0) {
      double m = s[lo];
      for (int t = lo + 1; t <= hi; ++t)
        if (s[t] > m) m = s[t];
      out[j] = m;
    } else {
      double a = 0.0;
      for (int t = lo; t <= hi; ++t) a += s[t];
      out[j] = a / (double)k;
    }
  }
  return 0;
}

typedef struct {
  double v;
  int32_t i;
} oracle_pair;

static int cmp_desc_value_then_index(const void* a, const void* b) {
  const oracle_pair* x = (const oracle_pair*)a;
  const oracle_pair* y = (const oracle_pair*)b;
  if (x->v > y->v) return -1;
  if (x->v < y->v) return 1;
  return (x->i > y->i) - (x->i < y->i);
}

static int cmp_int32(const void* a, const void* b) {
  const int32_t x = *(const int32_t*)a, y = *(const int32_t*)b;
  return (x > y) - (x < y);
}

/*
 * Top-n_take positions of v[0..n) by value; equal values: lower position wins.
 * Full sort of (value descending, position ascending), first n_take taken, then
 * returned in ascending position.  *thresh receives the smallest selected value.
 */
static int select_top(const double* v, int n, int n_take, int32_t* out, double* thresh) {
  if (n_take > n) n_take = n;
  if (n_take <= 0) { if (thresh) *thresh = INFINITY; return 0; }
  oracle_pair* p = (oracle_pair*)malloc(sizeof(oracle_pair) * (size_t)n);
  if (!p) return -1;
  for (int j = 0; j < n; ++j) { p[j].v = v[j]; p[j].i = j; }
  qsort(p, (size_t)n, sizeof(oracle_pair), cmp_desc_value_then_index);
  for (int c = 0; c < n_take; ++c) out[c] = p[c].i;
  if (thresh) *thresh = p[n_take - 1].v;
  free(p);
  qsort(out, (size_t)n_take, sizeof(int32_t), cmp_int32);
  return n_take;
}

/*
 * Pool + top-C per (sequence, layer, KV head) (Algorithm 1 lines 10 and 13).
 *
 * With e = n - min(n_forced_tail, n) eligible positions [0, e): pool the scores of
 * the eligible range (window clipped to it), keep the min(c_max - forced, e)
 * best, add the forced tail [e, n) (Algorithm 1 line 13: the last n_window KV
 * pairs are always kept), emit ascending sequence-local positions; unused slots
 * are -1 and count_out holds the number of valid entries.
 *
 * scores [L, Hkv, T]; idx_out [n_seq, L, Hkv, c_max]; count_out [n_seq, L, Hkv];
 * pooled_out (optional) [L, Hkv, T]; thresh_out (optional) [n_seq, L, Hkv] = pooled
 * value of the weakest selected eligible position (+inf if none).
 */
int oracle_pool_topk(const double* scores, int n_seq, const int32_t* cu, int L, int Hkv, int64_t T,
                     int pool, int k, int c_max, int n_forced_tail, int32_t* idx_out,
                     int32_t* count_out, double* pooled_out, double* thresh_out) {
  if (c_max < 1 || n_forced_tail < 0 || n_forced_tail > c_max || k < 1) return -1;
  const int64_t n_units = (int64_t)n_seq * L * Hkv;
  int fail = 0;
#pragma omp parallel for schedule(dynamic, 1)
  for (int64_t u = 0; u < n_units; ++u) {
    const int s = (int)(u / ((int64_t)L * Hkv));
    const int l = (int)((u / Hkv) % L);
    const int h = (int)(u % Hkv);
    const int64_t b = cu[s];
    const int n = cu[s + 1] - cu[s];
    int32_t* idx = idx_out + u * (int64_t)c_max;
    for (int c = 0; c < c_max; ++c) idx[c] = -1;
    const int forced = n_forced_tail < n ? n_forced_tail : n;
    const int e = n - forced;
    int count = 0;
    double th = INFINITY;
    if (e > 0) {
      const double* sc = scores + ((int64_t)l * Hkv + h) * T + b;
      double* pooled = (double*)malloc(sizeof(double) * (size_t)e);
      if (!pooled) { fail = 1; continue; }
      oracle_pool(sc, e, pool, k, pooled);
      if (pooled_out) memcpy(pooled_out + ((int64_t)l * Hkv + h) * T + b, pooled, sizeof(double) * (size_t)e);
      int r = select_top(pooled, e, c_max - forced, idx, &th);
      if (r < 0) fail = 1; else count = r;
      free(pooled);
    }
    for (int t = 0; t < forced; ++t) idx[count++] = e + t;
    if (count_out) count_out[u] = count;
    if (thresh_out) thresh_out[u] = th;
  }
  return fail ? -2 : 0;
}

/*
 * K/V compaction (Algorithm 1 line 15): row c of the compacted cache of
 * (sequence s, layer l, KV head h) is the source row cu[s] + idx[s,l,h,c]; rows
 * with idx == -1 are zero.  Rows are d bf16 values copied as bytes.
 *
 * block_table == NULL : dst [n_seq, L, Hkv, c_max, d]
 * else                : dst [L, n_pages, Hkv, page_size, d], slot c of sequence s
 *                       lives in page block_table[s, c / page_size], row c % page_size.
 */
int oracle_compact(const uint16_t* src, int64_t st_layer, int64_t st_head, int64_t st_token,
                   int n_seq, const int32_t* cu, int L, int Hkv, int d, const int32_t* idx, int c_max,
                   uint16_t* dst, const int32_t* block_table, int page_size, int n_pages) {
  const int ppseq = block_table ? (c_max + page_size - 1) / page_size : 0;
  for (int s = 0; s < n_seq; ++s)
    for (int l = 0; l < L; ++l)
      for (int h = 0; h < Hkv; ++h)
        for (int c = 0; c < c_max; ++c) {
          const int32_t i = idx[(((int64_t)s * L + l) * Hkv + h) * c_max + c];
          uint16_t* out;
          if (block_table) {
            const int32_t page = block_table[(int64_t)s * ppseq + c / page_size];
            if (page < 0 || page >= n_pages) return -1;
            out = dst + ((((int64_t)l * n_pages + page) * Hkv + h) * page_size + c % page_size) * d;
          } else {
            out = dst + ((((int64_t)s * L + l) * Hkv + h) * c_max + c) * d;
          }
          if (i < 0) {
            memset(out, 0, sizeof(uint16_t) * (size_t)d);
          } else {
            if (i >= cu[s + 1] - cu[s]) return -1;
            const uint16_t* in = src + (int64_t)l * st_layer + (int64_t)h * st_head + ((int64_t)cu[s] + i) * st_token;
            memcpy(out, in, sizeof(uint16_t) * (size_t)d);
          }
        }
  return 0;
}

/*
 * SpecPC keep set (Algorithm 2 lines 7-10, with the aggregation, pooling and
 * neighbour handling selected by arguments).
 *
 * Per sequence: t[j] = reduce over all (layer, KV head) of scores[l,h,cu[s]+j]
 * (reduce 0 = sum in (l, h) order, 1 = max; Algorithm 2 line 7 uses max), pool over
 * the eligible range [0, n - forced) (pool 2: the printed order of Algorithm 2 lines
 * 8-9, average pool of k then max pool of n_neighbor, and no widening below), keep
 * the c_max best (Algorithm 2 line 10),
 * widen every kept position i to [i - n_neighbor, i + n_neighbor] clipped to the
 * eligible range, add the forced tail (the always-kept window), and return the
 * ascending list of distinct positions.
 *
 * keep_out [n_seq, keep_capacity] (-1 padded), n_keep_out [n_seq],
 * token_out (optional) [T] pooled token scores, thresh_out (optional) [n_seq].
 */
int oracle_specpc_select(const double* scores, int n_seq, const int32_t* cu, int L, int Hkv, int64_t T,
                         int reduce, int pool, int k, int c_max, int n_neighbor, int n_forced_tail,
                         int32_t* keep_out, int keep_capacity, int32_t* n_keep_out, double* token_out,
                         double* thresh_out) {
  if (c_max < 1 || n_neighbor < 0 || n_forced_tail < 0 || k < 1) return -1;
  for (int s = 0; s < n_seq; ++s) {
    const int64_t b = cu[s];
    const int n = cu[s + 1] - cu[s];
    int32_t* keep = keep_out + (int64_t)s * keep_capacity;
    for (int c = 0; c < keep_capacity; ++c) keep[c] = -1;
    n_keep_out[s] = 0;
    if (thresh_out) thresh_out[s] = INFINITY;
    if (n <= 0) continue;
    const int forced = n_forced_tail < n ? n_forced_tail : n;
    const int e = n - forced;
    unsigned char* mark = (unsigned char*)calloc((size_t)n, 1);
    if (!mark) return -2;
    if (e > 0) {
      double* t = (double*)malloc(sizeof(double) * (size_t)e);
      double* pooled = (double*)malloc(sizeof(double) * (size_t)e);
      int32_t* top = (int32_t*)malloc(sizeof(int32_t) * (size_t)(c_max < e ? c_max : e));
      if (!t || !pooled || !top) return -2;
      for (int j = 0; j < e; ++j) {
        double a = reduce == 0 ? 0.0 : -INFINITY;
        for (int l = 0; l < L; ++l)
          for (int h = 0; h < Hkv; ++h) {
            const double v = scores[((int64_t)l * Hkv + h) * T + b + j];
            if (reduce == 0) a += v;
            else if (v > a) a = v;
          }
        t[j] = a;
      }
      int widen = n_neighbor;
      if (pool == 2) {
        /* Algorithm 2 lines 8-9 in the printed order: AvgPool1D(k), then MaxPool1D(n_neighbor)
         * before the selection; nothing is widened afterwards. */
        double* avg = (double*)malloc(sizeof(double) * (size_t)e);
        if (!avg) return -2;
        oracle_pool(t, e, 1, k, avg);
        oracle_pool(avg, e, 0, n_neighbor > 1 ? n_neighbor : 1, pooled);
        free(avg);
        widen = 0;
      } else {
        oracle_pool(t, e, pool, k, pooled);
      }
      if (token_out) memcpy(token_out + b, pooled, sizeof(double) * (size_t)e);
      double th;
      const int n_top = select_top(pooled, e, c_max, top, &th);
      if (n_top < 0) return -2;
      if (thresh_out) thresh_out[s] = th;
      for (int c = 0; c < n_top; ++c) {
        int lo = top[c] - widen, hi = top[c] + widen;
        if (lo < 0) lo = 0;
        if (hi > e - 1) hi = e - 1;
        for (int j = lo; j <= hi; ++j) mark[j] = 1;
      }
      free(t); free(pooled); free(top);
    }
    for (int j = e; j < n; ++j) mark[j] = 1;
    int cnt = 0;
    for (int j = 0; j < n; ++j)
      if (mark[j]) {
        if (cnt >= keep_capacity) { free(mark); return -3; }
        keep[cnt++] = j;
      }
    n_keep_out[s] = cnt;
    free(mark);
  }
  return 0;
}
