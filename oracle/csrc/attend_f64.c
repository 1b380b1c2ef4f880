/* Oracle attention in plain C, float64 (test infrastructure only).
 *
 * Same definition as oracle/attention.py, written as scalar loops so that it
 * can be read against the definition and still finish on full-size batches:
 * for a batch row (task, q_len n, ctx_len L) with preserved prefix p = L - n,
 * query i sits at position p + i and attends keys 0..p+i of the task's
 * preserved cache (the state Continuous Task Batching keeps across pauses,
 * paper Section 4); query head h reads KV head h / G.
 *
 *   s_j = scale * <q, k_j>, m = max s_j, l = sum exp(s_j - m),
 *   O = sum exp(s_j - m) v_j / l, LSE = m + ln l.
 *
 * Keys and values are read through a page table from token-major pools
 * [page][slot][kv_head][d] of raw bf16 bits (this oracle's own layout).
 * No blocking, no fusion: two passes over the keys per (query, head).
 * OpenMP only spreads independent (query, head) pairs over cores.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

static inline double bf16_to_f64(uint16_t bits) {
  uint32_t u = ((uint32_t)bits) << 16;
  float f;
  memcpy(&f, &u, sizeof f);
  return (double)f;
}

int tide_oracle_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

/* Returns 0, or -1 on a bad argument / allocation failure.
 *   pool_k, pool_v   [num_pages][S][Hkv][D] uint16
 *   page_tables      [n_rows][max_pages] int32, row b's logical page -> physical page
 *   row_qlen/ctx     [n_rows]; row_qoff[b] = index of row b's first query in q
 *   q                [sum q_len][Hq][D] uint16
 *   items            n_items pairs (item_row[k], item_qidx[k]) = which queries to compute
 *   out              [n_items][Hq][D] float64;  lse [n_items][Hq] float64
 */
int tide_oracle_attend_f64(const uint16_t* pool_k, const uint16_t* pool_v, int64_t num_pages,
                           int S, int Hkv, int D, int Hq,
                           const int32_t* page_tables, int max_pages, int n_rows,
                           const int32_t* row_qlen, const int32_t* row_ctx, const int64_t* row_qoff,
                           const uint16_t* q, double scale,
                           int64_t n_items, const int32_t* item_row, const int32_t* item_qidx,
                           double* out, double* lse, int n_threads) {
  if (S <= 0 || Hkv <= 0 || D <= 0 || Hq <= 0 || Hq % Hkv != 0 || n_rows < 0 || n_items < 0) return -1;
  const int G = Hq / Hkv;
  int max_ctx = 1;
  for (int b = 0; b < n_rows; ++b) {
    if (row_qlen[b] < 1 || row_ctx[b] < row_qlen[b]) return -1;
    if ((int64_t)(row_ctx[b] + S - 1) / S > max_pages) return -1;
    if (row_ctx[b] > max_ctx) max_ctx = row_ctx[b];
    for (int lp = 0; lp < (row_ctx[b] + S - 1) / S; ++lp) {
      const int64_t page = page_tables[(size_t)b * max_pages + lp];
      if (page < 0 || page >= num_pages) return -1;
    }
  }
  for (int64_t k = 0; k < n_items; ++k) {
    int b = item_row[k];
    if (b < 0 || b >= n_rows || item_qidx[k] < 0 || item_qidx[k] >= row_qlen[b]) return -1;
  }
#ifdef _OPENMP
  if (n_threads > 0) omp_set_num_threads(n_threads);
#endif
  int failed = 0;
#pragma omp parallel
  {
    double* s = (double*)malloc(sizeof(double) * (size_t)max_ctx);
    double* qv = (double*)malloc(sizeof(double) * (size_t)D);
    double* acc = (double*)malloc(sizeof(double) * (size_t)D);
    if (!s || !qv || !acc) {
#pragma omp atomic write
      failed = 1;
    }
#pragma omp barrier
    if (!failed) {
#pragma omp for schedule(dynamic, 1) collapse(2)
      for (int64_t k = 0; k < n_items; ++k) {
        for (int h = 0; h < Hq; ++h) {
          const int b = item_row[k], i = item_qidx[k];
          const int g = h / G;
          const int n = row_qlen[b], L = row_ctx[b];
          const int last = (L - n) + i; /* keys 0..last are visible */
          const int32_t* table = page_tables + (size_t)b * max_pages;
          const uint16_t* qp = q + ((size_t)(row_qoff[b] + i) * Hq + h) * D;
          for (int d = 0; d < D; ++d) qv[d] = bf16_to_f64(qp[d]);
          double m = -INFINITY;
          for (int j = 0; j <= last; ++j) {
            const int64_t page = table[j / S];
            const uint16_t* kp = pool_k + (((size_t)page * S + (j % S)) * Hkv + g) * D;
            double dot = 0.0;
            for (int d = 0; d < D; ++d) dot += qv[d] * bf16_to_f64(kp[d]);
            s[j] = scale * dot;
            if (s[j] > m) m = s[j];
          }
          double l = 0.0;
          for (int d = 0; d < D; ++d) acc[d] = 0.0;
          for (int j = 0; j <= last; ++j) {
            const int64_t page = table[j / S];
            const double w = exp(s[j] - m);
            l += w;
            const uint16_t* vp = pool_v + (((size_t)page * S + (j % S)) * Hkv + g) * D;
            for (int d = 0; d < D; ++d) acc[d] += w * bf16_to_f64(vp[d]);
          }
          double* op = out + ((size_t)k * Hq + h) * D;
          for (int d = 0; d < D; ++d) op[d] = acc[d] / l;
          lse[(size_t)k * Hq + h] = m + log(l);
        }
      }
    }
    free(s); free(qv); free(acc);
  }
  return failed ? -1 : 0;
}
