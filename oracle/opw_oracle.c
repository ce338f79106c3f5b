/*
 * CPU oracle for the decode-time core-attention stage (TEST INFRASTRUCTURE ONLY).
 *
 * This file is the slow, plain, fp64 statement of what the stage computes.  It is
 * used by the tests, by the smoke check and by the benchmark's CPU-baseline leg and
 * by nothing else; the product path never calls it.  It shares no code, header,
 * table or helper with the CUDA path: the pool indexing below is re-derived from
 * the documented layout formula, not included from the library.
 *
 * What the paper fixes (and what it leaves open):
 *   - The stage is "core attention only": projections, position encoding and the
 *     output projection live in other stages (Section 4, the CAD template; Section
 *     3.4 "From Bounds to Plans").  So q, k_new, v_new arrive ready to use.
 *   - The KV cache is paged and resident on the stage; only token, position and
 *     KV-cache metadata change between iterations (Section 6, first paragraph).
 *   - Layer types: full attention reads the KV cache of the entire context, a
 *     sliding-window layer reads a bounded window (Section 3.4, second limitation).
 *   - The paper prints no formula for attention itself.  The result is the textbook
 *     softmax attention, so the oracle is that definition written out:
 *         s_j = scale * <q_h, K_j>,  out_h = sum_j softmax(s)_j V_j,
 *         lse_h = log sum_j exp(s_j)
 *     over the visible keys j in [lo, n), with grouped-query heads h -> kv head
 *     h / G (contiguous groups), n = number of keys after this step's append,
 *     lo = 0 for a full layer and max(0, n - W) for a window of W keys that
 *     includes the current token.
 *
 * Parity pins (tests marked "not gpu"): pure-Python brute force on tiny inputs,
 * torch's float64 scaled_dot_product_attention on dense contiguous pages, the
 * closed forms for a single key and for identical keys, q = 0 coverage probes,
 * page-permutation invariance, window == full attention over the truncated cache.
 * The GQA head map, the softmax scale and the window convention are conventions
 * the paper does not state; they are pinned only by agreement with the torch
 * routine and the probes (declared readings, not paper values).
 *
 * Pool layout (one layer), 16-bit elements.  Element (page p, kv head g,
 * kv in {K=0, V=1}, slot t, dim d) lives at
 *     ((((p*Hkv + g)*2 + kv)*P + t)*D) + (((d/8) ^ (t & 7))*8) + (d % 8)
 * i.e. each (page, head) owns one contiguous K tile followed by one V tile, each
 * P rows of D elements, and inside a row the 16-byte groups are permuted by an
 * XOR with the low three bits of the slot.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

/* bf16 (upper 16 bits of an IEEE float) widened exactly to double. */
static double bf16_to_f64(uint16_t h) {
  uint32_t u = ((uint32_t)h) << 16;
  float f;
  memcpy(&f, &u, sizeof f);
  return (double)f;
}

int64_t opw_oracle_pool_index(int64_t Hkv, int64_t P, int64_t D, int64_t p, int64_t g,
                              int64_t kv, int64_t t, int64_t d) {
  int64_t row = (((p * Hkv + g) * 2 + kv) * P + t) * D;
  int64_t grp = (d / 8) ^ (t & 7);
  return row + grp * 8 + (d % 8);
}

int opw_oracle_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

/*
 * Naive append (Section 6: KV-cache metadata and contents change every iteration).
 * For every batch row with positions[b] >= 0 the new key and value rows are copied,
 * as raw 16-bit words, into slot positions[b] % P of page
 * page_table[b][positions[b] / P].  Returns 0, or -1 if a referenced page id is
 * outside [0, num_pages) (nothing is written for that row).
 */
int opw_oracle_kv_append(uint16_t *pool, int64_t num_pages, int64_t Hkv, int64_t D, int64_t P,
                         int64_t B, const uint16_t *k_new, const uint16_t *v_new,
                         const int32_t *positions, const int32_t *page_table,
                         int64_t max_pages_per_seq) {
  int rc = 0;
  for (int64_t b = 0; b < B; ++b) {
    int64_t pos = positions[b];
    if (pos < 0) continue;
    int64_t lp = pos / P;
    if (lp >= max_pages_per_seq) { rc = -1; continue; }
    int64_t pg = page_table[b * max_pages_per_seq + lp];
    int64_t t = pos % P;
    if (pg < 0 || pg >= num_pages) { rc = -1; continue; }
    for (int64_t g = 0; g < Hkv; ++g)
      for (int64_t d = 0; d < D; ++d) {
        pool[opw_oracle_pool_index(Hkv, P, D, pg, g, 0, t, d)] = k_new[(b * Hkv + g) * D + d];
        pool[opw_oracle_pool_index(Hkv, P, D, pg, g, 1, t, d)] = v_new[(b * Hkv + g) * D + d];
      }
  }
  return rc;
}

/*
 * Softmax attention of one query token per sequence over that sequence's pages.
 *   kv_lens[b] = n_b, keys visible after the append (<= 0: inactive row, out = 0,
 *   lse = -inf).  window = 0: full; window = W > 0: keys [max(0, n-W), n).
 * out is [B, Hq, D] and lse is [B, Hq], both double.  Only rows listed in
 * rows[0..n_rows) are computed when rows != NULL (used to sample huge batches);
 * the others are left untouched.
 * Returns 0, or -1 if a page id inside a visible range is out of bounds.
 */
int opw_oracle_decode_attention(const uint16_t *pool, int64_t num_pages, int64_t Hq, int64_t Hkv,
                                int64_t D, int64_t P, int64_t B, const uint16_t *q,
                                const int32_t *kv_lens, const int32_t *page_table,
                                int64_t max_pages_per_seq, int64_t window, double scale,
                                const int32_t *rows, int64_t n_rows, double *out, double *lse) {
  const int64_t G = Hq / Hkv;
  const int64_t nb = rows ? n_rows : B;
  int rc = 0;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
  for (int64_t bi = 0; bi < nb; ++bi) {
    for (int64_t h = 0; h < Hq; ++h) {
      const int64_t b = rows ? rows[bi] : bi;
      const int64_t n = kv_lens[b];
      double *o = out + (b * Hq + h) * D;
      if (n <= 0) {
        for (int64_t d = 0; d < D; ++d) o[d] = 0.0;
        lse[b * Hq + h] = -INFINITY;
        continue;
      }
      const int64_t g = h / G;
      const int64_t lo = (window > 0 && n > window) ? n - window : 0;
      const int64_t cnt = n - lo;
      double *s = (double *)malloc(sizeof(double) * (size_t)cnt);
      double *acc = (double *)calloc((size_t)D, sizeof(double));
      int bad = 0;
      /* scores */
      double m = -INFINITY;
      for (int64_t j = lo; j < n; ++j) {
        int64_t pg = page_table[b * max_pages_per_seq + j / P];
        if (pg < 0 || pg >= num_pages) { bad = 1; break; }
        int64_t t = j % P;
        double dot = 0.0;
        for (int64_t d = 0; d < D; ++d)
          dot += bf16_to_f64(q[(b * Hq + h) * D + d]) *
                 bf16_to_f64(pool[opw_oracle_pool_index(Hkv, P, D, pg, g, 0, t, d)]);
        s[j - lo] = scale * dot;
        if (s[j - lo] > m) m = s[j - lo];
      }
      if (bad) {
#pragma omp atomic write
        rc = -1;
        for (int64_t d = 0; d < D; ++d) o[d] = NAN;
        lse[b * Hq + h] = NAN;
        free(s);
        free(acc);
        continue;
      }
      /* softmax weights and the weighted sum of values */
      double l = 0.0;
      for (int64_t j = lo; j < n; ++j) {
        double pj = exp(s[j - lo] - m);
        l += pj;
        int64_t pg = page_table[b * max_pages_per_seq + j / P];
        int64_t t = j % P;
        for (int64_t d = 0; d < D; ++d)
          acc[d] += pj * bf16_to_f64(pool[opw_oracle_pool_index(Hkv, P, D, pg, g, 1, t, d)]);
      }
      for (int64_t d = 0; d < D; ++d) o[d] = acc[d] / l;
      lse[b * Hq + h] = m + log(l);
      free(s);
      free(acc);
    }
  }
  return rc;
}
