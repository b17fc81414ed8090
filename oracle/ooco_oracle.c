/*
 * ooco_oracle.c -- plain, slow, fp64 CPU statement of what the paged decode
 * path computes.  TEST INFRASTRUCTURE ONLY: it is called by the tests, by the
 * smoke check and by the benchmark's cpu_baseline / reference legs; the
 * product library never links, loads or calls it, and it shares no code with
 * the CUDA sources (own bf16 decoder, own indexing).
 *
 * Parity status of each function
 *   oracle_decode_attention  pinned: brute force without max-subtraction on
 *                            gathered contiguous K/V, a library softmax
 *                            attention in fp64, and the invariants
 *                            (T = 1 returns V, equal keys give the mean of V,
 *                            block permutation, weights sum to 1, key shift,
 *                            partition merge) -- see tests/test_oracle_pins.py
 *   oracle_kv_append         pinned: definition is a verbatim word copy; the
 *                            tests check the one written slot and that every
 *                            other word is untouched, against numpy indexing
 *   oracle_bytes_model       pinned: literal enumeration of the addressed
 *                            cache slots, the Hq = Hkv case of the printed
 *                            table entry, and hand-computed golden values
 *
 * What is computed (section 2.1: decode feeds only the newest token and reuses
 * the KV cache held in a non-contiguous pool; section 2.3: every cached token
 * of every request is read, GQA shares one kv head among Hq/Hkv query heads;
 * section 3.3.1 and the operator figure: softmax attention, one fused
 * operator): for sequence b, query head hq, kv head hk = hq / (Hq / Hkv),
 *     s_t = scale * sum_i q[b,hq,i] * K[b,t,hk,i]       t = 0 .. T_b - 1
 *     w_t = exp(s_t - max s) / sum_t exp(s_t - max s)
 *     out[b,hq,:] = sum_t w_t * V[b,t,hk,:]
 * with token t of sequence b stored in slot t % bs of physical block
 * block_table[b][t / bs].  bf16 inputs are widened exactly; every product and
 * sum is fp64.  No tiling, no splitting, no reordering.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* bf16 is the upper half of an IEEE binary32: widen by placing the 16 bits on top. */
static double bf16_to_f64(uint16_t bits) {
  uint32_t w = ((uint32_t)bits) << 16;
  float f;
  memcpy(&f, &w, sizeof f);
  return (double)f;
}

int oracle_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

/*
 * pairs: optional list of n_pairs (b, hq) index pairs (int32, interleaved) to
 * compute; NULL computes all B*Hq.  Outputs are indexed [b][hq] regardless:
 *   out   fp64 [B, Hq, D]     lse  fp64 [B, Hq]  (natural log of sum_t exp(s_t))
 *   wsum  fp64 [B, Hq]        (sum of the normalised weights, ideally 1)
 * Rows that are not computed are left untouched.  T_b = 0 gives zeros, lse = -inf.
 * Returns 0, or -1 on a bad argument, -2 if a needed table entry is outside
 * [0, num_blocks).
 */
int oracle_decode_attention(int32_t B, int32_t Hq, int32_t Hkv, int32_t D, int32_t bs,
                            int32_t num_blocks, int32_t MB, int64_t block_stride,
                            int64_t head_stride, int64_t token_stride, const uint16_t* q,
                            const uint16_t* k_cache, const uint16_t* v_cache,
                            const int32_t* block_table, const int32_t* context_lens,
                            double scale, const int32_t* pairs, int64_t n_pairs, double* out,
                            double* lse, double* wsum) {
  if (B <= 0 || Hq <= 0 || Hkv <= 0 || D <= 0 || bs <= 0 || MB <= 0 || Hq % Hkv) return -1;
  const int32_t G = Hq / Hkv;
  const int64_t n_work = pairs ? n_pairs : (int64_t)B * Hq;
  int status = 0;

#pragma omp parallel for schedule(dynamic, 1)
  for (int64_t wi = 0; wi < n_work; ++wi) {
    const int32_t b = pairs ? pairs[2 * wi] : (int32_t)(wi / Hq);
    const int32_t hq = pairs ? pairs[2 * wi + 1] : (int32_t)(wi % Hq);
    const int32_t hk = hq / G;
    int32_t T = context_lens[b];
    if (T < 0) T = 0;
    if ((int64_t)T > (int64_t)MB * bs) T = MB * bs;
    double* o = out + ((int64_t)b * Hq + hq) * D;
    for (int32_t i = 0; i < D; ++i) o[i] = 0.0;
    if (T == 0) {
      lse[(int64_t)b * Hq + hq] = -INFINITY;
      wsum[(int64_t)b * Hq + hq] = 0.0;
      continue;
    }
    const uint16_t* qv = q + ((int64_t)b * Hq + hq) * D;
    double* s = (double*)malloc(sizeof(double) * (size_t)T);
    int bad = 0;

    /* scores */
    double smax = -INFINITY;
    for (int32_t t = 0; t < T; ++t) {
      const int32_t blk = block_table[(int64_t)b * MB + t / bs];
      if (blk < 0 || blk >= num_blocks) { bad = 1; break; }
      const uint16_t* kv = k_cache + (int64_t)blk * block_stride + (int64_t)hk * head_stride +
                           (int64_t)(t % bs) * token_stride;
      double dot = 0.0;
      for (int32_t i = 0; i < D; ++i) dot += bf16_to_f64(qv[i]) * bf16_to_f64(kv[i]);
      s[t] = scale * dot;
      if (s[t] > smax) smax = s[t];
    }
    if (bad) {
#pragma omp atomic write
      status = -2;
      free(s);
      continue;
    }
    /* softmax weights */
    double denom = 0.0;
    for (int32_t t = 0; t < T; ++t) {
      s[t] = exp(s[t] - smax);
      denom += s[t];
    }
    double ws = 0.0;
    /* weighted sum of values */
    for (int32_t t = 0; t < T; ++t) {
      const double w = s[t] / denom;
      ws += w;
      const int32_t blk = block_table[(int64_t)b * MB + t / bs];
      const uint16_t* vv = v_cache + (int64_t)blk * block_stride + (int64_t)hk * head_stride +
                           (int64_t)(t % bs) * token_stride;
      for (int32_t i = 0; i < D; ++i) o[i] += w * bf16_to_f64(vv[i]);
    }
    lse[(int64_t)b * Hq + hq] = smax + log(denom);
    wsum[(int64_t)b * Hq + hq] = ws;
    free(s);
  }
  return status;
}

/*
 * KV append (section 2.1, "expands the KV cache"): the head_dim 16-bit words
 * of k_new[b,h,:] / v_new[b,h,:] go, unchanged, to slot positions[b] % bs of
 * block block_table[b][positions[b] / bs].  A sequence whose position is
 * negative or beyond the table, or whose table entry is outside the pool, is
 * skipped.  Returns the number of sequences written.
 */
int64_t oracle_kv_append(int32_t B, int32_t Hkv, int32_t D, int32_t bs, int32_t num_blocks,
                         int32_t MB, int64_t block_stride, int64_t head_stride,
                         int64_t token_stride, const uint16_t* k_new, const uint16_t* v_new,
                         uint16_t* k_cache, uint16_t* v_cache, const int32_t* block_table,
                         const int32_t* positions) {
  int64_t written = 0;
  for (int32_t b = 0; b < B; ++b) {
    const int32_t pos = positions[b];
    if (pos < 0 || (int64_t)pos >= (int64_t)MB * bs) continue;
    const int32_t blk = block_table[(int64_t)b * MB + pos / bs];
    if (blk < 0 || blk >= num_blocks) continue;
    for (int32_t h = 0; h < Hkv; ++h) {
      const int64_t dst = (int64_t)blk * block_stride + (int64_t)h * head_stride +
                          (int64_t)(pos % bs) * token_stride;
      const int64_t src = ((int64_t)b * Hkv + h) * D;
      for (int32_t i = 0; i < D; ++i) {
        k_cache[dst + i] = k_new[src + i];
        v_cache[dst + i] = v_new[src + i];
      }
    }
    ++written;
  }
  return written;
}

/*
 * Attention row of Table "Operator Modeling" per sequence, S_q = 1, S_kv = T_b,
 * D_h = Hq * D (the FLOP entry 4 * D_h * S_q * S_kv carries no separate head
 * factor, so D_h spans all query heads):
 *     flops    = 4 * D_h * T_b
 *     memory   = 2 d (S_q D_h + S_kv D_h * Hkv / Hq)
 * The table prints the ratio as Hq / Hkv; that reading would make GQA raise
 * KV traffic, against section 2.3, so the ratio is taken as Hkv / Hq.  The
 * first term is q plus out (d * D_h each), the second K plus V.
 * cost[7] = { flops, bytes_q, bytes_out, bytes_kv, bytes_index, bytes_paper, total_tokens }.
 */
int oracle_bytes_model(int32_t B, int32_t Hq, int32_t Hkv, int32_t D, int32_t bs,
                       const int32_t* context_lens, int32_t d, int64_t* cost) {
  if (B <= 0 || Hq <= 0 || Hkv <= 0 || D <= 0 || bs <= 0 || d <= 0 || Hq % Hkv) return -1;
  for (int i = 0; i < 7; ++i) cost[i] = 0;
  const int64_t Dh = (int64_t)Hq * D;
  for (int32_t b = 0; b < B; ++b) {
    const int64_t T = context_lens[b] > 0 ? context_lens[b] : 0;
    cost[0] += 4 * Dh * 1 * T;
    cost[1] += (int64_t)d * 1 * Dh;
    cost[2] += (int64_t)d * 1 * Dh;
    cost[3] += 2 * (int64_t)d * T * (Dh * Hkv / Hq);
    cost[4] += 4 * (1 + (T + bs - 1) / bs);
    cost[6] += T;
  }
  cost[5] = cost[1] + cost[2] + cost[3];
  return 0;
}
