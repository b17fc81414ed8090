/*
 * ooco_oracle_fp8.c -- fp64 CPU statement of the paged decode path over an 8-bit (E4M3) KV cache.
 * TEST INFRASTRUCTURE ONLY, like ooco_oracle.c; shares no code with the CUDA sources.
 *
 * The paper's operator model carries the bytes per stored value as the parameter d (Table "Symbol
 * definitions"); d = 1 halves the KV traffic of the memory-bound decode attention (section 3.3.3).
 * Stored values are OCP 8-bit floating point E4M3 (the "fn" variant: no infinities, one NaN
 * mantissa pattern), written out from the format's definition:
 *     code = s eeee mmm,  bias 7
 *     e = 0        : (-1)^s * 2^-6 * (m / 8)                     (zero and subnormals)
 *     e = 15, m = 7: NaN
 *     otherwise    : (-1)^s * 2^(e - 7) * (1 + m / 8)            (largest finite: 448 = 0x7E)
 * A cache word stands for  decode(code) * tensor_scale  (one fp32 scale for K, one for V).
 *
 * Parity status
 *   oracle_e4m3_decode / oracle_e4m3_encode   pinned: all 256 codes and random / midpoint / saturating
 *       inputs against an independent library conversion, plus hand-worked ties
 *   oracle_decode_attention_fp8               pinned: bit-equal to oracle_decode_attention on a bf16 pool
 *       holding the dequantised values (exact for power-of-two scales)
 *   oracle_kv_append_fp8                      pinned: encode pins + the one-slot / untouched-words checks
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

static double bf16_to_f64(uint16_t bits) {
  uint32_t w = ((uint32_t)bits) << 16;
  float f;
  memcpy(&f, &w, sizeof f);
  return (double)f;
}

double oracle_e4m3_decode(uint8_t code) {
  const int s = code >> 7, e = (code >> 3) & 15, m = code & 7;
  double v;
  if (e == 15 && m == 7) return NAN;
  if (e == 0) v = ldexp((double)m / 8.0, -6);
  else v = ldexp(1.0 + (double)m / 8.0, e - 7);
  return s ? -v : v;
}

/*
 * Nearest E4M3 code of x, ties to the even code, magnitudes beyond the largest finite value
 * saturate to it, the sign is kept (also on zero), NaN gives the NaN code.  Brute force over the
 * 127 finite magnitudes, so there is no rounding logic to get wrong.
 */
uint8_t oracle_e4m3_encode(float x) {
  if (isnan(x)) return 0x7F;
  const uint8_t sign = signbit(x) ? 0x80 : 0x00;
  const double a = fabs((double)x);
  int best = 0;
  double best_err = INFINITY;
  for (int c = 0; c <= 0x7E; ++c) {
    const double err = fabs(oracle_e4m3_decode((uint8_t)c) - a);
    if (err < best_err || (err == best_err && (c & 1) == 0)) {
      best = c;
      best_err = err;
    }
  }
  return (uint8_t)(sign | best);
}

/* Same contract as oracle_decode_attention with 8-bit pools (strides in elements = bytes). */
int oracle_decode_attention_fp8(int32_t B, int32_t Hq, int32_t Hkv, int32_t D, int32_t bs,
                                int32_t num_blocks, int32_t MB, int64_t block_stride, int64_t head_stride,
                                int64_t token_stride, const uint16_t* q, const uint8_t* k_cache,
                                const uint8_t* v_cache, const int32_t* block_table,
                                const int32_t* context_lens, double scale, float k_scale, float v_scale,
                                const int32_t* pairs, int64_t n_pairs, double* out, double* lse, double* wsum) {
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
    double smax = -INFINITY;
    for (int32_t t = 0; t < T; ++t) {
      const int32_t blk = block_table[(int64_t)b * MB + t / bs];
      if (blk < 0 || blk >= num_blocks) { bad = 1; break; }
      const uint8_t* kv = k_cache + (int64_t)blk * block_stride + (int64_t)hk * head_stride +
                          (int64_t)(t % bs) * token_stride;
      double dot = 0.0;
      for (int32_t i = 0; i < D; ++i) dot += bf16_to_f64(qv[i]) * (oracle_e4m3_decode(kv[i]) * (double)k_scale);
      s[t] = scale * dot;
      if (s[t] > smax) smax = s[t];
    }
    if (bad) {
#pragma omp atomic write
      status = -2;
      free(s);
      continue;
    }
    double denom = 0.0;
    for (int32_t t = 0; t < T; ++t) {
      s[t] = exp(s[t] - smax);
      denom += s[t];
    }
    double ws = 0.0;
    for (int32_t t = 0; t < T; ++t) {
      const double w = s[t] / denom;
      ws += w;
      const int32_t blk = block_table[(int64_t)b * MB + t / bs];
      const uint8_t* vv = v_cache + (int64_t)blk * block_stride + (int64_t)hk * head_stride +
                          (int64_t)(t % bs) * token_stride;
      for (int32_t i = 0; i < D; ++i) o[i] += w * (oracle_e4m3_decode(vv[i]) * (double)v_scale);
    }
    lse[(int64_t)b * Hq + hq] = smax + log(denom);
    wsum[(int64_t)b * Hq + hq] = ws;
    free(s);
  }
  return status;
}

/*
 * Append into an 8-bit cache: the stored code of a new bf16 value x is
 *     encode( (float)x / scale )        -- one IEEE binary32 division, then nearest-even E4M3, saturating
 * Everything else as oracle_kv_append.  Returns the number of sequences written.
 */
int64_t oracle_kv_append_fp8(int32_t B, int32_t Hkv, int32_t D, int32_t bs, int32_t num_blocks, int32_t MB,
                             int64_t block_stride, int64_t head_stride, int64_t token_stride,
                             const uint16_t* k_new, const uint16_t* v_new, uint8_t* k_cache, uint8_t* v_cache,
                             const int32_t* block_table, const int32_t* positions, float k_scale, float v_scale) {
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
        const volatile float kq = (float)bf16_to_f64(k_new[src + i]) / k_scale;
        const volatile float vq = (float)bf16_to_f64(v_new[src + i]) / v_scale;
        k_cache[dst + i] = oracle_e4m3_encode(kq);
        v_cache[dst + i] = oracle_e4m3_encode(vq);
      }
    }
    ++written;
  }
  return written;
}
