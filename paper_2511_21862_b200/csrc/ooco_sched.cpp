// Host side of ooco_sched.h: Roofline latency predictor and the step-level scheduling decisions
// built on it.  Plain C++ on 64-bit integers and doubles; no CUDA.
//
// For a decode batch every operator count is an affine function of the batch size n and of the
// total number of cached tokens, so L(B) is evaluated in O(1) from (n, tokens): the selection
// algorithms keep those two integers as running sums and never rebuild a batch.
#include <algorithm>
#include <cmath>
#include <cstdint>
#include <numeric>
#include <vector>

#include "../../include/ooco.h"
#include "../../include/ooco_sched.h"

namespace {

struct Predictor {
  const ooco_model_t* m;
  const ooco_hw_params_t* hw;
  int64_t hq, hkv, D_h;

  bool init(const ooco_model_t* model, const ooco_hw_params_t* h) {
    m = model;
    hw = h;
    if (!m || !hw) return false;
    if (m->num_layers <= 0 || m->hidden <= 0 || m->num_q_heads <= 0 || m->num_kv_heads <= 0 || m->head_dim <= 0 ||
        m->intermediate <= 0 || m->vocab <= 0 || m->bytes_per_value <= 0 || m->tp <= 0)
      return false;
    if (m->num_q_heads % m->num_kv_heads || m->num_q_heads % m->tp || m->num_kv_heads % m->tp) return false;
    if (m->intermediate % m->tp || m->vocab % m->tp) return false;
    if (!(hw->F_g > 0) || !(hw->F_ad > 0) || !(hw->M_g > 0) || !(hw->M_a > 0) || !(hw->O_d >= 0)) return false;
    if (m->tp > 1 && !(hw->B_c > 0)) return false;
    hq = m->num_q_heads / m->tp;
    hkv = m->num_kv_heads / m->tp;
    D_h = hq * m->head_dim;
    return true;
  }

  // One GEMM of Table "Operator Modeling": adds its latency to `t`, its two roofline terms to fl / by.
  void gemm(double N, double Din, double Dout, double& t, double& fl, double& by) const {
    const double f = 2.0 * N * Din * Dout / hw->F_g;
    const double b = m->bytes_per_value * (N * Din + Din * Dout + N * Dout) / hw->M_g;
    t += std::max(f, b);
    fl += f;
    by += b;
  }

  void eval(int64_t n, int64_t tokens, ooco_latency_t* o) const {
    o->gemm = o->attention = o->comm = 0.0;
    o->overhead = hw->O_d;
    o->gemm_compute_bound = o->attention_compute_bound = 0;
    if (n > 0) {
      const double N = (double)n, d = m->bytes_per_value;
      double layer = 0.0, fl = 0.0, by = 0.0;
      gemm(N, m->hidden, (double)(hq + 2 * hkv) * m->head_dim, layer, fl, by);
      gemm(N, (double)D_h, m->hidden, layer, fl, by);
      gemm(N, m->hidden, (double)(m->gated_mlp ? 2 : 1) * m->intermediate / m->tp, layer, fl, by);
      gemm(N, (double)m->intermediate / m->tp, m->hidden, layer, fl, by);
      double head = 0.0, hfl = 0.0, hby = 0.0;
      gemm(N, m->hidden, (double)m->vocab / m->tp, head, hfl, hby);
      o->gemm = layer * m->num_layers + head;
      o->gemm_compute_bound = fl * m->num_layers + hfl >= by * m->num_layers + hby;
      // attention row, S_q = 1, summed over the batch; K/V width D_h * Hkv / Hq
      const double a_fl = 4.0 * (double)D_h * (double)tokens / hw->F_ad;
      const double a_by = 2.0 * d * ((double)n * D_h + (double)tokens * (double)(hkv * m->head_dim)) / hw->M_a;
      o->attention = std::max(a_fl, a_by) * m->num_layers;
      o->attention_compute_bound = a_fl >= a_by;
      if (m->tp > 1) o->comm = 2.0 * m->num_layers * (N * m->hidden * d / hw->B_c);
    }
    o->total = o->gemm + o->attention + o->comm + o->overhead;
  }

  double L(int64_t n, int64_t tokens) const {
    ooco_latency_t o;
    eval(n, tokens, &o);
    return o.total;
  }
};

inline int64_t clamp_len(int32_t t) { return t > 0 ? t : 0; }

}  // namespace

extern "C" {

int ooco_predict_decode_latency(const ooco_model_t* model, const ooco_hw_params_t* hw, int64_t batch_size,
                                int64_t total_tokens, ooco_latency_t* out) {
  if (!model || !hw || !out) return OOCO_E_NULLPTR;
  Predictor p;
  if (!p.init(model, hw) || batch_size < 0 || total_tokens < 0) return OOCO_E_SHAPE;
  p.eval(batch_size, total_tokens, out);
  return OOCO_OK;
}

int ooco_predict_prefill_latency(const ooco_model_t* model, const ooco_hw_params_t* hw, const int32_t* prompt_lens,
                                 int32_t n, ooco_latency_t* out) {
  if (!model || !hw || !out || (n > 0 && !prompt_lens)) return OOCO_E_NULLPTR;
  Predictor p;
  if (!p.init(model, hw) || n < 0 || !(hw->F_ap > 0) || !(hw->O_p >= 0)) return OOCO_E_SHAPE;
  const ooco_model_t* m = model;
  double N = 0.0, sq = 0.0, reqs = 0.0;  // prompt tokens, sum of squared prompt lengths, requests
  for (int32_t i = 0; i < n; ++i) {
    if (prompt_lens[i] <= 0) continue;
    N += prompt_lens[i];
    sq += (double)prompt_lens[i] * prompt_lens[i];
    reqs += 1.0;
  }
  out->gemm = out->attention = out->comm = 0.0;
  out->overhead = hw->O_p;
  out->gemm_compute_bound = out->attention_compute_bound = 0;
  if (reqs > 0) {
    const double d = m->bytes_per_value;
    double layer = 0.0, fl = 0.0, by = 0.0;
    p.gemm(N, m->hidden, (double)(p.hq + 2 * p.hkv) * m->head_dim, layer, fl, by);
    p.gemm(N, (double)p.D_h, m->hidden, layer, fl, by);
    p.gemm(N, m->hidden, (double)(m->gated_mlp ? 2 : 1) * m->intermediate / m->tp, layer, fl, by);
    p.gemm(N, (double)m->intermediate / m->tp, m->hidden, layer, fl, by);
    double head = 0.0, hfl = 0.0, hby = 0.0;
    p.gemm(reqs, m->hidden, (double)m->vocab / m->tp, head, hfl, hby);  // last token of each request only
    out->gemm = layer * m->num_layers + head;
    out->gemm_compute_bound = fl * m->num_layers + hfl >= by * m->num_layers + hby;
    // attention row with S_q = S_kv = prompt length, summed over the requests (one fused operator)
    const double a_fl = 4.0 * (double)p.D_h * sq / hw->F_ap;
    const double a_by = 2.0 * d * (N * p.D_h + N * (double)(p.hkv * m->head_dim)) / hw->M_a;
    out->attention = std::max(a_fl, a_by) * m->num_layers;
    out->attention_compute_bound = a_fl >= a_by;
    if (m->tp > 1) out->comm = 2.0 * m->num_layers * (N * m->hidden * d / hw->B_c);
  }
  out->total = out->gemm + out->attention + out->comm + out->overhead;
  return OOCO_OK;
}

int64_t ooco_compute_saturated_batch(const ooco_model_t* model, const ooco_hw_params_t* hw) {
  Predictor p;
  if (!p.init(model, hw)) return 0;
  // the FLOP share grows with N, so "compute-bound as a whole" is monotone in N: bisection
  auto bound = [&](int64_t n) {
    ooco_latency_t o;
    p.eval(n, n, &o);
    return o.gemm_compute_bound != 0;
  };
  int64_t hi = 1;
  while (!bound(hi)) {
    if (hi >= ((int64_t)1 << 40)) return hi;
    hi *= 2;
  }
  int64_t lo = hi / 2;  // bound(lo) is false (or lo = 0)
  while (hi - lo > 1) {
    const int64_t mid = lo + (hi - lo) / 2;
    if (bound(mid)) hi = mid; else lo = mid;
  }
  return hi;
}

int ooco_mix_decoding_select(const ooco_model_t* model, const ooco_hw_params_t* hw, const int32_t* online_lens,
                             int32_t n_on, const int32_t* offline_lens, int32_t n_off, double slo_seconds,
                             const int32_t* probe_order, int32_t K, uint8_t* selected_out,
                             int32_t* n_selected_out, double* latency_out, int32_t* over_slo_out) {
  if (!model || !hw || (n_on > 0 && !online_lens) || (n_off > 0 && (!offline_lens || !selected_out)) ||
      (K > 0 && !probe_order))
    return OOCO_E_NULLPTR;
  Predictor p;
  if (!p.init(model, hw) || n_on < 0 || n_off < 0) return OOCO_E_SHAPE;
  int64_t n = n_on, tokens = 0;
  for (int32_t i = 0; i < n_on; ++i) tokens += clamp_len(online_lens[i]);
  const bool over = p.L(n, tokens) > slo_seconds;
  std::vector<uint8_t> tested((size_t)n_off, 0);
  int32_t picked = 0;
  for (int32_t r = 0; r < n_off; ++r) selected_out[r] = 0;
  // random probes (at most K draws)
  for (int32_t k = 0; k < K; ++k) {
    const int32_t r = probe_order[k];
    if (r < 0 || r >= n_off || tested[r]) continue;
    tested[r] = 1;
    const int64_t t = clamp_len(offline_lens[r]);
    if (p.L(n + 1, tokens + t) <= slo_seconds) {
      ++n;
      tokens += t;
      selected_out[r] = 1;
      ++picked;
    }
  }
  // the untested rest: ascending length, longest feasible prefix by bisection
  std::vector<int32_t> rest;
  for (int32_t r = 0; r < n_off; ++r)
    if (!tested[r]) rest.push_back(r);
  if (!rest.empty() && p.L(n, tokens) < slo_seconds) {
    std::sort(rest.begin(), rest.end(), [&](int32_t a, int32_t b) {
      const int64_t la = clamp_len(offline_lens[a]), lb = clamp_len(offline_lens[b]);
      return la != lb ? la < lb : a < b;
    });
    std::vector<int64_t> prefix(rest.size() + 1, 0);
    for (size_t i = 0; i < rest.size(); ++i) prefix[i + 1] = prefix[i] + clamp_len(offline_lens[rest[i]]);
    size_t lo = 0, hi = rest.size();  // invariant: prefix of length lo fits; (hi + 1) does not or does not exist
    while (lo < hi) {
      const size_t mid = lo + (hi - lo + 1) / 2;
      if (p.L(n + (int64_t)mid, tokens + prefix[mid]) <= slo_seconds) lo = mid; else hi = mid - 1;
    }
    for (size_t i = 0; i < lo; ++i) selected_out[rest[i]] = 1;
    n += (int64_t)lo;
    tokens += prefix[lo];
    picked += (int32_t)lo;
  }
  if (n_selected_out) *n_selected_out = picked;
  if (latency_out) *latency_out = p.L(n, tokens);
  if (over_slo_out) *over_slo_out = over ? 1 : 0;
  return OOCO_OK;
}

int ooco_migration_length_preference(const ooco_model_t* model, const ooco_hw_params_t* hw, int64_t batch_size,
                                     int64_t total_tokens, int32_t all_included, double slo_seconds,
                                     int64_t bs_sat, int64_t capacity_tokens, int32_t len_min, int32_t len_max,
                                     int32_t* pref_out) {
  if (!model || !hw || !pref_out) return OOCO_E_NULLPTR;
  Predictor p;
  if (!p.init(model, hw) || batch_size < 0 || total_tokens < 0 || len_min < 0 || len_max < len_min)
    return OOCO_E_SHAPE;
  *pref_out = -1;
  if (!(p.L(batch_size, total_tokens) < slo_seconds) || !all_included) return OOCO_OK;
  // largest l in [len_min, len_max] with fits(l), fits being monotone (true ... true false ... false)
  auto largest = [&](auto fits) -> int32_t {
    if (!fits(len_min)) return -1;
    int64_t lo = len_min, hi = len_max;
    while (lo < hi) {
      const int64_t mid = lo + (hi - lo + 1) / 2;
      if (fits(mid)) lo = mid; else hi = mid - 1;
    }
    return (int32_t)lo;
  };
  if (batch_size >= bs_sat) {
    // compute-saturated: fill the memory capacity with the longest request the SLO allows
    *pref_out = largest([&](int64_t l) {
      return p.L(batch_size + 1, total_tokens + l) <= slo_seconds && total_tokens + l <= capacity_tokens;
    });
    return OOCO_OK;
  }
  const int64_t g = bs_sat - batch_size;
  auto group_fits = [&](int64_t l) { return p.L(batch_size + g, total_tokens + g * l) <= slo_seconds; };
  const int32_t l = largest(group_fits);
  *pref_out = l >= 0 ? l : len_min;  // saturation out of reach: ask for the shortest requests
  return OOCO_OK;
}

int ooco_select_closest_to_preference(const int32_t* offline_lens, int32_t n, int32_t pref, int32_t count,
                                      int32_t* picked_out, int32_t* n_picked_out) {
  if ((n > 0 && !offline_lens) || !n_picked_out || (count > 0 && n > 0 && !picked_out)) return OOCO_E_NULLPTR;
  if (n < 0) return OOCO_E_SHAPE;
  std::vector<int32_t> order((size_t)n);
  std::iota(order.begin(), order.end(), 0);
  const int32_t take = std::max(0, std::min(count, n));
  auto key_less = [&](int32_t a, int32_t b) {
    const int64_t da = std::llabs((int64_t)offline_lens[a] - pref), db = std::llabs((int64_t)offline_lens[b] - pref);
    if (da != db) return da < db;
    if (offline_lens[a] != offline_lens[b]) return offline_lens[a] < offline_lens[b];
    return a < b;
  };
  std::partial_sort(order.begin(), order.begin() + take, order.end(), key_less);
  for (int32_t i = 0; i < take; ++i) picked_out[i] = order[i];
  *n_picked_out = take;
  return OOCO_OK;
}

int ooco_select_evictions(const int32_t* offline_lens, int32_t n, int64_t need_tokens, int32_t compute_bound,
                          uint8_t* evicted_out, int64_t* freed_out) {
  if ((n > 0 && (!offline_lens || !evicted_out)) || !freed_out) return OOCO_E_NULLPTR;
  if (n < 0) return OOCO_E_SHAPE;
  std::vector<int32_t> order((size_t)n);
  std::iota(order.begin(), order.end(), 0);
  std::sort(order.begin(), order.end(), [&](int32_t a, int32_t b) {
    if (offline_lens[a] != offline_lens[b])
      return compute_bound ? offline_lens[a] > offline_lens[b] : offline_lens[a] < offline_lens[b];
    return a < b;
  });
  int64_t freed = 0;
  for (int32_t i = 0; i < n; ++i) evicted_out[i] = 0;
  for (int32_t i = 0; i < n && freed < need_tokens; ++i) {
    evicted_out[order[i]] = 1;
    freed += offline_lens[order[i]];
  }
  *freed_out = freed;
  return OOCO_OK;
}

int ooco_fit_bandwidth(const double* bytes, const double* seconds, int32_t n, double* M_out, double* overhead_out) {
  if (!bytes || !seconds || !M_out || !overhead_out) return OOCO_E_NULLPTR;
  if (n < 2) return OOCO_E_SHAPE;
  double mx = 0, my = 0;
  for (int32_t i = 0; i < n; ++i) {
    mx += bytes[i];
    my += seconds[i];
  }
  mx /= n;
  my /= n;
  double sxx = 0, sxy = 0;
  for (int32_t i = 0; i < n; ++i) {
    sxx += (bytes[i] - mx) * (bytes[i] - mx);
    sxy += (bytes[i] - mx) * (seconds[i] - my);
  }
  if (!(sxx > 0) || sxy == 0) return OOCO_E_SHAPE;
  const double slope = sxy / sxx;
  *M_out = 1.0 / slope;
  *overhead_out = my - slope * mx;
  return OOCO_OK;
}

}  // extern "C"
