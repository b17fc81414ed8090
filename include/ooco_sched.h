/*
 * ooco_sched.h -- host-side C ABI of the Roofline performance model and of the step-level
 * scheduling decisions built on it (section 3.3 "Performance Model", section 3.4 "Scheduling
 * Logic").  Everything here is plain host arithmetic: no device is touched, nothing is allocated
 * that outlives the call, every function is re-entrant.  All pointers are HOST pointers owned by
 * the caller.  Return value: OOCO_OK (0) or a negative OOCO_E_* code of ooco.h.
 *
 * The latency predictor L(.) is the operator-level simulator of section 3.3: it walks the GEMM,
 * attention and communication operators of one decode iteration of a decoder-only transformer,
 * takes each operator's FLOPs and bytes from Table "Operator Modeling", turns them into a time with
 *     op latency = max(FLOPs / F, bytes / M)                      (Eq. "op_latency")
 * and adds the static overhead O_d.  For a decode batch the result depends on the batch only
 * through its size and its total number of cached tokens.
 */
#ifndef OOCO_SCHED_H_
#define OOCO_SCHED_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* Table "Parameters for latency modeling".  Rates in FLOP/s and bytes/s, times in seconds. */
typedef struct {
  double F_g;  /* achievable FLOP/s of GEMM operators                          */
  double F_ap; /* achievable FLOP/s of prefill attention (unused by decode)    */
  double F_ad; /* achievable FLOP/s of decode attention                        */
  double M_g;  /* achievable memory bandwidth of GEMM operators                */
  double M_a;  /* achievable memory bandwidth of attention operators           */
  double O_p;  /* static overhead of a prefill iteration (unused by decode)    */
  double O_d;  /* static overhead of a decode iteration                        */
  double B_c;  /* effective bandwidth of communication operators (tp > 1)      */
} ooco_hw_params_t;

/*
 * The model structure the simulator walks ("the structure of common LLMs is relatively fixed").
 * One decode iteration with N requests runs, per layer and per tensor-parallel rank:
 *   GEMM  N x hidden -> (Hq + 2 Hkv) * head_dim / tp              (QKV projection)
 *   attention, D_h = Hq * head_dim / tp, S_q = 1                    (one fused operator)
 *   GEMM  N x Hq * head_dim / tp -> hidden                          (output projection)
 *   GEMM  N x hidden -> (gated ? 2 : 1) * intermediate / tp         (MLP up, gate fused)
 *   GEMM  N x intermediate / tp -> hidden                           (MLP down)
 *   tp > 1: two all-reduces of N * hidden * d bytes each, at B_c
 * and once per iteration GEMM N x hidden -> vocab / tp (LM head).  Normalisation, rotary and
 * activation kernels are not modelled (the paper models GEMM, attention and communication).
 */
typedef struct {
  int32_t num_layers;
  int32_t hidden;
  int32_t num_q_heads;
  int32_t num_kv_heads;
  int32_t head_dim;
  int32_t intermediate;
  int32_t vocab;
  int32_t bytes_per_value; /* the table's d (2 for bf16) */
  int32_t tp;              /* tensor-parallel degree >= 1; must divide the head counts */
  int32_t gated_mlp;       /* 1: gate and up projections (SwiGLU), 0: a single up projection */
} ooco_model_t;

typedef struct {
  double total;     /* seconds: gemm + attention + comm + overhead */
  double gemm;
  double attention;
  double comm;
  double overhead;  /* O_d */
  int32_t gemm_compute_bound;      /* 1 when the summed GEMM FLOP time >= the summed GEMM byte time */
  int32_t attention_compute_bound; /* 1 when the attention operator's FLOP time >= its byte time */
} ooco_latency_t;

/*
 * L(B) of a decode iteration (section 3.3.2) for a batch of `batch_size` requests holding
 * `total_tokens` cached tokens in all.  The attention operator is one fused operator per layer
 * over the whole batch: FLOPs 4 * D_h * total_tokens, bytes 2d * (batch_size * D_h + total_tokens
 * * D_h * Hkv / Hq) -- the table prints Hq / Hkv in the K/V term; with D_h the width of all query
 * heads the K/V width is D_h * Hkv / Hq, which is what is used (at Hq = Hkv both agree).
 * An empty batch (batch_size = 0) costs O_d.
 */
int ooco_predict_decode_latency(const ooco_model_t* model, const ooco_hw_params_t* hw, int64_t batch_size,
                                int64_t total_tokens, ooco_latency_t* out);

/*
 * Latency of a prefill iteration over the given prompts (sections 3.3.1 / 3.3.2; host pointer
 * prompt_lens [n], non-positive lengths are ignored): the linear layers see all prompt tokens
 * (N = their sum), the attention operator of a layer is one fused operator over the requests with
 * S_q = S_kv = the prompt length (the table's row as printed, no causal discount), timed against
 * F_ap and M_a, only the last token of each request passes through the LM head, plus O_p.
 */
int ooco_predict_prefill_latency(const ooco_model_t* model, const ooco_hw_params_t* hw, const int32_t* prompt_lens,
                                 int32_t n, ooco_latency_t* out);

/*
 * bs_sat of Algorithm "Offline Request Migration Decision": the smallest decode batch size at
 * which the GEMM operators of an iteration are compute-bound as a whole (summed FLOP time >=
 * summed byte time).  The paper takes the threshold as given; this derives it from the same
 * operator model.  Returns 0 on bad arguments.
 */
int64_t ooco_compute_saturated_batch(const ooco_model_t* model, const ooco_hw_params_t* hw);

/*
 * Algorithm "Mix Decoding Selection": choose the offline requests that decode together with all
 * online requests of a latency-strict instance so that the predicted step latency stays within
 * the TPOT bound S.
 *   1. B <- all online requests.
 *   2. For each of the first K entries of probe_order (the caller's random draws, indices into the
 *      offline set; an index seen before or out of range is passed over and does not count as
 *      tested): add the request when L(B + r) <= S, otherwise discard it.
 *   3. If untested requests remain and L(B) < S: sort the untested ones by ascending length (equal
 *      lengths by ascending index) and add the longest prefix R' of that order with L(B + R') <= S
 *      (binary search; L is monotone in the prefix).
 *   online_lens [n_on], offline_lens [n_off]   context lengths (cached tokens) of the requests
 *   selected_out [n_off]                       1 = decodes in this step, 0 = does not
 *   latency_out                                L(B) of the selected batch (may be NULL)
 * When the online requests alone exceed S the call still returns OOCO_OK with no offline request
 * selected (best-effort mode: every online request decodes anyway) and *over_slo_out = 1.
 */
int ooco_mix_decoding_select(const ooco_model_t* model, const ooco_hw_params_t* hw, const int32_t* online_lens,
                             int32_t n_on, const int32_t* offline_lens, int32_t n_off, double slo_seconds,
                             const int32_t* probe_order, int32_t K, uint8_t* selected_out,
                             int32_t* n_selected_out, double* latency_out, int32_t* over_slo_out);

/*
 * Algorithm "Offline Request Migration Decision", run on a latency-strict instance after its mix
 * decoding selection: decides whether to pull offline requests from a latency-relaxed instance
 * and which length to ask for.
 *   batch_size, total_tokens   the current decoding batch B
 *   all_included               1 when the last selection took every request on the instance
 *   bs_sat                     compute-saturated batch size threshold
 *   capacity_tokens            KV-cache capacity in tokens (U_mem = tokens / capacity_tokens)
 *   len_min, len_max           shortest / longest request length that can be asked for
 * Result *pref_out:
 *   -1  no migration (L(B) >= S, or requests were left out of B)
 *   if batch_size >= bs_sat: the largest l in [len_min, len_max] with L(B + one request of length
 *       l) <= S and U_mem <= 1, or -1 when even len_min does not fit;
 *   else, with g = bs_sat - batch_size: if g requests of length len_min fit under S, the largest l
 *       such that g requests of length l fit under S (the group that reaches saturation); else
 *       len_min (shortest requests, to grow the batch as far as possible).
 */
int ooco_migration_length_preference(const ooco_model_t* model, const ooco_hw_params_t* hw, int64_t batch_size,
                                     int64_t total_tokens, int32_t all_included, double slo_seconds,
                                     int64_t bs_sat, int64_t capacity_tokens, int32_t len_min, int32_t len_max,
                                     int32_t* pref_out);

/*
 * The latency-relaxed side of the pull (last step of the same algorithm): among its decoding
 * offline requests pick the `count` whose lengths are closest to `pref` (ties: shorter first, then
 * lower index).  picked_out [min(count, n)] receives their indices in order of closeness.
 */
int ooco_select_closest_to_preference(const int32_t* offline_lens, int32_t n, int32_t pref, int32_t count,
                                      int32_t* picked_out, int32_t* n_picked_out);

/*
 * Eviction choice of section 3.4.1: free at least need_tokens of KV space on a latency-strict
 * instance by evicting offline requests.  When the instance's bottleneck is computation
 * (compute_bound != 0) longer requests go first, so the decode batch shrinks as little as
 * possible; otherwise shorter requests go first, which costs the least recomputation.  Ties by
 * ascending index.  evicted_out [n]: 1 = evict.  *freed_out = tokens freed (< need_tokens only when
 * everything was evicted).
 */
int ooco_select_evictions(const int32_t* offline_lens, int32_t n, int64_t need_tokens, int32_t compute_bound,
                          uint8_t* evicted_out, int64_t* freed_out);

/*
 * Profiling fit of section 3.3.2 ("parameters ... obtained through a small amount of profiling
 * data") for a memory-bound operator: least-squares line seconds = overhead + bytes / M through n
 * measurements.  Needs n >= 2 and two distinct byte counts.
 */
int ooco_fit_bandwidth(const double* bytes, const double* seconds, int32_t n, double* M_out, double* overhead_out);

#ifdef __cplusplus
}
#endif
#endif /* OOCO_SCHED_H_ */
