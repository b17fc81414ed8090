/*
 * ooco.h -- C ABI of the B200 (sm_100a) paged decode-attention library.
 *
 * The library implements the one operator that dominates a decode step in an
 * online/offline co-located LLM serving instance: grouped-query attention of
 * one new query token per sequence over that sequence's paged KV cache, plus
 * the append of the new token's K/V into the cache, plus the Roofline byte /
 * FLOP count a bottleneck-aware scheduler feeds its latency predictor with.
 * Around that core: the same operations over an 8-bit cache (*_fp8) and for
 * several query tokens per sequence, up to a prefill chunk (*_mq), the movement of cache blocks that a
 * request migration needs (ooco_kv_*_blocks), and a variant with built-in
 * scratch memory (ooco_decode_attention_static).  The host-side latency model
 * and scheduling decisions are declared in ooco_sched.h.
 *
 * Conventions that hold for every entry point
 *   - "device" pointers are CUDA global-memory addresses valid on the current
 *     device; "host" pointers are ordinary CPU addresses.  The caller owns
 *     every buffer.  Entry points in this header never allocate device memory.
 *   - bf16 tensors are passed as `const void*` / `void*` to 16-bit words.
 *   - `cuda_stream` is a `cudaStream_t` cast to `void*` (NULL = legacy default
 *     stream).  All device work is enqueued on it; no entry point synchronises
 *     with the host unless its comment says so.
 *   - Return value: OOCO_OK (0) or a negative OOCO_E_* code.  Argument
 *     validation (pointers, shape, sizes, alignment, the fit of the chosen
 *     kernel's shared memory) happens on the host before anything is enqueued:
 *     a call that returns OOCO_E_NULLPTR, _SHAPE, _UNSUPPORTED or _WORKSPACE
 *     has enqueued nothing and touched no buffer.  OOCO_E_CUDA reports a
 *     failing CUDA call or launch; launches of the same call that preceded it
 *     (the plan, a fused append) may already be enqueued.
 *   - `scale` (the softmax scale) must be positive and finite (OOCO_E_SHAPE
 *     otherwise).
 */
#ifndef OOCO_H_
#define OOCO_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define OOCO_VERSION 1

enum {
  OOCO_OK = 0,
  OOCO_E_NULLPTR = -1,     /* a required pointer is NULL                          */
  OOCO_E_SHAPE = -2,       /* an extent is <= 0, Hq % Hkv != 0, bad stride, ...   */
  OOCO_E_UNSUPPORTED = -3, /* legal shape outside what the kernels are built for  */
  OOCO_E_WORKSPACE = -4,   /* workspace / staging buffer too small or misaligned  */
  OOCO_E_CUDA = -5,        /* a CUDA runtime / driver call or a launch failed     */
  OOCO_E_DEVICE = -6       /* the device-side status word reports a problem       */
};

/*
 * Shape of one attention operator invocation (one transformer layer).
 * Symbols follow the paper's symbol table (Table "Symbol definitions"):
 * Hq = num_q_heads, Hkv = num_kv_heads; the table's D_h ("hidden dim for
 * attention") equals Hq * head_dim.  All extents count elements, not bytes.
 *
 * The KV pool is the non-contiguous KV-cache memory pool of section 2.1
 * (continuous batching): `num_blocks` physical blocks of `block_size` token
 * slots each.  Element (block n, kv head h, slot s, dim i) of k_cache and of
 * v_cache lives at
 *     n * kv_block_stride + h * kv_head_stride + s * kv_token_stride + i.
 * The tuned layout is head-major [num_blocks, Hkv, block_size, head_dim]
 * (kv_token_stride = head_dim, kv_head_stride = block_size * head_dim); a
 * token-major pool [num_blocks, block_size, Hkv, head_dim] is accepted too.
 *
 * Supported by the kernels: head_dim in {64, 128}; block_size in
 * {16, 32, 64, 128, 256}; 1 <= Hq / Hkv <= 16; every stride a multiple of 8
 * elements (16 bytes) and the cache, q and out base addresses 16-byte aligned
 * (OOCO_E_UNSUPPORTED otherwise: the kernels use vector loads and stores).
 */
typedef struct {
  int32_t batch;              /* B: sequences in the decode batch                  */
  int32_t num_q_heads;        /* Hq                                                */
  int32_t num_kv_heads;       /* Hkv; query head hq reads kv head hq / (Hq / Hkv)  */
  int32_t head_dim;           /* per-head dimension                                */
  int32_t block_size;         /* token slots per physical block                    */
  int32_t num_blocks;         /* physical blocks in the pool                       */
  int32_t max_blocks_per_seq; /* row width of block_table                          */
  int32_t reserved;           /* must be 0                                         */
  int64_t kv_block_stride;
  int64_t kv_head_stride;
  int64_t kv_token_stride;
} ooco_shape_t;

/*
 * Roofline cost of one decode-attention invocation (Table "Operator
 * Modeling", attention row, with S_q = 1 and S_kv = context length, summed
 * over the batch).  bytes_paper = bytes_q + bytes_out + bytes_kv is the
 * table's memory entry; bytes_index (block table and length reads) is not in
 * the paper's model and is reported beside it.
 */
typedef struct {
  int64_t flops;        /* sum_b 4 * Hq * head_dim * T_b                            */
  int64_t bytes_q;      /* d * B * Hq * head_dim                                    */
  int64_t bytes_out;    /* d * B * Hq * head_dim                                    */
  int64_t bytes_kv;     /* sum_b 2 * d * Hkv * head_dim * T_b                       */
  int64_t bytes_index;  /* 4 * (B + sum_b ceil(T_b / block_size))                   */
  int64_t bytes_paper;  /* bytes_q + bytes_out + bytes_kv                           */
  int64_t total_tokens; /* sum_b T_b                                                */
} ooco_cost_t;

/*
 * KV-cache append (section 2.1: a decode execution "reuses and expands" the
 * KV cache).  For every sequence b and kv head h the head_dim 16-bit words of
 * k_new[b, h, :] are copied verbatim to slot positions[b] % block_size of
 * physical block block_table[b, positions[b] / block_size] of k_cache, and
 * likewise for V.  No other word of either cache is written.
 *
 *   k_new, v_new   device, bf16 [B, Hkv, head_dim], contiguous, read-only
 *   k_cache,v_cache device, bf16 pool (layout: see ooco_shape_t), written
 *   block_table    device, int32 [B, max_blocks_per_seq], read-only
 *   positions      device, int32 [B], read-only; a sequence with a negative
 *                  position or one at or beyond max_blocks_per_seq * block_size
 *                  is skipped, as is one whose table entry is outside
 *                  [0, num_blocks)
 * No two sequences may target the same (block, slot).
 */
int ooco_kv_append(const ooco_shape_t* shape, const void* k_new, const void* v_new,
                   void* k_cache, void* v_cache, const int32_t* block_table,
                   const int32_t* positions, void* cuda_stream);

/*
 * Upper bound, in bytes, of the workspace ooco_decode_attention needs for
 * `shape` whatever the context lengths are.  Host arithmetic only.  Returns 0
 * for an invalid or unsupported shape.
 */
size_t ooco_decode_workspace_bytes(const ooco_shape_t* shape);

/*
 * Paged decode attention (sections 2.1 and 2.3: one query token per sequence,
 * the whole cached context of every sequence is read, GQA; section 3.3.1: the
 * operator is one fused kernel whose score matrix stays on chip).
 * For every sequence b, query head hq, with kv head h = hq / (Hq / Hkv):
 *     s_t   = scale * <q[b, hq, :], K_b,t,h>          t in [0, T_b)
 *     w     = softmax_t(s)
 *     out[b, hq, :] = sum_t w_t * V_b,t,h
 * where token t of sequence b lives in slot t % block_size of physical block
 * block_table[b, t / block_size] and T_b = context_lens[b].  Inputs are bf16,
 * products and sums are accumulated in fp32, the result is rounded to bf16
 * (round to nearest even).  T_b = 0 gives out[b] = 0.
 *
 *   q              device, bf16 [B, Hq, head_dim], contiguous
 *   k_cache,v_cache device, bf16 pool, read-only (blocks may be shared
 *                  between sequences)
 *   block_table    device, int32 [B, max_blocks_per_seq]; only the first
 *                  ceil(T_b / block_size) entries of row b are read
 *   context_lens   device, int32 [B]; values are clamped to
 *                  [0, max_blocks_per_seq * block_size]
 *   out            device, bf16 [B, Hq, head_dim], written
 *   workspace      device, >= ooco_decode_workspace_bytes(shape) bytes,
 *                  256-byte aligned; scratch, contents undefined afterwards
 *                  except for the status word ooco_workspace_status reads.
 *                  Calls that may overlap on the GPU need separate workspaces.
 * Pool slots at or beyond T_b and table entries beyond the last used block
 * are never interpreted (they may hold NaN / garbage).  A table entry outside
 * [0, num_blocks) that IS needed reads as zeros and never faults.
 * Three launches are enqueued (plan, split-KV partial attention, LSE merge);
 * the call is asynchronous.
 */
int ooco_decode_attention(const ooco_shape_t* shape, const void* q, const void* k_cache,
                          const void* v_cache, const int32_t* block_table,
                          const int32_t* context_lens, float scale, void* out,
                          void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * One decode step of this operator with DEVICE buffers: the KV append of ooco_kv_append
 * (the new token's K / V written at positions[b]) fused into the first launch of
 * ooco_decode_attention, which then attends over context_lens[b] tokens; a serving step
 * passes context_lens = positions + 1 (section 2.1: decode reuses and expands the cache).
 * Same arguments, layouts, ownership and errors as the two calls it replaces; three
 * launches instead of four.  The attention sees the appended rows.
 */
int ooco_decode_step(const ooco_shape_t* shape, const void* q, const void* k_new, const void* v_new,
                     void* k_cache, void* v_cache, const int32_t* block_table,
                     const int32_t* positions, const int32_t* context_lens, float scale, void* out,
                     void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Several query tokens per sequence (the attention row of Table "Operator Modeling" with S_q > 1:
 * multi-token decode, or a chunk of a prefill running next to decodes).  The q_len query
 * tokens of sequence b are the LAST q_len tokens of its context: their K / V must already be in the
 * cache (ooco_kv_append_mq writes them), context_lens[b] counts them, and query token i attends to
 * tokens [0, T_b - q_len + i + 1) -- causal attention over the cache.  A query token that sees no
 * token at all (T_b - q_len + i + 1 <= 0) gives a zero row.
 *   q, out          device, bf16 [B, q_len, Hq, head_dim], contiguous
 *   k_new, v_new    device, bf16 [B, q_len, Hkv, head_dim]; token i of sequence b is written at
 *                   position positions[b] + i (ooco_kv_append_mq); positions beyond the block table
 *                   are skipped, as in ooco_kv_append
 *   workspace       >= ooco_decode_workspace_bytes_mq(shape, q_len)
 * Supported: 1 <= q_len <= 8192 (OOCO_E_UNSUPPORTED beyond).  Up to 16 score columns per
 * (sequence, kv head), (Hq / Hkv) * q_len <= 16, run the decode kernels (HBM-bound: the cache is
 * read once); more columns run a prefill-chunk kernel, which cuts the columns into row tiles of
 * up to 128, reads the cache once per row tile (the repeats hit L2) and never loads tokens a tile
 * cannot see; it becomes bound by the tensor pipe beyond 128 columns.  At head_dim 128 that kernel
 * runs on tcgen05 (scores and output in tensor memory; over a bf16 cache one CTA per SM with two
 * 128-row tiles taking turns on the tensor pipe, or, up to 128 columns, one tile whose scores run a
 * stage ahead of its softmax), otherwise on mma.sync.  Over the 8-bit cache
 * (ooco_decode_step_mq_fp8) every chunk of more than 16 columns runs a tcgen05 kernel whose spare
 * warps widen each 8-bit stage to f16 in shared memory first (up to 128 columns the one-CTA-per-SM
 * kernel in its one-tile mode, beyond that the kernel with two CTAs per SM).  The workspace grows with q_len: one fp32
 * partial row per (split item, score column).  q_len = 1 is ooco_decode_attention /
 * ooco_kv_append exactly.  Everything else as for those two.
 */
size_t ooco_decode_workspace_bytes_mq(const ooco_shape_t* shape, int32_t q_len);
int ooco_decode_attention_mq(const ooco_shape_t* shape, int32_t q_len, const void* q, const void* k_cache,
                             const void* v_cache, const int32_t* block_table, const int32_t* context_lens,
                             float scale, void* out, void* workspace, size_t workspace_bytes,
                             void* cuda_stream);
int ooco_kv_append_mq(const ooco_shape_t* shape, int32_t q_len, const void* k_new, const void* v_new,
                      void* k_cache, void* v_cache, const int32_t* block_table, const int32_t* positions,
                      void* cuda_stream);
/* ooco_kv_append_mq fused into the first launch of ooco_decode_attention_mq (three launches), as
 * ooco_decode_step does for one token; a serving step passes context_lens = positions + q_len. */
int ooco_decode_step_mq(const ooco_shape_t* shape, int32_t q_len, const void* q, const void* k_new,
                        const void* v_new, void* k_cache, void* v_cache, const int32_t* block_table,
                        const int32_t* positions, const int32_t* context_lens, float scale, void* out,
                        void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * The same three operations over an 8-bit KV cache (the operator model's d, "byte per value", set
 * to 1 for K and V: Table "Symbol definitions"; decode attention is memory-bound, section 3.3.3, so
 * halving the stored bytes halves its time).  k_cache / v_cache hold OCP E4M3 codes (1 sign, 4
 * exponent bits with bias 7, 3 mantissa bits, no infinities, S.1111.111 = NaN, largest finite 448),
 * one byte per value, same four-index layout with the strides of `shape` counted in bytes; a code
 * stands for decode(code) * k_scale (v_scale), one positive fp32 scale per tensor.  q, k_new,
 * v_new and out stay bf16.
 *   ooco_kv_append_fp8        stores e4m3(x / scale) for every new value x: one fp32 division,
 *                             round to nearest even, magnitudes beyond 448 saturate to 448.
 *   ooco_decode_attention_fp8 attention as ooco_decode_attention with K = decode(code) * k_scale,
 *                             V = decode(code) * v_scale; codes are widened exactly to f16, q and
 *                             the softmax weights are rounded to f16, accumulation is fp32.
 *   ooco_decode_step_fp8      the fused append + attention step, as ooco_decode_step.
 * Restrictions beyond ooco_shape_t's: head_dim = 128, strides multiples of 16 bytes; a NaN code
 * inside the attended range is not propagated as NaN (it reads as a finite value).  Workspace,
 * status word, launches, ownership and errors as for the bf16 entry points.
 */
int ooco_kv_append_fp8(const ooco_shape_t* shape, const void* k_new, const void* v_new, void* k_cache,
                       void* v_cache, const int32_t* block_table, const int32_t* positions, float k_scale,
                       float v_scale, void* cuda_stream);
int ooco_decode_attention_fp8(const ooco_shape_t* shape, const void* q, const void* k_cache, const void* v_cache,
                              const int32_t* block_table, const int32_t* context_lens, float scale,
                              float k_scale, float v_scale, void* out, void* workspace, size_t workspace_bytes,
                              void* cuda_stream);
int ooco_decode_step_fp8(const ooco_shape_t* shape, const void* q, const void* k_new, const void* v_new,
                         void* k_cache, void* v_cache, const int32_t* block_table, const int32_t* positions,
                         const int32_t* context_lens, float scale, float k_scale, float v_scale, void* out,
                         void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Both variants at once: q_len query tokens per sequence over an 8-bit cache.  With k_new and v_new
 * (bf16 [B, q_len, Hkv, head_dim]) the quantising append of the q_len new tokens at positions[b] + i
 * is fused into the first launch, as in ooco_decode_step_mq; with both NULL (positions may be NULL
 * too) only the attention runs.  Restrictions: those of the two variants together (head_dim 128,
 * 1 <= q_len <= 8192); codes are widened exactly to f16, q and the softmax weights are rounded to
 * f16, accumulation is fp32 -- for every q_len.
 */
int ooco_decode_step_mq_fp8(const ooco_shape_t* shape, int32_t q_len, const void* q, const void* k_new,
                            const void* v_new, void* k_cache, void* v_cache, const int32_t* block_table,
                            const int32_t* positions, const int32_t* context_lens, float scale, float k_scale,
                            float v_scale, void* out, void* workspace, size_t workspace_bytes,
                            void* cuda_stream);

/*
 * Paged decode attention for callers that cannot allocate device memory.  (The paper has no
 * counterpart; this is a packaging variant of ooco_decode_attention.)
 *
 * Who needs it: an inference engine that hands the whole device to its KV-cache pool at
 * start-up has nothing left for cudaMalloc to give; a latency-critical decode loop cannot
 * afford the device-wide synchronisation an allocation or a free implies; and a plug-in
 * running under a host framework may be forbidden to allocate outside that framework's own
 * pool.  Such a caller cannot provide the workspace ooco_decode_attention asks for.
 *
 * This entry point takes the same inputs and output but no workspace: the scratch is an
 * array of OOCO_STATIC_SCRATCH_BYTES built into the library's device image (every GPU that
 * loads the library holds it until the process exits).  The call allocates nothing, neither
 * through cudaMalloc / cudaFree nor through any allocating library routine, and computes
 * exactly what ooco_decode_attention computes, with the same launches.
 *
 *   - A shape whose ooco_decode_workspace_bytes exceeds OOCO_STATIC_SCRATCH_BYTES is refused
 *     with OOCO_E_WORKSPACE before anything is launched, and ooco_last_error_detail names
 *     both sizes.  The exact test is ooco_decode_workspace_bytes(shape) <=
 *     OOCO_STATIC_SCRATCH_BYTES; with the default tuning, head_dim 128 and block tables of up
 *     to 8 K tokens that admits about 500 sequences of 32 q / 8 kv heads and about 50 of
 *     64 q / 8 kv heads.  The bound moves with ooco_set_tuning knobs 4 and 5, which change
 *     ooco_decode_workspace_bytes.
 *   - The first call on each device looks up the array's device address (that device must be
 *     current, as for every call); make that first call outside any stream capture.  With
 *     CUDA's lazy module loading that first call is also when the device receives the
 *     library's code and the array itself: "allocates nothing" holds from the second call on,
 *     so make one warm-up call per device BEFORE handing the rest of the device's memory to a
 *     pool; a first call on a device that is already full can fail with OOCO_E_CUDA.
 *   - All calls on a device share the one array: two calls that may overlap on the GPU (other
 *     streams, other host threads) race on it and corrupt each other's results.  Calls on one
 *     stream are ordered and safe.  The array keeps the previous call's contents; nothing in
 *     it needs to start at zero, because the first kernel of each call rewrites every field
 *     that is read later.
 *   - The device status word of this variant is not exposed.
 */
#define OOCO_STATIC_SCRATCH_BYTES (16u << 20)
int ooco_decode_attention_static(const ooco_shape_t* shape, const void* q, const void* k_cache,
                                 const void* v_cache, const int32_t* block_table,
                                 const int32_t* context_lens, float scale, void* out,
                                 void* cuda_stream);

/*
 * Paged KV block movement (section 3.4.3 "Offline Request Migration": an offline request's KV
 * cache is transferred from a latency-relaxed to a latency-strict instance; section 3.4.1: space
 * is freed on a latency-strict instance by evicting offline requests; section 4: the KV cache is
 * what travels between instances).  The transport wants one contiguous buffer per transfer, the
 * pool is non-contiguous, so a migration is gather (sender) -> transfer -> scatter (receiver).
 *
 * ooco_kv_gather_blocks   packs the n listed pool blocks, in list order, into
 *                         k_packed / v_packed, bf16 [n, Hkv, block_size, head_dim] contiguous.
 * ooco_kv_scatter_blocks  is the inverse: block i of the packed buffers is written to pool
 *                         block block_ids[i].
 * ooco_kv_copy_blocks     copies pool block src_ids[i] to pool block dst_ids[i] (pool
 *                         compaction, copy-on-write of a shared prefix block).
 * All copy 16-bit words verbatim; every word of a listed destination block is written, nothing
 * else is.
 *
 *   shape            the pool's shape (num_kv_heads, head_dim, block_size, num_blocks and the three
 *                    strides are used; the other fields must merely be valid)
 *   block_ids, src_ids, dst_ids   device, int32 [n]; n = 0 is legal and launches nothing
 *   k_packed, v_packed            device, 16-byte aligned, n * Hkv * block_size * head_dim words each
 *   status           device int32, may be NULL.  Bits are OR-ed in, never cleared: 4 = an id was
 *                    outside [0, num_blocks) (that list entry is skipped), 2 = a bounded wait in
 *                    the kernel gave up.  The caller zeroes it and reads it back when it wants to.
 * Destination ids must be distinct, and in ooco_kv_copy_blocks no block may be both a source and
 * a destination.  One launch, asynchronous on `cuda_stream`.  The tuned case is a pool whose
 * (block, kv head) tiles are contiguous (kv_token_stride = head_dim); other strides are moved
 * row by row.
 */
int ooco_kv_gather_blocks(const ooco_shape_t* shape, const void* k_cache, const void* v_cache,
                          const int32_t* block_ids, int32_t n, void* k_packed, void* v_packed,
                          int32_t* status, void* cuda_stream);
int ooco_kv_scatter_blocks(const ooco_shape_t* shape, const void* k_packed, const void* v_packed,
                           const int32_t* block_ids, int32_t n, void* k_cache, void* v_cache,
                           int32_t* status, void* cuda_stream);
int ooco_kv_copy_blocks(const ooco_shape_t* shape, void* k_cache, void* v_cache, const int32_t* src_ids,
                        const int32_t* dst_ids, int32_t n, int32_t* status, void* cuda_stream);

/*
 * Reads back the device-side status word an earlier ooco_decode_attention /
 * ooco_decode_step_host call left in `workspace`.  SYNCHRONISES `cuda_stream`.
 * *status_host is 0 when every kernel ran to completion, otherwise a bit mask
 * (1: plan overflowed the work list, 2: a bounded wait inside the attention
 * kernel gave up).  Returns OOCO_E_DEVICE when *status_host != 0.
 */
int ooco_workspace_status(const void* workspace, void* cuda_stream, int32_t* status_host);

/*
 * Attention row of the paper's operator model (Table "Operator Modeling"),
 * summed over the batch with S_q = 1, S_kv = context_lens_host[b]; this is the
 * attention term of the latency predictor L(.) of Algorithms "Offline Request
 * Migration Decision" and "Mix Decoding Selection".  Pure host arithmetic on
 * 64-bit integers; touches no device.
 *
 *   context_lens_host  HOST, int32 [B]; negative lengths count as 0
 *   bytes_per_value    the table's d (2 for bf16)
 *   cost_out           HOST, written
 * The printed table multiplies the K/V term by Hq / Hkv; with D_h = Hq *
 * head_dim that cannot be right (GQA would increase traffic), so the K/V term
 * here is 2 * d * S_kv * D_h * Hkv / Hq, which equals the bytes of the cache
 * slots the operator addresses and coincides with the printed formula when
 * Hq = Hkv.
 */
int ooco_decode_bytes_model(const ooco_shape_t* shape, const int32_t* context_lens_host,
                            int32_t bytes_per_value, ooco_cost_t* cost_out);

/*
 * The same row of Table "Operator Modeling" with S_q = q_len query tokens per sequence, as printed
 * (no causal discount): flops = sum_b 4 D_h q_len T_b; bytes_q = bytes_out = d q_len D_h per
 * sequence; the K / V and index terms do not depend on q_len.  q_len = 1 is ooco_decode_bytes_model.
 */
int ooco_attention_bytes_model(const ooco_shape_t* shape, int32_t q_len, const int32_t* context_lens_host,
                               int32_t bytes_per_value, ooco_cost_t* cost_out);

/*
 * Bytes of device staging memory ooco_decode_step_host needs for `shape`
 * (0 for an invalid shape).  Host arithmetic only.
 */
size_t ooco_step_staging_bytes(const ooco_shape_t* shape);

/*
 * One whole decode step of this operator driven from HOST buffers: copies the
 * step's inputs to the device, appends the new token's K/V at positions[b]
 * and attends over context_lens[b] tokens (ooco_decode_step; a serving step
 * passes context_lens = positions + 1, section 2.1), and copies `out` back.  Everything is enqueued on
 * `cuda_stream` in that order and the call returns after the stream has been
 * SYNCHRONISED, so out_host is valid on return.
 *
 * When all six input buffers are page-locked and 16-byte aligned (cudaHostAlloc / cudaHostRegister,
 * e.g. torch pinned memory) the step's first launch reads them through their device mapping (the
 * planning and append CTAs directly, extra CTAs staging the block table and the lengths for the
 * attention kernel), the attention kernel fetches each work item's q rows from the host mapping
 * itself (with up to 8 query heads per kv head; otherwise q is staged too), and a page-locked
 * out_host is written by the attention kernels directly: three launches, no copy-engine transfer,
 * and q and out cross the host link while the attention runs.  Pageable buffers are detected and
 * go through one cudaMemcpyAsync each.  The results are the same.
 *
 *   q_host, k_new_host, v_new_host   HOST (pinned for full copy speed), bf16
 *                                    [B,Hq,D], [B,Hkv,D], [B,Hkv,D]
 *   block_table_host                 HOST int32 [B, max_blocks_per_seq]
 *   positions_host, context_lens_host HOST int32 [B]
 *   k_cache, v_cache                 DEVICE pool (the persistent serving state)
 *   out_host                         HOST bf16 [B,Hq,D], written
 *   staging                          DEVICE scratch, >= ooco_step_staging_bytes
 *   workspace                        DEVICE, as for ooco_decode_attention
 */
int ooco_decode_step_host(const ooco_shape_t* shape, const void* q_host,
                          const void* k_new_host, const void* v_new_host,
                          const int32_t* block_table_host, const int32_t* positions_host,
                          const int32_t* context_lens_host, void* k_cache, void* v_cache,
                          float scale, void* out_host, void* staging, size_t staging_bytes,
                          void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Where the host time of the last successful ooco_decode_step_host call on this thread went:
 * *enqueue_ns = from entry until everything was enqueued (validation, pointer queries, tensor-map
 * encoding, launches), *wait_ns = the wait for the stream after that.  Host clocks; for benchmarks.
 */
int ooco_last_host_step_ns(int64_t* enqueue_ns, int64_t* wait_ns);

/*
 * Number of kernels the last successful ooco_decode_attention call on this
 * thread enqueued (for launch accounting in benchmarks); 0 before any call.
 */
int ooco_last_launch_count(void);

/*
 * Per-kernel timing of ooco_decode_attention for benchmarks.  ooco_profile_enable(n > 0)
 * creates CUDA events for up to n calls (process-wide; host objects only, no device
 * memory) and makes every later ooco_decode_attention call record four events on its
 * stream: before the plan kernel, before the attention kernel, after it, after the merge
 * kernel; n = 0 switches recording off and destroys the events.  ooco_profile_read
 * SYNCHRONISES on the recorded events, writes for each recorded call, oldest first, the
 * three durations in milliseconds (plan, attention, merge) to ms_out[3 * i + 0..2] for at
 * most max_records calls, stores the number written in *n_out and forgets all records.
 * Do not enable while a stream is being captured into a graph.
 */
int ooco_profile_enable(int max_records);
int ooco_profile_read(float* ms_out, int max_records, int* n_out);

/*
 * Launch-shape override for benchmark sweeps (process-wide; the defaults are the tuned
 * values).  knob: 0 consumer warps per CTA {2,4,8}; 1 pipeline stages (0 = as many as
 * fit); 2 CTAs per SM {1..4}; 3 / 4 minimum / maximum split-KV chunk in tokens (multiples
 * of 128); 5 target work items per CTA; 6 non-zero = one TMA copy per 64-dim half;
 * 7 16-token tiles per consumer warp and stage {1,2}; 8 non-zero = launch the attention and
 * merge kernels with programmatic dependent launch (their prologues overlap the predecessor);
 * 9 CTAs per SM of the block-movement kernel {1..3}; 10 non-zero = ooco_decode_step_host reads
 * page-locked inputs through their device mapping and lets the kernels write a page-locked result
 * directly (zero = always one copy per buffer; 2 = as 1, but q is staged on the device by the first launch
 * instead of being fetched from the host mapping by the attention kernel); 11 non-zero = 9 to 16 score columns per
 * (sequence, kv head) run the kernel whose warps share 16 score rows and split the tokens of a
 * stage (zero = the decode kernel with two 8-column tiles); 12 = which prefill chunks (more than 16 score
 * columns) run the tcgen05 kernels at head_dim 128 over a bf16 cache: 1 = all of them (default), n in
 * [17, 65536] = those with n or more score columns, 0 = none (the mma.sync kernel of the prefill-chunk path).
 * 13 non-zero = diagnostic fp32 output: `out` of the attention entry points is then fp32 (same
 * shape, 4 bytes per value) and holds the values the kernels would otherwise round to bf16 (every
 * row goes through the partial-result and merge path; an unsplit row passes it unchanged), so a
 * test can separate the arithmetic's error from the output format's rounding; not for the host-buffer
 * step (OOCO_E_UNSUPPORTED).  14 non-zero = the decode kernel over the 8-bit cache (8 consumer warps)
 * computes its scores on tcgen05 from the stored codes (zero = mma.sync on codes widened in registers).
 * 15 = the tcgen05 kernel with one CTA per SM and two 128-row tiles per CTA (head_dim 128): 2 (default) = every
 * chunk that knob 12 sends to tcgen05 (with 128 score columns or fewer the kernel runs one tile and gives the
 * second tile's score buffer and issuing warp to it; over the 8-bit cache only these chunks, its idle warps
 * widening the codes), 1 = only chunks of more than 128 score columns over a bf16 cache, 0 = never (one tile per
 * CTA, two CTAs per SM).
 * Changing knobs 4 or 5 changes ooco_decode_workspace_bytes.  Returns OOCO_E_SHAPE for an
 * unknown knob or a value outside its range.  ooco_get_tuning returns a knob's current value
 * (OOCO_E_SHAPE, which is negative, for an unknown knob).
 */
int ooco_set_tuning(int knob, int value);
int ooco_get_tuning(int knob);

/*
 * The checked build.  Compiling the library with -DOOCO_CHECKS (build.py writes it to
 * libooco_checked.so) makes the kernels range-check every index they derive from device data: each
 * block-table entry they read, the fields of each work item, each partial-result slot and output
 * row, and the shared-memory destination of each asynchronous copy.  A violation is OR-ed into the
 * status word ooco_workspace_status reads (8: table entry outside [0, num_blocks), 16: work-item
 * field out of range, 32: partial-slot / work-list / output index out of range, 64: shared-memory
 * destination outside its region) and the access is skipped (a bad table entry reads as zeros); the
 * kernels never trap.  It stands in for a memory checker on machines where none can be run; the
 * release build compiles the checks to nothing.
 *   ooco_checked_build     1 in the checked build, 0 otherwise.
 *   ooco_check_predicate   evaluates one of the range predicates on the HOST (for unit tests of the
 *                          predicates themselves): which = 0 table entry {id, num_blocks};
 *                          1 index {i, n}; 2 work item {sequence, slot, first token, end token, B,
 *                          max items, table capacity in tokens}; 3 span {offset, bytes, lo, hi}.
 *                          Returns 1 / 0, or a negative OOCO_E_* for a NULL pointer or unknown `which`.
 */
int ooco_checked_build(void);
int ooco_check_predicate(int which, const int64_t* args_host);

/*
 * Text about the last OOCO_E_CUDA or OOCO_E_WORKSPACE on this thread ("" if none yet): the CUDA
 * call that failed with its error code, or, from ooco_decode_attention_static, the scratch size
 * the shape needs next to the size of the built-in array.  The pointer stays valid for the
 * thread's lifetime.
 */
const char* ooco_last_error_detail(void);

/* Static, human-readable name of a status code.  Never NULL. */
const char* ooco_status_string(int status);

/* OOCO_VERSION the library was built from. */
int ooco_version(void);

#ifdef __cplusplus
}
#endif
#endif /* OOCO_H_ */
