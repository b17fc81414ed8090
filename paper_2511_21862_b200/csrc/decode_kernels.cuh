// Paged decode attention for sm_100a: plan -> split-KV partial attention -> LSE merge.
//
// Work item = (sequence b, kv head h, token chunk [t0, t1)).  One CTA processes an item with
// a producer warp that streams K / V tiles global -> shared through TMA (128-byte swizzle)
// into a ring of stages (at head_dim 128 a second warp issues the V copies, from a descriptor
// the first posts per stage), and NCW consumer warps that each own 16 tokens of every stage:
//   S[16 tok x 8 heads]  = K_tile (A, ldmatrix) x Q^T (B, registers)          mma.sync bf16
//   online softmax over tokens (warp shuffles), P packed to bf16, transposed by movmatrix
//   O^T[D x 8 heads]    += V_tile^T (A, ldmatrix.trans) x P (B)               mma.sync bf16
// so every K / V byte is read from HBM once, by one CTA, for the whole GQA group.
// CTAs are persistent and pull items from a device-side list through an atomic counter.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_fp8.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "ptx.cuh"

namespace ooco {

constexpr int kStatusPlanOverflow = 1;
constexpr int kStatusWaitTimeout = 2;
// Reported by the checked build only (compiled with -DOOCO_CHECKS):
constexpr int kStatusBadTableEntry = 8;   // a block-table entry that is read lies outside [0, num_blocks)
constexpr int kStatusBadItem = 16;        // a work-item field outside its range
constexpr int kStatusBadIndex = 32;       // a partial-result slot, work-list or output index outside its buffer
constexpr int kStatusBadSmem = 64;        // a shared-memory destination outside the region it belongs to

// ------------------------------------------------------------------------------------ checked build
// With -DOOCO_CHECKS every index the kernels derive from device data (table entries, work items,
// partial-result slots) and every shared-memory destination of a copy is range-checked; a violation
// sets a bit of the workspace's status word and the access is skipped (or, for a table entry, replaced
// by an id the tensor-map bounds check turns into zeros).  Nothing traps.  Without the macro the
// checks compile to nothing.
#ifdef OOCO_CHECKS
constexpr bool kChecked = true;
#else
constexpr bool kChecked = false;
#endif
__host__ __device__ inline bool chk_table_entry(long long blk, long long num_blocks) { return blk >= 0 && blk < num_blocks; }
__host__ __device__ inline bool chk_index(long long i, long long n) { return i >= 0 && i < n; }
// item = {sequence, partial slot, first token, end token}
__host__ __device__ inline bool chk_item(long long b, long long slot, long long t0, long long t1, long long B,
                                         long long max_items, long long cap_tokens) {
  return b >= 0 && b < B && slot >= 0 && slot < max_items && t0 >= 0 && t0 <= t1 && t1 <= cap_tokens;
}
__host__ __device__ inline bool chk_span(long long off, long long bytes, long long lo, long long hi) {
  return off >= lo && bytes >= 0 && off + bytes <= hi;
}
// true = proceed.  In the checked build a failed predicate is recorded and answers false.
__device__ __forceinline__ bool checked(bool ok, int32_t* status, int bit) {
  if (kChecked && !ok) {
    atomicOr(status, bit);
    return false;
  }
  return true;
}
constexpr uint64_t kWaitLimitNs = 2000000000ull;  // every in-kernel wait gives up after 2 s

struct WsHeader {  // first 256 bytes of the workspace
  int32_t status;
  int32_t n_items;
  int32_t next_item;
  int32_t chunk_tokens;
  int32_t pad[60];
};
static_assert(sizeof(WsHeader) == 256, "header is 256 bytes");

struct DecodeParams {
  const __nv_bfloat16* q;
  __nv_bfloat16* out;
  const int32_t* block_table;
  const int32_t* context_lens;
  WsHeader* hdr;
  int4* items;            // [max_items] {b, partial slot = chunk index * Hkv + h, t0, t1}, longest first
  int32_t* seq_first;     // [B + 1] first chunk index of each sequence (exclusive scan)
  float* part_o;          // [max_items, GQ, D] normalised partial outputs
  float* part_lse;        // [max_items, GQ] log2-domain log-sum-exp of each partial
  int32_t B, Hq, Hkv, G, D, bs, MB;
  int32_t NB;             // physical blocks in the pool (read by the checked build only)
  int32_t out_f32;        // diagnostic: `out` holds fp32 and every row goes through the partial + merge path
  int32_t Sq;             // query tokens per sequence (the last Sq tokens of its context); 1 = decode
  int32_t GQ;             // G * Sq: score columns of one (sequence, kv head), column = query * G + head
  int32_t max_items;
  int32_t tile_rows;      // token rows per TMA box = min(bs, stage tokens)
  int32_t split_halves;   // 1: one 4-d TMA per 64-dim half; 0: one 5-d TMA per box
  int32_t nstages;
  int32_t nstages_raw;    // 8-bit prefill-chunk kernel: stages of its ring of 8-bit copies
  int32_t grid_main;      // CTAs the plan sizes the chunks for
  int32_t next_item_init; // start of the dynamic work counter = CTAs of the attention grid (they take the first units statically)
  int32_t chunk_min, chunk_max, items_per_cta;
  float scale_log2e;        // softmax scale * log2(e) (* the K tensor scale of an 8-bit cache)
  float v_scale;            // V tensor scale of an 8-bit cache (1 for bf16)
};

// ------------------------------------------------------------------------------------ append
struct AppendParams {
  const uint4* k_new;   // NULL: no append in this launch
  const uint4* v_new;
  uint16_t* k_cache;
  uint16_t* v_cache;
  const int32_t* block_table;
  const int32_t* positions;
  int32_t B, Hkv, D, bs, NB, MB;
  int32_t Sq;               // new tokens per sequence: k_new / v_new are [B, Sq, Hkv, D], token i goes to positions[b] + i
  int64_t bstr, hstr, tstr;
  int32_t kv8;              // 1: the caches hold 8-bit E4M3 codes (k_cache / v_cache are byte arrays)
  float k_scale, v_scale;   // tensor scales of an 8-bit cache: stored code = e4m3(x / scale)
};

// Eight bf16 values -> eight E4M3 codes: one IEEE fp32 division by the tensor scale, then round to
// nearest even, saturating at the largest finite code.
__device__ __forceinline__ uint2 quantize_e4m3x8(const uint4 w, float scale) {
  const uint32_t in[4] = {w.x, w.y, w.z, w.w};
  uint32_t out[2] = {0u, 0u};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float lo = __fdiv_rn(__uint_as_float(in[i] << 16), scale);
    const float hi = __fdiv_rn(__uint_as_float(in[i] & 0xffff0000u), scale);
    const uint32_t c = (uint32_t)__nv_cvt_float_to_fp8(lo, __NV_SATFINITE, __NV_E4M3) |
                       ((uint32_t)__nv_cvt_float_to_fp8(hi, __NV_SATFINITE, __NV_E4M3) << 8);
    out[i >> 1] |= c << (16 * (i & 1));
  }
  return make_uint2(out[0], out[1]);
}

// Copies the new K / V rows into their slots, one thread per 16-byte vector; `block` of
// `nblocks` CTAs cooperate grid-stride.
__device__ __forceinline__ void kv_append_body(const AppendParams& a, int block, int nblocks) {
  const int vec_per_row = a.D / 8;
  const long long n = (long long)a.B * a.Sq * a.Hkv * vec_per_row;
  for (long long i = block * (long long)blockDim.x + threadIdx.x; i < n; i += (long long)nblocks * blockDim.x) {
    const int v = (int)(i % vec_per_row);
    const int h = (int)((i / vec_per_row) % a.Hkv);
    const long long tok = i / ((long long)vec_per_row * a.Hkv);  // (sequence, new token) index
    const int b = (int)(tok / a.Sq);
    const long long pos64 = (long long)a.positions[b] + (tok % a.Sq);
    const int pos = pos64 > 0x7fffffffLL ? -1 : (int)pos64;
    if (pos < 0 || (long long)pos >= (long long)a.MB * a.bs) continue;
    const int blk = a.block_table[(size_t)b * a.MB + pos / a.bs];
    if (blk < 0 || blk >= a.NB) continue;
    const int64_t dst = (int64_t)blk * a.bstr + (int64_t)h * a.hstr + (int64_t)(pos % a.bs) * a.tstr + 8 * v;
    if (a.kv8) {
      *reinterpret_cast<uint2*>(reinterpret_cast<uint8_t*>(a.k_cache) + dst) = quantize_e4m3x8(a.k_new[i], a.k_scale);
      *reinterpret_cast<uint2*>(reinterpret_cast<uint8_t*>(a.v_cache) + dst) = quantize_e4m3x8(a.v_new[i], a.v_scale);
    } else {
      *reinterpret_cast<uint4*>(a.k_cache + dst) = a.k_new[i];
      *reinterpret_cast<uint4*>(a.v_cache + dst) = a.v_new[i];
    }
  }
}

__global__ void __launch_bounds__(256) kv_append_kernel(const AppendParams a) {
  kv_append_body(a, blockIdx.x, gridDim.x);
}

// ------------------------------------------------------------------------------------ host staging
// Host -> device staging of inputs that live in page-locked host memory: the CTAs read the host
// buffers through their device mapping (16-byte loads over the host link) instead of one copy-engine
// transfer per buffer, each of which costs several microseconds of fixed latency.
constexpr int kStageBuffers = 3;
struct HostStageParams {
  const uint8_t* src[kStageBuffers];  // device-visible addresses of page-locked host buffers
  uint8_t* dst[kStageBuffers];        // 256-byte aligned device buffers
  uint32_t bytes[kStageBuffers];      // multiples of 4; 0 = unused
};
__device__ __forceinline__ void host_stage_body(const HostStageParams& p, int block, int nblocks) {
  const uint32_t tid = block * blockDim.x + threadIdx.x, nthr = nblocks * blockDim.x;
#pragma unroll 1
  for (int k = 0; k < kStageBuffers; ++k) {
    const uint32_t n = p.bytes[k];
    if (((uintptr_t)p.src[k] & 15) == 0) {
      const uint32_t n16 = n / 16;
      for (uint32_t i = tid; i < n16; i += nthr)
        reinterpret_cast<uint4*>(p.dst[k])[i] = reinterpret_cast<const uint4*>(p.src[k])[i];
      for (uint32_t i = n16 * 4 + tid; i < n / 4; i += nthr)
        reinterpret_cast<uint32_t*>(p.dst[k])[i] = reinterpret_cast<const uint32_t*>(p.src[k])[i];
    } else {
      for (uint32_t i = tid; i < n / 4; i += nthr)
        reinterpret_cast<uint32_t*>(p.dst[k])[i] = reinterpret_cast<const uint32_t*>(p.src[k])[i];
    }
  }
}

// ------------------------------------------------------------------------------------ plan
// CTA 0 plans; CTAs 1 .. n_append (present only in the fused step) do the KV append; any further CTAs
// (host-buffer step only) stage the inputs the attention kernel reads.  The plan chooses the chunk
// length from the total work, splits every sequence into near-equal chunks that are multiples of
// `stage_tok`, and writes the item list.
template <int kThreads>
__global__ void __launch_bounds__(kThreads) plan_kernel(DecodeParams p, int stage_tok, int first_in_smem,
                                                        const AppendParams ap, int n_append,
                                                        const HostStageParams hs) {
  extern __shared__ int s_first[];  // when they fit (first_in_smem): seq_first [B + 1], then clamped lengths [B]
  // Launched programmatically: nothing of the caller's buffers or of the workspace may be touched
  // before the preceding work in the stream (which may still read the workspace, or still
  // produce this call's inputs) is complete.
  grid_dep_wait();
  grid_dep_launch();
  if (blockIdx.x > 0) {
    if ((int)blockIdx.x <= n_append)
      kv_append_body(ap, blockIdx.x - 1, n_append);
    else
      host_stage_body(hs, blockIdx.x - 1 - n_append, gridDim.x - 1 - n_append);
    return;
  }
  __shared__ long long s_red[kThreads / 32];
  __shared__ int s_scan[kThreads / 32];
  __shared__ long long s_total;
  __shared__ int s_run;
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const long long cap = (long long)p.MB * p.bs;

  int* s_len = s_first + p.B + 1;
  auto len_of = [&](int b) -> long long {  // context length clamped to [0, table capacity]
    if (first_in_smem) return s_len[b];
    const long long t = p.context_lens[b];
    return t < 0 ? 0 : (t > cap ? cap : t);
  };
  long long acc = 0;
  for (int b = tid; b < p.B; b += kThreads) {
    long long t = p.context_lens[b];
    t = t < 0 ? 0 : (t > cap ? cap : t);
    if (first_in_smem) s_len[b] = (int)t;
    acc += t;
  }
  for (int o = 16; o; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
  if (lane == 0) s_red[wid] = acc;
  __syncthreads();
  if (tid == 0) {
    long long t = 0;
    for (int i = 0; i < kThreads / 32; ++i) t += s_red[i];
    s_total = t;
    s_run = 0;
  }
  __syncthreads();
  // chunk length: about items_per_cta items per CTA, within [chunk_min, chunk_max]
  long long want = (s_total * p.Hkv) / ((long long)p.grid_main * p.items_per_cta) + 1;
  want = ((want + stage_tok - 1) / stage_tok) * stage_tok;
  if (want < p.chunk_min) want = p.chunk_min;
  if (want > p.chunk_max) want = p.chunk_max;
  const int chunk = (int)want;

  // exclusive scan of chunks per sequence, kThreads sequences at a time
  for (int base = 0; base < p.B; base += kThreads) {
    const int b = base + tid;
    int n = 0;
    if (b < p.B) n = (int)((len_of(b) + chunk - 1) / chunk);
    int inc = n;
    for (int o = 1; o < 32; o <<= 1) {
      int v = __shfl_up_sync(0xffffffffu, inc, o);
      if (lane >= o) inc += v;
    }
    if (lane == 31) s_scan[wid] = inc;
    __syncthreads();
    if (wid == 0) {
      int v = lane < kThreads / 32 ? s_scan[lane] : 0;
      int w = v;
      for (int o = 1; o < 32; o <<= 1) {
        int u = __shfl_up_sync(0xffffffffu, w, o);
        if (lane >= o) w += u;
      }
      if (lane < kThreads / 32) s_scan[lane] = w - v;  // exclusive warp offsets
    }
    __syncthreads();
    const int run = s_run;
    if (b < p.B) {
      const int f = run + s_scan[wid] + inc - n;
      p.seq_first[b] = f;
      if (first_in_smem) s_first[b] = f;
    }
    __syncthreads();
    if (tid == kThreads - 1) s_run = run + s_scan[wid] + inc;
    __syncthreads();
  }
  const int n_chunks = s_run;
  if (tid == 0) {
    p.seq_first[p.B] = n_chunks;
    if (first_in_smem) s_first[p.B] = n_chunks;
  }
  __syncthreads();
  const int* first = first_in_smem ? s_first : p.seq_first;
  long long n_items = (long long)n_chunks * p.Hkv;
  const bool overflow = n_items > p.max_items;
  if (overflow) n_items = 0;
  if (tid == 0) {
    p.hdr->status = overflow ? kStatusPlanOverflow : 0;
    p.hdr->n_items = (int)n_items;
    p.hdr->next_item = p.next_item_init;
    p.hdr->chunk_tokens = chunk;
  }
  // Items in order of decreasing length (longest first keeps the tail of the dynamic schedule
  // short): counting sort of the chunks by length in stages.  An item carries its partial-result
  // slot (chunk index * Hkv + head), which does not depend on the order.
  __shared__ int s_hist[kThreads];    // bucket r = kThreads - 1 - min(stages, kThreads - 1)
  __shared__ int s_cursor[kThreads];
  s_hist[tid] = 0;
  __syncthreads();
  const int n_chunks_ok = overflow ? 0 : n_chunks;
  auto chunk_of = [&](int ci, int& b, int& t0, int& t1) {
    int lo = 0, hi = p.B;  // largest b with first[b] <= ci
    while (hi - lo > 1) {
      const int mid = (lo + hi) >> 1;
      if (first[mid] <= ci) lo = mid; else hi = mid;
    }
    b = lo;
    const int T = (int)len_of(b);
    const int n = first[b + 1] - first[b];
    const int c = ci - first[b];
    int len = (T + n - 1) / n;                              // near-equal chunks ...
    len = ((len + stage_tok - 1) / stage_tok) * stage_tok;  // ... in whole stages
    t0 = c * len;
    t1 = t0 + len;
    if (t0 > T) t0 = T;
    if (t1 > T) t1 = T;
    const int stages = (t1 - t0 + stage_tok - 1) / stage_tok;
    return kThreads - 1 - (stages < kThreads - 1 ? stages : kThreads - 1);
  };
  for (int ci = tid; ci < n_chunks_ok; ci += kThreads) {
    int b, t0, t1;
    atomicAdd(&s_hist[chunk_of(ci, b, t0, t1)], 1);
  }
  __syncthreads();
  {  // exclusive scan of the histogram (bucket 0 = longest)
    const int v = s_hist[tid];
    int inc = v;
    for (int o = 1; o < 32; o <<= 1) {
      int u = __shfl_up_sync(0xffffffffu, inc, o);
      if (lane >= o) inc += u;
    }
    if (lane == 31) s_scan[wid] = inc;
    __syncthreads();
    if (wid == 0) {
      int w0 = lane < kThreads / 32 ? s_scan[lane] : 0;
      int w = w0;
      for (int o = 1; o < 32; o <<= 1) {
        int u = __shfl_up_sync(0xffffffffu, w, o);
        if (lane >= o) w += u;
      }
      if (lane < kThreads / 32) s_scan[lane] = w - w0;
    }
    __syncthreads();
    s_cursor[tid] = s_scan[wid] + inc - v;
  }
  __syncthreads();
  for (int ci = tid; ci < n_chunks_ok; ci += kThreads) {
    int b, t0, t1;
    const int r = chunk_of(ci, b, t0, t1);
    const long long pos = atomicAdd(&s_cursor[r], 1);
    for (int h = 0; h < p.Hkv; ++h)
      if (checked(chk_index(pos * p.Hkv + h, p.max_items), &p.hdr->status, kStatusBadIndex))
        p.items[pos * p.Hkv + h] = make_int4(b, ci * p.Hkv + h, t0, t1);
  }
  // sequences without context produce zeros
  const int row = p.Sq * p.Hq * p.D;
  for (int b = wid; b < p.B; b += kThreads / 32) {
    if (len_of(b) > 0) continue;
    if (p.out_f32) {
      for (int i = lane; i < row; i += 32) reinterpret_cast<float*>(p.out)[(size_t)b * row + i] = 0.f;
    } else {
      for (int i = lane; i < row; i += 32) p.out[(size_t)b * row + i] = __float2bfloat16(0.f);
    }
  }
}

// Bounded mbarrier wait whose verdict is the same in every lane of the (converged) warp.
__device__ __forceinline__ bool warp_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  return __all_sync(0xffffffffu, mbar_wait_bounded(bar, parity, abort_flag, kWaitLimitNs));
}

// ------------------------------------------------------------------------------------ main
// Shared-memory carve-up, shared by host (sizing) and device.  TPW = 16-token tiles each
// consumer warp owns per stage.
// KVM: 0 = bf16 cache; 1 = 8-bit cache, scores on mma.sync from codes widened in registers; 2 = 8-bit cache,
// scores on tcgen05 (kind::f8f6f4) straight from the stage, read back from tensor memory.
template <int D, int NCW, int NT, int TPW, int KVM = 0>
struct SmemLayout {
  static constexpr int kStageTok = 16 * NCW * TPW;
  static constexpr int kTileBytes = kStageTok * D * (KVM ? 1 : 2);  // K (or V) bytes of one stage
  static constexpr int kStageBytes = 2 * kTileBytes;
  static constexpr int kHeads = NT * 8;
  static constexpr int kOStride = 64 + 4;                    // floats per head row of one 64-dim pass
  static constexpr int kMergeOBytes = NCW * kHeads * kOStride * 4;
  static constexpr int kMergeBytes = kMergeOBytes + NCW * kHeads * 2 * 4;
  // KVM 2: K and V have rings of their own.  The K tile of a stage is dead as soon as its score MMAs are complete
  // (the scores wait in tensor memory, kTcSBuffers stages of them), so kTcKSlots slots keep the K stream going and
  // the rest of the shared memory gives the V ring (`nstages` slots) the depth the consumers' latency needs.
  // Besides: the query of a work item as two E4M3 terms ([2 * kHeads rows][128 bytes], 1024-byte aligned), two
  // such tiles (consecutive items alternate), and beside every score buffer the inverse row scales of its item.
  static constexpr int kTcKSlots = 2, kTcSBuffers = 8;
  // A second producer warp issues the V copies of every stage (the first hands it a descriptor per stage): one
  // warp issuing all copies of a stage is the limit with small boxes.  Present for the 8-bit tcgen05 mode and for
  // the bf16 cache at head_dim 128 (at head_dim 64 the extra warp would cost the fourth CTA per SM).
  static constexpr bool kVProducer = KVM == 2 || (KVM == 0 && D == 128);
  static constexpr int kWarps = NCW + 1 + (KVM == 2 ? 1 : 0) + (kVProducer ? 1 : 0);  // consumers, producer, [MMA], [V producer]
  static constexpr int kVDescBytes = 96;  // what the V producer warp needs for one stage (see VStageDesc)
  static constexpr int kQSplitBytes = KVM == 2 ? 2 * kHeads * 128 : 0;
  static constexpr int kTcSColumns = 2 * kHeads;             // tensor-memory columns of one stage's scores
  __host__ __device__ static int q_slot_bytes(int G) { return ((G * D * 2 + 127) / 128) * 128; }
  __host__ __device__ static size_t total(int nstages, int G) {
    if (KVM == 2)
      return 1024 + (size_t)kTcKSlots * (kTileBytes + q_slot_bytes(G) + 16 + 16) +
             (size_t)nstages * (kTileBytes + 16 + 16 + kVDescBytes + 8) + kMergeBytes + 64 + 2 * kQSplitBytes +
             kTcSBuffers * (kHeads * 4 + 8) + 32;
    return 1024 + (size_t)nstages * (kStageBytes + q_slot_bytes(G) + 16 + 16 + (kVProducer ? kVDescBytes + 8 : 0)) +
           kMergeBytes + 64;
  }
};

// One consumer warp's work on its TPW tiles of a stage.  kTail: some of the warp's rows lie
// beyond the chunk (`valid` < 16 * TPW of them count); masked rows get weight 0 and their V
// words are cleared in registers, so NaN / stale bytes there never reach an accumulator.
template <int D, int NT, int TPW, bool kTail>
__device__ __forceinline__ void consume_tiles(uint32_t kst, uint32_t vst, const uint32_t (&tile_k)[TPW],
                                              const uint32_t (&tile_v)[TPW], const uint32_t (&kpat)[D / 16],
                                              const uint32_t (&vpat)[D / 16],
                                              const uint32_t (&qf)[NT][D / 16][2], float (&m_run)[NT][2],
                                              float (&l_run)[NT][2], float (&o_acc)[NT][D / 16][4],
                                              float scale_log2e, int valid, int g, int t, int lim_w = 0,
                                              const int (*qi_col)[2] = nullptr) {
  // kTail only: lim_w = rows of this warp the first query token may see (causal limit, several query
  // tokens per sequence), qi_col[nt][c] = query token of the lane's score column c of tile nt.
  constexpr int KS = D / 16;
  constexpr int NACC = TPW == 1 ? 2 : 1;  // a lone tile splits its k-steps over two accumulators
  // ---- scores: S = K_tile x Q^T
  float sc[TPW][NT][NACC][4];
#pragma unroll
  for (int u = 0; u < TPW; ++u)
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
      for (int a = 0; a < NACC; ++a)
#pragma unroll
        for (int e = 0; e < 4; ++e) sc[u][nt][a][e] = 0.f;
#pragma unroll
  for (int k = 0; k < KS; ++k) {
#pragma unroll
    for (int u = 0; u < TPW; ++u) {
      if (kTail && valid <= 16 * u) continue;
      uint32_t a0, a1, a2, a3;
      ldmatrix_x4(kst + tile_k[u] + kpat[k], a0, a1, a2, a3);
#pragma unroll
      for (int nt = 0; nt < NT; ++nt)
        mma_bf16(sc[u][nt][k % NACC], a0, a1, a2, a3, qf[nt][k][0], qf[nt][k][1]);
    }
  }
  uint32_t pb[TPW][NT][2];
#pragma unroll
  for (int nt = 0; nt < NT; ++nt) {
    float s[TPW][4];  // [u]: (token g, head 2t) (token g, head 2t+1) (token g+8, 2t) (token g+8, 2t+1)
    float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
    for (int u = 0; u < TPW; ++u) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        float v = sc[u][nt][0][e];
        if (NACC == 2) v += sc[u][nt][NACC - 1][e];
        s[u][e] = v * scale_log2e;
      }
      if (kTail) {
        const int l0 = min(valid, lim_w + qi_col[nt][0]), l1 = min(valid, lim_w + qi_col[nt][1]);
        if (16 * u + g >= l0) s[u][0] = -INFINITY;
        if (16 * u + g >= l1) s[u][1] = -INFINITY;
        if (16 * u + g + 8 >= l0) s[u][2] = -INFINITY;
        if (16 * u + g + 8 >= l1) s[u][3] = -INFINITY;
      }
      mx0 = fmaxf(mx0, fmaxf(s[u][0], s[u][2]));
      mx1 = fmaxf(mx1, fmaxf(s[u][1], s[u][3]));
    }
#pragma unroll
    for (int o = 4; o < 32; o <<= 1) {
      mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, o));
      mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, o));
    }
    const float mo0 = m_run[nt][0], mo1 = m_run[nt][1];
    float mn0 = fmaxf(mo0, mx0), mn1 = fmaxf(mo1, mx1);
    m_run[nt][0] = mn0;
    m_run[nt][1] = mn1;
    if (kTail) {  // a column that has seen nothing yet (causal limit): keep the exponents finite
      mn0 = mn0 == -INFINITY ? 0.f : mn0;
      mn1 = mn1 == -INFINITY ? 0.f : mn1;
    }
    const float al0 = ex2(mo0 - mn0), al1 = ex2(mo1 - mn1);
    float add0 = 0.f, add1 = 0.f;
#pragma unroll
    for (int u = 0; u < TPW; ++u) {
      const uint32_t p01 = pack_bf16x2(ex2(s[u][0] - mn0), ex2(s[u][1] - mn1));  // token g
      const uint32_t p23 = pack_bf16x2(ex2(s[u][2] - mn0), ex2(s[u][3] - mn1));  // token g+8
      // sums use the rounded weights, so numerator and denominator agree exactly
      add0 += __uint_as_float(p01 << 16) + __uint_as_float(p23 << 16);
      add1 += __uint_as_float(p01 & 0xffff0000u) + __uint_as_float(p23 & 0xffff0000u);
      pb[u][nt][0] = movmatrix_trans(p01);  // tokens 2t,2t+1 of head g
      pb[u][nt][1] = movmatrix_trans(p23);  // tokens 2t+8,2t+9 of head g
    }
    l_run[nt][0] = l_run[nt][0] * al0 + add0;
    l_run[nt][1] = l_run[nt][1] * al1 + add1;
    if (__any_sync(0xffffffffu, (al0 != 1.f) | (al1 != 1.f))) {
#pragma unroll
      for (int k = 0; k < KS; ++k) {
        o_acc[nt][k][0] *= al0;
        o_acc[nt][k][1] *= al1;
        o_acc[nt][k][2] *= al0;
        o_acc[nt][k][3] *= al1;
      }
    }
  }
  // ---- values: O^T += V_tile^T x P
#pragma unroll
  for (int u = 0; u < TPW; ++u) {
    if (kTail && valid <= 16 * u) continue;
    uint32_t mk01 = 0xffffffffu, mk23 = 0xffffffffu;
    if (kTail) {
      const int v = valid - 16 * u;
      mk01 = (2 * t < v ? 0x0000ffffu : 0u) | (2 * t + 1 < v ? 0xffff0000u : 0u);
      mk23 = (2 * t + 8 < v ? 0x0000ffffu : 0u) | (2 * t + 9 < v ? 0xffff0000u : 0u);
    }
#pragma unroll
    for (int k = 0; k < KS; ++k) {
      uint32_t a0, a1, a2, a3;
      ldmatrix_x4_trans(vst + tile_v[u] + vpat[k], a0, a1, a2, a3);
      if (kTail) {
        a0 &= mk01;
        a1 &= mk01;
        a2 &= mk23;
        a3 &= mk23;
      }
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) mma_bf16(o_acc[nt][k], a0, a1, a2, a3, pb[u][nt][0], pb[u][nt][1]);
    }
  }
}

// ---- 8-bit (E4M3) cache: one consumer warp's work on its 16-token tile of a stage.
// A token row is D = 128 bytes.  The codes are widened to f16 in registers (exactly, up to the fixed
// factor 2^-8: see e4m3x2_to_f16x2) and both contractions run as f16 MMAs; the tensor scales and
// that factor are applied outside (K's is folded into the softmax scale, V's multiplies the output).
// (The 8-bit mma.sync shapes were measured slower than widening plus f16 MMAs on this part.)
// Fragment bookkeeping:
//   scores  ldmatrix (16-bit units) hands lane (g, t) the four codes of dims 4t .. 4t+3 of a 16-dim
//           chunk; they fill the MMA's k slots (2t, 2t+1) and (2t+8, 2t+9).  The contraction does not
//           care about the order of k as long as Q uses the same one (it does: see the q fragments).
//   values  ldmatrix.trans hands lane (g, t) dims (2g, 2g+1) of tokens (2t, 2t+1); a byte permute
//           regroups them per dim, so MMA row g is dim 2g and row g + 8 is dim 2g + 1 of the chunk
//           (the epilogue writes the accumulators back in that order).
// Two E4M3 codes (bytes of `x` picked by the byte-permute selector `sel`, which must also zero the
// upper byte of each 16-bit lane) -> f16x2 holding their values / 256, exactly, with integer
// operations only (the conversion instruction runs on the slow special-function pipe): with the code
// c in the low byte of a lane, (c + (c & 0x80)) << 7 moves the sign to bit 15 and the 7 magnitude bits
// to bits 7..13, i.e. exponent and mantissa land in the f16 fields with the exponent read against
// bias 15 instead of 7 (hence the factor 2^-8; subnormal codes become f16 subnormals of the same
// relative value).  The NaN codes come out as the finite +-480 / 256.
template <uint32_t sel>
__device__ __forceinline__ uint32_t e4m3x2_to_f16x2(uint32_t x) {
  const uint32_t c = __byte_perm(x, 0u, sel);
  return (c + (c & 0x00800080u)) << 7;
}
constexpr uint32_t kSelB0B1 = 0x4140, kSelB2B3 = 0x4342;  // consecutive codes (score operand)
constexpr uint32_t kSelB0B2 = 0x4240, kSelB1B3 = 0x4341;  // codes two apart (value operand: regroup per dim)
constexpr float kE4m3WidenFactor = 256.f;                  // what the widened values must be multiplied by
__device__ __forceinline__ float f16_lo(uint32_t x) { return __half2float(__ushort_as_half((unsigned short)(x & 0xffffu))); }
__device__ __forceinline__ float f16_hi(uint32_t x) { return __half2float(__ushort_as_half((unsigned short)(x >> 16))); }

// Softmax and value part of a 16-token tile over the 8-bit cache; `sv[nt]` holds the tile's scaled scores (log2
// domain) in the MMA accumulator layout: (token g, head 2t) (token g, head 2t+1) (token g+8, 2t) (token g+8, 2t+1).
template <int D, int NT, bool kTail>
__device__ __forceinline__ void kv8_softmax_values(uint32_t vst, uint32_t tile_off, const uint32_t (&pat)[D / 16],
                                                   float (&sv)[NT][4], float (&m_run)[NT][2], float (&l_run)[NT][2],
                                                   float (&o_acc)[NT][D / 16][4], int valid, int g, int t, int lim_w,
                                                   const int (*qi_col)[2]);

template <int D, int NT, bool kTail>
__device__ __forceinline__ void consume_tile_kv8(uint32_t kst, uint32_t vst, uint32_t tile_off,
                                                 const uint32_t (&pat)[D / 16], const uint32_t (&qf)[NT][D / 16][2],
                                                 float (&m_run)[NT][2], float (&l_run)[NT][2],
                                                 float (&o_acc)[NT][D / 16][4], float scale_log2e, int valid,
                                                 int g, int t, int lim_w = 0, const int (*qi_col)[2] = nullptr) {
  // kTail only: lim_w / qi_col carry the causal limit of several query tokens, as in consume_tiles
  constexpr int KS = D / 16;  // 16-dim chunks
  float sc[NT][2][4];
#pragma unroll
  for (int nt = 0; nt < NT; ++nt)
#pragma unroll
    for (int a = 0; a < 2; ++a)
#pragma unroll
      for (int e = 0; e < 4; ++e) sc[nt][a][e] = 0.f;
#pragma unroll
  for (int j = 0; j < KS / 2; ++j) {
    uint32_t r0, r1, r2, r3;  // (tokens 0-7, chunk 2j) (tokens 8-15, 2j) (tokens 0-7, 2j+1) (tokens 8-15, 2j+1)
    ldmatrix_x4(kst + tile_off + pat[j], r0, r1, r2, r3);
    const uint32_t a0 = e4m3x2_to_f16x2<kSelB0B1>(r0), a2 = e4m3x2_to_f16x2<kSelB2B3>(r0);
    const uint32_t a1 = e4m3x2_to_f16x2<kSelB0B1>(r1), a3 = e4m3x2_to_f16x2<kSelB2B3>(r1);
    const uint32_t c0 = e4m3x2_to_f16x2<kSelB0B1>(r2), c2 = e4m3x2_to_f16x2<kSelB2B3>(r2);
    const uint32_t c1 = e4m3x2_to_f16x2<kSelB0B1>(r3), c3 = e4m3x2_to_f16x2<kSelB2B3>(r3);
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      mma_f16(sc[nt][0], a0, a1, a2, a3, qf[nt][2 * j][0], qf[nt][2 * j][1]);
      mma_f16(sc[nt][1], c0, c1, c2, c3, qf[nt][2 * j + 1][0], qf[nt][2 * j + 1][1]);
    }
  }
  float sv[NT][4];
#pragma unroll
  for (int nt = 0; nt < NT; ++nt)
#pragma unroll
    for (int e = 0; e < 4; ++e) sv[nt][e] = (sc[nt][0][e] + sc[nt][1][e]) * scale_log2e;
  kv8_softmax_values<D, NT, kTail>(vst, tile_off, pat, sv, m_run, l_run, o_acc, valid, g, t, lim_w, qi_col);
}

template <int D, int NT, bool kTail>
__device__ __forceinline__ void kv8_softmax_values(uint32_t vst, uint32_t tile_off, const uint32_t (&pat)[D / 16],
                                                   float (&sv)[NT][4], float (&m_run)[NT][2], float (&l_run)[NT][2],
                                                   float (&o_acc)[NT][D / 16][4], int valid, int g, int t, int lim_w,
                                                   const int (*qi_col)[2]) {
  constexpr int KS = D / 16;
  uint32_t pb[NT][2];
#pragma unroll
  for (int nt = 0; nt < NT; ++nt) {
    float (&s)[4] = sv[nt];
    if (kTail) {
      const int l0 = min(valid, lim_w + qi_col[nt][0]), l1 = min(valid, lim_w + qi_col[nt][1]);
      if (g >= l0) s[0] = -INFINITY;
      if (g >= l1) s[1] = -INFINITY;
      if (g + 8 >= l0) s[2] = -INFINITY;
      if (g + 8 >= l1) s[3] = -INFINITY;
    }
    float mx0 = fmaxf(s[0], s[2]), mx1 = fmaxf(s[1], s[3]);
#pragma unroll
    for (int o = 4; o < 32; o <<= 1) {
      mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, o));
      mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, o));
    }
    const float mo0 = m_run[nt][0], mo1 = m_run[nt][1];
    float mn0 = fmaxf(mo0, mx0), mn1 = fmaxf(mo1, mx1);
    m_run[nt][0] = mn0;
    m_run[nt][1] = mn1;
    if (kTail) {  // a column that has seen nothing yet (causal limit): keep the exponents finite
      mn0 = mn0 == -INFINITY ? 0.f : mn0;
      mn1 = mn1 == -INFINITY ? 0.f : mn1;
    }
    const float al0 = ex2(mo0 - mn0), al1 = ex2(mo1 - mn1);
    const uint32_t p01 = pack_f16x2(ex2(s[0] - mn0), ex2(s[1] - mn1));  // token g
    const uint32_t p23 = pack_f16x2(ex2(s[2] - mn0), ex2(s[3] - mn1));  // token g+8
    // sums use the rounded weights, so numerator and denominator agree exactly
    l_run[nt][0] = l_run[nt][0] * al0 + f16_lo(p01) + f16_lo(p23);
    l_run[nt][1] = l_run[nt][1] * al1 + f16_hi(p01) + f16_hi(p23);
    pb[nt][0] = movmatrix_trans(p01);  // tokens 2t,2t+1 of head g
    pb[nt][1] = movmatrix_trans(p23);  // tokens 2t+8,2t+9 of head g
    if (__any_sync(0xffffffffu, (al0 != 1.f) | (al1 != 1.f))) {
#pragma unroll
      for (int k = 0; k < KS; ++k) {
        o_acc[nt][k][0] *= al0;
        o_acc[nt][k][1] *= al1;
        o_acc[nt][k][2] *= al0;
        o_acc[nt][k][3] *= al1;
      }
    }
  }
  uint32_t mk01 = 0xffffffffu, mk23 = 0xffffffffu;
  if (kTail) {
    mk01 = (2 * t < valid ? 0x0000ffffu : 0u) | (2 * t + 1 < valid ? 0xffff0000u : 0u);
    mk23 = (2 * t + 8 < valid ? 0x0000ffffu : 0u) | (2 * t + 9 < valid ? 0xffff0000u : 0u);
  }
#pragma unroll
  for (int j = 0; j < KS / 2; ++j) {
    uint32_t r0, r1, r2, r3;  // transposed: lane (g, t) holds dims (2g, 2g+1) x tokens (2t, 2t+1) of each matrix
    ldmatrix_x4_trans(vst + tile_off + pat[j], r0, r1, r2, r3);
#pragma unroll
    for (int half = 0; half < 2; ++half) {
      const uint32_t lo = half ? r2 : r0, hi = half ? r3 : r1;  // tokens 0-7 / 8-15 of chunk 2j + half
      uint32_t a0 = e4m3x2_to_f16x2<kSelB0B2>(lo);  // dim 2g,   tokens 2t, 2t+1
      uint32_t a1 = e4m3x2_to_f16x2<kSelB1B3>(lo);  // dim 2g+1, tokens 2t, 2t+1
      uint32_t a2 = e4m3x2_to_f16x2<kSelB0B2>(hi);  // dim 2g,   tokens 2t+8, 2t+9
      uint32_t a3 = e4m3x2_to_f16x2<kSelB1B3>(hi);  // dim 2g+1, tokens 2t+8, 2t+9
      if (kTail) {
        a0 &= mk01;
        a1 &= mk01;
        a2 &= mk23;
        a3 &= mk23;
      }
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) mma_f16(o_acc[nt][2 * j + half], a0, a1, a2, a3, pb[nt][0], pb[nt][1]);
    }
  }
}

// D[tmem] (+)= A[smem] x B[smem] with 8-bit floating-point operands (the formats are in the instruction descriptor).
__device__ __forceinline__ void umma_f8_ss(uint32_t d_tmem, uint64_t a, uint64_t b, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
      "l"(a), "l"(b), "r"(idesc), "r"(accumulate)
      : "memory");
}
// 16 lanes x (8 * N) fp32 columns of tensor memory in the accumulator layout of mma.sync m16n8: for column
// block i, registers 4i .. 4i + 3 of lane (g = lane / 4, t = lane % 4) hold (row g, columns 2t, 2t + 1) and
// (row g + 8, columns 2t, 2t + 1).  The lane field of the address may be the warp's lane quarter base or 16 more.
__device__ __forceinline__ void tmem_ld_frag(uint32_t taddr, uint32_t (&r)[8]) {
  asm volatile("tcgen05.ld.sync.aligned.16x256b.x2.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
               : "r"(taddr));
}
__device__ __forceinline__ void tmem_ld_frag(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.16x256b.x4.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr));
}
// Two fp32 -> two E4M3 codes (round to nearest even, saturating); `lo` lands in the low byte.
__device__ __forceinline__ uint32_t pack_e4m3x2(float lo, float hi) {
  uint16_t d;
  asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(d) : "f"(hi), "f"(lo));
  return d;
}

// KVM 2: one stage's V copies as the K producer hands them to the V producer warp (one slot per V ring slot).
struct VStageDesc {
  int32_t nbox;      // boxes (TMA copies) of the stage; -1 = end marker: arrive on the stage's barrier and stop
  int32_t h;         // kv head
  int32_t pad[2];
  int32_t blk[8];    // physical block of box i (8 boxes of 16 rows fill a 128-token stage)
  int32_t c_tok[8];  // first token row of box i inside its block
  int32_t pad2[4];
};
static_assert(sizeof(VStageDesc) == 96, "descriptor slot is 96 bytes");

// The 8-bit path is bound by the consumer warps' instruction latency, not by HBM, so its 8-warp shape
// is compiled for two CTAs per SM (16 consumer warps), which caps it at 112 registers per thread (102 with the
// extra MMA warp of KVM 2).
//
// KVM 2 -- scores of the 8-bit cache on the 5th-generation tensor cores.  A stage is 128 tokens = the M of one
// tcgen05.mma: one more warp (NCW + 1) waits for each stage, splits the stage's query rows into two E4M3 terms
// (q * a = hi + lo / 16 with a power-of-two row scale a: as precise as the bf16 query) in a swizzled [16 x 128 B]
// tile and issues S[128 tok x 16] = K_stage . Qsplit^T (4 MMAs of K 32, kind::f8f6f4, both operands straight from
// shared memory, K as the TMA wrote it) into the stage's own tensor-memory columns.  The consumer warps load their
// 16-token tile of S in the mma.sync accumulator layout and go on with the softmax and the value MMAs as in KVM 1;
// the codes of K are never widened.
template <int D, int NCW, int NT, int TPW, int KVM>
__device__ __forceinline__ uint32_t decode_main_body(const CUtensorMap& tm_k, const CUtensorMap& tm_v,
                                                     const DecodeParams& p, uint8_t* smem_raw) {
  constexpr bool KV8 = KVM != 0, KVTC = KVM == 2;
  constexpr bool VP = SmemLayout<D, NCW, NT, TPW, KVM>::kVProducer;  // the V copies are issued by a warp of their own
  constexpr int kVProducerWarp = NCW + (KVTC ? 2 : 1);
  using L = SmemLayout<D, NCW, NT, TPW, KVM>;
  static_assert(!KV8 || (D == 128 && TPW == 1), "the 8-bit path is built for head_dim 128, one tile per warp");
  static_assert(!KVTC || NCW == 8, "a stage must hold the 128 tokens of one tcgen05 MMA");
  constexpr int kStageTok = L::kStageTok;
  constexpr int KS = D / 16;  // k-steps of the score MMA = m-tiles of the value MMA

  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* gen = smem_raw + (base - raw);
  const int nst = p.nstages;
  const int qslot = L::q_slot_bytes(p.GQ);
  constexpr int kNK = L::kTcKSlots, kNS = L::kTcSBuffers;
  // stages: [nst][K tile, V tile]; KVM 2: K ring [kNK][K tile], then V ring [nst][V tile] (full / empty / meta below
  // are the V ring's, i.e. what the consumer warps see, in every mode)
  const uint32_t s_stage = base;
  const uint32_t s_vring = s_stage + (uint32_t)kNK * L::kTileBytes;
  const uint32_t s_qs = KVTC ? s_vring + (uint32_t)nst * L::kTileBytes
                             : s_stage + (uint32_t)nst * L::kStageBytes;  // KVM 2: two split query tiles (1024-byte aligned)
  const uint32_t s_q = s_qs + 2u * L::kQSplitBytes;
  const uint32_t s_merge = s_q + (uint32_t)(KVTC ? kNK : nst) * qslot;  // (KVM 2: the query rows travel with the K tile)
  const uint32_t s_meta = s_merge + L::kMergeBytes;
  const uint32_t s_kmeta = s_meta + (uint32_t)nst * 16;
  const uint32_t s_full = s_kmeta + (KVTC ? kNK * 16u : 0u);
  const uint32_t s_empty = s_full + (uint32_t)nst * 8;
  const uint32_t s_mbar = s_empty + (uint32_t)nst * 8;
  const uint32_t s_inva = s_mbar + 16;                     // KVM 2: [kNS][heads] inverse row scales, one set per score buffer
  const uint32_t s_sready = s_inva + (uint32_t)kNS * L::kHeads * 4;  // KVM 2: [kNS] the stage's scores are in tensor memory
  const uint32_t s_drain = s_sready + (uint32_t)kNS * 8;
  const uint32_t s_tslot = s_drain + 8;
  const uint32_t s_qfree = s_tslot + 8;                     // KVM 2: [2] the MMAs that read split tile i are complete
  const uint32_t s_kfull = s_qfree + 16;                    // KVM 2: [kNK] the K tile (and the item's query rows) has landed
  const uint32_t s_kempty = s_kfull + (uint32_t)kNK * 8;    // KVM 2: [kNK] the MMAs that read the K tile are complete
  const uint32_t s_vdfull = KVTC ? s_kempty + (uint32_t)kNK * 8 : s_mbar + 16;  // [nst] the stage's V descriptor is posted
  const uint32_t s_vdesc = s_vdfull + (uint32_t)nst * 8;    // [nst] VStageDesc
  VStageDesc* g_vdesc = reinterpret_cast<VStageDesc*>(gen + (s_vdesc - base));
  int4* g_kmeta = reinterpret_cast<int4*>(gen + (s_kmeta - base));
  float* g_merge = reinterpret_cast<float*>(gen + (s_merge - base));
  int4* g_meta = reinterpret_cast<int4*>(gen + (s_meta - base));
  uint8_t* g_q = gen + (s_q - base);
  volatile int* s_abort = reinterpret_cast<volatile int*>(gen + (s_mbar + 8 - base));

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    *s_abort = 0;
    for (int i = 0; i < nst; ++i) {
      mbar_init(s_full + 8 * i, 1);
      mbar_init(s_empty + 8 * i, NCW);
    }
    mbar_init(s_mbar, NCW * 32);
    if (VP)
      for (int i = 0; i < nst; ++i) mbar_init(s_vdfull + 8 * i, 1);
    if (KVTC) {
      for (int i = 0; i < kNS; ++i) mbar_init(s_sready + 8 * i, 1);
      for (int i = 0; i < kNK; ++i) {
        mbar_init(s_kfull + 8 * i, 1);
        mbar_init(s_kempty + 8 * i, 1);
      }
      mbar_init(s_drain, 1);
      mbar_init(s_qfree, 1);
      mbar_init(s_qfree + 8, 1);
    }
    fence_mbar_init();
  }
  uint32_t tmem = 0;
  if (KVTC) {
    if (warp == NCW + 1) {
      tmem_alloc(s_tslot, kNS * L::kTcSColumns);  // 128 or 256 columns
    }
    tc_fence_before_sync();
  }
  __syncthreads();
  if (KVTC) {
    tc_fence_after_sync();
    tmem = *reinterpret_cast<volatile uint32_t*>(gen + (s_tslot - base));
  }
  grid_dep_wait();    // the plan (and a fused append) must have completed
  grid_dep_launch();  // the merge kernel may queue up behind this grid
  const int n_items = p.hdr->n_items;

  if (KVTC && warp == NCW + 1) {
    // ================================================================= score MMA warp (KVM 2)
    // kind::f8f6f4: E4M3 x E4M3 -> fp32, both operands K-major, M = 128 tokens, N = 2 * heads (high and low term)
    const uint32_t idesc = (1u << 4) | ((uint32_t)(L::kTcSColumns >> 3) << 17) | ((uint32_t)(kStageTok >> 4) << 24);
    bool issued = false;
    // items seen so far; item n (counted from 1) uses split tile (n - 1) & 1, as that tile's use number (n - 1) >> 1.
    // A tile is rewritten only once the MMAs of its previous use are complete: the item's last stage commits to
    // the tile's own barrier.
    uint32_t n_item = 0;
    float my_inva = 0.f;  // lane r: the inverse scale of row r of the current item
    for (uint32_t it = 0;; ++it) {
      const uint32_t slot = it % kNK, sbuf = it % kNS;  // K ring slot (the query rows share it), score buffer
      if (!warp_wait(s_kfull + 8 * slot, (it / kNK) & 1u, s_abort)) {
        if (lane == 0) atomicOr(&p.hdr->status, kStatusWaitTimeout);
        break;
      }
      const int4 meta = g_kmeta[slot];
      if (meta.x < 0) break;
      const bool first = (meta.w >> 16) & 1, last = (meta.w >> 17) & 1;
      if (first) ++n_item;
      const uint32_t qb = (n_item - 1) & 1, q_use = (n_item - 1) >> 1;
      if (first && !warp_wait(s_qfree + 8 * qb, (q_use & 1u) ^ 1u, s_abort)) {  // passes at once for a tile's first use
        if (lane == 0) atomicOr(&p.hdr->status, kStatusWaitTimeout);
        break;
      }
      // ---- at the item's first stage: its query rows, row r as hi + lo / 16, scaled by a power of two that
      // brings the row's largest magnitude into [128, 256) (E4M3 goes up to 448); lane l owns dims 4l .. 4l + 3
      const uint8_t* qs = g_q + (size_t)slot * qslot;
      uint8_t* qd = gen + (s_qs - base) + (size_t)qb * L::kQSplitBytes;
#pragma unroll 2
      for (int hr = 0; first && hr < L::kHeads; ++hr) {
        float x[4] = {0.f, 0.f, 0.f, 0.f};
        if (hr < p.GQ) {
          const uint2 w = *reinterpret_cast<const uint2*>(qs + ((size_t)hr * D + 4 * lane) * 2);
          x[0] = __uint_as_float(w.x << 16);
          x[1] = __uint_as_float(w.x & 0xffff0000u);
          x[2] = __uint_as_float(w.y << 16);
          x[3] = __uint_as_float(w.y & 0xffff0000u);
        }
        float mx = fmaxf(fmaxf(fabsf(x[0]), fabsf(x[1])), fmaxf(fabsf(x[2]), fabsf(x[3])));
#pragma unroll
        for (int o = 16; o; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        if (!(mx <= 3.0e38f)) mx = 0.f;  // a row holding NaN or infinity is outside the contract: keep the scale finite
        // a = 2^(7 - exponent of mx), its biased exponent clamped to the normal range; 1 for an all-zero row
        int ae = 127 + 7 + 127 - (int)((__float_as_uint(mx) >> 23) & 0xffu);
        ae = mx > 0.f ? (ae > 254 ? 254 : ae) : 127;
        const float a = __uint_as_float((uint32_t)ae << 23), inv_a = __uint_as_float((uint32_t)(254 - ae) << 23);
        const uint32_t h01 = pack_e4m3x2(x[0] * a, x[1] * a), h23 = pack_e4m3x2(x[2] * a, x[3] * a);
        const uint32_t f01 = e4m3x2_to_f16x2<kSelB0B1>(h01), f23 = e4m3x2_to_f16x2<kSelB0B1>(h23);  // values / 256
        const uint32_t l01 = pack_e4m3x2((x[0] * a - f16_lo(f01) * kE4m3WidenFactor) * 16.f,
                                         (x[1] * a - f16_hi(f01) * kE4m3WidenFactor) * 16.f);
        const uint32_t l23 = pack_e4m3x2((x[2] * a - f16_lo(f23) * kE4m3WidenFactor) * 16.f,
                                         (x[3] * a - f16_hi(f23) * kE4m3WidenFactor) * 16.f);
        const uint32_t off = (uint32_t)hr * 128 + ((((uint32_t)lane >> 2) ^ ((uint32_t)hr & 7)) << 4) + ((uint32_t)lane & 3) * 4;
        *reinterpret_cast<uint32_t*>(qd + off) = h01 | (h23 << 16);
        *reinterpret_cast<uint32_t*>(qd + L::kHeads * 128 + off) = l01 | (l23 << 16);
        if (lane == hr) my_inva = inv_a;
      }
      if (first) fence_proxy_async_smem();  // the tile is read by the MMAs through the async proxy
      // the row scales travel with the stage's score buffer (the consumer warps may be several stages, and items,
      // behind this warp): written and fenced before the MMAs whose completion the consumers wait for are issued
      if (lane < L::kHeads) reinterpret_cast<float*>(gen + (s_inva - base))[sbuf * L::kHeads + lane] = my_inva;
      __threadfence_block();
      __syncwarp();
      if (lane == 0) {
        const uint32_t kst = s_stage + slot * L::kTileBytes, qst = s_qs + qb * L::kQSplitBytes;
#pragma unroll
        for (int k = 0; k < D / 32; ++k)  // 32 contraction bytes per MMA
          umma_f8_ss(tmem + sbuf * L::kTcSColumns, umma_smem_desc(kst + k * 32, 0, 1024),
                     umma_smem_desc(qst + k * 32, 0, 1024), idesc, k ? 1u : 0u);
        umma_commit(s_sready + 8 * sbuf);
        umma_commit(s_kempty + 8 * slot);  // the K tile (and the query rows beside it) may be refilled
        if (last) umma_commit(s_qfree + 8 * qb);
      }
      __syncwarp();
      issued = true;
    }
    if (issued) {  // the tensor memory must not be released under MMAs in flight
      if (lane == 0) umma_commit(s_drain);
      __syncwarp();
      int dummy = 0;
      mbar_wait_bounded(s_drain, 0u, &dummy, kWaitLimitNs / 8);
    }
    return tmem;
  }

  if (VP && warp == kVProducerWarp) {
    // ================================================================= V producer warp
    // With blocks of 16 tokens a stage is 4 to 8 K boxes and as many V boxes of 2 to 4 KiB; one warp issuing every
    // copy of every stage does not keep up with HBM, so the producer below posts each stage's V boxes here.
    if (lane == 0) prefetch_tmap(&tm_v);
    const uint32_t vbox_bytes = (uint32_t)p.tile_rows * D * (KV8 ? 1 : 2);
    int it = 0;
    bool ok = true;
    for (;; ++it) {
      const int slot = it % nst;
      if (!warp_wait(s_vdfull + 8 * slot, (uint32_t)(it / nst) & 1u, s_abort)) {
        ok = false;
        break;
      }
      const VStageDesc& vd = g_vdesc[slot];
      const int nbox = vd.nbox;
      const uint32_t full = s_full + 8 * slot;
      if (nbox < 0) {  // end marker (KVM 2: the consumer warps see it through the V ring's barrier, arrived on here)
        if (KVTC && lane == 0) mbar_arrive(full);
        break;
      }
      // (bf16: the producer has armed the stage's barrier for the K, V and q bytes together)
      if (KVTC && lane == 0) mbar_arrive_expect_tx(full, (uint32_t)nbox * vbox_bytes);
      __syncwarp();
      if (lane < nbox && lane < 8) {
        const uint32_t dv = (KVTC ? s_vring + (uint32_t)slot * L::kTileBytes
                                  : s_stage + (uint32_t)slot * L::kStageBytes + L::kTileBytes) + lane * vbox_bytes;
        const int c_tok = vd.c_tok[lane], h = vd.h, blk = vd.blk[lane];
        if (KV8) {
          tma_load_4d(dv, &tm_v, full, 0, c_tok, h, blk);
        } else if (D == 128 && !p.split_halves) {
          tma_load_5d(dv, &tm_v, full, 0, c_tok, 0, h, blk);
        } else {
#pragma unroll
          for (int j = 0; j < D / 64; ++j) tma_load_4d(dv + j * (vbox_bytes / (D / 64)), &tm_v, full, 64 * j, c_tok, h, blk);
        }
      }
    }
    if (!ok) {  // stop path: wait (bounded) until every V copy already issued has landed
      if (lane == 0) atomicOr(&p.hdr->status, kStatusWaitTimeout);
      int dummy_abort = 0;
      for (int k = 0; k < (it < nst ? it : nst); ++k) {
        const int j = it - 1 - k;
        mbar_wait_bounded(s_full + 8 * (j % nst), (uint32_t)(j / nst) & 1u, &dummy_abort, kWaitLimitNs / 8);
      }
    }
    return tmem;
  }

  if (warp == NCW) {
    // ================================================================= producer warp
    if (lane == 0) {
      prefetch_tmap(&tm_k);
      if (!VP) prefetch_tmap(&tm_v);
    }
    const int boxes_per_stage = kStageTok / p.tile_rows;
    const uint32_t box_bytes = (uint32_t)p.tile_rows * D * (KV8 ? 1 : 2);
    int it = 0;
    int item = blockIdx.x;
    int4 d = make_int4(0, 0, 0, 0);
    int blk_cur = 0;
    int T_cur = 0;  // context length of the item's sequence (only read when there are several query tokens)
    const long long cap_tokens = (long long)p.MB * p.bs;
    auto seq_len = [&](int b) {
      const long long T = p.context_lens[b];
      return (int)(T < 0 ? 0 : (T > cap_tokens ? cap_tokens : T));
    };
    // checked build: an item whose fields are out of range is never dereferenced; a table entry outside
    // the pool is recorded and replaced by an id beyond the tensor map (the copy then delivers zeros)
    auto item_ok = [&](const int4& x) {
      return checked(chk_item(x.x, x.y, x.z, x.w, p.B, p.max_items, cap_tokens), &p.hdr->status, kStatusBadItem);
    };
    auto table_entry = [&](const int32_t* e) {
      const int v = *e;
      return checked(chk_table_entry(v, p.NB), &p.hdr->status, kStatusBadTableEntry) ? v : p.NB;
    };
    bool violated = false;
    if (item < n_items) {
      d = p.items[item];
      if (item_ok(d)) {
        const int tb = d.z + lane * p.tile_rows;
        if (lane < boxes_per_stage && tb < d.w) blk_cur = table_entry(p.block_table + (size_t)d.x * p.MB + tb / p.bs);
        if (p.Sq > 1) T_cur = seq_len(d.x);
      }
    }
    bool ok = true;
    while (item < n_items && ok) {
      if (kChecked && !item_ok(d)) {  // stop the CTA: the consumers leave through the abort flag
        *s_abort = 1;
        violated = true;
        ok = false;
        break;
      }
      int nxt = 0;
      if (lane == 0) nxt = atomicAdd(&p.hdr->next_item, 1);
      int4 nd = make_int4(0, 0, 0, 0);
      int blk_nxt_item = 0, T_nxt = 0;
      const int b = d.x, slot_id = d.y, h = d.y % p.Hkv, t0 = d.z, t1 = d.w;
      const int nstage_item = (t1 - t0 + kStageTok - 1) / kStageTok;
      const int32_t* row = p.block_table + (size_t)b * p.MB;
      for (int s = 0; s < nstage_item; ++s, ++it) {
        const int tok0 = t0 + s * kStageTok;
        const int ntok = min(kStageTok, t1 - tok0);
        const int nbox = (ntok + p.tile_rows - 1) / p.tile_rows;
        // table entries of the following stage, one stage ahead of their use
        int blk_n = 0;
        {
          const int tb = tok0 + kStageTok + lane * p.tile_rows;
          if (s + 1 < nstage_item && lane < boxes_per_stage && tb < t1) blk_n = table_entry(row + tb / p.bs);
        }
        const int slot = it % nst;
        const uint32_t ph = (uint32_t)(it / nst) & 1u;
        const int kslot = KVTC ? it % kNK : slot;  // KVM 2: the K tile and the query rows go to the K ring
        if (!warp_wait(s_empty + 8 * slot, ph ^ 1u, s_abort) ||
            (KVTC && !warp_wait(s_kempty + 8 * kslot, (((uint32_t)it / kNK) & 1u) ^ 1u, s_abort))) {
          ok = false;
          break;
        }
        const uint32_t full = s_full + 8 * slot;
        const uint32_t kfull = KVTC ? s_kfull + 8 * kslot : full;
        if (lane == 0) {
          const int flags = (s == 0 ? 1 : 0) | (s == nstage_item - 1 ? 2 : 0);
          // rows of this stage the first query token may see, biased by 16 and clipped to 10 bits
          // (one query token: everything)
          int cm = 1023;
          if (p.Sq > 1) {
            const long long lim0 = (long long)T_cur - p.Sq + 1 - tok0 + 16;
            cm = lim0 < 0 ? 0 : (lim0 > 1023 ? 1023 : (int)lim0);
          }
          const int4 meta = make_int4(slot_id, b, h, ntok | (flags << 16) | (cm << 18));
          g_meta[slot] = meta;
          const uint32_t qbytes = s == 0 ? (uint32_t)p.GQ * D * 2 : 0u;
          if (KVTC) {  // (the V producer warp arms the stage's own barrier)
            g_kmeta[kslot] = meta;
            mbar_arrive_expect_tx(kfull, nbox * box_bytes + qbytes);
            g_vdesc[slot].nbox = nbox;
            g_vdesc[slot].h = h;
          } else {
            mbar_arrive_expect_tx(full, 2u * nbox * box_bytes + qbytes);
            if (VP) {
              g_vdesc[slot].nbox = nbox;
              g_vdesc[slot].h = h;
            }
          }
        }
        __syncwarp();
        bool span_ok = true;  // checked build: every copy lands inside its stage (and the q rows inside their slot)
        if (lane < nbox) {
          const int tb = tok0 + lane * p.tile_rows;
          const int c_tok = tb % p.bs;
          const uint32_t k0 = KVTC ? s_stage + (uint32_t)kslot * L::kTileBytes : s_stage + (uint32_t)slot * L::kStageBytes;
          const uint32_t v0 = KVTC ? s_vring + (uint32_t)slot * L::kTileBytes : k0 + L::kTileBytes;
          const uint32_t dk = k0 + lane * box_bytes, dv = v0 + lane * box_bytes;
          span_ok = checked(chk_span(dk, box_bytes, k0, (long long)k0 + L::kTileBytes) &&
                                chk_span(dv, box_bytes, v0, (long long)v0 + L::kTileBytes) && chk_span(slot, 1, 0, nst) &&
                                chk_span(kslot, 1, 0, KVTC ? kNK : nst),
                            &p.hdr->status, kStatusBadSmem);
          if (!span_ok) {
            // skipped
          } else if (KVTC) {  // the K box here, the V box through the V producer warp
            tma_load_4d(dk, &tm_k, kfull, 0, c_tok, h, blk_cur);
            g_vdesc[slot].blk[lane & 7] = blk_cur;
            g_vdesc[slot].c_tok[lane & 7] = c_tok;
          } else if (KV8) {  // a token row is one 128-byte swizzle row: one 4-d copy per box
            tma_load_4d(dk, &tm_k, kfull, 0, c_tok, h, blk_cur);
            tma_load_4d(dv, &tm_v, full, 0, c_tok, h, blk_cur);
          } else if (D == 128 && !p.split_halves) {
            tma_load_5d(dk, &tm_k, full, 0, c_tok, 0, h, blk_cur);
            if (!VP) tma_load_5d(dv, &tm_v, full, 0, c_tok, 0, h, blk_cur);
          } else {
#pragma unroll
            for (int j = 0; j < D / 64; ++j) {
              tma_load_4d(dk + j * (box_bytes / (D / 64)), &tm_k, full, 64 * j, c_tok, h, blk_cur);
              if (!VP) tma_load_4d(dv + j * (box_bytes / (D / 64)), &tm_v, full, 64 * j, c_tok, h, blk_cur);
            }
          }
          if (VP && !KVTC && span_ok) {  // the V box goes through the V producer warp
            g_vdesc[slot].blk[lane & 7] = blk_cur;
            g_vdesc[slot].c_tok[lane & 7] = c_tok;
          }
        }
        if (s == 0 && lane < p.Sq) {  // one run of G heads per query token, side by side: [query][head][D]
          const uint32_t dq = s_q + (uint32_t)kslot * qslot + (uint32_t)lane * p.G * D * 2;
          if (checked(chk_span(dq, (long long)p.G * D * 2, s_q + (long long)kslot * qslot, s_q + (long long)(kslot + 1) * qslot),
                      &p.hdr->status, kStatusBadSmem))
            bulk_g2s(dq, p.q + (((size_t)b * p.Sq + lane) * p.Hq + (size_t)h * p.G) * D, (uint32_t)p.G * D * 2, kfull);
          else
            span_ok = false;
        }
        if (kChecked && !__all_sync(0xffffffffu, span_ok)) {  // a skipped copy leaves the stage incomplete: stop
          *s_abort = 1;
          violated = true;
          ok = false;
          break;
        }
        if (VP) {  // hand the stage's V boxes to the V producer warp
          __syncwarp();
          if (lane == 0) mbar_arrive(s_vdfull + 8 * slot);
        }
        // look ahead to the next item: its descriptor, then its first table entries
        if (s == 0) {
          nxt = __shfl_sync(0xffffffffu, nxt, 0);
          if (nxt < n_items) nd = p.items[nxt];
        }
        if (s == (nstage_item > 1 ? 1 : 0) && nxt < n_items && (!kChecked || item_ok(nd))) {
          const int tb = nd.z + lane * p.tile_rows;
          if (lane < boxes_per_stage && tb < nd.w) blk_nxt_item = table_entry(p.block_table + (size_t)nd.x * p.MB + tb / p.bs);
          if (p.Sq > 1) T_nxt = seq_len(nd.x);
        }
        blk_cur = blk_n;
      }
      if (nstage_item <= 0) nxt = __shfl_sync(0xffffffffu, nxt, 0);  // (items are never empty)
      item = nxt;
      d = nd;
      blk_cur = blk_nxt_item;
      T_cur = T_nxt;
    }
    // end marker (one stage, seen by every consumer warp)
    if (ok) {
      const int slot = it % nst, kslot = it % kNK;
      const uint32_t ph = (uint32_t)(it / nst) & 1u;
      if (warp_wait(s_empty + 8 * slot, ph ^ 1u, s_abort) &&
          (!KVTC || warp_wait(s_kempty + 8 * kslot, (((uint32_t)it / kNK) & 1u) ^ 1u, s_abort))) {
        if (lane == 0) {
          g_meta[slot] = make_int4(-1, 0, 0, 0);
          if (KVTC) {  // the consumers' marker travels through the V producer warp, which stops on it too
            g_vdesc[slot].nbox = -1;
            mbar_arrive(s_vdfull + 8 * slot);
            g_kmeta[kslot] = make_int4(-1, 0, 0, 0);
            mbar_arrive(s_kfull + 8 * kslot);
          } else {
            mbar_arrive(s_full + 8 * slot);
            if (VP) {  // the V producer warp stops on the marker too
              g_vdesc[slot].nbox = -1;
              mbar_arrive(s_vdfull + 8 * slot);
            }
          }
        }
        ++it;
      } else {
        ok = false;
      }
    }
    if (!ok) {
      // stop path: record it, then wait (bounded) until every copy already issued has landed
      if (lane == 0 && !violated) atomicOr(&p.hdr->status, kStatusWaitTimeout);
      int dummy_abort = 0;
      const int pending = KVTC ? 0 : (it < nst ? it : nst);  // (KVM 2: the V producer warp drains the V ring)
      for (int k = 0; k < pending; ++k) {
        const int j = it - 1 - k;
        mbar_wait_bounded(s_full + 8 * (j % nst), (uint32_t)(j / nst) & 1u, &dummy_abort, kWaitLimitNs / 8);
      }
      for (int k = 0; KVTC && k < (it < kNK ? it : kNK); ++k) {
        const int j = it - 1 - k;
        mbar_wait_bounded(s_kfull + 8 * (j % kNK), (uint32_t)(j / kNK) & 1u, &dummy_abort, kWaitLimitNs / 8);
      }
    }
    return tmem;
  }

  // =================================================================== consumer warps
  const int g = lane >> 2, t = lane & 3;
  float m_run[NT][2], l_run[NT][2];
  float o_acc[NT][KS][4];
  uint32_t qf[NT][KS][2];
#pragma unroll
  for (int nt = 0; nt < NT; ++nt) {
    m_run[nt][0] = m_run[nt][1] = -INFINITY;
    l_run[nt][0] = l_run[nt][1] = 0.f;
#pragma unroll
    for (int k = 0; k < KS; ++k) {
      o_acc[nt][k][0] = o_acc[nt][k][1] = o_acc[nt][k][2] = o_acc[nt][k][3] = 0.f;
      qf[nt][k][0] = qf[nt][k][1] = 0u;
    }
  }
  // Per-lane byte offsets of the ldmatrix rows inside a stage's K / V tile.  A box holds
  // [D/64 halves][tile_rows][64 dims] with the 128-byte swizzle (16-byte chunk ^= row & 7).
  // first token row of this warp inside a stage (KVM 2: a warp reads tensor memory in its own lane quarter only)
  const int r0 = KVTC ? 32 * (warp & 3) + 16 * (warp >> 2) : 16 * TPW * warp;
  const uint32_t box_bytes = (uint32_t)p.tile_rows * D * (KV8 ? 1 : 2);
  const uint32_t half_bytes = (uint32_t)p.tile_rows * 128;
  const int lr_k = (lane & 7) + ((lane >> 3) & 1) * 8, cs_k = lane >> 4;
  // 8-bit tiles are read with the K pattern for V too (matrices: tokens 0-7 / 8-15 of chunk c, then c + 1)
  const int lr_v = KV8 ? lr_k : (lane & 7) + (lane >> 4) * 8, cs_v = KV8 ? cs_k : (lane >> 3) & 1;
  uint32_t tile_k[TPW], tile_v[TPW], kpat[KS], vpat[KS];
#pragma unroll
  for (int u = 0; u < TPW; ++u) {
    const int r = r0 + 16 * u;
    const uint32_t bo = (uint32_t)(r / p.tile_rows) * box_bytes;
    tile_k[u] = bo + (uint32_t)(r % p.tile_rows + lr_k) * 128;
    tile_v[u] = bo + (uint32_t)(r % p.tile_rows + lr_v) * 128;
  }
#pragma unroll
  for (int k = 0; k < KS; ++k) {
    const int ck = 2 * k + cs_k, cv = 2 * k + cs_v;
    kpat[k] = (uint32_t)(ck >> 3) * half_bytes + (uint32_t)(((ck & 7) ^ (lr_k & 7)) << 4);
    vpat[k] = (uint32_t)(cv >> 3) * half_bytes + (uint32_t)(((cv & 7) ^ (lr_v & 7)) << 4);
  }
  int qi_col[NT][2];  // query token of this lane's score columns 8 nt + 2t, + 1 (column = query * G + head)
#pragma unroll
  for (int nt = 0; nt < NT; ++nt) {
    qi_col[nt][0] = p.Sq > 1 ? (8 * nt + 2 * t) / p.G : 0;
    qi_col[nt][1] = p.Sq > 1 ? (8 * nt + 2 * t + 1) / p.G : 0;
  }
  uint32_t mphase = 0;  // parity of the next merge-barrier phase to wait for
  bool merge_pending_read = false;

  int slot = -1;
  uint32_t full_phase = 1u;  // slot / phase of stage `it` without dividing by the runtime stage count
  for (int it = 0;; ++it) {
    if (++slot == nst) slot = 0;
    if (slot == 0) full_phase ^= 1u;
    if (!warp_wait(s_full + 8 * slot, full_phase, s_abort)) {
      if (lane == 0) atomicOr(&p.hdr->status, kStatusWaitTimeout);
      return tmem;
    }
    const int4 meta = g_meta[slot];
    if (meta.x < 0) break;
    const int ntok = meta.w & 0xffff;
    const bool first = (meta.w >> 16) & 1, last = (meta.w >> 17) & 1;
    if (first) {
      const uint8_t* qs = g_q + (size_t)slot * qslot;
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
        const int head = 8 * nt + g;
        m_run[nt][0] = m_run[nt][1] = -INFINITY;
        l_run[nt][0] = l_run[nt][1] = 0.f;
#pragma unroll
        for (int k = 0; k < KS; ++k) {
          o_acc[nt][k][0] = o_acc[nt][k][1] = o_acc[nt][k][2] = o_acc[nt][k][3] = 0.f;
          uint32_t v0 = 0u, v1 = 0u;
          if (!KVTC && head < p.GQ) {
            if (KV8) {  // dims 16k + 4t .. + 3 as two f16 pairs (the k order of the 8-bit score MMA)
              const uint2 w = *reinterpret_cast<const uint2*>(qs + ((size_t)head * D + 16 * k + 4 * t) * 2);
              v0 = pack_f16x2(__uint_as_float(w.x << 16), __uint_as_float(w.x & 0xffff0000u));
              v1 = pack_f16x2(__uint_as_float(w.y << 16), __uint_as_float(w.y & 0xffff0000u));
            } else {
              const uint8_t* src = qs + ((size_t)head * D + 16 * k + 2 * t) * 2;
              v0 = *reinterpret_cast<const uint32_t*>(src);
              v1 = *reinterpret_cast<const uint32_t*>(src + 16);
            }
          }
          qf[nt][k][0] = v0;
          qf[nt][k][1] = v1;
        }
      }
    }
    const int valid = ntok - r0;  // this warp's rows [0, valid) of 16 * TPW hold tokens of the chunk
    if (valid > 0) {
      const uint32_t kst = s_stage + (uint32_t)slot * L::kStageBytes;  // (not read with KVM 2)
      const uint32_t vst = KVTC ? s_vring + (uint32_t)slot * L::kTileBytes : kst + L::kTileBytes;
      // rows of this warp the first query token may see; with one query token that is all of them
      const int lim_w = ((meta.w >> 18) & 1023) - 16 - r0;
      if (KVTC) {
        // this warp's 16 x (2 * heads) tile of the stage's scores, in the accumulator layout of mma.sync
        const uint32_t sbuf = (uint32_t)it % kNS;
        if (!warp_wait(s_sready + 8 * sbuf, ((uint32_t)it / kNS) & 1u, s_abort)) {
          if (lane == 0) atomicOr(&p.hdr->status, kStatusWaitTimeout);
          return tmem;
        }
        tc_fence_after_sync();
        uint32_t f[8 * NT];
        tmem_ld_frag(tmem + ((uint32_t)r0 << 16) + sbuf * L::kTcSColumns, f);
        tmem_ld_wait();
        const float* inva = reinterpret_cast<const float*>(gen + (s_inva - base)) + sbuf * L::kHeads;
        float sv[NT][4];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
          const float2 ia = *reinterpret_cast<const float2*>(inva + 8 * nt + 2 * t);
          const float m0 = ia.x * p.scale_log2e, m1 = ia.y * p.scale_log2e;
#pragma unroll
          for (int e = 0; e < 4; ++e)  // high term + low term / 16
            sv[nt][e] = fmaf(__uint_as_float(f[4 * (NT + nt) + e]), 0.0625f, __uint_as_float(f[4 * nt + e])) * ((e & 1) ? m1 : m0);
        }
        if (valid >= 16 && lim_w >= 16)
          kv8_softmax_values<D, NT, false>(vst, tile_k[0], kpat, sv, m_run, l_run, o_acc, valid, g, t, 0, nullptr);
        else
          kv8_softmax_values<D, NT, true>(vst, tile_k[0], kpat, sv, m_run, l_run, o_acc, valid, g, t, lim_w, qi_col);
      } else if (KV8) {
        if (valid >= 16 && lim_w >= 16)
          consume_tile_kv8<D, NT, false>(kst, vst, tile_k[0], kpat, qf, m_run, l_run, o_acc, p.scale_log2e, valid, g, t);
        else
          consume_tile_kv8<D, NT, true>(kst, vst, tile_k[0], kpat, qf, m_run, l_run, o_acc, p.scale_log2e, valid, g, t,
                                        lim_w, qi_col);
      } else {
        if (valid >= 16 * TPW && lim_w >= 16 * TPW)
          consume_tiles<D, NT, TPW, false>(kst, vst, tile_k, tile_v, kpat, vpat, qf, m_run, l_run, o_acc,
                                           p.scale_log2e, valid, g, t);
        else
          consume_tiles<D, NT, TPW, true>(kst, vst, tile_k, tile_v, kpat, vpat, qf, m_run, l_run, o_acc,
                                          p.scale_log2e, valid, g, t, lim_w, qi_col);
      }
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(s_empty + 8 * slot);

    if (last) {
      // ---- combine the NCW warps' running states (64 dims per pass), then write the item's result
      const int item = meta.x, b = meta.y, h = meta.z;
      // checked build: the partial slot and the sequence index address the workspace and `out`
      const bool dst_ok = checked(chk_index(item, p.max_items) && chk_index(b, p.B) && chk_index(h, p.Hkv),
                                  &p.hdr->status, kStatusBadIndex);
      const int n_chunks = dst_ok ? p.seq_first[b + 1] - p.seq_first[b] : 1;
      float* mo = g_merge + (size_t)warp * L::kHeads * L::kOStride;
      float* all_m = g_merge + L::kMergeOBytes / 4;
      float lsum[NT][2];
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
        float l0 = l_run[nt][0], l1 = l_run[nt][1];
#pragma unroll
        for (int o = 4; o < 32; o <<= 1) {
          l0 += __shfl_xor_sync(0xffffffffu, l0, o);
          l1 += __shfl_xor_sync(0xffffffffu, l1, o);
        }
        lsum[nt][0] = l0;
        lsum[nt][1] = l1;
      }
#pragma unroll
      for (int pass = 0; pass < D / 64; ++pass) {
        if (merge_pending_read) {  // earlier readers must be done with the buffer
          if (!warp_wait(s_mbar, mphase, s_abort)) {
            if (lane == 0) atomicOr(&p.hdr->status, kStatusWaitTimeout);
            return tmem;
          }
          mphase ^= 1u;
        }
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
          const int h0 = 8 * nt + 2 * t;
          if (pass == 0 && g == 0) {
            float* mm = all_m + ((size_t)warp * L::kHeads + h0) * 2;
            mm[0] = m_run[nt][0];
            mm[1] = lsum[nt][0];
            mm[2] = m_run[nt][1];
            mm[3] = lsum[nt][1];
          }
#pragma unroll
          for (int kk = 0; kk < 4; ++kk) {
            const int k = 4 * pass + kk;
            // accumulator rows g / g + 8 hold dims g / g + 8 of the chunk (bf16) or 2g / 2g + 1 (8-bit)
            const int d_lo = 16 * kk + (KV8 ? 2 * g : g), d_hi = 16 * kk + (KV8 ? 2 * g + 1 : g + 8);
            mo[(size_t)h0 * L::kOStride + d_lo] = o_acc[nt][k][0];
            mo[(size_t)(h0 + 1) * L::kOStride + d_lo] = o_acc[nt][k][1];
            mo[(size_t)h0 * L::kOStride + d_hi] = o_acc[nt][k][2];
            mo[(size_t)(h0 + 1) * L::kOStride + d_hi] = o_acc[nt][k][3];
          }
        }
        mbar_arrive(s_mbar);
        if (!warp_wait(s_mbar, mphase, s_abort)) {
          if (lane == 0) atomicOr(&p.hdr->status, kStatusWaitTimeout);
          return tmem;
        }
        mphase ^= 1u;
        for (int idx = threadIdx.x; idx < p.GQ * 64; idx += NCW * 32) {
          const int col = idx >> 6, dl = idx & 63, dim = 64 * pass + dl;  // column = query * G + head
          float M = -INFINITY;
#pragma unroll
          for (int w = 0; w < NCW; ++w) M = fmaxf(M, all_m[(w * L::kHeads + col) * 2]);
          const float Ms = M == -INFINITY ? 0.f : M;  // a query that saw nothing of this chunk (causal limit)
          float den = 0.f, num = 0.f;
#pragma unroll
          for (int w = 0; w < NCW; ++w) {
            const float sw = ex2(all_m[(w * L::kHeads + col) * 2] - Ms);
            den += sw * all_m[(w * L::kHeads + col) * 2 + 1];
            num += sw * g_merge[((size_t)w * L::kHeads + col) * L::kOStride + dl];
          }
          float o = den > 0.f ? num / den : 0.f;
          if (KV8) o *= p.v_scale;
          if (kChecked && !dst_ok) continue;
          if (n_chunks == 1 && !p.out_f32) {
            const int qi = p.Sq > 1 ? col / p.G : 0, head = col - qi * p.G;
            p.out[(((size_t)b * p.Sq + qi) * p.Hq + (size_t)h * p.G + head) * D + dim] = __float2bfloat16_rn(o);
          } else {
            p.part_o[((size_t)item * p.GQ + col) * D + dim] = o;
            if (dim == 0) p.part_lse[(size_t)item * p.GQ + col] = den > 0.f ? M + lg2(den) : -INFINITY;
          }
        }
        mbar_arrive(s_mbar);
        merge_pending_read = true;
      }
    }
  }
  return tmem;
}

template <int D, int NCW, int NT, int TPW, int KVM = 0>
__global__ void __launch_bounds__(SmemLayout<D, NCW, NT, TPW, KVM>::kWarps * 32, (KVM && NCW == 8 && NT == 1) ? 2 : 1)
decode_main_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                   const DecodeParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t tmem = decode_main_body<D, NCW, NT, TPW, KVM>(tm_k, tm_v, p, smem_raw);
  if (KVM == 2) {  // common exit: release the tensor memory once every warp is done with it
    tc_fence_before_sync();
    __syncthreads();
    if ((threadIdx.x >> 5) == NCW + 1) {
      using L = SmemLayout<D, NCW, NT, TPW, KVM>;
      tmem_dealloc(tmem, L::kTcSBuffers * L::kTcSColumns);
    }
  }
}

// ------------------------------------------------------------------------------------ merge
// LSE merge of the partial results of split sequences.  `wpu` warps (1, 2, 4 or 8, all in one CTA)
// share a (sequence, query token, query head) unit: each takes a contiguous share of the unit's
// chunks, 32 chunks at a time (one lse per lane), lanes own D / 32 consecutive dims,
//   out = sum_c 2^(lse_c - M) o_c / sum_c 2^(lse_c - M),  M = max_c lse_c,
// and the first warp of the unit combines the shares through shared memory.  Units of unsplit
// sequences have nothing to do.  The host picks wpu > 1 when there are too few units to fill the GPU
// (a handful of very long sequences).
template <int D>
__global__ void __launch_bounds__(256) lse_merge_kernel(const DecodeParams p, const int wpu_log2) {
  constexpr int V = D / 32;  // dims per lane
  __shared__ float s_part[8][D + 2];  // per warp: its share's accumulator, running maximum, denominator
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int wpu = 1 << wpu_log2, units_per_block = 8 >> wpu_log2, sub = warp & (wpu - 1);
  const int per_seq = p.Sq * p.Hq;  // (query token, query head) rows of one sequence
  const int n_units = p.B * per_seq;
  // The chunk scan was written by the plan kernel, which had completed before the attention grid
  // (the grid this launch depends on) passed its own dependency wait, so it may be read before
  // the wait below; only the partial results need the attention grid to be complete.
  int first = 0, n = 0;
  grid_dep_launch();  // a programmatically launched successor may start its own prologue
  {
    const int u = blockIdx.x * units_per_block + (warp >> wpu_log2);
    if (u < n_units) {
      first = p.seq_first[u / per_seq];
      n = p.seq_first[u / per_seq + 1] - first;
    }
  }
  // (also on the overflow path: this grid's completion must imply the attention grid's, because the next
  // call's first kernel waits on this grid only before it rewrites the workspace and the cache)
  grid_dep_wait();
  if (p.hdr->status & kStatusPlanOverflow) return;  // no work list, no partials (status is reported)
  for (int ub = blockIdx.x * units_per_block; ub < n_units; ub += gridDim.x * units_per_block, first = -1) {
    const int u = ub + (warp >> wpu_log2);
    const bool live = u < n_units;
    const int b = live ? u / per_seq : 0, rem = live ? u % per_seq : 0;
    const int qi = rem / p.Hq, hq = rem % p.Hq;
    const int h = hq / p.G, head = qi * p.G + hq % p.G;  // `head` = score column of (query, head) in its group
    if (live && first < 0) {
      first = p.seq_first[b];
      n = p.seq_first[b + 1] - first;
    }
    // unsplit (or empty) sequence: the attention kernel wrote the row itself -- except with fp32 output, where
    // every row is a partial (an unsplit row passes through unchanged: one chunk of weight 1)
    bool work = live && (n > 1 || (p.out_f32 && n == 1));
    if (work && !checked(chk_index((long long)(first + n) * p.Hkv - 1, p.max_items) && first >= 0, &p.hdr->status,
                         kStatusBadIndex))
      work = false;
    float M = -INFINITY, den = 0.f, acc[V];
#pragma unroll
    for (int i = 0; i < V; ++i) acc[i] = 0.f;
    if (work) {
      const int c_lo = (int)(((long long)n * sub) >> wpu_log2), c_hi = (int)(((long long)n * (sub + 1)) >> wpu_log2);
      for (int c0 = c_lo; c0 < c_hi; c0 += 32) {
        const int cnt = min(32, c_hi - c0);
        float lse = -INFINITY;
        if (lane < cnt) lse = p.part_lse[((size_t)(first + c0 + lane) * p.Hkv + h) * p.GQ + head];
        float gm = lse;
#pragma unroll
        for (int o = 16; o; o >>= 1) gm = fmaxf(gm, __shfl_xor_sync(0xffffffffu, gm, o));
        const float Mn = fmaxf(M, gm);
        const float Ms = Mn == -INFINITY ? 0.f : Mn;  // nothing seen so far (causal limit): keep exponents finite
        const float resc = exp2f(M - Ms);
        M = Mn;
        const float w_lane = exp2f(lse - Ms);  // 0 for lanes beyond cnt
        float ws = w_lane;
#pragma unroll
        for (int o = 16; o; o >>= 1) ws += __shfl_xor_sync(0xffffffffu, ws, o);
        den = den * resc + ws;
#pragma unroll
        for (int i = 0; i < V; ++i) acc[i] *= resc;
        const float* src = p.part_o + (((size_t)(first + c0) * p.Hkv + h) * p.GQ + head) * D + lane * V;
        const size_t cstride = (size_t)p.Hkv * p.GQ * D;
#pragma unroll 8
        for (int j = 0; j < cnt; ++j) {
          const float w = __shfl_sync(0xffffffffu, w_lane, j);
          if (V == 4) {
            const float4 o = *reinterpret_cast<const float4*>(src + j * cstride);
            acc[0] += w * o.x; acc[1] += w * o.y; acc[2] += w * o.z; acc[V - 1] += w * o.w;
          } else {
            const float2 o = *reinterpret_cast<const float2*>(src + j * cstride);
            acc[0] += w * o.x; acc[V - 1] += w * o.y;
          }
        }
      }
    }
    if (wpu > 1) {  // the unit's first warp folds in the other shares (block-uniform control flow)
      if (sub != 0) {
#pragma unroll
        for (int i = 0; i < V; ++i) s_part[warp][lane * V + i] = acc[i];
        if (lane == 0) {
          s_part[warp][D] = M;
          s_part[warp][D + 1] = den;
        }
      }
      __syncthreads();
      if (work && sub == 0) {
        for (int w = 1; w < wpu; ++w) {
          const float Mw = s_part[warp + w][D], dw = s_part[warp + w][D + 1];
          const float Mn = fmaxf(M, Mw);
          const float Ms = Mn == -INFINITY ? 0.f : Mn;
          const float ra = exp2f(M - Ms), rb = exp2f(Mw - Ms);
          M = Mn;
          den = den * ra + dw * rb;
#pragma unroll
          for (int i = 0; i < V; ++i) acc[i] = acc[i] * ra + s_part[warp + w][lane * V + i] * rb;
        }
      }
      __syncthreads();  // the shares are consumed before the next round overwrites them
    }
    if (work && sub == 0) {
      const size_t at = (((size_t)b * p.Sq + qi) * p.Hq + hq) * D + lane * V;
      const float inv = den > 0.f ? 1.f / den : 0.f;  // den = 0: the query saw no token at all
      if (p.out_f32) {
#pragma unroll
        for (int i = 0; i < V; ++i) reinterpret_cast<float*>(p.out)[at + i] = acc[i] * inv;
      } else {
#pragma unroll
        for (int i = 0; i < V; i += 2)
          *reinterpret_cast<__nv_bfloat162*>(p.out + at + i) = __floats2bfloat162_rn(acc[i] * inv, acc[i + 1] * inv);
      }
    }
  }
}

}  // namespace ooco
