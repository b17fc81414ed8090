// Host side of the ooco_* C ABI: argument validation, tensor-map encoding, launches.
#include <cuda.h>
#include <cuda_runtime.h>

#include <atomic>
#include <chrono>
#include <cstdint>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <utility>
#include <vector>

#include "../../include/ooco.h"
#include "block_copy_kernels.cuh"
#include "chunk_kernels.cuh"
#include "chunk_tc_kernels.cuh"
#include "chunk_tc2_kernels.cuh"
#include "decode_kernels.cuh"

namespace ooco {

// ------------------------------------------------------------------------------------ tuning
// Launch-shape knobs (benchmark sweeps); defaults are the tuned configuration.
enum Knob { kKnobWarps = 0, kKnobStages, kKnobCtasPerSm, kKnobChunkMin, kKnobChunkMax, kKnobItemsPerCta,
            kKnobSplitHalves, kKnobTilesPerWarp, kKnobPdl, kKnobCopyCtasPerSm, kKnobHostStageKernel, kKnobRowLayout16, kKnobChunkTcgen05, kKnobOutF32, kKnobKv8Tcgen05, kKnobChunkTwoTiles, kKnobCount };
static std::atomic<int> g_knobs[kKnobCount] = {{4}, {0}, {2}, {256}, {8192}, {6}, {0}, {1}, {1}, {1}, {1}, {1}, {1}, {0}, {1}, {2}};
static std::atomic<int> g_overridden[kKnobCount];  // knob set through ooco_set_tuning
constexpr int kGridCap = 592;  // 148 SMs x 4 CTAs: most CTAs any launch shape uses (host-only workspace bound)

static thread_local int tl_last_launches = 0;
static thread_local bool tl_events_between_kernels = false;  // profiling: no programmatic overlap
static thread_local char tl_detail[160] = "";
static thread_local int64_t tl_host_ns[2] = {0, 0};  // last host-buffer step: host work before the wait, the wait

// Remembers where a CUDA-side failure happened (read back through ooco_last_error_detail).
static int fail_cuda(const char* where, long code) {
  snprintf(tl_detail, sizeof tl_detail, "%s failed with code %ld", where, code);
  return OOCO_E_CUDA;
}

// Optional per-call kernel timing (benchmarks): 4 events per ooco_decode_attention call.
struct Profiler {
  std::mutex mu;
  std::vector<cudaEvent_t> ev;  // 4 per record: before plan, before attention, after attention, after merge
  int capacity = 0, used = 0;
};
static Profiler g_prof;
static std::atomic<int> g_prof_on{0};

struct DeviceInfo {
  int sm_count = 0;
  int smem_optin = 0;
};
static DeviceInfo device_info(int dev) {
  static DeviceInfo cache[64];
  static std::atomic<int> ready[64];
  if (dev >= 0 && dev < 64 && ready[dev].load(std::memory_order_acquire)) return cache[dev];
  DeviceInfo d;
  cudaDeviceGetAttribute(&d.sm_count, cudaDevAttrMultiProcessorCount, dev);
  cudaDeviceGetAttribute(&d.smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
  if (dev >= 0 && dev < 64) {
    cache[dev] = d;
    ready[dev].store(1, std::memory_order_release);
  }
  return d;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);
static EncodeTiledFn encode_fn() {
  static std::atomic<EncodeTiledFn> fn{nullptr};
  EncodeTiledFn f = fn.load(std::memory_order_acquire);
  if (f) return f;
  void* ptr = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) != cudaSuccess ||
      qres != cudaDriverEntryPointSuccess || !ptr)
    return nullptr;
  f = reinterpret_cast<EncodeTiledFn>(ptr);
  fn.store(f, std::memory_order_release);
  return f;
}

static bool supported_block(int bs) { return bs == 16 || bs == 32 || bs == 64 || bs == 128 || bs == 256; }

static int validate_shape(const ooco_shape_t* s) {
  if (!s) return OOCO_E_NULLPTR;
  if (s->batch <= 0 || s->num_q_heads <= 0 || s->num_kv_heads <= 0 || s->head_dim <= 0 ||
      s->block_size <= 0 || s->num_blocks <= 0 || s->max_blocks_per_seq <= 0 || s->reserved != 0)
    return OOCO_E_SHAPE;
  if (s->num_q_heads % s->num_kv_heads) return OOCO_E_SHAPE;
  if (s->kv_block_stride <= 0 || s->kv_head_stride <= 0 || s->kv_token_stride < s->head_dim)
    return OOCO_E_SHAPE;
  if (s->head_dim != 64 && s->head_dim != 128) return OOCO_E_UNSUPPORTED;
  if (!supported_block(s->block_size)) return OOCO_E_UNSUPPORTED;
  if (s->num_q_heads / s->num_kv_heads > 16) return OOCO_E_UNSUPPORTED;
  if ((s->kv_block_stride | s->kv_head_stride | s->kv_token_stride) & 7) return OOCO_E_UNSUPPORTED;
  if ((int64_t)s->max_blocks_per_seq * s->block_size > (int64_t)1 << 30) return OOCO_E_UNSUPPORTED;
  return OOCO_OK;
}

// More than 16 score columns per (sequence, kv head) go to the prefill-chunk kernel; consumer warps of
// its CTA (16 columns each) for a given number of columns.
constexpr int kDecodeMaxColumns = 16;
constexpr int kMaxQLen = 8192;
static int chunk_warps(int columns) { return columns <= 32 ? 2 : (columns <= 64 ? 4 : 8); }
static int chunk_row_tiles(int columns) { return (columns + 16 * chunk_warps(columns) - 1) / (16 * chunk_warps(columns)); }

// Work items the plan aims at per CTA: many short ones balance the HBM-bound decode kernels; the chunk
// kernels pay a query load, an epilogue and a partial row per score column for every item, and want few.
static int plan_items_per_cta(int columns) {
  if (columns > kDecodeMaxColumns && !g_overridden[kKnobItemsPerCta].load()) return 2;
  return g_knobs[kKnobItemsPerCta].load();
}

// Workspace carve-up (all offsets multiples of 256 bytes).
struct WsLayout {
  size_t off_first, off_items, off_lse, off_o, total;
  int max_items;
};
static WsLayout ws_layout(const ooco_shape_t* s, int q_len = 1) {
  const int G = s->num_q_heads / s->num_kv_heads * q_len;  // score columns per (sequence, kv head)
  const int64_t cmax = g_knobs[kKnobChunkMax].load();
  const int64_t ipc = plan_items_per_cta(G);
  const int64_t per_seq = ((int64_t)s->max_blocks_per_seq * s->block_size + cmax - 1) / cmax;
  int64_t extra = (int64_t)s->num_kv_heads * s->batch * per_seq;
  // the plan cuts the sequences into about (CTAs it sizes for) x ipc items; the chunk path sizes for the
  // CTAs divided by the row tiles of an item, since every item is worked on once per row tile
  const int64_t sized_ctas = G > kDecodeMaxColumns ? (kGridCap + chunk_row_tiles(G) - 1) / chunk_row_tiles(G) : kGridCap;
  if (extra < sized_ctas * ipc) extra = sized_ctas * ipc;
  // (the bound needs no slack; a partial row per score column makes chunk-path items large, so theirs is small)
  const int64_t max_items = (int64_t)s->num_kv_heads * s->batch + extra + (G > kDecodeMaxColumns ? 8 : 64);
  auto up = [](size_t x) { return (x + 255) & ~(size_t)255; };
  WsLayout w;
  w.max_items = (int)(max_items > INT32_MAX ? INT32_MAX : max_items);
  w.off_first = 256;
  w.off_items = w.off_first + up(((size_t)s->batch + 1) * 4);
  w.off_lse = w.off_items + up((size_t)w.max_items * 16);
  w.off_o = w.off_lse + up((size_t)w.max_items * G * 4);
  w.total = w.off_o + up((size_t)w.max_items * G * s->head_dim * 4);
  return w;
}

static int encode_kv_map(CUtensorMap* tm, const ooco_shape_t* s, const void* base, int tile_rows,
                         bool five_d) {
  EncodeTiledFn enc = encode_fn();
  if (!enc) return fail_cuda("cudaGetDriverEntryPoint(cuTensorMapEncodeTiled)", -1);
  const cuuint64_t es = 2;
  CUresult r;
  if (five_d) {  // (64 dims, token, half, head, block): one box = [2][tile_rows][64]
    cuuint64_t dims[5] = {64, (cuuint64_t)s->block_size, (cuuint64_t)s->head_dim / 64,
                          (cuuint64_t)s->num_kv_heads, (cuuint64_t)s->num_blocks};
    cuuint64_t strides[4] = {(cuuint64_t)s->kv_token_stride * es, 64 * es, (cuuint64_t)s->kv_head_stride * es,
                             (cuuint64_t)s->kv_block_stride * es};
    cuuint32_t box[5] = {64, (cuuint32_t)tile_rows, (cuuint32_t)s->head_dim / 64, 1, 1};
    cuuint32_t estr[5] = {1, 1, 1, 1, 1};
    r = enc(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  } else {  // (dims, token, head, block): one box = [tile_rows][64]
    cuuint64_t dims[4] = {(cuuint64_t)s->head_dim, (cuuint64_t)s->block_size, (cuuint64_t)s->num_kv_heads,
                          (cuuint64_t)s->num_blocks};
    cuuint64_t strides[3] = {(cuuint64_t)s->kv_token_stride * es, (cuuint64_t)s->kv_head_stride * es,
                             (cuuint64_t)s->kv_block_stride * es};
    cuuint32_t box[4] = {64, (cuuint32_t)tile_rows, 1, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    r = enc(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  }
  return r == CUDA_SUCCESS ? OOCO_OK : fail_cuda(five_d ? "cuTensorMapEncodeTiled(5d)" : "cuTensorMapEncodeTiled(4d)", (long)r);
}

// 8-bit pool: (128 bytes of a token row, token, head, block), one box = [tile_rows][128 B].
static int encode_kv8_map(CUtensorMap* tm, const ooco_shape_t* s, const void* base, int tile_rows) {
  EncodeTiledFn enc = encode_fn();
  if (!enc) return fail_cuda("cudaGetDriverEntryPoint(cuTensorMapEncodeTiled)", -1);
  cuuint64_t dims[4] = {(cuuint64_t)s->head_dim, (cuuint64_t)s->block_size, (cuuint64_t)s->num_kv_heads,
                        (cuuint64_t)s->num_blocks};
  cuuint64_t strides[3] = {(cuuint64_t)s->kv_token_stride, (cuuint64_t)s->kv_head_stride,
                           (cuuint64_t)s->kv_block_stride};
  cuuint32_t box[4] = {(cuuint32_t)s->head_dim, (cuuint32_t)tile_rows, 1, 1};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  CUresult r = enc(tm, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<void*>(base), dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? OOCO_OK : fail_cuda("cuTensorMapEncodeTiled(8-bit)", (long)r);
}

// Launch with the programmatic-stream-serialization attribute (the kernel itself waits for its
// predecessor with griddepcontrol.wait) when `pdl`, else an ordinary launch.
template <typename... KArgs, typename... Args>
static cudaError_t launch_ex(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                             bool pdl, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kern, std::forward<Args>(args)...);
}

template <int D, int NCW, int NT, int TPW, int KVM = 0>
static int launch_main(const CUtensorMap& tk, const CUtensorMap& tv, DecodeParams& p, const DeviceInfo& di,
                       int ctas_per_sm, int want_stages, cudaStream_t st, int dev, bool dry) {
  using L = SmemLayout<D, NCW, NT, TPW, KVM>;
  auto kern = decode_main_kernel<D, NCW, NT, TPW, KVM>;
  // the opt-in limit covers static + dynamic shared memory of the kernel
  static std::atomic<int> static_smem{-1};
  if (static_smem.load() < 0) {
    cudaFuncAttributes fa;
    cudaError_t e = cudaFuncGetAttributes(&fa, kern);
    if (e != cudaSuccess) return fail_cuda("cudaFuncGetAttributes", (long)e);
    static_smem.store((int)fa.sharedSizeBytes);
  }
  const size_t dyn_max = (size_t)di.smem_optin - (size_t)static_smem.load();
  // per-CTA share of the SM's shared memory (1 KiB per CTA is reserved by the system)
  const size_t budget = ctas_per_sm > 1 ? ((size_t)di.smem_optin + 1024) / ctas_per_sm - 1024 - static_smem.load()
                                        : dyn_max;
  int nst = want_stages > 0 ? want_stages : 32;
  if (KVM == 2 && nst > 8) nst = 8;  // every stage owns tensor-memory columns for its scores
  while (nst > 2 && L::total(nst, p.GQ) > budget) --nst;
  if (L::total(nst, p.GQ) > dyn_max) return OOCO_E_UNSUPPORTED;
  p.nstages = nst;
  const size_t smem = L::total(nst, p.GQ);
  static std::atomic<size_t> configured[64];
  if (dev < 0 || dev >= 64 || configured[dev].load() < smem) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn_max);
    if (e != cudaSuccess) return fail_cuda("cudaFuncSetAttribute(max dynamic smem)", (long)e);
    if (dev >= 0 && dev < 64) configured[dev].store(dyn_max);
  }
  if (dry) return OOCO_OK;  // sizing and attributes only: the caller launches nothing before these have passed
  cudaError_t e = launch_ex(kern, dim3(p.next_item_init), dim3(L::kWarps * 32), smem, st,
                            g_knobs[kKnobPdl].load() != 0 && !tl_events_between_kernels, tk, tv, p);
  if (e == cudaSuccess) e = cudaGetLastError();
  return e == cudaSuccess ? OOCO_OK : fail_cuda("launch of the attention kernel", (long)e);
}

template <int D, int NCW, int TPW>
static int launch_main_nt(const CUtensorMap& tk, const CUtensorMap& tv, DecodeParams& p, const DeviceInfo& di,
                          int cps, int stages, cudaStream_t st, int dev, bool dry) {
  if (p.GQ <= 8) return launch_main<D, NCW, 1, TPW>(tk, tv, p, di, cps, stages, st, dev, dry);
  return launch_main<D, NCW, 2, TPW>(tk, tv, p, di, cps, stages, st, dev, dry);
}

// 8-bit cache: head_dim 128, one tile per warp.  `tc`: the 8-warp shape with the scores on tcgen05.
static int launch_main_kv8(int ncw, bool tc, const CUtensorMap& tk, const CUtensorMap& tv, DecodeParams& p,
                           const DeviceInfo& di, int cps, int stages, cudaStream_t st, int dev, bool dry) {
  const bool wide = p.GQ > 8;
  if (tc && ncw == 8)
    return wide ? launch_main<128, 8, 2, 1, 2>(tk, tv, p, di, cps, stages, st, dev, dry)
                : launch_main<128, 8, 1, 1, 2>(tk, tv, p, di, cps, stages, st, dev, dry);
  switch (ncw) {
    case 2:
      return wide ? launch_main<128, 2, 2, 1, 1>(tk, tv, p, di, cps, stages, st, dev, dry)
                  : launch_main<128, 2, 1, 1, 1>(tk, tv, p, di, cps, stages, st, dev, dry);
    case 8:
      return wide ? launch_main<128, 8, 2, 1, 1>(tk, tv, p, di, cps, stages, st, dev, dry)
                  : launch_main<128, 8, 1, 1, 1>(tk, tv, p, di, cps, stages, st, dev, dry);
    default:
      return wide ? launch_main<128, 4, 2, 1, 1>(tk, tv, p, di, cps, stages, st, dev, dry)
                  : launch_main<128, 4, 1, 1, 1>(tk, tv, p, di, cps, stages, st, dev, dry);
  }
}

template <int D>
static int launch_main_ncw(int ncw, int tpw, const CUtensorMap& tk, const CUtensorMap& tv, DecodeParams& p,
                           const DeviceInfo& di, int cps, int stages, cudaStream_t st, int dev, bool dry) {
  if (tpw == 2) {
    switch (ncw) {
      case 2: return launch_main_nt<D, 2, 2>(tk, tv, p, di, cps, stages, st, dev, dry);
      default: return launch_main_nt<D, 4, 2>(tk, tv, p, di, cps, stages, st, dev, dry);
    }
  }
  switch (ncw) {
    case 2: return launch_main_nt<D, 2, 1>(tk, tv, p, di, cps, stages, st, dev, dry);
    case 8: return launch_main_nt<D, 8, 1>(tk, tv, p, di, cps, stages, st, dev, dry);
    default: return launch_main_nt<D, 4, 1>(tk, tv, p, di, cps, stages, st, dev, dry);
  }
}

// Prefill-chunk kernel: as many 64-token stages as the CTA's share of shared memory holds (at most 8).
template <int D, int NCW>
static int launch_chunk(const CUtensorMap& tk, const CUtensorMap& tv, DecodeParams& p, const DeviceInfo& di,
                        int ctas_per_sm, cudaStream_t st, int dev, bool dry) {
  using L = ChunkSmem<D>;
  auto kern = chunk_main_kernel<D, NCW>;
  static std::atomic<int> static_smem{-1};
  if (static_smem.load() < 0) {
    cudaFuncAttributes fa;
    cudaError_t e = cudaFuncGetAttributes(&fa, kern);
    if (e != cudaSuccess) return fail_cuda("cudaFuncGetAttributes", (long)e);
    static_smem.store((int)fa.sharedSizeBytes);
  }
  const size_t dyn_max = (size_t)di.smem_optin - (size_t)static_smem.load();
  const size_t budget = ctas_per_sm > 1 ? ((size_t)di.smem_optin + 1024) / ctas_per_sm - 1024 - static_smem.load()
                                        : dyn_max;
  int nst = 8;
  while (nst > 2 && L::total(nst) > budget) --nst;
  if (L::total(nst) > dyn_max) return OOCO_E_UNSUPPORTED;
  p.nstages = nst;
  const size_t smem = L::total(nst);
  static std::atomic<size_t> configured[64];
  if (dev < 0 || dev >= 64 || configured[dev].load() < smem) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn_max);
    if (e != cudaSuccess) return fail_cuda("cudaFuncSetAttribute(max dynamic smem)", (long)e);
    if (dev >= 0 && dev < 64) configured[dev].store(dyn_max);
  }
  if (dry) return OOCO_OK;  // sizing and attributes only: the caller launches nothing before these have passed
  cudaError_t e = launch_ex(kern, dim3(p.next_item_init), dim3((NCW + 1) * 32), smem, st,
                            g_knobs[kKnobPdl].load() != 0 && !tl_events_between_kernels, tk, tv, p);
  if (e == cudaSuccess) e = cudaGetLastError();
  return e == cudaSuccess ? OOCO_OK : fail_cuda("launch of the chunk attention kernel", (long)e);
}

// Prefill chunk on tcgen05 with one 128-row tile per CTA and two CTAs per SM (head_dim 128): what the 8-bit cache
// runs, and the bf16 cache when the kernel below is switched off.
template <bool KV8>
static int launch_chunk_tc(const CUtensorMap& tk, const CUtensorMap& tv, DecodeParams& p, const DeviceInfo& di,
                           int ctas_per_sm, cudaStream_t st, int dev, bool dry) {
  auto kern = chunk_tc_kernel<KV8>;
  static std::atomic<int> static_smem{-1};
  if (static_smem.load() < 0) {
    cudaFuncAttributes fa;
    cudaError_t e = cudaFuncGetAttributes(&fa, kern);
    if (e != cudaSuccess) return fail_cuda("cudaFuncGetAttributes", (long)e);
    static_smem.store((int)fa.sharedSizeBytes);
  }
  const size_t dyn_max = (size_t)di.smem_optin - (size_t)static_smem.load();
  const size_t budget = ctas_per_sm > 1 ? ((size_t)di.smem_optin + 1024) / ctas_per_sm - 1024 - static_smem.load()
                                        : dyn_max;
  // 8-bit cache: two 16-bit stages (the MMAs' double buffer) and as many 8-bit stages as fit beside them
  int nst = KV8 ? 2 : 6, nraw = KV8 ? 4 : 0;
  while (!KV8 && nst > 2 && ChunkTcSmem::total(nst) > budget) --nst;
  while (KV8 && nraw > 2 && ChunkTcSmem::total(nst, nraw) > budget) --nraw;
  if (ChunkTcSmem::total(nst, nraw) > dyn_max) return OOCO_E_UNSUPPORTED;
  p.nstages = nst;
  p.nstages_raw = nraw;
  const size_t smem = ChunkTcSmem::total(nst, nraw);
  static std::atomic<size_t> configured[64];
  if (dev < 0 || dev >= 64 || configured[dev].load() < smem) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn_max);
    if (e != cudaSuccess) return fail_cuda("cudaFuncSetAttribute(max dynamic smem)", (long)e);
    if (dev >= 0 && dev < 64) configured[dev].store(dyn_max);
  }
  if (dry) return OOCO_OK;  // sizing and attributes only: the caller launches nothing before these have passed
  cudaError_t e = launch_ex(kern, dim3(p.next_item_init), dim3(KV8 ? 256 : 192), smem, st,
                            g_knobs[kKnobPdl].load() != 0 && !tl_events_between_kernels, tk, tv, p);
  if (e == cudaSuccess) e = cudaGetLastError();
  return e == cudaSuccess ? OOCO_OK : fail_cuda("launch of the tcgen05 chunk attention kernel", (long)e);
}

// Prefill chunk on tcgen05, one persistent CTA per SM, 512 tensor-memory columns, 128-token K / V slots (head_dim 128,
// bf16 cache): two 128-row tiles per CTA beyond 128 score columns; up to 128 columns its one-tile mode, in which the
// second tile's resources (score columns, issuing warp, Q region) pipeline the one tile -- it beats the one-tile
// kernel and the mma.sync kernel on every workload measured, from 17 columns on.  KV8: the one-tile mode over the 8-bit
// cache (the idle softmax warps widen the codes), 1.25 to 1.5 times as fast as the two-CTA kernel on these shapes.
template <bool KV8>
static int launch_chunk_tc2(const CUtensorMap& tk, const CUtensorMap& tv, DecodeParams& p, const DeviceInfo& di,
                            cudaStream_t st, int dev, bool dry) {
  auto kern = chunk_tc2_kernel<KV8>;
  static std::atomic<int> static_smem{-1};
  if (static_smem.load() < 0) {
    cudaFuncAttributes fa;
    cudaError_t e = cudaFuncGetAttributes(&fa, kern);
    if (e != cudaSuccess) return fail_cuda("cudaFuncGetAttributes", (long)e);
    static_smem.store((int)fa.sharedSizeBytes);
  }
  const size_t dyn_max = (size_t)di.smem_optin - (size_t)static_smem.load();
  const size_t smem = ChunkTc2Smem::total();
  if (smem > dyn_max) return OOCO_E_UNSUPPORTED;
  static std::atomic<size_t> configured[64];
  if (dev < 0 || dev >= 64 || configured[dev].load() < smem) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn_max);
    if (e != cudaSuccess) return fail_cuda("cudaFuncSetAttribute(max dynamic smem)", (long)e);
    if (dev >= 0 && dev < 64) configured[dev].store(dyn_max);
  }
  if (dry) return OOCO_OK;  // sizing and attributes only: the caller launches nothing before these have passed
  cudaError_t e = launch_ex(kern, dim3(p.next_item_init), dim3(kTc2Threads), smem, st,
                            g_knobs[kKnobPdl].load() != 0 && !tl_events_between_kernels, tk, tv, p);
  if (e == cudaSuccess) e = cudaGetLastError();
  return e == cudaSuccess ? OOCO_OK : fail_cuda("launch of the two-tile tcgen05 chunk attention kernel", (long)e);
}

// 9 .. 16 score columns: the warps of a CTA share one 16-row tile and split the tokens of a stage.
template <int D>
static int launch_row16(const CUtensorMap& tk, const CUtensorMap& tv, DecodeParams& p, const DeviceInfo& di,
                        int ctas_per_sm, cudaStream_t st, int dev, bool dry) {
  constexpr int NCW = 4;
  using M = Row16Smem<NCW>;
  auto kern = row16_main_kernel<D, NCW>;
  static std::atomic<int> static_smem{-1};
  if (static_smem.load() < 0) {
    cudaFuncAttributes fa;
    cudaError_t e = cudaFuncGetAttributes(&fa, kern);
    if (e != cudaSuccess) return fail_cuda("cudaFuncGetAttributes", (long)e);
    static_smem.store((int)fa.sharedSizeBytes);
  }
  const size_t dyn_max = (size_t)di.smem_optin - (size_t)static_smem.load();
  const size_t budget = ctas_per_sm > 1 ? ((size_t)di.smem_optin + 1024) / ctas_per_sm - 1024 - static_smem.load()
                                        : dyn_max;
  int nst = 8;
  while (nst > 2 && M::template total<D>(nst) > budget) --nst;
  if (M::template total<D>(nst) > dyn_max) return OOCO_E_UNSUPPORTED;
  p.nstages = nst;
  const size_t smem = M::template total<D>(nst);
  static std::atomic<size_t> configured[64];
  if (dev < 0 || dev >= 64 || configured[dev].load() < smem) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn_max);
    if (e != cudaSuccess) return fail_cuda("cudaFuncSetAttribute(max dynamic smem)", (long)e);
    if (dev >= 0 && dev < 64) configured[dev].store(dyn_max);
  }
  if (dry) return OOCO_OK;  // sizing and attributes only: the caller launches nothing before these have passed
  cudaError_t e = launch_ex(kern, dim3(p.next_item_init), dim3((NCW + 1) * 32), smem, st,
                            g_knobs[kKnobPdl].load() != 0 && !tl_events_between_kernels, tk, tv, p);
  if (e == cudaSuccess) e = cudaGetLastError();
  return e == cudaSuccess ? OOCO_OK : fail_cuda("launch of the 16-row attention kernel", (long)e);
}

template <int D>
static int launch_chunk_ncw(int ncw, const CUtensorMap& tk, const CUtensorMap& tv, DecodeParams& p,
                            const DeviceInfo& di, int cps, cudaStream_t st, int dev, bool dry) {
  switch (ncw) {
    case 2: return launch_chunk<D, 2>(tk, tv, p, di, cps, st, dev, dry);
    case 4: return launch_chunk<D, 4>(tk, tv, p, di, cps, st, dev, dry);
    default: return launch_chunk<D, 8>(tk, tv, p, di, cps, st, dev, dry);
  }
}

static AppendParams make_append_params(const ooco_shape_t* s, const void* k_new, const void* v_new,
                                       void* k_cache, void* v_cache, const int32_t* block_table,
                                       const int32_t* positions) {
  AppendParams a;
  a.k_new = (const uint4*)k_new;
  a.v_new = (const uint4*)v_new;
  a.k_cache = (uint16_t*)k_cache;
  a.v_cache = (uint16_t*)v_cache;
  a.block_table = block_table;
  a.positions = positions;
  a.B = s->batch;
  a.Hkv = s->num_kv_heads;
  a.D = s->head_dim;
  a.bs = s->block_size;
  a.NB = s->num_blocks;
  a.MB = s->max_blocks_per_seq;
  a.bstr = s->kv_block_stride;
  a.hstr = s->kv_head_stride;
  a.tstr = s->kv_token_stride;
  a.Sq = 1;
  a.kv8 = 0;
  a.k_scale = a.v_scale = 1.f;
  return a;
}

static int append_blocks(const ooco_shape_t* s, int threads, int q_len = 1) {
  const long long n = (long long)s->batch * q_len * s->num_kv_heads * (s->head_dim / 8);
  long long blocks = (n + threads - 1) / threads;
  return (int)(blocks > 2048 ? 2048 : blocks);
}

// Built-in scratch for ooco_decode_attention_static: it lives in the library's device image, so
// using it needs no allocation call.  In host code the name below is only a stand-in for the
// symbol; the device address comes from cudaGetSymbolAddress (static_scratch_ptr).
static __device__ __align__(256) unsigned char g_static_scratch[OOCO_STATIC_SCRATCH_BYTES];

// Device address of g_static_scratch on the current device, looked up once per device.
static int static_scratch_ptr(void** ptr_out) {
  static std::mutex mu;
  static void* cache[64];
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return fail_cuda("cudaGetDevice", (long)e);
  std::lock_guard<std::mutex> lk(mu);
  if (dev >= 0 && dev < 64 && cache[dev]) {
    *ptr_out = cache[dev];
    return OOCO_OK;
  }
  void* ptr = nullptr;
  e = cudaGetSymbolAddress((void**)&ptr, g_static_scratch);
  if (e != cudaSuccess || !ptr) return fail_cuda("cudaGetSymbolAddress(built-in scratch)", (long)e);
  if (dev >= 0 && dev < 64) cache[dev] = ptr;
  *ptr_out = ptr;
  return OOCO_OK;
}

static int current_device(int* dev) { return cudaGetDevice(dev) == cudaSuccess ? OOCO_OK : OOCO_E_CUDA; }

// Device-visible address of a page-locked (pinned / registered) host buffer on the current device,
// or nullptr when `host` is ordinary pageable memory (which a kernel must never be given).
static void* mapped_host_pointer(const void* host) {
  cudaPointerAttributes a;
  if (cudaPointerGetAttributes(&a, host) != cudaSuccess) {
    cudaGetLastError();
    return nullptr;
  }
  if (a.type != cudaMemoryTypeHost || !a.devicePointer) return nullptr;
  return a.devicePointer;
}

// Largest contiguous run of a side: 0 = whole block, 1 = one kv head of a block, 2 = one token row.
static int run_level(int64_t hstr, int64_t tstr, int bs, int D) {
  if (tstr != D) return 2;
  return hstr == (int64_t)bs * D ? 0 : 1;
}

static BlockSide pool_side(const ooco_shape_t* s, const void* k, const void* v, const int32_t* ids) {
  BlockSide b;
  b.k = (uint16_t*)k;
  b.v = (uint16_t*)v;
  b.ids = ids;
  b.bstr = s->kv_block_stride;
  b.hstr = s->kv_head_stride;
  b.tstr = s->kv_token_stride;
  b.nb = s->num_blocks;
  return b;
}

static BlockSide packed_side(const ooco_shape_t* s, const void* k, const void* v, int n) {
  BlockSide b;
  b.k = (uint16_t*)k;
  b.v = (uint16_t*)v;
  b.ids = nullptr;
  b.tstr = s->head_dim;
  b.hstr = (int64_t)s->block_size * s->head_dim;
  b.bstr = b.hstr * s->num_kv_heads;
  b.nb = n;
  return b;
}

// Moves n listed blocks from `src` to `dst` (K and V) with the bulk-copy kernel.
static int launch_block_copy(const ooco_shape_t* s, const BlockSide& src, const BlockSide& dst, int n,
                             int32_t* status, void* cuda_stream) {
  if (n == 0) return OOCO_OK;
  int dev = 0, rc;
  if ((rc = current_device(&dev))) return rc;
  const DeviceInfo di = device_info(dev);
  if (di.sm_count <= 0) return OOCO_E_CUDA;
  BlockCopyParams p;
  memset(&p, 0, sizeof p);
  p.src = src;
  p.dst = dst;
  p.n = n;
  p.Hkv = s->num_kv_heads;
  p.bs = s->block_size;
  p.D = s->head_dim;
  const int ls = run_level(src.hstr, src.tstr, p.bs, p.D), ld = run_level(dst.hstr, dst.tstr, p.bs, p.D);
  p.run_level = ls > ld ? ls : ld;
  p.runs_per_block = p.run_level == 0 ? 1 : (p.run_level == 1 ? p.Hkv : p.Hkv * p.bs);
  p.run_bytes = 2 * p.Hkv * p.bs * p.D / p.runs_per_block;
  p.pieces_per_run = (p.run_bytes + kCopyPieceBytes - 1) / kCopyPieceBytes;
  p.status = status;
  const long long total = (long long)n * p.runs_per_block * p.pieces_per_run * 2;
  const long long cap = (long long)di.sm_count * g_knobs[kKnobCopyCtasPerSm].load();
  const int grid = (int)(total < cap ? total : cap);
  const size_t smem = (size_t)kCopyStages * kCopyPieceBytes + 128;
  static std::atomic<int> configured[64];
  if (dev < 0 || dev >= 64 || !configured[dev].load()) {
    cudaError_t e = cudaFuncSetAttribute(block_copy_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return fail_cuda("cudaFuncSetAttribute(block copy smem)", (long)e);
    if (dev >= 0 && dev < 64) configured[dev].store(1);
  }
  cudaError_t e = launch_ex(block_copy_kernel, dim3(grid), dim3(32), smem, (cudaStream_t)cuda_stream,
                            g_knobs[kKnobPdl].load() != 0, p);
  if (e == cudaSuccess) e = cudaGetLastError();
  return e == cudaSuccess ? OOCO_OK : fail_cuda("launch of the block copy kernel", (long)e);
}

}  // namespace ooco

using namespace ooco;

extern "C" {

int ooco_version(void) { return OOCO_VERSION; }

const char* ooco_status_string(int status) {
  switch (status) {
    case OOCO_OK: return "ok";
    case OOCO_E_NULLPTR: return "null pointer argument";
    case OOCO_E_SHAPE: return "invalid shape";
    case OOCO_E_UNSUPPORTED: return "shape not supported by the kernels";
    case OOCO_E_WORKSPACE: return "workspace or staging buffer too small or misaligned";
    case OOCO_E_CUDA: return "CUDA call or launch failed";
    case OOCO_E_DEVICE: return "device-side status word reports a problem";
    default: return "unknown status";
  }
}

int ooco_last_launch_count(void) { return tl_last_launches; }

const char* ooco_last_error_detail(void) { return tl_detail; }

int ooco_profile_enable(int max_records) {
  if (max_records < 0 || max_records > (1 << 20)) return OOCO_E_SHAPE;
  std::lock_guard<std::mutex> lk(g_prof.mu);
  g_prof_on.store(0, std::memory_order_release);
  for (cudaEvent_t e : g_prof.ev) cudaEventDestroy(e);
  g_prof.ev.clear();
  g_prof.capacity = g_prof.used = 0;
  if (max_records == 0) return OOCO_OK;
  g_prof.ev.resize(4 * (size_t)max_records);
  for (auto& e : g_prof.ev)
    if (cudaEventCreate(&e) != cudaSuccess) return fail_cuda("cudaEventCreate", -1);
  g_prof.capacity = max_records;
  g_prof_on.store(1, std::memory_order_release);
  return OOCO_OK;
}

int ooco_profile_read(float* ms_out, int max_records, int* n_out) {
  if (!ms_out || !n_out) return OOCO_E_NULLPTR;
  std::lock_guard<std::mutex> lk(g_prof.mu);
  int n = g_prof.used < max_records ? g_prof.used : max_records;
  for (int i = 0; i < n; ++i) {
    cudaEvent_t* e = &g_prof.ev[4 * (size_t)i];
    if (cudaEventSynchronize(e[3]) != cudaSuccess) return fail_cuda("cudaEventSynchronize", -1);
    for (int k = 0; k < 3; ++k)
      if (cudaEventElapsedTime(&ms_out[3 * i + k], e[k], e[k + 1]) != cudaSuccess)
        return fail_cuda("cudaEventElapsedTime", -1);
  }
  *n_out = n;
  g_prof.used = 0;
  return OOCO_OK;
}

int ooco_set_tuning(int knob, int value) {
  if (knob < 0 || knob >= kKnobCount) return OOCO_E_SHAPE;
  if (knob == kKnobWarps && value != 2 && value != 4 && value != 8) return OOCO_E_SHAPE;
  if (knob == kKnobStages && (value < 0 || value > 64)) return OOCO_E_SHAPE;
  if (knob == kKnobCtasPerSm && (value < 1 || value > 4)) return OOCO_E_SHAPE;
  if ((knob == kKnobChunkMin || knob == kKnobChunkMax) && (value < 128 || value > (1 << 20) || value % 128))
    return OOCO_E_SHAPE;
  if (knob == kKnobItemsPerCta && (value < 1 || value > 64)) return OOCO_E_SHAPE;
  if (knob == kKnobTilesPerWarp && value != 1 && value != 2) return OOCO_E_SHAPE;
  if (knob == kKnobCopyCtasPerSm && (value < 1 || value > 3)) return OOCO_E_SHAPE;
  if ((knob == kKnobOutF32 || knob == kKnobKv8Tcgen05) && value != 0 && value != 1) return OOCO_E_SHAPE;
  if (knob == kKnobChunkTwoTiles && (value < 0 || value > 2)) return OOCO_E_SHAPE;
  if (knob == kKnobChunkTcgen05 && value != 0 && value != 1 && (value < 17 || value > 65536)) return OOCO_E_SHAPE;
  g_knobs[knob].store(value);
  g_overridden[knob].store(1);
  return OOCO_OK;
}

int ooco_get_tuning(int knob) {
  if (knob < 0 || knob >= kKnobCount) return OOCO_E_SHAPE;
  return g_knobs[knob].load();
}

int ooco_checked_build(void) { return kChecked ? 1 : 0; }

int ooco_check_predicate(int which, const int64_t* a) {
  if (!a) return OOCO_E_NULLPTR;
  switch (which) {
    case 0: return chk_table_entry(a[0], a[1]) ? 1 : 0;
    case 1: return chk_index(a[0], a[1]) ? 1 : 0;
    case 2: return chk_item(a[0], a[1], a[2], a[3], a[4], a[5], a[6]) ? 1 : 0;
    case 3: return chk_span(a[0], a[1], a[2], a[3]) ? 1 : 0;
    default: return OOCO_E_SHAPE;
  }
}

int ooco_kv_append(const ooco_shape_t* s, const void* k_new, const void* v_new, void* k_cache, void* v_cache,
                   const int32_t* block_table, const int32_t* positions, void* cuda_stream) {
  int rc = validate_shape(s);
  if (rc) return rc;
  if (!k_new || !v_new || !k_cache || !v_cache || !block_table || !positions) return OOCO_E_NULLPTR;
  if (((uintptr_t)k_new | (uintptr_t)v_new | (uintptr_t)k_cache | (uintptr_t)v_cache) & 15)
    return OOCO_E_UNSUPPORTED;
  const AppendParams ap = make_append_params(s, k_new, v_new, k_cache, v_cache, block_table, positions);
  kv_append_kernel<<<append_blocks(s, 256), 256, 0, (cudaStream_t)cuda_stream>>>(ap);
  cudaError_t e = cudaGetLastError();
  return e == cudaSuccess ? OOCO_OK : fail_cuda("launch of the append kernel", (long)e);
}

size_t ooco_decode_workspace_bytes(const ooco_shape_t* s) {
  if (validate_shape(s)) return 0;
  return ws_layout(s).total;
}

// Plan (+ optional fused append) -> split-KV attention -> LSE merge on `cuda_stream`.
// Query tokens per sequence: the score columns of a (sequence, kv head) pair, G * q_len, must fit the
// two 8-column MMA tiles of the kernel.
static int validate_q_len(const ooco_shape_t* s, int q_len, bool kv8 = false) {
  if (q_len < 1) return OOCO_E_SHAPE;
  if (q_len == 1) return OOCO_OK;
  if (q_len > kMaxQLen) return OOCO_E_UNSUPPORTED;
  (void)s;
  (void)kv8;  // the 8-bit cache runs the decode kernel up to 16 score columns and the tcgen05 chunk kernel beyond
  return OOCO_OK;
}

struct Kv8Scales {  // present: the caches hold E4M3 codes, a code stands for decode(code) * scale
  float k_scale, v_scale;
};

static int validate_kv8(const ooco_shape_t* s, const Kv8Scales* kv8) {
  if (!kv8) return OOCO_OK;
  if (!(kv8->k_scale > 0.f) || !(kv8->v_scale > 0.f)) return OOCO_E_SHAPE;
  if (s->head_dim != 128) return OOCO_E_UNSUPPORTED;
  if ((s->kv_block_stride | s->kv_head_stride | s->kv_token_stride) & 15) return OOCO_E_UNSUPPORTED;
  return OOCO_OK;
}

static int decode_core(const ooco_shape_t* s, const void* q, const void* k_cache, const void* v_cache,
                       const int32_t* block_table, const int32_t* context_lens, float scale, void* out,
                       void* workspace, size_t workspace_bytes, void* cuda_stream, const AppendParams* append,
                       const Kv8Scales* kv8 = nullptr, int q_len = 1, const HostStageParams* host_stage = nullptr,
                       const int32_t* plan_context_lens = nullptr) {
  // host_stage / plan_context_lens (host-buffer step): extra CTAs of the first launch stage q and the
  // block table for the attention kernel while its planning CTA reads the lengths, and its append CTAs
  // the new rows, straight from the mapped host buffers.
  int rc = validate_shape(s);
  if (rc) return rc;
  if ((rc = validate_kv8(s, kv8))) return rc;
  if ((rc = validate_q_len(s, q_len, kv8 != nullptr))) return rc;
  if (!(scale > 0.f) || !(scale <= 3.0e38f)) return OOCO_E_SHAPE;  // positive and finite (NaN fails both)
  if (!q || !k_cache || !v_cache || !block_table || !context_lens || !out || !workspace) return OOCO_E_NULLPTR;
  if (((uintptr_t)k_cache | (uintptr_t)v_cache | (uintptr_t)q | (uintptr_t)out) & 15) return OOCO_E_UNSUPPORTED;
  const WsLayout w = ws_layout(s, q_len);
  if (workspace_bytes < w.total || ((uintptr_t)workspace & 255)) return OOCO_E_WORKSPACE;
  int dev = 0;
  if ((rc = current_device(&dev))) return rc;
  const DeviceInfo di = device_info(dev);
  if (di.sm_count <= 0) return OOCO_E_CUDA;
  cudaStream_t st = (cudaStream_t)cuda_stream;

  // Launch shape of the decode kernel: 4 consumer warps x 2 CTAs per SM; the 8-bit path wants 16 consumer
  // warps per SM (it is latency-bound): 8 x 2; more than 8 score columns need two MMA column tiles and too
  // many registers for two CTAs of any shape: 8 x 1 (bf16 caches leave the decode kernel there, see below).
  // A knob set by the caller wins.
  const int G_ = s->num_q_heads / s->num_kv_heads * q_len;
  int ncw = g_knobs[kKnobWarps].load(), cps = g_knobs[kKnobCtasPerSm].load();
  if (!g_overridden[kKnobWarps].load() && (kv8 || G_ > 8)) ncw = 8;
  if (!g_overridden[kKnobCtasPerSm].load() && G_ > 8) cps = 1;
  // head_dim 64 halves the bytes per token, not the per-token work of the consumers: four smaller CTAs per
  // SM (16 consumer warps) keep up with HBM where two do not (4.9 -> 6.8 TB/s)
  if (!g_overridden[kKnobCtasPerSm].load() && !g_overridden[kKnobWarps].load() && G_ <= 8 && s->head_dim == 64)
    cps = 4;
  int tpw = g_knobs[kKnobTilesPerWarp].load();
  if (ncw == 8 || kv8) tpw = 1;
  // prefill chunk: 64-token stages; 8 warps (128 columns) x 1 CTA per SM, fewer columns: smaller CTAs x 2
  const bool chunk = G_ > kDecodeMaxColumns;
  // 9 .. 16 columns: the row layout with the tokens of a stage split over 4 warps x 2 CTAs per SM (the
  // column layout of the decode kernel needs a second MMA tile and a transposition per tile there)
  const bool row16 = !chunk && !kv8 && G_ > 8 && g_knobs[kKnobRowLayout16].load() != 0;
  // (the 8-bit cache has no mma.sync chunk kernel: every chunk over it runs the tcgen05 kernel)
  // (knob 12: 0 = never; 1 = every prefill chunk, i.e. from 17 score columns; n >= 17 = from n columns)
  const int tc_knob = g_knobs[kKnobChunkTcgen05].load();
  const int tc_from = tc_knob == 1 ? 17 : tc_knob;
  const bool chunk_tc = chunk && s->head_dim == 128 && (kv8 || (tc_knob != 0 && G_ >= tc_from));
  // (more than one 128-row tile per item, bf16: the kernel that keeps two tiles per CTA on the tensor pipe in turns)
  const int two_tiles = g_knobs[kKnobChunkTwoTiles].load();  // 1: beyond 128 columns only; 2: its one-tile mode below, too
  // (8-bit cache: only the one-tile mode has a variant that widens the codes, so up to 128 columns)
  const bool chunk_tc2 = chunk_tc && two_tiles != 0 && (kv8 ? (G_ <= kTcRows && two_tiles == 2) : (G_ > kTcRows || two_tiles == 2));
  if (chunk) {
    ncw = chunk_warps(G_);
    cps = (ncw == 8 && !chunk_tc) ? 1 : 2;
    if (chunk_tc && g_overridden[kKnobCtasPerSm].load()) cps = g_knobs[kKnobCtasPerSm].load() > 1 ? 2 : 1;
    if (chunk_tc2) cps = 1;
  } else if (row16) {
    ncw = 4;
    cps = 2;
  }
  const int stage_tok = chunk_tc2 ? kTc2StageTok : ((chunk || row16) ? kChunkStageTok : 16 * ncw * tpw);
  DecodeParams p;
  memset(&p, 0, sizeof p);
  uint8_t* ws = (uint8_t*)workspace;
  p.q = (const __nv_bfloat16*)q;
  p.out = (__nv_bfloat16*)out;
  p.block_table = block_table;
  p.context_lens = context_lens;
  p.hdr = (WsHeader*)ws;
  p.seq_first = (int32_t*)(ws + w.off_first);
  p.items = (int4*)(ws + w.off_items);
  p.part_lse = (float*)(ws + w.off_lse);
  p.part_o = (float*)(ws + w.off_o);
  p.B = s->batch;
  p.Hq = s->num_q_heads;
  p.Hkv = s->num_kv_heads;
  p.G = p.Hq / p.Hkv;
  p.Sq = q_len;
  p.GQ = p.G * q_len;
  p.D = s->head_dim;
  p.bs = s->block_size;
  p.MB = s->max_blocks_per_seq;
  p.NB = s->num_blocks;
  p.out_f32 = g_knobs[kKnobOutF32].load() != 0;
  p.max_items = w.max_items;
  p.tile_rows = s->block_size < stage_tok ? s->block_size : stage_tok;
  p.grid_main = di.sm_count * cps;
  if (p.grid_main > kGridCap) p.grid_main = kGridCap;
  p.next_item_init = p.grid_main;
  if (chunk_tc2)
    p.grid_main = (p.grid_main + (G_ + kTc2Rows - 1) / kTc2Rows - 1) / ((G_ + kTc2Rows - 1) / kTc2Rows);
  else if (chunk)
    p.grid_main = (p.grid_main + chunk_row_tiles(G_) - 1) / chunk_row_tiles(G_);
  p.chunk_min = g_knobs[kKnobChunkMin].load();
  p.chunk_max = g_knobs[kKnobChunkMax].load();
  if (p.chunk_max < p.chunk_min) p.chunk_max = p.chunk_min;
  p.items_per_cta = plan_items_per_cta(G_);
  // the 8-bit path widens codes to value / 256 (kE4m3WidenFactor): both scales carry the factor back (K's only
  // where K is widened: the tcgen05 score path multiplies the codes' own values)
  const bool kv8_tc = kv8 && !chunk && ncw == 8 && g_knobs[kKnobKv8Tcgen05].load() != 0;
  p.scale_log2e = scale * 1.4426950408889634f * (kv8 ? kv8->k_scale * (kv8_tc ? 1.f : kE4m3WidenFactor) : 1.f);
  p.v_scale = kv8 ? kv8->v_scale * kE4m3WidenFactor : 1.f;

  CUtensorMap tk, tv;
  bool five_d = !kv8 && !chunk && !row16 && s->head_dim == 128 && !g_knobs[kKnobSplitHalves].load();
  if (five_d && encode_kv_map(&tk, s, k_cache, p.tile_rows, true) != OOCO_OK) five_d = false;
  if (kv8) {
    if ((rc = encode_kv8_map(&tk, s, k_cache, p.tile_rows))) return rc;
    if ((rc = encode_kv8_map(&tv, s, v_cache, p.tile_rows))) return rc;
  } else if (five_d) {
    if ((rc = encode_kv_map(&tv, s, v_cache, p.tile_rows, true))) return rc;
  } else {
    if ((rc = encode_kv_map(&tk, s, k_cache, p.tile_rows, false))) return rc;
    if ((rc = encode_kv_map(&tv, s, v_cache, p.tile_rows, false))) return rc;
  }
  p.split_halves = five_d ? 0 : 1;

  // Everything of the attention launch that can refuse the call (shared-memory fit, function attributes) runs
  // once without launching, before the first kernel of the call is enqueued.
  const int stages = g_knobs[kKnobStages].load();
  auto launch_attention = [&](bool dry) -> int {
    if (chunk_tc2)
      return kv8 ? launch_chunk_tc2<true>(tk, tv, p, di, st, dev, dry) : launch_chunk_tc2<false>(tk, tv, p, di, st, dev, dry);
    if (chunk_tc)
      return kv8 ? launch_chunk_tc<true>(tk, tv, p, di, cps, st, dev, dry)
                 : launch_chunk_tc<false>(tk, tv, p, di, cps, st, dev, dry);
    if (chunk)
      return s->head_dim == 128 ? launch_chunk_ncw<128>(ncw, tk, tv, p, di, cps, st, dev, dry)
                                : launch_chunk_ncw<64>(ncw, tk, tv, p, di, cps, st, dev, dry);
    if (row16)
      return s->head_dim == 128 ? launch_row16<128>(tk, tv, p, di, cps, st, dev, dry)
                                : launch_row16<64>(tk, tv, p, di, cps, st, dev, dry);
    if (kv8) return launch_main_kv8(ncw, kv8_tc, tk, tv, p, di, cps, stages, st, dev, dry);
    return s->head_dim == 128 ? launch_main_ncw<128>(ncw, tpw, tk, tv, p, di, cps, stages, st, dev, dry)
                              : launch_main_ncw<64>(ncw, tpw, tk, tv, p, di, cps, stages, st, dev, dry);
  };
  if ((rc = launch_attention(true))) return rc;

  cudaEvent_t* pe = nullptr;
  if (g_prof_on.load(std::memory_order_acquire)) {
    std::lock_guard<std::mutex> lk(g_prof.mu);
    if (g_prof.used < g_prof.capacity) pe = &g_prof.ev[4 * (size_t)g_prof.used++];
  }
  tl_events_between_kernels = pe != nullptr;
  if (pe) cudaEventRecord(pe[0], st);
  const size_t first_bytes = (2 * (size_t)p.B + 1) * 4;  // chunk scan + clamped lengths
  const int first_in_smem = first_bytes <= 32 * 1024;    // static + dynamic shared memory stay under 48 KiB
  AppendParams ap;
  memset(&ap, 0, sizeof ap);
  if (append) ap = *append;
  const int n_append = append ? append_blocks(s, 1024, append->Sq) : 0;
  HostStageParams hs;
  memset(&hs, 0, sizeof hs);
  int n_stage = 0;
  if (host_stage) {
    hs = *host_stage;
    size_t total = 0;
    for (int k = 0; k < kStageBuffers; ++k) total += hs.bytes[k];
    n_stage = (int)((total / 16 + 1023) / 1024);
    n_stage = n_stage < 1 ? 1 : (n_stage > 256 ? 256 : n_stage);
  }
  const bool pdl_on = g_knobs[kKnobPdl].load() != 0 && !pe;
  DecodeParams pp = p;  // the planning CTA may read the lengths from another (host-mapped) copy
  if (plan_context_lens) pp.context_lens = plan_context_lens;
  cudaError_t e = launch_ex(plan_kernel<1024>, dim3(1 + n_append + n_stage), dim3(1024),
                            first_in_smem ? first_bytes : 0, st, pdl_on, pp, stage_tok, first_in_smem, ap, n_append,
                            hs);
  if (e == cudaSuccess) e = cudaGetLastError();
  if (e != cudaSuccess) return fail_cuda("launch of the plan kernel", (long)e);
  if (pe) cudaEventRecord(pe[1], st);
  rc = launch_attention(false);
  if (rc) return rc;
  if (pe) cudaEventRecord(pe[2], st);
  {
    const long long units = (long long)p.B * p.Sq * p.Hq;  // (sequence, query token, query head)
    int wpu_log2 = 0;  // warps per unit: more when the units alone cannot fill the SMs (few, very long sequences)
    while (wpu_log2 < 3 && (units << (wpu_log2 + 1)) <= (long long)di.sm_count * 8) ++wpu_log2;
    const long long need = ((units << wpu_log2) + 7) / 8;
    const int blocks = (int)(need < (long long)di.sm_count * 8 ? need : (long long)di.sm_count * 8);
    const bool pdl = g_knobs[kKnobPdl].load() != 0 && !pe;
    if (s->head_dim == 128)
      e = launch_ex(lse_merge_kernel<128>, dim3(blocks), dim3(256), 0, st, pdl, p, wpu_log2);
    else
      e = launch_ex(lse_merge_kernel<64>, dim3(blocks), dim3(256), 0, st, pdl, p, wpu_log2);
  }
  if (e == cudaSuccess) e = cudaGetLastError();
  if (e != cudaSuccess) return fail_cuda("launch of the merge kernel", (long)e);
  if (pe) cudaEventRecord(pe[3], st);
  tl_last_launches = 3;
  return OOCO_OK;
}

int ooco_decode_attention(const ooco_shape_t* s, const void* q, const void* k_cache, const void* v_cache,
                          const int32_t* block_table, const int32_t* context_lens, float scale, void* out,
                          void* workspace, size_t workspace_bytes, void* cuda_stream) {
  return decode_core(s, q, k_cache, v_cache, block_table, context_lens, scale, out, workspace, workspace_bytes,
                     cuda_stream, nullptr);
}

int ooco_decode_step(const ooco_shape_t* s, const void* q, const void* k_new, const void* v_new, void* k_cache,
                     void* v_cache, const int32_t* block_table, const int32_t* positions,
                     const int32_t* context_lens, float scale, void* out, void* workspace,
                     size_t workspace_bytes, void* cuda_stream) {
  int rc = validate_shape(s);
  if (rc) return rc;
  if (!k_new || !v_new || !k_cache || !v_cache || !block_table || !positions) return OOCO_E_NULLPTR;
  if (((uintptr_t)k_new | (uintptr_t)v_new | (uintptr_t)k_cache | (uintptr_t)v_cache) & 15)
    return OOCO_E_UNSUPPORTED;
  const AppendParams ap = make_append_params(s, k_new, v_new, k_cache, v_cache, block_table, positions);
  return decode_core(s, q, k_cache, v_cache, block_table, context_lens, scale, out, workspace, workspace_bytes,
                     cuda_stream, &ap);
}

int ooco_kv_append_fp8(const ooco_shape_t* s, const void* k_new, const void* v_new, void* k_cache, void* v_cache,
                       const int32_t* block_table, const int32_t* positions, float k_scale, float v_scale,
                       void* cuda_stream) {
  int rc = validate_shape(s);
  if (rc) return rc;
  const Kv8Scales sc = {k_scale, v_scale};
  if ((rc = validate_kv8(s, &sc))) return rc;
  if (!k_new || !v_new || !k_cache || !v_cache || !block_table || !positions) return OOCO_E_NULLPTR;
  if (((uintptr_t)k_new | (uintptr_t)v_new | (uintptr_t)k_cache | (uintptr_t)v_cache) & 15)
    return OOCO_E_UNSUPPORTED;
  AppendParams ap = make_append_params(s, k_new, v_new, k_cache, v_cache, block_table, positions);
  ap.kv8 = 1;
  ap.k_scale = k_scale;
  ap.v_scale = v_scale;
  kv_append_kernel<<<append_blocks(s, 256), 256, 0, (cudaStream_t)cuda_stream>>>(ap);
  cudaError_t e = cudaGetLastError();
  return e == cudaSuccess ? OOCO_OK : fail_cuda("launch of the append kernel", (long)e);
}

int ooco_decode_attention_fp8(const ooco_shape_t* s, const void* q, const void* k_cache, const void* v_cache,
                              const int32_t* block_table, const int32_t* context_lens, float scale, float k_scale,
                              float v_scale, void* out, void* workspace, size_t workspace_bytes,
                              void* cuda_stream) {
  const Kv8Scales sc = {k_scale, v_scale};
  return decode_core(s, q, k_cache, v_cache, block_table, context_lens, scale, out, workspace, workspace_bytes,
                     cuda_stream, nullptr, &sc);
}

int ooco_decode_step_fp8(const ooco_shape_t* s, const void* q, const void* k_new, const void* v_new, void* k_cache,
                         void* v_cache, const int32_t* block_table, const int32_t* positions,
                         const int32_t* context_lens, float scale, float k_scale, float v_scale, void* out,
                         void* workspace, size_t workspace_bytes, void* cuda_stream) {
  int rc = validate_shape(s);
  if (rc) return rc;
  const Kv8Scales sc = {k_scale, v_scale};
  if ((rc = validate_kv8(s, &sc))) return rc;
  if (!k_new || !v_new || !k_cache || !v_cache || !block_table || !positions) return OOCO_E_NULLPTR;
  if (((uintptr_t)k_new | (uintptr_t)v_new | (uintptr_t)k_cache | (uintptr_t)v_cache) & 15)
    return OOCO_E_UNSUPPORTED;
  AppendParams ap = make_append_params(s, k_new, v_new, k_cache, v_cache, block_table, positions);
  ap.kv8 = 1;
  ap.k_scale = k_scale;
  ap.v_scale = v_scale;
  return decode_core(s, q, k_cache, v_cache, block_table, context_lens, scale, out, workspace, workspace_bytes,
                     cuda_stream, &ap, &sc);
}

size_t ooco_decode_workspace_bytes_mq(const ooco_shape_t* s, int32_t q_len) {
  if (validate_shape(s) || validate_q_len(s, q_len)) return 0;
  return ws_layout(s, q_len).total;
}

int ooco_decode_attention_mq(const ooco_shape_t* s, int32_t q_len, const void* q, const void* k_cache,
                             const void* v_cache, const int32_t* block_table, const int32_t* context_lens,
                             float scale, void* out, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  return decode_core(s, q, k_cache, v_cache, block_table, context_lens, scale, out, workspace, workspace_bytes,
                     cuda_stream, nullptr, nullptr, q_len);
}

int ooco_kv_append_mq(const ooco_shape_t* s, int32_t q_len, const void* k_new, const void* v_new, void* k_cache,
                      void* v_cache, const int32_t* block_table, const int32_t* positions, void* cuda_stream) {
  int rc = validate_shape(s);
  if (rc) return rc;
  if (q_len < 1) return OOCO_E_SHAPE;
  if (!k_new || !v_new || !k_cache || !v_cache || !block_table || !positions) return OOCO_E_NULLPTR;
  if (((uintptr_t)k_new | (uintptr_t)v_new | (uintptr_t)k_cache | (uintptr_t)v_cache) & 15)
    return OOCO_E_UNSUPPORTED;
  AppendParams ap = make_append_params(s, k_new, v_new, k_cache, v_cache, block_table, positions);
  ap.Sq = q_len;
  kv_append_kernel<<<append_blocks(s, 256, q_len), 256, 0, (cudaStream_t)cuda_stream>>>(ap);
  cudaError_t e = cudaGetLastError();
  return e == cudaSuccess ? OOCO_OK : fail_cuda("launch of the append kernel", (long)e);
}

int ooco_decode_step_mq(const ooco_shape_t* s, int32_t q_len, const void* q, const void* k_new, const void* v_new,
                        void* k_cache, void* v_cache, const int32_t* block_table, const int32_t* positions,
                        const int32_t* context_lens, float scale, void* out, void* workspace,
                        size_t workspace_bytes, void* cuda_stream) {
  int rc = validate_shape(s);
  if (rc) return rc;
  if ((rc = validate_q_len(s, q_len))) return rc;
  if (!k_new || !v_new || !k_cache || !v_cache || !block_table || !positions) return OOCO_E_NULLPTR;
  if (((uintptr_t)k_new | (uintptr_t)v_new | (uintptr_t)k_cache | (uintptr_t)v_cache) & 15)
    return OOCO_E_UNSUPPORTED;
  AppendParams ap = make_append_params(s, k_new, v_new, k_cache, v_cache, block_table, positions);
  ap.Sq = q_len;
  return decode_core(s, q, k_cache, v_cache, block_table, context_lens, scale, out, workspace, workspace_bytes,
                     cuda_stream, &ap, nullptr, q_len);
}

int ooco_decode_step_mq_fp8(const ooco_shape_t* s, int32_t q_len, const void* q, const void* k_new,
                            const void* v_new, void* k_cache, void* v_cache, const int32_t* block_table,
                            const int32_t* positions, const int32_t* context_lens, float scale, float k_scale,
                            float v_scale, void* out, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  int rc = validate_shape(s);
  if (rc) return rc;
  const Kv8Scales sc = {k_scale, v_scale};
  if ((rc = validate_kv8(s, &sc))) return rc;
  if ((rc = validate_q_len(s, q_len))) return rc;
  if (!k_cache || !v_cache || !block_table) return OOCO_E_NULLPTR;
  if (!k_new && !v_new)  // attention only
    return decode_core(s, q, k_cache, v_cache, block_table, context_lens, scale, out, workspace, workspace_bytes,
                       cuda_stream, nullptr, &sc, q_len);
  if (!k_new || !v_new || !positions) return OOCO_E_NULLPTR;
  if (((uintptr_t)k_new | (uintptr_t)v_new | (uintptr_t)k_cache | (uintptr_t)v_cache) & 15)
    return OOCO_E_UNSUPPORTED;
  AppendParams ap = make_append_params(s, k_new, v_new, k_cache, v_cache, block_table, positions);
  ap.Sq = q_len;
  ap.kv8 = 1;
  ap.k_scale = k_scale;
  ap.v_scale = v_scale;
  return decode_core(s, q, k_cache, v_cache, block_table, context_lens, scale, out, workspace, workspace_bytes,
                     cuda_stream, &ap, &sc, q_len);
}

int ooco_decode_attention_static(const ooco_shape_t* s, const void* q, const void* k_cache,
                                 const void* v_cache, const int32_t* block_table,
                                 const int32_t* context_lens, float scale, void* out, void* cuda_stream) {
  int rc = validate_shape(s);
  if (rc) return rc;
  const size_t need = ws_layout(s).total;
  if (need > (size_t)OOCO_STATIC_SCRATCH_BYTES) {
    snprintf(tl_detail, sizeof tl_detail,
             "shape needs %zu bytes of scratch, the built-in scratch holds %zu: use ooco_decode_attention",
             need, (size_t)OOCO_STATIC_SCRATCH_BYTES);
    return OOCO_E_WORKSPACE;
  }
  void* scratch = nullptr;
  if ((rc = static_scratch_ptr(&scratch))) return rc;
  return ooco_decode_attention(s, q, k_cache, v_cache, block_table, context_lens, scale, out, scratch,
                               (size_t)OOCO_STATIC_SCRATCH_BYTES, cuda_stream);
}

static int check_block_args(const ooco_shape_t* s, int32_t n, const void* a, const void* b, const void* c,
                            const void* d, bool ids_ok) {
  int rc = validate_shape(s);
  if (rc) return rc;
  if (n < 0) return OOCO_E_SHAPE;
  if (!a || !b || !c || !d || (!ids_ok && n > 0)) return OOCO_E_NULLPTR;
  if (((uintptr_t)a | (uintptr_t)b | (uintptr_t)c | (uintptr_t)d) & 15) return OOCO_E_UNSUPPORTED;
  return OOCO_OK;
}

int ooco_kv_gather_blocks(const ooco_shape_t* s, const void* k_cache, const void* v_cache,
                          const int32_t* block_ids, int32_t n, void* k_packed, void* v_packed, int32_t* status,
                          void* cuda_stream) {
  int rc = check_block_args(s, n, k_cache, v_cache, k_packed, v_packed, block_ids != nullptr);
  if (rc) return rc;
  return launch_block_copy(s, pool_side(s, k_cache, v_cache, block_ids), packed_side(s, k_packed, v_packed, n), n,
                           status, cuda_stream);
}

int ooco_kv_scatter_blocks(const ooco_shape_t* s, const void* k_packed, const void* v_packed,
                           const int32_t* block_ids, int32_t n, void* k_cache, void* v_cache, int32_t* status,
                           void* cuda_stream) {
  int rc = check_block_args(s, n, k_cache, v_cache, k_packed, v_packed, block_ids != nullptr);
  if (rc) return rc;
  return launch_block_copy(s, packed_side(s, k_packed, v_packed, n), pool_side(s, k_cache, v_cache, block_ids), n,
                           status, cuda_stream);
}

int ooco_kv_copy_blocks(const ooco_shape_t* s, void* k_cache, void* v_cache, const int32_t* src_ids,
                        const int32_t* dst_ids, int32_t n, int32_t* status, void* cuda_stream) {
  int rc = check_block_args(s, n, k_cache, v_cache, k_cache, v_cache, src_ids && dst_ids);
  if (rc) return rc;
  return launch_block_copy(s, pool_side(s, k_cache, v_cache, src_ids), pool_side(s, k_cache, v_cache, dst_ids), n,
                           status, cuda_stream);
}

int ooco_workspace_status(const void* workspace, void* cuda_stream, int32_t* status_host) {
  if (!workspace || !status_host) return OOCO_E_NULLPTR;
  int32_t v = 0;
  if (cudaMemcpyAsync(&v, workspace, sizeof v, cudaMemcpyDeviceToHost, (cudaStream_t)cuda_stream) != cudaSuccess)
    return OOCO_E_CUDA;
  if (cudaStreamSynchronize((cudaStream_t)cuda_stream) != cudaSuccess) return OOCO_E_CUDA;
  *status_host = v;
  return v == 0 ? OOCO_OK : OOCO_E_DEVICE;
}

int ooco_decode_bytes_model(const ooco_shape_t* s, const int32_t* context_lens_host, int32_t bytes_per_value,
                            ooco_cost_t* c) {
  return ooco_attention_bytes_model(s, 1, context_lens_host, bytes_per_value, c);
}

int ooco_attention_bytes_model(const ooco_shape_t* s, int32_t q_len, const int32_t* context_lens_host,
                               int32_t bytes_per_value, ooco_cost_t* c) {
  if (!s || !context_lens_host || !c) return OOCO_E_NULLPTR;
  if (s->batch <= 0 || s->num_q_heads <= 0 || s->num_kv_heads <= 0 || s->head_dim <= 0 || s->block_size <= 0 ||
      bytes_per_value <= 0 || s->num_q_heads % s->num_kv_heads || q_len < 1)
    return OOCO_E_SHAPE;
  const int64_t d = bytes_per_value;
  const int64_t q_row = (int64_t)s->num_q_heads * s->head_dim;     // D_h of the operator table
  const int64_t kv_row = (int64_t)s->num_kv_heads * s->head_dim;   // D_h * Hkv / Hq
  int64_t tokens = 0, blocks = 0;
  for (int32_t b = 0; b < s->batch; ++b) {
    const int64_t t = context_lens_host[b] > 0 ? context_lens_host[b] : 0;
    tokens += t;
    blocks += (t + s->block_size - 1) / s->block_size;
  }
  c->total_tokens = tokens;
  c->flops = 4 * q_row * q_len * tokens;          // 4 D_h S_q S_kv
  c->bytes_q = d * s->batch * q_len * q_row;      // d S_q D_h per sequence
  c->bytes_out = c->bytes_q;
  c->bytes_kv = 2 * d * kv_row * tokens;
  c->bytes_index = 4 * ((int64_t)s->batch + blocks);
  c->bytes_paper = c->bytes_q + c->bytes_out + c->bytes_kv;
  return OOCO_OK;
}

size_t ooco_step_staging_bytes(const ooco_shape_t* s) {
  if (validate_shape(s)) return 0;
  auto up = [](size_t x) { return (x + 255) & ~(size_t)255; };
  const size_t qb = (size_t)s->batch * s->num_q_heads * s->head_dim * 2;
  const size_t kb = (size_t)s->batch * s->num_kv_heads * s->head_dim * 2;
  return up(qb) * 2 + up(kb) * 2 + up((size_t)s->batch * s->max_blocks_per_seq * 4) + 2 * up((size_t)s->batch * 4);
}

int ooco_decode_step_host(const ooco_shape_t* s, const void* q_host, const void* k_new_host,
                          const void* v_new_host, const int32_t* block_table_host,
                          const int32_t* positions_host, const int32_t* context_lens_host, void* k_cache,
                          void* v_cache, float scale, void* out_host, void* staging, size_t staging_bytes,
                          void* workspace, size_t workspace_bytes, void* cuda_stream) {
  int rc = validate_shape(s);
  if (rc) return rc;
  if (!q_host || !k_new_host || !v_new_host || !block_table_host || !positions_host || !context_lens_host ||
      !k_cache || !v_cache || !out_host || !staging || !workspace)
    return OOCO_E_NULLPTR;
  if (staging_bytes < ooco_step_staging_bytes(s) || ((uintptr_t)staging & 255)) return OOCO_E_WORKSPACE;
  if (workspace_bytes < ws_layout(s).total || ((uintptr_t)workspace & 255)) return OOCO_E_WORKSPACE;
  if (!(scale > 0.f) || !(scale <= 3.0e38f)) return OOCO_E_SHAPE;
  if (((uintptr_t)k_cache | (uintptr_t)v_cache) & 15) return OOCO_E_UNSUPPORTED;
  if (g_knobs[kKnobOutF32].load()) return OOCO_E_UNSUPPORTED;  // the staging and the host result are sized for bf16
  const auto t_enter = std::chrono::steady_clock::now();
  auto up = [](size_t x) { return (x + 255) & ~(size_t)255; };
  cudaStream_t st = (cudaStream_t)cuda_stream;
  const size_t qb = (size_t)s->batch * s->num_q_heads * s->head_dim * 2;
  const size_t kb = (size_t)s->batch * s->num_kv_heads * s->head_dim * 2;
  const size_t tb = (size_t)s->batch * s->max_blocks_per_seq * 4;
  const size_t lb = (size_t)s->batch * 4;
  uint8_t* base = (uint8_t*)staging;
  uint8_t* d_q = base;
  uint8_t* d_out = d_q + up(qb);
  uint8_t* d_kn = d_out + up(qb);
  uint8_t* d_vn = d_kn + up(kb);
  uint8_t* d_tab = d_vn + up(kb);
  uint8_t* d_pos = d_tab + up(tb);
  uint8_t* d_len = d_pos + up(lb);
  const void* hsrc[6] = {q_host, k_new_host, v_new_host, block_table_host, positions_host, context_lens_host};
  uint8_t* ddst[6] = {d_q, d_kn, d_vn, d_tab, d_pos, d_len};
  const size_t nbytes[6] = {qb, kb, kb, tb, lb, lb};
  // Page-locked inputs (all six, each under 4 GiB) are read through their device mapping inside the
  // step's first launch: the planning CTA reads the lengths, the append CTAs the new rows, positions and
  // table entries, and extra CTAs stage q, the block table and the lengths for the attention kernel.
  // Otherwise one copy per buffer.
  const void* msrc[6];
  bool mapped = g_knobs[kKnobHostStageKernel].load() != 0;
  for (int k = 0; k < 6 && mapped; ++k) {
    msrc[k] = mapped_host_pointer(hsrc[k]);
    mapped = msrc[k] != nullptr && nbytes[k] < ((size_t)1 << 32) && ((uintptr_t)msrc[k] & 15) == 0;
  }
  // A page-locked result buffer is written by the kernels themselves, through its device mapping.
  void* out_mapped = g_knobs[kKnobHostStageKernel].load() != 0 ? mapped_host_pointer(out_host) : nullptr;
  if (out_mapped && ((uintptr_t)out_mapped & 15)) out_mapped = nullptr;
  void* out_dev = out_mapped ? out_mapped : (void*)d_out;
  if (mapped) {
    HostStageParams hs;
    memset(&hs, 0, sizeof hs);
    const int pick[kStageBuffers] = {0, 3, 5};  // q, block table, lengths
    for (int k = 0; k < kStageBuffers; ++k) {
      hs.src[k] = (const uint8_t*)msrc[pick[k]];
      hs.dst[k] = ddst[pick[k]];
      hs.bytes[k] = (uint32_t)nbytes[pick[k]];
    }
    // The decode kernel (up to 8 query heads per kv head) fetches the q rows of a work item with one bulk copy
    // beside the item's first K / V stage: it takes them from the host mapping itself, so q crosses the host link
    // while the attention runs instead of in front of it.  (The 16-row kernel loads q with plain loads at the
    // start of an item and keeps the staged copy.)
    const bool q_direct = s->num_q_heads / s->num_kv_heads <= 8 && g_knobs[kKnobHostStageKernel].load() != 2;
    if (q_direct) hs.bytes[0] = 0;
    const AppendParams ap = make_append_params(s, msrc[1], msrc[2], k_cache, v_cache, (const int32_t*)msrc[3],
                                               (const int32_t*)msrc[4]);
    if ((rc = decode_core(s, q_direct ? msrc[0] : (const void*)d_q, k_cache, v_cache, (const int32_t*)d_tab, (const int32_t*)d_len, scale, out_dev,
                          workspace, workspace_bytes, st, &ap, nullptr, 1, &hs, (const int32_t*)msrc[5])))
      return rc;
  } else {
    bool ok = true;
    for (int k = 0; k < 6; ++k)
      ok &= cudaMemcpyAsync(ddst[k], hsrc[k], nbytes[k], cudaMemcpyHostToDevice, st) == cudaSuccess;
    if (!ok) return fail_cuda("cudaMemcpyAsync(host to device)", -1);
    if ((rc = ooco_decode_step(s, d_q, d_kn, d_vn, k_cache, v_cache, (const int32_t*)d_tab, (const int32_t*)d_pos,
                               (const int32_t*)d_len, scale, out_dev, workspace, workspace_bytes, st)))
      return rc;
  }
  if (!out_mapped && cudaMemcpyAsync(out_host, d_out, qb, cudaMemcpyDeviceToHost, st) != cudaSuccess)
    return fail_cuda("cudaMemcpyAsync(device to host)", -1);
  const auto t_enqueued = std::chrono::steady_clock::now();
  if (cudaStreamSynchronize(st) != cudaSuccess) return fail_cuda("cudaStreamSynchronize", -1);
  const auto t_done = std::chrono::steady_clock::now();
  tl_host_ns[0] = std::chrono::duration_cast<std::chrono::nanoseconds>(t_enqueued - t_enter).count();
  tl_host_ns[1] = std::chrono::duration_cast<std::chrono::nanoseconds>(t_done - t_enqueued).count();
  return OOCO_OK;
}

int ooco_last_host_step_ns(int64_t* enqueue_ns, int64_t* wait_ns) {
  if (!enqueue_ns || !wait_ns) return OOCO_E_NULLPTR;
  *enqueue_ns = tl_host_ns[0];
  *wait_ns = tl_host_ns[1];
  return OOCO_OK;
}

}  // extern "C"
