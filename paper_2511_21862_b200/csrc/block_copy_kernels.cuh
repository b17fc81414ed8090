// Paged KV block movement for sm_100a: pack pool blocks into a contiguous buffer (migration send,
// eviction to a staging area), unpack them into other pool blocks (migration receive, restore) and
// copy blocks inside a pool.  One kernel serves all three: a list entry i names a source block and
// a destination block; each side is either the pool (block id looked up in a list) or a packed
// buffer (block i of [n, Hkv, bs, D]).
//
// The work is a plain HBM-bound copy, so it runs on the copy engines of the SM: one lane per CTA
// drives a ring of shared-memory stages with 1-D bulk async copies (global -> shared, completion on
// an mbarrier; shared -> global, completion by bulk groups).  No data passes through registers.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "decode_kernels.cuh"  // status bits
#include "ptx.cuh"

namespace ooco {

constexpr int kCopyStages = 4;
constexpr int kCopyPieceBytes = 16 * 1024;
constexpr int kCopyAddrRing = 64;            // two batches of 32 piece descriptors
constexpr int kStatusBadBlockId = 4;         // a listed block id was outside its pool (entry skipped)
constexpr uint64_t kCopyWaitLimitNs = 2000000000ull;

struct BlockSide {
  uint16_t* k;          // K base (pool or packed buffer)
  uint16_t* v;          // V base
  const int32_t* ids;   // [n] block ids, or NULL: entry i is block i of a packed buffer
  int64_t bstr, hstr, tstr;  // element strides of (block, kv head, token slot)
  int32_t nb;           // blocks on this side (ids outside [0, nb) are skipped and reported)
};

struct BlockCopyParams {
  BlockSide src, dst;
  int32_t n;              // list entries
  int32_t Hkv, bs, D;
  int32_t run_level;      // contiguous run: 0 = whole block, 1 = (block, head), 2 = (block, head, token)
  int32_t runs_per_block;
  int32_t run_bytes;
  int32_t pieces_per_run; // a run is moved in pieces of at most kCopyPieceBytes
  int32_t* status;        // device status word (may be NULL): bits are OR-ed in, never cleared
};

__device__ __forceinline__ void bulk_s2g(void* dst, uint32_t src, uint32_t bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst), "r"(src), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// Until at most `N` of the most recent bulk groups are still reading their shared-memory source.
template <int N>
__device__ __forceinline__ void bulk_wait_read() {
  asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

// Element offset of run `r` of block `blk` on one side.
__device__ __forceinline__ int64_t run_offset(const BlockSide& s, int level, int bs, int64_t blk, int r) {
  if (level == 0) return blk * s.bstr;
  if (level == 1) return blk * s.bstr + (int64_t)r * s.hstr;
  return blk * s.bstr + (int64_t)(r / bs) * s.hstr + (int64_t)(r % bs) * s.tstr;
}

__global__ void __launch_bounds__(32) block_copy_kernel(const BlockCopyParams p) {
  extern __shared__ uint8_t copy_smem_raw[];
  __shared__ uint64_t s_src[kCopyAddrRing];   // 0: nothing to move for this piece
  __shared__ uint64_t s_dst[kCopyAddrRing];
  __shared__ uint32_t s_bytes[kCopyAddrRing];
  __shared__ __align__(8) uint64_t s_full[kCopyStages];
  __shared__ int s_abort;

  const uint32_t raw = smem_u32(copy_smem_raw);
  const uint32_t stage0 = (raw + 127u) & ~127u;
  const int lane = threadIdx.x;
  const long long total = (long long)p.n * p.runs_per_block * p.pieces_per_run * 2;
  // pieces of this CTA: blockIdx.x, blockIdx.x + gridDim.x, ...
  const long long mine = total > blockIdx.x ? (total - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;

  if (lane == 0) {
    s_abort = 0;
    for (int i = 0; i < kCopyStages; ++i) mbar_init(smem_u32(&s_full[i]), 1);
    fence_mbar_init();
  }
  __syncwarp();
  grid_dep_wait();    // launched programmatically: the preceding work may still produce the inputs
  grid_dep_launch();

  // Descriptors of pieces [t0, t0 + 32) of this CTA into the ring (one per lane).
  auto describe = [&](long long t0) {
    const long long t = t0 + lane;
    uint64_t sa = 0, da = 0;
    uint32_t nbytes = 0;
    if (t < mine) {
      const long long g = blockIdx.x + t * (long long)gridDim.x;
      const int q = (int)(g % p.pieces_per_run);
      const int r = (int)((g / p.pieces_per_run) % p.runs_per_block);
      const int kv = (int)((g / ((long long)p.pieces_per_run * p.runs_per_block)) & 1);
      const int i = (int)(g / ((long long)p.pieces_per_run * p.runs_per_block * 2));
      const int64_t sb = p.src.ids ? p.src.ids[i] : i;
      const int64_t db = p.dst.ids ? p.dst.ids[i] : i;
      if (sb >= 0 && sb < p.src.nb && db >= 0 && db < p.dst.nb) {
        const int64_t piece_off = (int64_t)q * (kCopyPieceBytes / 2);
        const uint16_t* sbase = kv ? p.src.v : p.src.k;
        uint16_t* dbase = kv ? p.dst.v : p.dst.k;
        sa = (uint64_t)(sbase + run_offset(p.src, p.run_level, p.bs, sb, r) + piece_off);
        da = (uint64_t)(dbase + run_offset(p.dst, p.run_level, p.bs, db, r) + piece_off);
        const int left = p.run_bytes - q * kCopyPieceBytes;
        nbytes = (uint32_t)(left < kCopyPieceBytes ? left : kCopyPieceBytes);
      } else if (p.status) {
        atomicOr(p.status, kStatusBadBlockId);
      }
    }
    const int e = (int)(t % kCopyAddrRing);
    s_src[e] = sa;
    s_dst[e] = da;
    s_bytes[e] = nbytes;
  };

  // lane 0: start the load of piece t (its stage is free)
  auto issue_load = [&](long long t) {
    const int e = (int)(t % kCopyAddrRing), slot = (int)(t % kCopyStages);
    const uint32_t bar = smem_u32(&s_full[slot]);
    if (s_src[e]) {
      mbar_arrive_expect_tx(bar, s_bytes[e]);
      bulk_g2s(stage0 + (uint32_t)slot * kCopyPieceBytes, (const void*)s_src[e], s_bytes[e], bar);
    } else {
      mbar_arrive(bar);  // skipped entry: the phase completes with nothing in the stage
    }
  };

  describe(0);
  describe(32);
  __syncwarp();
  constexpr int kAhead = kCopyStages - 1;
  bool ok = true;
  long long loads_issued = 0;
  if (lane == 0)
    for (long long t = 0; t < kAhead && t < mine; ++t, ++loads_issued) issue_load(t);

  for (long long t = 0; t < mine; ++t) {
    if (t > 0 && (t & 31) == 0) {  // entering a new batch: describe the one after it
      __syncwarp();                // lane 0 is done with the ring entries about to be overwritten
      describe(t + 32);
      __syncwarp();
    }
    if (lane == 0 && ok) {
      const int e = (int)(t % kCopyAddrRing), slot = (int)(t % kCopyStages);
      if (!mbar_wait_bounded(smem_u32(&s_full[slot]), (uint32_t)(t / kCopyStages) & 1u, &s_abort,
                             kCopyWaitLimitNs)) {
        ok = false;
      } else {
        if (s_src[e]) {
          fence_proxy_async_smem();
          bulk_s2g((void*)s_dst[e], stage0 + (uint32_t)slot * kCopyPieceBytes, s_bytes[e]);
        }
        bulk_commit();  // one group per piece (empty for a skipped entry) keeps the group count in step
        const long long tn = t + kAhead;
        if (tn < mine) {
          bulk_wait_read<1>();  // the store issued one piece ago has drained the stage piece tn reuses
          issue_load(tn);
          ++loads_issued;
        }
      }
    }
  }
  if (lane == 0) {
    if (!ok) {
      // a wait gave up: report it, then wait (bounded) for the loads still in flight
      if (p.status) atomicOr(p.status, kStatusWaitTimeout);
      int dummy = 0;
      for (long long t = loads_issued > kCopyStages ? loads_issued - kCopyStages : 0; t < loads_issued; ++t)
        mbar_wait_bounded(smem_u32(&s_full[t % kCopyStages]), (uint32_t)(t / kCopyStages) & 1u, &dummy,
                          kCopyWaitLimitNs / 8);
    }
    bulk_wait_all();
  }
}

}  // namespace ooco
