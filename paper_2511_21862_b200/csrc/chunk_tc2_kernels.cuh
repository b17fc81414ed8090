// Prefill-chunk attention over the paged cache on tcgen05, two row tiles per CTA (head_dim 128, bf16 cache, more than
// 128 score columns per (sequence, kv head)).  Same plan, merge and work items as chunk_tc_kernel
// (chunk_tc_kernels.cuh); a unit of work is (item, PAIR of 128-row tiles), one persistent CTA of 20 warps per SM:
//
//   warps 0..7    softmax of tile 0, warps 8..15 of tile 1: a warp owns 16 score rows (tensor-memory lanes), four
//                 threads share a row (16-lane tensor-memory shapes, quad shuffles)
//   warp 16       K producer: walks the units, TMA copies of the K slots (128 tokens: [half][128 tok][64 dims],
//                 128-byte swizzle), posts each stage's meta words and a descriptor of its V boxes
//   warp 17       V producer: TMA copies of the V slots from those descriptors
//   warps 18, 19  one lane of warp 18 + t issues the MMAs of tile t into the 512 tensor-memory columns:
//                   S_t[128 x 128]   = Q_t[128 x 128] . K_slot^T    8 x tcgen05.mma M128 N128 K16, both operands shared memory
//                   O_t[128 x 128] (+)= P_t[128 x 128] . V_slot      8 x tcgen05.mma M128 N128 K16, P from tensor memory,
//                                                                    V MN-major from the slot
//                 columns of tile t: S_t at 256 t (P_t, two bf16 per column, over its first 64 once the softmax
//                 threads have read S_t), O_t at 256 t + 128.  Q_t lives in shared memory (32 KiB per tile).
//
// Why this shape.  One thread gets an MMA issued about every 110 cycles whatever its size (measured: N 64 or 128, either
// operand source; N 256: 165), so MMAs should be as large as tensor memory allows (128-token slots: N = 128 for the
// scores) and each tile needs an issuing thread of its own (two issuers run side by side: one N = 128 MMA per 70
// cycles).  A tile's chain per stage is  scores -> softmax -> P.V -> next scores  (S_t(n+1) overwrites P_t(n), and the
// pipe executes one thread's MMAs in order, so P.V_t(n) is issued first; it also means P.V_t(n-1) is complete whenever
// S_t(n) is: a softmax thread may rescale its rows of O_t as soon as it holds the scores).  The chain is latency-bound,
// so the two tiles run half a stage apart -- the issuing warps keep the order S_0(n), S_1(n), S_0(n+1), ... -- and one
// tile's softmax runs beside the other tile's MMAs.  The tiles share every K / V slot.  Every wait is bounded; on a
// wait that gives up the CTA stops issuing, drains and releases the tensor memory.
#pragma once
#include "chunk_tc_kernels.cuh"

namespace ooco {

constexpr int kTc2StageTok = 128;                    // tokens of K (or V) per slot
constexpr int kTc2HalfBytes = kTc2StageTok * 128;    // [128 tok][64 dims] bf16
constexpr int kTc2SlotBytes = 2 * kTc2HalfBytes;     // K (or V) of one stage: 32 KiB
constexpr int kTc2QBytes = 2 * kTcRows * 128;        // one tile's queries: [half][128 rows][64 dims] bf16, 32 KiB
constexpr int kTc2Rows = 2 * kTcRows;                // score rows of a unit
constexpr int kTc2TmemCols = 512;
constexpr int kTc2KSlots = 2, kTc2VSlots = 3, kTc2MetaRing = 8;
constexpr int kTc2Threads = 20 * 32;               // 16 softmax warps, K producer, V producer, one MMA warp per tile
constexpr int kTc2RawSlotBytes = kTc2StageTok * 128;  // 8-bit cache: K (or V) codes of one stage, one 128-byte row per token

struct ChunkTc2Smem {
  __host__ __device__ static size_t total() {
    return 1024 + 2 * (size_t)kTc2QBytes + (size_t)(kTc2KSlots + kTc2VSlots) * kTc2SlotBytes + kTc2MetaRing * 32 +
           kTc2VSlots * sizeof(VStageDesc) + 512;
  }
};

// Barrier bookkeeping.  Stage number n (counted over the whole kernel, bookkeeping stages and the end marker
// included) uses K slot n % 2, V slot n % 3 (n % 2 over the 8-bit cache), meta entry n % 8 and, for each tile, barrier n & 1 of the pairs
// [2] below with phase parity (n >> 1) & 1 -- every tile takes a turn of its barriers on every stage, with or
// without work, so nobody can be overtaken by two completions of a barrier it waits on.
//
// KV8 (the caches hold E4M3 codes; one-tile mode only, the host launches nothing else): the TMA copies land 8-bit
// stages ([128 tok][128 B] of K, of V) in rings of their own -- two K slots in tile 1's Q region, two V slots in what
// is the third V slot otherwise -- and the eight warps that would be tile 1's softmax warps widen every stage into the
// 16-bit slot layout, exactly, to f16 holding value / 256 (e4m3x2_to_f16x2; the factor is part of the softmax scale
// and of the output scale), so both contractions run as kind::f16 MMAs with f16 operands (Q and P rounded to f16).
template <bool KV8>
__global__ void __launch_bounds__(kTc2Threads, 1)
chunk_tc2_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                 const DecodeParams p) {
  constexpr int D = 128;
  constexpr int NK = kTc2KSlots, NV = KV8 ? 2 : kTc2VSlots, NM = kTc2MetaRing;
  // One-tile mode: no work item has rows for tile 1 (at most 128 score columns).  The kernel is then bound by HBM,
  // not by the tensor pipe, and what would idle serves the one tile: tile 1's score columns are a second S buffer
  // and tile 1's issuing warp issues the P.V MMAs (see the MMA warps).  (Over a bf16 cache tile 1's Q region and
  // softmax warps stay idle: the region as a third K slot, and the warps taking half of every row's tokens, were
  // built and measured no faster.  Over the 8-bit cache they hold and widen the 8-bit slots.)
  const bool solo = p.GQ <= kTcRows;
  constexpr int kWarpK = 16, kWarpV = 17, kWarpM = 18;  // warps 0 .. 15: softmax; 18, 19: MMA of tile 0, 1
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* gen = smem_raw + (base - raw);
  const uint32_t s_q = base;                                       // [2] Q tiles
  const uint32_t s_k = s_q + 2u * kTc2QBytes;                      // [NK] K slots
  const uint32_t s_v = s_k + (uint32_t)NK * kTc2SlotBytes;         // [NV] V slots
  const uint32_t s_rk = s_q + kTc2QBytes;                          // KV8: [NK] 8-bit K slots (tile 1's Q region)
  const uint32_t s_rv = s_v + (uint32_t)NV * kTc2SlotBytes;        // KV8: [NV] 8-bit V slots (the third V slot's place)
  const uint32_t s_meta = s_v + (uint32_t)kTc2VSlots * kTc2SlotBytes;  // [NM] two int4 per stage
  const uint32_t s_vdesc = s_meta + (uint32_t)NM * 32;             // [NV] VStageDesc
  const uint32_t s_bar = s_vdesc + (uint32_t)kTc2VSlots * sizeof(VStageDesc);
  const uint32_t s_kfull = s_bar;                  // [NK] the K slot has landed                          (TMA)
  const uint32_t s_kempty = s_kfull + NK * 8;      // [NK] the score MMAs that read it are complete       (MMA commit)
  const uint32_t s_vfull = s_kempty + NK * 8;      // [NV] the V slot has landed                          (TMA)
  const uint32_t s_vempty = s_vfull + NV * 8;      // [NV] the P.V MMAs that read it are complete         (MMA commit)
  const uint32_t s_vdfull = s_vempty + NV * 8;     // [NV] the stage's V descriptor is posted             (K producer)
  const uint32_t s_mfull = s_vdfull + NV * 8;      // [NM] the stage's meta words are posted              (K producer)
  const uint32_t s_sready = s_mfull + NM * 8;      // [2 tiles][2] S_t holds the stage's scores            (MMA commit)
  const uint32_t s_pready = s_sready + 32;         // [2 tiles][2] P_t written, O_t rescaled, V rows clean (256 threads)
  const uint32_t s_pvdone = s_pready + 32;         // [2 tiles] the unit's last P.V_t is complete          (MMA commit)
  const uint32_t s_qready = s_pvdone + 16;         // [2 tiles] Q_t of the unit is in shared memory        (256 threads)
  const uint32_t s_pvstage = s_qready + 16;       // [2] one-tile mode: the stage's P.V is complete              (MMA commit)
  const uint32_t s_rkfull = s_pvstage + 16;       // KV8 [NK] the 8-bit K slot has landed                         (TMA)
  const uint32_t s_rkempty = s_rkfull + 16;       // KV8 [NK] the 8-bit K slot has been widened                   (256 threads)
  const uint32_t s_rvfull = s_rkempty + 16;       // KV8 [NV] the 8-bit V slot has landed                         (TMA)
  const uint32_t s_rvempty = s_rvfull + 16;       // KV8 [NV] the 8-bit V slot has been widened                   (256 threads)
  const uint32_t s_drain = s_rvempty + 16;
  const uint32_t s_slot = s_drain + 16;
  int4* g_meta = reinterpret_cast<int4*>(gen + (s_meta - base));
  VStageDesc* g_vdesc = reinterpret_cast<VStageDesc*>(gen + (s_vdesc - base));
  volatile uint32_t* g_slot = reinterpret_cast<volatile uint32_t*>(gen + (s_slot - base));
  volatile int* s_abort = reinterpret_cast<volatile int*>(gen + (s_slot + 4 - base));
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    *s_abort = 0;
    for (int i = 0; i < NK; ++i) {
      mbar_init(s_kfull + 8 * i, KV8 ? 256 : 1);  // (KV8: filled by the widening threads, not by TMA)
      mbar_init(s_kempty + 8 * i, solo ? 1 : 2);  // one arrival per MMA warp that reads K
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(s_rkfull + 8 * i, 1);
      mbar_init(s_rkempty + 8 * i, 256);
      mbar_init(s_rvfull + 8 * i, 1);
      mbar_init(s_rvempty + 8 * i, 256);
    }
    for (int i = 0; i < NV; ++i) {
      mbar_init(s_vfull + 8 * i, KV8 ? 256 : 1);
      mbar_init(s_vempty + 8 * i, solo ? 1 : 2);
      mbar_init(s_vdfull + 8 * i, 1);
    }
    for (int i = 0; i < NM; ++i) mbar_init(s_mfull + 8 * i, 1);
    for (int i = 0; i < 4; ++i) {
      mbar_init(s_sready + 8 * i, 1);
      mbar_init(s_pready + 8 * i, 256);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(s_pvdone + 8 * i, 1);
      mbar_init(s_qready + 8 * i, 256);
      mbar_init(s_pvstage + 8 * i, 1);
    }
    mbar_init(s_drain, 1);
    mbar_init(s_drain + 8, 1);
    fence_mbar_init();
  }
  if (warp == kWarpM) tmem_alloc(s_slot, kTc2TmemCols);
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = *g_slot;
  grid_dep_wait();    // the plan (and a fused append) must have completed
  grid_dep_launch();  // the merge kernel may queue up behind this grid

  const int nrt = (p.GQ + kTc2Rows - 1) / kTc2Rows;  // tile pairs per work item
  const long long cap_tokens = (long long)p.MB * p.bs;

  if (warp == kWarpK) {
    // ================================================================= K producer (and the walk over the units)
    if (lane == 0) prefetch_tmap(&tm_k);
    const long long n_units = (long long)p.hdr->n_items * nrt;
    const int boxes_per_stage = kTc2StageTok / p.tile_rows;   // at most 8 (blocks of 16 tokens)
    const uint32_t box_rows_bytes = (uint32_t)p.tile_rows * 128;
    int it = 0;
    bool ok = true, violated = false;
    long long unit = blockIdx.x;
    auto table_entry = [&](const int32_t* e) {
      const int v = *e;
      return checked(chk_table_entry(v, p.NB), &p.hdr->status, kStatusBadTableEntry) ? v : p.NB;
    };
    // waits until K slot, V slot (and with it the V descriptor) of stage `it` are free; false when a wait gave up
    auto acquire = [&]() {
      // (KV8: the slots the copies land in are the 8-bit ones, free once they have been widened)
      return warp_wait((KV8 ? s_rkempty : s_kempty) + 8 * (it % NK), (((uint32_t)(it / NK)) & 1u) ^ 1u, s_abort) &&
             warp_wait((KV8 ? s_rvempty : s_vempty) + 8 * (it % NV), (((uint32_t)(it / NV)) & 1u) ^ 1u, s_abort);
    };
    while (unit < n_units && ok) {
      int nxt = 0;
      if (lane == 0) nxt = atomicAdd(&p.hdr->next_item, 1);
      nxt = __shfl_sync(0xffffffffu, nxt, 0);
      // the last tile pair of an item sees the most tokens: it goes first (longest work first)
      const int item = (int)(unit / nrt), rt = nrt - 1 - (int)(unit - (long long)item * nrt);
      const int4 d = p.items[item];
      if (!checked(chk_item(d.x, d.y, d.z, d.w, p.B, p.max_items, cap_tokens), &p.hdr->status, kStatusBadItem)) {
        *s_abort = 1;
        violated = true;
        ok = false;
        break;
      }
      const int b = d.x, h = d.y % p.Hkv, t0 = d.z, t1 = d.w;
      long long T = p.context_lens[b];
      T = T < 0 ? 0 : (T > cap_tokens ? cap_tokens : T);
      const int lim_base = (int)T - p.Sq + 1;                      // tokens the first query token sees
      const int col_hi = min(p.GQ, (rt + 1) * kTc2Rows) - 1;
      const int t1e = min(t1, lim_base + col_hi / p.G);             // nothing beyond is visible to this tile pair
      const int nstage = t1e > t0 ? (t1e - t0 + kTc2StageTok - 1) / kTc2StageTok : 0;
      const int32_t* row = p.block_table + (size_t)b * p.MB;
      int blk_cur = 0;
      {
        const int tb = t0 + lane * p.tile_rows;
        if (lane < boxes_per_stage && tb < t1e) blk_cur = table_entry(row + tb / p.bs);
      }
      // a pair that sees nothing of this chunk passes one stage without tokens, which carries the bookkeeping
      for (int s = 0; s < (nstage > 0 ? nstage : 1); ++s, ++it) {
        const int tok0 = t0 + s * kTc2StageTok;
        const int ntok = nstage > 0 ? min(kTc2StageTok, t1e - tok0) : 0;
        const int nbox = (ntok + p.tile_rows - 1) / p.tile_rows;
        int blk_n = 0;  // table entries of the following stage, one stage ahead of their use
        {
          const int tb = tok0 + kTc2StageTok + lane * p.tile_rows;
          if (s + 1 < nstage && lane < boxes_per_stage && tb < t1e) blk_n = table_entry(row + tb / p.bs);
        }
        if (!acquire()) {
          ok = false;
          break;
        }
        const int ks = it % NK, vs = it % NV, ms = it % NM;
        const uint32_t kfull = (KV8 ? s_rkfull : s_kfull) + 8 * ks;
        if (lane == 0) {
          const int flags = (s == 0 ? 1 : 0) | (s == (nstage > 0 ? nstage : 1) - 1 ? 2 : 0);
          g_meta[2 * ms] = make_int4(d.y, b, h, ntok | (flags << 16));
          g_meta[2 * ms + 1] = make_int4(tok0, lim_base, t1, rt);
          g_vdesc[vs].nbox = nbox;
          g_vdesc[vs].h = h;
          if (nbox > 0)
            mbar_arrive_expect_tx(kfull, (KV8 ? 1u : 2u) * (uint32_t)nbox * box_rows_bytes);
          else
            mbar_arrive(kfull);
        }
        __syncwarp();
        bool span_ok = true;
        if (lane < nbox) {
          const int tb = tok0 + lane * p.tile_rows;
          const int c_tok = tb % p.bs;
          const uint32_t k0 = KV8 ? s_rk + (uint32_t)ks * kTc2RawSlotBytes : s_k + (uint32_t)ks * kTc2SlotBytes;
          const uint32_t dk = k0 + (uint32_t)lane * box_rows_bytes;
          span_ok = checked(chk_span(dk, box_rows_bytes, k0, (long long)k0 + kTc2HalfBytes) && chk_span(lane, 1, 0, 8),
                            &p.hdr->status, kStatusBadSmem);
          if (span_ok) {
            tma_load_4d(dk, &tm_k, kfull, 0, c_tok, h, blk_cur);  // (KV8: the row's 128 codes; else its first 64 dims)
            if (!KV8) tma_load_4d(dk + kTc2HalfBytes, &tm_k, kfull, 64, c_tok, h, blk_cur);
            g_vdesc[vs].blk[lane & 7] = blk_cur;
            g_vdesc[vs].c_tok[lane & 7] = c_tok;
          }
        }
        if (kChecked && !__all_sync(0xffffffffu, span_ok)) {  // a skipped copy leaves the stage incomplete: stop
          *s_abort = 1;
          violated = true;
          ok = false;
          break;
        }
        __syncwarp();
        if (lane == 0) {
          mbar_arrive(s_vdfull + 8 * vs);  // the V producer takes over the stage's V boxes
          mbar_arrive(s_mfull + 8 * ms);   // the softmax threads may read the meta words
        }
        blk_cur = blk_n;
      }
      unit = nxt;
    }
    if (ok) {  // end marker: one more stage, seen by every other warp
      if (acquire()) {
        if (lane == 0) {
          g_meta[2 * (it % NM)] = make_int4(-1, 0, 0, 0);
          g_vdesc[it % NV].nbox = -1;
          mbar_arrive((KV8 ? s_rkfull : s_kfull) + 8 * (it % NK));
          mbar_arrive(s_vdfull + 8 * (it % NV));
          mbar_arrive(s_mfull + 8 * (it % NM));
        }
        ++it;
      } else {
        ok = false;
      }
    }
    if (!ok) {  // stop path: record it, then wait (bounded) until every K copy already issued has landed
      if (lane == 0 && !violated) atomicOr(&p.hdr->status, kStatusWaitTimeout);
      int dummy_abort = 0;
      for (int k = 0; k < (it < NK ? it : NK); ++k) {
        const int j = it - 1 - k;
        mbar_wait_bounded((KV8 ? s_rkfull : s_kfull) + 8 * (j % NK), (uint32_t)(j / NK) & 1u, &dummy_abort, kWaitLimitNs / 8);
      }
    }
  } else if (warp == kWarpV) {
    // ================================================================= V producer
    if (lane == 0) prefetch_tmap(&tm_v);
    const uint32_t box_rows_bytes = (uint32_t)p.tile_rows * 128;
    int it = 0;
    bool ok = true;
    for (;; ++it) {
      const int vs = it % NV;
      if (!warp_wait(s_vdfull + 8 * vs, (uint32_t)(it / NV) & 1u, s_abort)) {
        ok = false;
        break;
      }
      const VStageDesc& vd = g_vdesc[vs];
      const int nbox = vd.nbox;
      const uint32_t vfull = (KV8 ? s_rvfull : s_vfull) + 8 * vs;
      if (nbox <= 0) {  // a stage without tokens, or the end marker
        if (lane == 0) mbar_arrive(vfull);
        if (nbox < 0) break;
        continue;
      }
      if (lane == 0) mbar_arrive_expect_tx(vfull, (KV8 ? 1u : 2u) * (uint32_t)nbox * box_rows_bytes);
      __syncwarp();
      if (lane < nbox && lane < 8) {
        const uint32_t dv = (KV8 ? s_rv + (uint32_t)vs * kTc2RawSlotBytes : s_v + (uint32_t)vs * kTc2SlotBytes) +
                            (uint32_t)lane * box_rows_bytes;
        tma_load_4d(dv, &tm_v, vfull, 0, vd.c_tok[lane], vd.h, vd.blk[lane]);
        if (!KV8) tma_load_4d(dv + kTc2HalfBytes, &tm_v, vfull, 64, vd.c_tok[lane], vd.h, vd.blk[lane]);
      }
    }
    if (!ok) {
      if (lane == 0) atomicOr(&p.hdr->status, kStatusWaitTimeout);
      int dummy_abort = 0;
      for (int k = 0; k < (it < NV ? it : NV); ++k) {
        const int j = it - 1 - k;
        mbar_wait_bounded((KV8 ? s_rvfull : s_vfull) + 8 * (j % NV), (uint32_t)(j / NV) & 1u, &dummy_abort, kWaitLimitNs / 8);
      }
    }
  } else if (warp >= kWarpM && solo) {
    // ================================================================= MMA warps, one-tile mode
    // One thread issues an MMA about every 100 cycles, so a single issuing thread needs longer for the 16 MMAs of a
    // stage than HBM needs for the stage's bytes.  With one tile the two issuing warps split the stage instead: warp
    // kWarpM issues the scores S(n) = Q . K_slot^T into S buffer n & 1 (columns 256 (n & 1); buffer 1 is what tile 1's
    // scores would occupy), warp kWarpM + 1 the values O += P(n) . V_slot.  The pipe keeps no order between two
    // threads' MMAs, so each hand-over has a barrier: S(n) overwrites P(n - 2), hence waits for P.V(n - 2) to be
    // complete (s_pvstage, one completion per stage, with or without tokens); P.V(n) waits for the softmax threads'
    // P(n).  The scores of a stage are thus computed while the softmax threads still work on the one before.
    const int t = warp - kWarpM;
    bool issued = false, ok = true;
    if (t == 0) {
      const uint32_t idesc_s = umma_idesc_16bit(kTcRows, kTc2StageTok, 0, !KV8);  // (KV8: f16 operands)
      const uint64_t dq = umma_smem_desc(s_q, 0, 1024);
      uint32_t n_q = 0;  // units with tokens (uses of the q-ready barrier)
      for (uint32_t n = 0;; ++n) {
        const int ks = n % NK, ms = n % NM;
        if (!warp_wait(s_kfull + 8 * ks, (n / NK) & 1u, s_abort)) {
          ok = false;
          break;
        }
        const int4 meta = g_meta[2 * ms];
        const bool end = meta.x < 0;
        const int ntok = end ? 0 : (meta.w & 0xffff);
        const bool first = !end && ((meta.w >> 16) & 1);
        // The buffer's previous contents, P(n - 2), have been consumed.  Waited for on every stage, with or without
        // tokens (the end marker included): it also means that the softmax threads are past their wait for S(n - 2),
        // so this stage's completion of the score barrier n & 1 cannot overtake them.
        if (n >= 2 && !warp_wait(s_pvstage + 8 * (n & 1), ((n - 2) >> 1) & 1u, s_abort)) {
          ok = false;
          break;
        }
        if (ntok > 0) {
          if (first) {
            if (!warp_wait(s_qready, n_q & 1u, s_abort)) {
              ok = false;
              break;
            }
            ++n_q;
          }
          tc_fence_after_sync();
          if (lane == 0) {
            const uint64_t dk = umma_smem_desc(s_k + (uint32_t)ks * kTc2SlotBytes, 0, 1024);
            const uint32_t ts = tmem + 256u * (n & 1);
#pragma unroll
            for (int hh = 0; hh < 2; ++hh)
#pragma unroll
              for (int k = 0; k < 4; ++k) {  // 16 dims = 32 bytes further along the rows; the second 64 dims = the next half
                const uint64_t off = (uint64_t)((hh * kTc2HalfBytes + k * 32) >> 4);
                umma_ss(ts, dq + off, dk + off, idesc_s, (hh | k) ? 1u : 0u);
              }
            umma_commit(s_sready + 8 * (n & 1));
            umma_commit(s_kempty + 8 * ks);
          }
          __syncwarp();
          issued = true;
        } else {
          // no scores: the turn of the barriers is taken all the same (also wakes the softmax threads for the end marker)
          if (lane == 0) {
            mbar_arrive(s_sready + 8 * (n & 1));
            mbar_arrive(s_kempty + 8 * ks);
          }
          __syncwarp();
        }
        if (end) break;
      }
    } else {
      const uint32_t idesc_o = umma_idesc_16bit(kTcRows, D, 1, !KV8);
      for (uint32_t n = 0;; ++n) {
        const int vs = n % NV, ms = n % NM;
        if (!warp_wait(s_mfull + 8 * ms, (n / NM) & 1u, s_abort)) {
          ok = false;
          break;
        }
        const int4 meta = g_meta[2 * ms];
        if (meta.x < 0) break;
        const int ntok = meta.w & 0xffff;
        const bool first = (meta.w >> 16) & 1, last = (meta.w >> 17) & 1;
        // the V slot first (normally there already), so that nothing but the MMAs follows the softmax threads' hand-over
        if ((ntok > 0 && !warp_wait(s_vfull + 8 * vs, (n / NV) & 1u, s_abort)) ||
            !warp_wait(s_pready + 8 * (n & 1), (n >> 1) & 1u, s_abort)) {
          ok = false;
          break;
        }
        if (ntok > 0) {
          tc_fence_after_sync();
          if (lane == 0) {
            const uint64_t dv = umma_smem_desc(s_v + (uint32_t)vs * kTc2SlotBytes, kTc2HalfBytes, 1024);
            const uint32_t tp = tmem + 256u * (n & 1);
#pragma unroll
            for (int k = 0; k < kTc2StageTok / 16; ++k)  // 16 tokens: 8 columns of P, 16 rows of 128 bytes of V in either half
              umma_ts(tmem + 128, tp + 8 * k, dv + (uint64_t)(k * (2048 >> 4)), idesc_o, (first && k == 0) ? 0u : 1u);
            if (last) umma_commit(s_pvdone);
            umma_commit(s_pvstage + 8 * (n & 1));
            umma_commit(s_vempty + 8 * vs);
          }
          __syncwarp();
          issued = true;
        } else {
          if (lane == 0) {
            if (last) mbar_arrive(s_pvdone);  // a unit without tokens: nothing to wait for
            mbar_arrive(s_pvstage + 8 * (n & 1));
            mbar_arrive(s_vempty + 8 * vs);
          }
          __syncwarp();
        }
      }
    }
    if (!ok && lane == 0) atomicOr(&p.hdr->status, kStatusWaitTimeout);
    if (!ok && issued) {  // the tensor memory must not be released under MMAs in flight
      if (lane == 0) umma_commit(s_drain + 8 * t);
      __syncwarp();
      int dummy = 0;
      mbar_wait_bounded(s_drain + 8 * t, 0u, &dummy, kWaitLimitNs / 8);
    }
  } else if (warp >= kWarpM) {
    // ================================================================= MMA warps: warp kWarpM + t issues tile t's MMAs
    // One thread issues an MMA about every 110 to 130 cycles whatever its size (measured: M128 N64 or N128 K16, either
    // operand source), twice what the pipe needs for N = 128, and the pipe overlaps the MMAs of two threads (two
    // issuers: one N = 128 MMA per 70 cycles).  So each tile has an issuing warp of its own; the order inside a tile,
    // P.V_t(n - 1) before S_t(n), is the program order of its thread, and the tiles need no order between them.
    const int t = warp - kWarpM;
    const uint32_t idesc_s = umma_idesc_16bit(kTcRows, kTc2StageTok, 0, true);
    const uint32_t idesc_o = umma_idesc_16bit(kTcRows, D, 1, true);
    const uint32_t ts = tmem + 256u * t;
    const uint64_t dq = umma_smem_desc(s_q + (uint32_t)t * kTc2QBytes, 0, 1024);
    uint32_t n_q = 0;  // units in which the tile had rows and tokens (uses of its q-ready barrier)
    bool issued = false, ok = true;
    // what is known about the stage whose P.V MMAs are still to be issued
    bool p_valid = false, p_act = false, p_first = false, p_last = false;
    int p_ntok = 0;
    uint32_t p_n = 0;
    for (uint32_t n = 0;; ++n) {
      const int ks = n % NK, ms = n % NM;
      if (!warp_wait(s_kfull + 8 * ks, (n / NK) & 1u, s_abort)) {
        ok = false;
        break;
      }
      const int4 meta = g_meta[2 * ms], meta2 = g_meta[2 * ms + 1];
      const bool end = meta.x < 0;
      const int ntok = end ? 0 : (meta.w & 0xffff);
      const bool first = !end && ((meta.w >> 16) & 1), last = !end && ((meta.w >> 17) & 1);
      const int rt = end ? 0 : meta2.w;
      const bool act = !end && (t == 0 || rt * kTc2Rows + kTcRows < p.GQ);  // a unit always has rows in its first tile
      // Everything that is normally there already is waited for first (the pending stage's V slot, the other tile's
      // turn: see below), so that nothing but the MMAs themselves follows the softmax threads' hand-over.
      if (p_valid && p_act && p_ntok > 0 && !warp_wait(s_vfull + 8 * (p_n % NV), (p_n / NV) & 1u, s_abort)) {
        ok = false;
        break;
      }
      // The tiles take turns, half a stage apart: S_0(n), S_1(n), S_0(n + 1), ... in this order, so that one tile's
      // softmax runs beside the other tile's MMAs (P.V of the stage before, then these scores) instead of both tiles
      // doing the same thing at once.  Tile 1 waits for tile 0's scores of this stage, tile 0 for tile 1's of the
      // stage before -- on every stage, with or without work, so that neither warp can get two turns ahead of the
      // other on a barrier pair.
      if (t == 1 ? !warp_wait(s_sready + 8 * (n & 1), (n >> 1) & 1u, s_abort)
                 : (n > 0 && !warp_wait(s_sready + 8 * (2 + ((n - 1) & 1)), ((n - 1) >> 1) & 1u, s_abort))) {
        ok = false;
        break;
      }
      // ---- P.V of the pending stage: waits for the tile's softmax threads, then issues (or just takes the turn)
      if (p_valid) {
        const int vs = p_n % NV;
        if (!warp_wait(s_pready + 8 * (2 * t + (p_n & 1)), (p_n >> 1) & 1u, s_abort)) {
          ok = false;
          break;
        }
        if (p_act && p_ntok > 0) {
          tc_fence_after_sync();
          if (lane == 0) {
            const uint64_t dv = umma_smem_desc(s_v + (uint32_t)vs * kTc2SlotBytes, kTc2HalfBytes, 1024);
#pragma unroll
            for (int k = 0; k < kTc2StageTok / 16; ++k)  // 16 tokens: 8 columns of P, 16 rows of 128 bytes of V in either half
              umma_ts(ts + 128, ts + 8 * k, dv + (uint64_t)(k * (2048 >> 4)), idesc_o, (p_first && k == 0) ? 0u : 1u);
            if (p_last) umma_commit(s_pvdone + 8 * t);
            umma_commit(s_vempty + 8 * vs);  // (one of the two arrivals that free the V slot)
          }
          __syncwarp();
          issued = true;
        } else {
          if (lane == 0) {
            if (p_act && p_last) mbar_arrive(s_pvdone + 8 * t);  // a unit without tokens: nothing to wait for
            mbar_arrive(s_vempty + 8 * vs);
          }
          __syncwarp();
        }
      }
      // ---- scores of this stage
      if (act && ntok > 0) {
        if (first) {
          if (!warp_wait(s_qready + 8 * t, n_q & 1u, s_abort)) {
            ok = false;
            break;
          }
          ++n_q;
        }
        tc_fence_after_sync();
        if (lane == 0) {
          const uint64_t dk = umma_smem_desc(s_k + (uint32_t)ks * kTc2SlotBytes, 0, 1024);
#pragma unroll
          for (int hh = 0; hh < 2; ++hh)
#pragma unroll
            for (int k = 0; k < 4; ++k) {  // 16 dims = 32 bytes further along the rows; the second 64 dims = the next half
              const uint64_t off = (uint64_t)((hh * kTc2HalfBytes + k * 32) >> 4);
              umma_ss(ts, dq + off, dk + off, idesc_s, (hh | k) ? 1u : 0u);
            }
          umma_commit(s_sready + 8 * (2 * t + (n & 1)));
          umma_commit(s_kempty + 8 * ks);  // (one of the two arrivals that free the K slot)
        }
        __syncwarp();
        issued = true;
      } else {
        // no scores for this tile: the turn of its barriers is taken all the same (also wakes the softmax threads
        // for the end marker)
        if (lane == 0) {
          mbar_arrive(s_sready + 8 * (2 * t + (n & 1)));
          mbar_arrive(s_kempty + 8 * ks);
        }
        __syncwarp();
      }
      if (end) break;
      p_valid = true;
      p_act = act;
      p_first = first;
      p_last = last;
      p_ntok = ntok;
      p_n = n;
    }
    if (!ok && lane == 0) atomicOr(&p.hdr->status, kStatusWaitTimeout);
    if (!ok && issued) {  // the tensor memory must not be released under MMAs in flight
      if (lane == 0) umma_commit(s_drain + 8 * t);
      __syncwarp();
      int dummy = 0;
      mbar_wait_bounded(s_drain + 8 * t, 0u, &dummy, kWaitLimitNs / 8);
    }
  } else {
    // ================================================================= softmax warps
    // Tile t = warps 8 t .. 8 t + 7.  Warp (q = warp & 3, hf = (warp >> 2) & 1) owns the 16 score rows
    // 32 q + 16 hf .. + 15 of the tile (a warp reaches the 32 tensor-memory lanes of its quarter q only) and reads
    // them in the 16-lane shape: lane (g, tq) holds rows g and g + 8, columns 8 i + 2 tq, + 1 -- two threads would be
    // too few per row to hide the latency of the row's chain, four share it here and combine with quad shuffles.
    const int t = warp >> 3, q4 = warp & 3, hf = (warp >> 2) & 1;
    const int g = lane >> 2, tq = lane & 3;
    const int row0 = 32 * q4 + 16 * hf + g;  // this thread's rows of the tile: row0 and row0 + 8
    const uint32_t trow = tmem + ((uint32_t)(32 * q4 + 16 * hf) << 16) + 256u * t;  // the warp's lanes, the tile's columns
    const int tid_t = threadIdx.x & 255;     // index among the tile's 256 threads
    // Score column (query token x head) of a tile's row r: column 4 (r % 32) + r / 32 of the tile, so that the columns
    // of a tile that is not full spread over the four lane quarters -- the warps with hf = 0 take rows before those with
    // hf = 1, one busy warp per scheduler -- and a warp none of whose rows is a column skips the stage's arithmetic.
    auto tile_col = [](int r) { return 4 * (r & 31) + (r >> 5); };
    uint8_t* q_gen = gen + (size_t)t * kTc2QBytes;
    float m_ref[2] = {-INFINITY, -INFINITY};  // reference maximum per row (scaled, log2 domain)
    float l_part[2] = {0.f, 0.f};             // this thread's share of the row's sum of weights
    int lim_row[2] = {0, 0};
    uint32_t n_unit = 0;  // units in which this tile had rows
    bool ok = true;
    bool q_ahead = false;  // the Q rows of the unit that starts with the next stage are in shared memory already
    // Q of tile pair `rt_` of (sequence b_, kv head h_) into the swizzled K-major tile ([half][row][64 dims], 16-byte
    // chunk ^= row & 7): thread i of the tile writes 64 dims (half i & 1) of row i >> 1; then the q-ready arrival
    auto load_q = [&](int b_, int h_, int rt_) {
      const int r_ = tid_t >> 1, half_ = tid_t & 1;
      const int col_ = rt_ * kTc2Rows + t * kTcRows + tile_col(r_);
      const int qi_ = col_ / p.G, head_ = col_ - qi_ * p.G;
      const bool real_ = col_ < p.GQ;
      const uint4* src = reinterpret_cast<const uint4*>(
          p.q + (((size_t)b_ * p.Sq + (real_ ? qi_ : 0)) * p.Hq + (size_t)h_ * p.G + (real_ ? head_ : 0)) * D + 64 * half_);
#pragma unroll
      for (int c = 0; c < 8; ++c) {
        uint4 v = real_ ? src[c] : make_uint4(0u, 0u, 0u, 0u);
        if (KV8) v = make_uint4(bf16x2_to_f16x2(v.x), bf16x2_to_f16x2(v.y), bf16x2_to_f16x2(v.z), bf16x2_to_f16x2(v.w));
        *reinterpret_cast<uint4*>(q_gen + (size_t)half_ * kTc2HalfBytes + (size_t)r_ * 128 + ((c ^ (r_ & 7)) << 4)) = v;
      }
      fence_proxy_async_smem();  // the tile is read by the MMAs through the async proxy
      mbar_arrive(s_qready + 8 * t);
    };
    if (KV8 && t == 1) {
      // ================================================================= widening warps (8-bit cache, one-tile mode)
      // Stage n of the 8-bit rings becomes stage n of the 16-bit slots (stages without tokens and the end marker take
      // their turns too).  A unit of work is (token row r, 16-byte chunk c of the row's 128 codes): one 16-byte load,
      // sixteen codes widened, two 16-byte stores into the row's 64-dim half c / 4; 1024 units per slot, four per
      // thread.  K first: the scores need it a stage earlier than P.V needs V.
      auto widen = [&](const uint8_t* rsrc, uint8_t* sdst, int ntok_) {
#pragma unroll
        for (int i = 0; i < kTc2StageTok * 8 / 256; ++i) {
          const int u = i * 256 + tid_t;
          const int r = u >> 3, c = u & 7;
          if (r >= ntok_) continue;  // rows beyond the stage's tokens are never used (masked scores, cleared V rows)
          const uint4 w = *reinterpret_cast<const uint4*>(rsrc + (size_t)r * 128 + ((c ^ (r & 7)) << 4));
          uint8_t* drow = sdst + (size_t)(c >> 2) * kTc2HalfBytes + (size_t)r * 128;
          *reinterpret_cast<uint4*>(drow + (((2 * (c & 3)) ^ (r & 7)) << 4)) =
              make_uint4(e4m3x2_to_f16x2<kSelB0B1>(w.x), e4m3x2_to_f16x2<kSelB2B3>(w.x), e4m3x2_to_f16x2<kSelB0B1>(w.y),
                         e4m3x2_to_f16x2<kSelB2B3>(w.y));
          *reinterpret_cast<uint4*>(drow + (((2 * (c & 3) + 1) ^ (r & 7)) << 4)) =
              make_uint4(e4m3x2_to_f16x2<kSelB0B1>(w.z), e4m3x2_to_f16x2<kSelB2B3>(w.z), e4m3x2_to_f16x2<kSelB0B1>(w.w),
                         e4m3x2_to_f16x2<kSelB2B3>(w.w));
        }
      };
      for (uint32_t n = 0;; ++n) {
        const int ks = n % NK, vs = n % NV, ms = n % NM;
        // the 8-bit K slot has landed (its meta words were written before its barrier was armed), the 16-bit one is free
        if (!warp_wait(s_rkfull + 8 * ks, (n / NK) & 1u, s_abort) ||
            !warp_wait(s_kempty + 8 * ks, ((n / NK) & 1u) ^ 1u, s_abort)) {
          ok = false;
          break;
        }
        const int4 meta = g_meta[2 * ms];
        const bool end = meta.x < 0;
        const int ntok = end ? 0 : (meta.w & 0xffff);
        if (ntok > 0) {
          widen(gen + (s_rk - base) + (size_t)ks * kTc2RawSlotBytes, gen + (s_k - base) + (size_t)ks * kTc2SlotBytes, ntok);
          fence_proxy_async_smem();  // the widened slot is read by the MMAs through the async proxy
        }
        mbar_arrive(s_kfull + 8 * ks);
        mbar_arrive(s_rkempty + 8 * ks);
        if (end) break;
        if (!warp_wait(s_rvfull + 8 * vs, (n / NV) & 1u, s_abort) ||
            !warp_wait(s_vempty + 8 * vs, ((n / NV) & 1u) ^ 1u, s_abort)) {
          ok = false;
          break;
        }
        if (ntok > 0) {
          widen(gen + (s_rv - base) + (size_t)vs * kTc2RawSlotBytes, gen + (s_v - base) + (size_t)vs * kTc2SlotBytes, ntok);
          fence_proxy_async_smem();
        }
        mbar_arrive(s_vfull + 8 * vs);
        mbar_arrive(s_rvempty + 8 * vs);
      }
    }
    for (uint32_t n = 0; !(solo && t == 1); ++n) {  // (one-tile mode: the warps of tile 1 have nothing else to do)
      const int ms = n % NM;
      if (!warp_wait(s_mfull + 8 * ms, (n / NM) & 1u, s_abort)) {
        ok = false;
        break;
      }
      const int4 meta = g_meta[2 * ms], meta2 = g_meta[2 * ms + 1];
      const bool end = meta.x < 0;
      const int ntok = end ? 0 : (meta.w & 0xffff);
      const bool first = !end && ((meta.w >> 16) & 1), last = !end && ((meta.w >> 17) & 1);
      const int b = meta.y, h = meta.z, rt = end ? 0 : meta2.w, lim_base = meta2.y;
      const bool act = !end && (t == 0 || rt * kTc2Rows + kTcRows < p.GQ);
      const int col0 = rt * kTc2Rows + t * kTcRows + tile_col(row0);  // score column of row0; that of row0 + 8: col0 + 32
      const bool warp_rows = rt * kTc2Rows + t * kTcRows + tile_col(32 * q4 + 16 * hf) < p.GQ;  // the warp's first column exists
      if (first && act) {
#pragma unroll
        for (int rr = 0; rr < 2; ++rr) {
          m_ref[rr] = -INFINITY;
          l_part[rr] = 0.f;
          lim_row[rr] = lim_base + (col0 + 32 * rr) / p.G;
        }
        if (ntok > 0 && !q_ahead) load_q(b, h, rt);
        q_ahead = false;
        ++n_unit;
      }
      if (!warp_wait(s_sready + 8 * (2 * t + (n & 1)), (n >> 1) & 1u, s_abort)) {
        ok = false;
        break;
      }
      if (end) break;
      if (act && ntok > 0 && warp_rows) {
        tc_fence_after_sync();
        // Two passes over the stage's scores, 64 tokens at a time (32 registers): the row maxima first, then, with the
        // reference maxima known, the weights.  Reading the scores twice costs little (tensor memory is close) and
        // keeps the threads clear of spills.  sh[4 i + 2 rr + c] = score of row (row0 + 8 rr), token 64 h2 + 8 i + 2 tq + c.
        // tokens [0, e) of the stage are visible to the row
        const int e0 = min(min(meta2.z, lim_row[0]) - meta2.x, ntok), e1 = min(min(meta2.z, lim_row[1]) - meta2.x, ntok);
        const bool masked = __any_sync(0xffffffffu, min(e0, e1) < kTc2StageTok);
        const uint32_t srow = trow + (solo ? 256u * (n & 1) : 0u);  // the stage's S (and P) columns
        auto load_half = [&](int h2, uint32_t (&sh)[32]) {
          tmem_ld_16x256b_x8(srow + 64 * h2, sh);
          tmem_ld_wait();
          if (masked) {
#pragma unroll
            for (int i = 0; i < 8; ++i)
#pragma unroll
              for (int c = 0; c < 2; ++c) {
                const int j = 64 * h2 + 8 * i + 2 * tq + c;
                if (j >= e0) sh[4 * i + c] = 0xff800000u;  // -inf
                if (j >= e1) sh[4 * i + 2 + c] = 0xff800000u;
              }
          }
        };
        float mxr[2] = {-INFINITY, -INFINITY};
#pragma unroll
        for (int h2 = 0; h2 < 2; ++h2) {
          uint32_t sh[32];
          load_half(h2, sh);
#pragma unroll
          for (int rr = 0; rr < 2; ++rr) {
            float ma = mxr[rr], mb = -INFINITY;
#pragma unroll
            for (int i = 0; i < 8; i += 2) {  // three-input maximum: two scores per instruction, two chains
              ma = fmax3(ma, __uint_as_float(sh[4 * i + 2 * rr]), __uint_as_float(sh[4 * i + 2 * rr + 1]));
              mb = fmax3(mb, __uint_as_float(sh[4 * i + 4 + 2 * rr]), __uint_as_float(sh[4 * i + 4 + 2 * rr + 1]));
            }
            mxr[rr] = fmaxf(ma, mb);
          }
        }
        float alpha[2] = {1.f, 1.f}, neg_mu[2];
        bool raise_any = false;
#pragma unroll
        for (int rr = 0; rr < 2; ++rr) {
          float mx = mxr[rr];
          mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
          mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
          mx *= p.scale_log2e;  // the scale is positive
          // reference maximum: raised only when the row maximum is more than kTcRescaleStep above it
          const bool raise = m_ref[rr] != -INFINITY && mx > m_ref[rr] + kTcRescaleStep;
          if (m_ref[rr] == -INFINITY) {
            m_ref[rr] = mx;  // nothing accumulated for this row so far
          } else if (raise) {
            alpha[rr] = ex2(m_ref[rr] - mx);
            m_ref[rr] = mx;
          }
          raise_any |= raise;
          neg_mu[rr] = m_ref[rr] == -INFINITY ? 0.f : -m_ref[rr];
        }
        if (__any_sync(0xffffffffu, raise_any)) {
          // P.V of the previous stage was issued before this stage's score MMAs, so it is complete: O may be rescaled
          // (one-tile mode: another thread issues it, so its own barrier is waited on; never on a unit's first stage)
          if (solo && !warp_wait(s_pvstage + 8 * ((n - 1) & 1), ((n - 1) >> 1) & 1u, s_abort)) {
            ok = false;
            break;
          }
          if (solo) tc_fence_after_sync();
#pragma unroll 1
          for (int c2 = 0; c2 < 2; ++c2) {
            uint32_t o[32];
            tmem_ld_16x256b_x8(trow + 128 + 64 * c2, o);
            tmem_ld_wait();
#pragma unroll
            for (int j = 0; j < 32; ++j) o[j] = __float_as_uint(__uint_as_float(o[j]) * alpha[(j >> 1) & 1]);
            tmem_st_16x256b_x8(trow + 128 + 64 * c2, o);
          }
          tmem_st_wait();
          l_part[0] *= alpha[0];
          l_part[1] *= alpha[1];
        }
        const float2 scale2 = make_float2(p.scale_log2e, p.scale_log2e);
        const float2 nm0 = make_float2(neg_mu[0], neg_mu[0]), nm1 = make_float2(neg_mu[1], neg_mu[1]);
        float2 add0 = {0.f, 0.f}, add1 = {0.f, 0.f};
#pragma unroll
        for (int h2 = 0; h2 < 2; ++h2) {  // 64 tokens at a time: 16 packed words of P per thread
          uint32_t sh[32];
          load_half(h2, sh);
          // (P of the first 64 tokens lands on score columns 0 .. 31, read by now; the second 64 tokens' scores, still
          // to be read, are columns 64 .. 127)
          uint32_t pw[16];  // pw[2 i + rr]: row (row0 + 8 rr), tokens 64 h2 + 8 i + 2 tq, + 1 = P column 32 h2 + 4 i + tq
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const int r = 4 * i;
            const float2 x0 = ffma2(make_float2(__uint_as_float(sh[r]), __uint_as_float(sh[r + 1])), scale2, nm0);
            const float2 x1 = ffma2(make_float2(__uint_as_float(sh[r + 2]), __uint_as_float(sh[r + 3])), scale2, nm1);
            const float2 w0 = make_float2(ex2(x0.x), ex2(x0.y)), w1 = make_float2(ex2(x1.x), ex2(x1.y));
            add0 = fadd2(add0, w0);
            add1 = fadd2(add1, w1);
            pw[2 * i] = KV8 ? pack_f16x2(w0.x, w0.y) : pack_bf16x2(w0.x, w0.y);
            pw[2 * i + 1] = KV8 ? pack_f16x2(w1.x, w1.y) : pack_bf16x2(w1.x, w1.y);
          }
          tmem_st_16x128b_x8(srow + 32 * h2, pw);
        }
        l_part[0] += add0.x + add0.y;
        l_part[1] += add1.x + add1.y;
        tmem_st_wait();
      }
      if (act && ntok > 0) {
        if (ntok < kTc2StageTok) {
          // V rows beyond the stage's tokens may hold anything (NaN included): clear them once the slot has landed
          const int vs = n % NV;
          if (!warp_wait(s_vfull + 8 * vs, (n / NV) & 1u, s_abort)) {
            ok = false;
            break;
          }
          uint8_t* vgen = gen + (s_v - base) + (size_t)vs * kTc2SlotBytes;
          for (int idx = tid_t; idx < (kTc2StageTok - ntok) * 16; idx += 256) {
            const int r = ntok + (idx >> 4), c = idx & 15;
            *reinterpret_cast<uint4*>(vgen + (size_t)(c >> 3) * kTc2HalfBytes + (size_t)r * 128 + ((c & 7) << 4)) =
                make_uint4(0u, 0u, 0u, 0u);
          }
          fence_proxy_async_smem();  // the cleared rows are read by the MMA through the async proxy
        }
        tc_fence_before_sync();
        __syncwarp();
      }
      mbar_arrive(s_pready + 8 * (2 * t + (n & 1)));

      if (last && act) {
        // The unit's last score MMAs are complete, so the tile's Q rows are free: when the next stage opens a unit
        // with rows in this tile, its Q goes to shared memory now and the score MMAs of that stage need not wait
        // for the epilogue below.
        {
          const int ms1 = (n + 1) % NM;
          if (!warp_wait(s_mfull + 8 * ms1, ((n + 1) / NM) & 1u, s_abort)) {
            ok = false;
            break;
          }
          const int4 nm = g_meta[2 * ms1], nm2 = g_meta[2 * ms1 + 1];
          if (nm.x >= 0 && (nm.w & 0xffff) > 0 && (t == 0 || nm2.w * kTc2Rows + kTcRows < p.GQ)) {
            load_q(nm.y, nm.z, nm2.w);
            q_ahead = true;
          }
        }
        // ---- the unit is complete: normalise the rows of O and write them
        const int slot_id = meta.x;
        const bool dst_ok = checked(chk_index(slot_id, p.max_items) && chk_index(b, p.B) && chk_index(h, p.Hkv),
                                    &p.hdr->status, kStatusBadIndex);
        const int n_chunks = dst_ok ? p.seq_first[b + 1] - p.seq_first[b] : 1;
        // use number n_unit - 1 of the tile's pv-done barrier
        if (!warp_wait(s_pvdone + 8 * t, (n_unit - 1) & 1u, s_abort)) {
          ok = false;
          break;
        }
        tc_fence_after_sync();
        const bool unit_has_tokens = ntok > 0;  // (a unit without tokens is one stage: nothing is in O)
        float inv[2], lse[2];
        __nv_bfloat16* orow[2];
        float* prow[2];
        bool write_row[2];
#pragma unroll
        for (int rr = 0; rr < 2; ++rr) {
          float l = l_part[rr];
          l += __shfl_xor_sync(0xffffffffu, l, 1);
          l += __shfl_xor_sync(0xffffffffu, l, 2);
          // l = 0: the row saw no token of this chunk; the 8-bit cache's V scale (and widening factor) comes in here
          inv[rr] = (l > 0.f ? 1.f / l : 0.f) * (KV8 ? p.v_scale : 1.f);
          lse[rr] = l > 0.f ? m_ref[rr] + lg2(l) : -INFINITY;
          const int col = col0 + 32 * rr;
          const int qi = col / p.G, head = col - qi * p.G;
          write_row[rr] = col < p.GQ && (!kChecked || dst_ok);
          orow[rr] = p.out + (((size_t)b * p.Sq + qi) * p.Hq + (size_t)h * p.G + head) * D;
          prow[rr] = p.part_o + ((size_t)slot_id * p.GQ + col) * D;
          if (write_row[rr] && tq == 0 && (n_chunks > 1 || p.out_f32)) p.part_lse[(size_t)slot_id * p.GQ + col] = lse[rr];
        }
#pragma unroll 1
        for (int c2 = 0; c2 < (warp_rows ? 2 : 0); ++c2) {
          uint32_t o[32];  // o[4 i + 2 rr + c] = row (row0 + 8 rr), dim 64 c2 + 8 i + 2 tq + c
          if (unit_has_tokens) {
            tmem_ld_16x256b_x8(trow + 128 + 64 * c2, o);
            tmem_ld_wait();
          } else {
#pragma unroll
            for (int j = 0; j < 32; ++j) o[j] = 0u;
          }
#pragma unroll
          for (int rr = 0; rr < 2; ++rr) {
            if (!write_row[rr]) continue;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              const float a = __uint_as_float(o[4 * i + 2 * rr]) * inv[rr], c = __uint_as_float(o[4 * i + 2 * rr + 1]) * inv[rr];
              const int dim = 64 * c2 + 8 * i + 2 * tq;
              if (n_chunks == 1 && !p.out_f32)
                *reinterpret_cast<uint32_t*>(orow[rr] + dim) = pack_bf16x2(a, c);
              else
                *reinterpret_cast<float2*>(prow[rr] + dim) = make_float2(a, c);
            }
          }
          __syncwarp();  // the tensor-memory loads are warp-wide: reconverge before the next one
        }
        tc_fence_before_sync();  // the next unit's first P.V overwrites O: ordered behind these reads by p-ready
      }
    }
    if (!ok && lane == 0) atomicOr(&p.hdr->status, kStatusWaitTimeout);
  }
  // ---- common exit: release the tensor memory once every warp is done with it
  tc_fence_before_sync();
  __syncthreads();
  if (warp == kWarpM) tmem_dealloc(tmem, kTc2TmemCols);
}

}  // namespace ooco
