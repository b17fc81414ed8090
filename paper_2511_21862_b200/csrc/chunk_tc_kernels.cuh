// Prefill-chunk attention over the paged cache on the 5th-generation tensor cores (tcgen05), head_dim 128, one
// 128-row tile per CTA and two CTAs per SM: every chunk over the 8-bit cache; over a bf16 cache the kernel of
// chunk_tc2_kernels.cuh runs by default and this one stays selectable.  Same units of work, producer warp, stage layout and
// meta words as chunk_main_kernel (chunk_kernels.cuh); row tiles are 128 score rows = the MMA's M.
//
//   warp 4      producer: TMA K / V stages of 64 tokens ([half][64 tok][64 dims], 128-byte swizzle)
//   warp 5      owns the tensor memory; one lane issues the MMAs, whose A operands live in tensor memory:
//                 S[128 x 64]   = Q[128 x 128] . K_stage^T      8 x tcgen05.mma M128 N64 K16, K K-major from the stage
//                 O[128 x 128] (+)= P[128 x 64] . V_stage        4 x tcgen05.mma M128 N128 K16, V MN-major from the stage
//               tensor-memory columns: S 0..63 (P, two bf16 per column, over its first 32 once the softmax
//               threads have read S), O 64..191, Q 192..255 -- shared memory holds nothing but the stages
//   warps 0..3  softmax: thread r owns score row r (tensor-memory lane r).  At the start of a unit it stores
//               its Q row into tensor memory.  Per stage it reads its S row, masks, keeps a reference maximum
//               that is only raised when the row maximum exceeds it by more than 8 (log2 units: the weights
//               stay below 2^8, and raising it means rescaling the row of O in tensor memory, which then
//               happens a few times per unit instead of once per stage), stores the bf16 weights as its P
//               row, and at the end of the unit normalises its O row and writes it.
// Every wait is bounded; on a wait that gives up the CTA stops issuing, drains and releases the tensor memory.
//
// KV8 (the caches hold E4M3 codes): the producer's TMA copies land the 8-bit stages ([64 tok][128 B] of K, then of
// V) in a ring of their own, and two more warps (6, 7) widen every stage into the 16-bit stage layout above --
// exactly, to f16 holding value / 256 (e4m3x2_to_f16x2; the factor goes into the softmax scale and the output
// scale) -- so both contractions run unchanged as kind::f16 MMAs with f16 operands (Q and P are rounded to f16, as
// in the 8-bit decode kernel).  The widening costs integer work on warps that do nothing else; the tensor pipe,
// not HBM, bounds this kernel, so the halved cache bytes buy capacity, not time.
#pragma once
#include "chunk_kernels.cuh"

namespace ooco {

constexpr int kTcRows = 128;        // score rows per row tile
constexpr int kTcTmemCols = 256;    // allocated columns (a power of two)
constexpr int kTcColS = 0, kTcColO = 64, kTcColQ = 192;
constexpr float kTcRescaleStep = 8.f;

constexpr int kTcRawStageBytes = 2 * kChunkStageTok * 128;  // 8-bit cache: K, then V, one 128-byte row per token
struct ChunkTcSmem {
  __host__ __device__ static size_t total(int nstages, int nraw = 0) {
    return 1024 + (size_t)nstages * (ChunkSmem<128>::kStageBytes + 32 + 16) + (size_t)nraw * (kTcRawStageBytes + 32 + 16) +
           128;
  }
};

// Barrier bookkeeping.  Barriers that come in pairs ([2]) are used alternately by consecutive stages, and use
// number n of a pair takes barrier n & 1 with phase parity (n >> 1) & 1: a waiter can then never be overtaken
// by two completions of the barrier it waits on (the completion after next needs the waiter's own progress).
template <bool KV8>
__global__ void __launch_bounds__(KV8 ? 256 : 192, 2)
chunk_tc_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                const DecodeParams p) {
  constexpr int D = 128;
  constexpr int kConvThreads = 64;  // KV8: warps 6 and 7
  using L = ChunkSmem<D>;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* gen = smem_raw + (base - raw);
  const int nst = p.nstages, nraw = KV8 ? p.nstages_raw : 0;
  const uint32_t s_stage = base;
  const uint32_t s_rstage = s_stage + (uint32_t)nst * L::kStageBytes;  // KV8: ring of 8-bit stages (1024-byte aligned)
  const uint32_t s_meta = s_rstage + (uint32_t)nraw * kTcRawStageBytes;
  const uint32_t s_rmeta = s_meta + (uint32_t)nst * 32;
  const uint32_t s_full = s_rmeta + (uint32_t)nraw * 32;
  const uint32_t s_empty = s_full + (uint32_t)nst * 8;
  const uint32_t s_rfull = s_empty + (uint32_t)nst * 8;   // KV8: the 8-bit stage has landed                (TMA)
  const uint32_t s_rempty = s_rfull + (uint32_t)nraw * 8;  // KV8: the 8-bit stage has been widened         (64 threads)
  const uint32_t s_sready = s_rempty + (uint32_t)nraw * 8;  // [2] S buffer holds the stage's scores       (MMA commit)
  const uint32_t s_sfree = s_sready + 16;                 // [2] S buffer has been read into registers  (128 softmax threads)
  const uint32_t s_pready = s_sfree + 16;                 // [2] meta words consumed, P written         (128 softmax threads)
  const uint32_t s_pvdone = s_pready + 16;                // [2] the stage's P.V is complete            (MMA commit)
  const uint32_t s_qready = s_pvdone + 16;                // Q of the unit is in shared memory          (128 softmax threads)
  const uint32_t s_drain = s_qready + 8;
  const uint32_t s_slot = s_drain + 8;
  int4* g_meta = reinterpret_cast<int4*>(gen + (s_meta - base));
  int4* g_rmeta = reinterpret_cast<int4*>(gen + (s_rmeta - base));
  volatile uint32_t* g_slot = reinterpret_cast<volatile uint32_t*>(gen + (s_slot - base));
  volatile int* s_abort = reinterpret_cast<volatile int*>(gen + (s_slot + 4 - base));
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    *s_abort = 0;
    for (int i = 0; i < nst; ++i) {
      mbar_init(s_full + 8 * i, KV8 ? kConvThreads : 1);  // KV8: filled by the widening threads, not by TMA
      mbar_init(s_empty + 8 * i, 1);
    }
    for (int i = 0; i < nraw; ++i) {
      mbar_init(s_rfull + 8 * i, 1);
      mbar_init(s_rempty + 8 * i, kConvThreads);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(s_sready + 8 * i, 1);
      mbar_init(s_sfree + 8 * i, 128);
      mbar_init(s_pready + 8 * i, 128);
      mbar_init(s_pvdone + 8 * i, 1);
    }
    mbar_init(s_qready, 128);
    mbar_init(s_drain, 1);
    fence_mbar_init();
  }
  if (warp == 5) tmem_alloc(s_slot, kTcTmemCols);
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = *g_slot;
  grid_dep_wait();    // the plan (and a fused append) must have completed
  grid_dep_launch();  // the merge kernel may queue up behind this grid

  if (warp == 4) {
    if (KV8)
      chunk_produce<D, true>(tm_k, tm_v, p, kTcRows, nraw, s_rstage, s_rfull, s_rempty, g_rmeta, s_abort, lane);
    else
      chunk_produce<D>(tm_k, tm_v, p, kTcRows, nst, s_stage, s_full, s_empty, g_meta, s_abort, lane);
  } else if (KV8 && warp >= 6) {
    // ================================================================= widening warps (8-bit cache only)
    // Stage number `it` of the 8-bit ring becomes stage number `it` of the 16-bit ring (bookkeeping stages and
    // the end marker included).  A unit of work is (tile K / V, token row r, 16-byte chunk c of the row's 128
    // codes): one 16-byte load, sixteen codes widened, two 16-byte stores into the row's 64-dim half c / 4.
    const int ctid = threadIdx.x - 192;
    const int nrw = KV8 ? nraw : 1;  // (this branch only exists for the 8-bit cache)
    bool ok = true;
    for (int it = 0;; ++it) {
      const int rs = it % nrw, slot = it % nst;
      if (!warp_wait(s_rfull + 8 * rs, (uint32_t)(it / nrw) & 1u, s_abort) ||
          !warp_wait(s_empty + 8 * slot, ((uint32_t)(it / nst) & 1u) ^ 1u, s_abort)) {
        ok = false;
        break;
      }
      const int4 meta = g_rmeta[2 * rs], meta2 = g_rmeta[2 * rs + 1];
      const int ntok = meta.x < 0 ? 0 : (meta.w & 0xffff);
      if (ntok > 0) {
        const uint8_t* rsrc = gen + (s_rstage - base) + (size_t)rs * kTcRawStageBytes;
        uint8_t* sdst = gen + (size_t)slot * L::kStageBytes;
#pragma unroll 4
        for (int i = 0; i < 2 * kChunkStageTok * 8 / kConvThreads; ++i) {
          const int u = i * kConvThreads + ctid;
          const int tile = u >> 9, r = (u >> 3) & 63, c = u & 7;
          if (r >= ntok) continue;  // rows beyond the stage's tokens are never used (masked scores, cleared V rows)
          const uint4 w = *reinterpret_cast<const uint4*>(rsrc + (size_t)tile * (kTcRawStageBytes / 2) + (size_t)r * 128 +
                                                          ((c ^ (r & 7)) << 4));
          uint8_t* drow = sdst + (size_t)tile * L::kTileBytes + (size_t)(c >> 2) * L::kHalfBytes + (size_t)r * 128;
          *reinterpret_cast<uint4*>(drow + (((2 * (c & 3)) ^ (r & 7)) << 4)) =
              make_uint4(e4m3x2_to_f16x2<kSelB0B1>(w.x), e4m3x2_to_f16x2<kSelB2B3>(w.x), e4m3x2_to_f16x2<kSelB0B1>(w.y),
                         e4m3x2_to_f16x2<kSelB2B3>(w.y));
          *reinterpret_cast<uint4*>(drow + (((2 * (c & 3) + 1) ^ (r & 7)) << 4)) =
              make_uint4(e4m3x2_to_f16x2<kSelB0B1>(w.z), e4m3x2_to_f16x2<kSelB2B3>(w.z), e4m3x2_to_f16x2<kSelB0B1>(w.w),
                         e4m3x2_to_f16x2<kSelB2B3>(w.w));
        }
      }
      if (ctid == 0) {
        g_meta[2 * slot] = meta;
        g_meta[2 * slot + 1] = meta2;
      }
      fence_proxy_async_smem();  // the widened stage is read by the MMAs through the async proxy
      mbar_arrive(s_full + 8 * slot);
      mbar_arrive(s_rempty + 8 * rs);
      if (meta.x < 0) break;
    }
    if (!ok && lane == 0) atomicOr(&p.hdr->status, kStatusWaitTimeout);
  } else if (warp == 5) {
    // ================================================================= MMA warp
    const uint32_t idesc_s = umma_idesc_16bit(kTcRows, kChunkStageTok, 0, !KV8);
    const uint32_t idesc_o = umma_idesc_16bit(kTcRows, D, 1, !KV8);
    uint32_t ph_q = 0, full_phase = 1u;
    uint32_t n_s = 0, n_p = 0, n_pv = 0;  // score MMAs issued, stages handed over by the softmax threads, P.V issued
    int slot = -1;
    bool issued = false, ok = true;
    // scores of the stage in `sl` (S also holds the previous stage's P: the tensor pipe runs in order, so these
    // MMAs start once the previous P.V has read it; the softmax threads have long read the previous scores)
    auto issue_scores = [&](int sl) {
      if (!warp_wait(s_sfree + 8 * (n_s & 1), ((n_s >> 1) & 1u) ^ 1u, s_abort)) return false;
      tc_fence_after_sync();
      if (lane == 0) {
        // (one descriptor per stage, advanced by adding to its address field: building one per MMA costs the issuing
        // thread more time than the MMA takes)
        const uint64_t dk = umma_smem_desc(s_stage + (uint32_t)sl * L::kStageBytes, 0, 1024);
#pragma unroll
        for (int h = 0; h < 2; ++h)
#pragma unroll
          for (int k = 0; k < 4; ++k)  // 16 dims of Q are 8 tensor-memory columns
            umma_ts(tmem + kTcColS, tmem + kTcColQ + 8 * (4 * h + k), dk + (uint64_t)((h * L::kHalfBytes + k * 32) >> 4), idesc_s,
                    (h | k) ? 1u : 0u);
        umma_commit(s_sready + 8 * (n_s & 1));
      }
      __syncwarp();
      ++n_s;
      issued = true;
      return true;
    };
    for (;;) {
      if (++slot == nst) slot = 0;
      if (slot == 0) full_phase ^= 1u;
      if (!warp_wait(s_full + 8 * slot, full_phase, s_abort)) {
        ok = false;
        break;
      }
      const int4 meta = g_meta[2 * slot];
      if (meta.x < 0) break;
      const int ntok = meta.w & 0xffff;
      const bool first = (meta.w >> 16) & 1;
      if (ntok > 0) {
        if (first) {
          if (!warp_wait(s_qready, ph_q, s_abort)) {
            ok = false;
            break;
          }
          ph_q ^= 1u;
        }
        if (!issue_scores(slot)) {
          ok = false;
          break;
        }
      }
      if (ntok == 0) {
        // a stage without tokens takes a turn of the S-buffer barriers as well, so that the softmax threads
        // can never be more than one stage ahead of this warp (see the note on barrier pairs)
        if (!warp_wait(s_sfree + 8 * (n_s & 1), ((n_s >> 1) & 1u) ^ 1u, s_abort)) {
          ok = false;
          break;
        }
        if (lane == 0) mbar_arrive(s_sready + 8 * (n_s & 1));
        __syncwarp();
        ++n_s;
      }
      // the softmax threads are done with this stage's meta words (and, with tokens, have written P)
      if (!warp_wait(s_pready + 8 * (n_p & 1), (n_p >> 1) & 1u, s_abort)) {
        ok = false;
        break;
      }
      ++n_p;
      if (ntok > 0) {
        tc_fence_after_sync();
        if (lane == 0) {
          const uint64_t dv = umma_smem_desc(s_stage + (uint32_t)slot * L::kStageBytes + L::kTileBytes, L::kHalfBytes, 1024);
#pragma unroll
          for (int k = 0; k < 4; ++k)  // 16 tokens: 8 columns of P, 16 rows of 128 bytes of V in either half
            umma_ts(tmem + kTcColO, tmem + kTcColS + 8 * k, dv + (uint64_t)(k * (2048 >> 4)), idesc_o,
                    (first && k == 0) ? 0u : 1u);
          umma_commit(s_empty + 8 * slot);
          umma_commit(s_pvdone + 8 * (n_pv & 1));
        }
        __syncwarp();
        ++n_pv;
      } else if (lane == 0) {
        mbar_arrive(s_empty + 8 * slot);
      }
    }
    if (!ok && lane == 0) atomicOr(&p.hdr->status, kStatusWaitTimeout);
    if (!ok && issued) {  // the tensor memory must not be released under MMAs in flight
      if (lane == 0) umma_commit(s_drain);
      __syncwarp();
      int dummy = 0;
      mbar_wait_bounded(s_drain, 0u, &dummy, kWaitLimitNs / 8);
    }
  } else {
    // ================================================================= softmax warps: thread = score row
    const int row = threadIdx.x;
    const uint32_t trow = tmem + ((uint32_t)(warp * 32) << 16);
    float m_ref = -INFINITY, l_run = 0.f;  // reference maximum (scaled, log2 domain), sum of the weights
    int lim_row = 0;
    uint32_t full_phase = 1u;
    uint32_t n_s = 0, n_pv = 0;  // stages seen so far (each takes a turn of the S and P barriers), stages with tokens
    int slot = -1;
    bool ok = true;
    // P.V number k is complete
    auto wait_pv = [&](uint32_t k) { return warp_wait(s_pvdone + 8 * (k & 1), (k >> 1) & 1u, s_abort); };
    for (;;) {
      if (++slot == nst) slot = 0;
      if (slot == 0) full_phase ^= 1u;
      if (!warp_wait(s_full + 8 * slot, full_phase, s_abort)) {
        ok = false;
        break;
      }
      const int4 meta = g_meta[2 * slot], meta2 = g_meta[2 * slot + 1];
      if (meta.x < 0) break;
      const int ntok = meta.w & 0xffff;
      const bool first = (meta.w >> 16) & 1, last = (meta.w >> 17) & 1;
      const int b = meta.y, h = meta.z, rt = meta2.w, lim_base = meta2.y;
      const int col = rt * kTcRows + row;
      const int qi = col / p.G, head = col - qi * p.G;
      const bool real_row = col < p.GQ;
      uint8_t* stage_gen = gen + (size_t)slot * L::kStageBytes;
      if (first) {
        m_ref = -INFINITY;
        l_run = 0.f;
        lim_row = lim_base + qi;
        if (ntok > 0) {  // this thread's Q row into the swizzled K-major tile
          const uint4* src = reinterpret_cast<const uint4*>(
              p.q + (((size_t)b * p.Sq + (real_row ? qi : 0)) * p.Hq + (size_t)h * p.G + (real_row ? head : 0)) * D);
#pragma unroll
          for (int half = 0; half < 2; ++half) {  // 64 dims = 32 columns of two bf16 each
            uint32_t qw[32];
#pragma unroll
            for (int c = 0; c < 8; ++c) {
              const uint4 v = real_row ? src[8 * half + c] : make_uint4(0u, 0u, 0u, 0u);
              qw[4 * c] = KV8 ? bf16x2_to_f16x2(v.x) : v.x;  // the widened codes are f16: so is the query
              qw[4 * c + 1] = KV8 ? bf16x2_to_f16x2(v.y) : v.y;
              qw[4 * c + 2] = KV8 ? bf16x2_to_f16x2(v.z) : v.z;
              qw[4 * c + 3] = KV8 ? bf16x2_to_f16x2(v.w) : v.w;
            }
            tmem_st32(trow + kTcColQ + 32 * half, qw);
          }
          tmem_st_wait();
          tc_fence_before_sync();
          mbar_arrive(s_qready);
        }
      }
      const uint32_t k_stage = n_s++;  // the stage is use k_stage of the S-buffer and P barriers
      if (!warp_wait(s_sready + 8 * (k_stage & 1), (k_stage >> 1) & 1u, s_abort)) {
        ok = false;
        break;
      }
      if (ntok == 0) mbar_arrive(s_sfree + 8 * (k_stage & 1));
      if (ntok > 0) {
        const uint32_t k_pv = n_pv++;  // this stage's P.V is number k_pv
        tc_fence_after_sync();
        uint32_t sr[2][32];
        tmem_ld32(trow + kTcColS, sr[0]);
        tmem_ld32(trow + kTcColS + 32, sr[1]);
        tmem_ld_wait();
        tc_fence_before_sync();
        mbar_arrive(s_sfree + 8 * (k_stage & 1));
        // tokens [0, e) of the stage are visible to this row
        const int e = min(min(meta2.z, lim_row) - meta2.x, ntok);
        if (e < kChunkStageTok) {
#pragma unroll
          for (int j = 0; j < 64; ++j)
            if (j >= e) sr[j >> 5][j & 31] = 0xff800000u;  // -inf
        }
        float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};  // four chains: the row is one thread's work
#pragma unroll
        for (int j = 0; j < 64; j += 2)  // three-input maximum: two scores per instruction
          mx4[(j >> 1) & 3] = fmax3(mx4[(j >> 1) & 3], __uint_as_float(sr[j >> 5][j & 31]),
                                    __uint_as_float(sr[(j + 1) >> 5][(j + 1) & 31]));
        const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * p.scale_log2e;  // the scale is positive
        // reference maximum: raised only when the row maximum is more than kTcRescaleStep above it
        const bool raise = m_ref != -INFINITY && mx > m_ref + kTcRescaleStep;
        float alpha = 1.f;
        if (m_ref == -INFINITY) {
          m_ref = mx;  // nothing accumulated for this row so far (its O row is 0 or not yet written)
        } else if (raise) {
          alpha = ex2(m_ref - mx);
          m_ref = mx;
        }
        if (__any_sync(0xffffffffu, raise)) {  // warp-uniform: the tensor-memory accesses are warp-wide
          if (!wait_pv(k_pv - 1)) {            // O must hold everything issued so far (never on a unit's first stage)
            ok = false;
            break;
          }
          tc_fence_after_sync();
#pragma unroll 1
          for (int c4 = 0; c4 < D / 32; ++c4) {
            uint32_t o[32];
            tmem_ld32(trow + kTcColO + 32 * c4, o);
            tmem_ld_wait();
#pragma unroll
            for (int j = 0; j < 32; ++j) o[j] = __float_as_uint(__uint_as_float(o[j]) * alpha);
            tmem_st32(trow + kTcColO + 32 * c4, o);
          }
          tmem_st_wait();
          l_run *= alpha;
        }
        const float neg_mu = m_ref == -INFINITY ? 0.f : -m_ref;
        float2 add4[4] = {{0.f, 0.f}, {0.f, 0.f}, {0.f, 0.f}, {0.f, 0.f}};
        const float2 scale2 = make_float2(p.scale_log2e, p.scale_log2e), neg_mu2 = make_float2(neg_mu, neg_mu);
        uint32_t pw[32];  // this row of P: 64 weights, two bf16 per word, in token order
#pragma unroll
        for (int i = 0; i < 32; ++i) {  // the scaling and the sums work on packed pairs: one instruction for two weights
          const int j = 2 * i;
          const float2 x = ffma2(make_float2(__uint_as_float(sr[j >> 5][j & 31]), __uint_as_float(sr[(j + 1) >> 5][(j + 1) & 31])),
                                 scale2, neg_mu2);
          const float2 w = make_float2(ex2(x.x), ex2(x.y));
          add4[i & 3] = fadd2(add4[i & 3], w);
          pw[i] = KV8 ? pack_f16x2(w.x, w.y) : pack_bf16x2(w.x, w.y);
        }
        {
          const float2 a01 = fadd2(add4[0], add4[1]), a23 = fadd2(add4[2], add4[3]);
          l_run += (a01.x + a01.y) + (a23.x + a23.y);
        }
        // over the first half of this row's scores (all of them are in registers by now)
        tmem_st32(trow + kTcColS, pw);
        tmem_st_wait();
        if (ntok < kChunkStageTok) {  // V rows beyond the stage's tokens may hold anything (NaN included): clear them
          uint8_t* vgen = stage_gen + L::kTileBytes;
          for (int idx = threadIdx.x; idx < (kChunkStageTok - ntok) * 16; idx += 128) {
            const int r = ntok + (idx >> 4), c = idx & 15;
            *reinterpret_cast<uint4*>(vgen + (size_t)(c >> 3) * L::kHalfBytes + (size_t)r * 128 + ((c & 7) << 4)) =
                make_uint4(0u, 0u, 0u, 0u);
          }
          fence_proxy_async_smem();  // the cleared rows are read by the MMA through the async proxy
        }
        tc_fence_before_sync();
        __syncwarp();
      }
      mbar_arrive(s_pready + 8 * (k_stage & 1));

      if (last) {
        // ---- the unit is complete: normalise this row of O and write it
        const int slot_id = meta.x;
        const bool dst_ok = checked(chk_index(slot_id, p.max_items) && chk_index(b, p.B) && chk_index(h, p.Hkv),
                                    &p.hdr->status, kStatusBadIndex);
        const int n_chunks = dst_ok ? p.seq_first[b + 1] - p.seq_first[b] : 1;
        const bool write_row = real_row && (!kChecked || dst_ok);
        if (ntok > 0) {
          if (!wait_pv(n_pv - 1)) {
            ok = false;
            break;
          }
          tc_fence_after_sync();
        }
        // l = 0: the row saw no token of this chunk; the 8-bit cache's V scale (and widening factor) comes in here
        const float inv = (l_run > 0.f ? 1.f / l_run : 0.f) * (KV8 ? p.v_scale : 1.f);
        __nv_bfloat16* orow = p.out + (((size_t)b * p.Sq + qi) * p.Hq + (size_t)h * p.G + head) * D;
        float* prow_o = p.part_o + ((size_t)slot_id * p.GQ + col) * D;
#pragma unroll 1
        for (int c4 = 0; c4 < D / 32; ++c4) {
          uint32_t o[32];
          if (ntok > 0) {
            tmem_ld32(trow + kTcColO + 32 * c4, o);
            tmem_ld_wait();
          } else {
#pragma unroll
            for (int j = 0; j < 32; ++j) o[j] = 0u;
          }
          if (write_row && n_chunks == 1 && !p.out_f32) {
#pragma unroll
            for (int v = 0; v < 4; ++v) {
              uint32_t w[4];
#pragma unroll
              for (int i = 0; i < 4; ++i)
                w[i] = pack_bf16x2(__uint_as_float(o[8 * v + 2 * i]) * inv, __uint_as_float(o[8 * v + 2 * i + 1]) * inv);
              *reinterpret_cast<uint4*>(orow + 32 * c4 + 8 * v) = make_uint4(w[0], w[1], w[2], w[3]);
            }
          } else if (write_row) {
#pragma unroll
            for (int v = 0; v < 8; ++v)
              *reinterpret_cast<float4*>(prow_o + 32 * c4 + 4 * v) =
                  make_float4(__uint_as_float(o[4 * v]) * inv, __uint_as_float(o[4 * v + 1]) * inv,
                              __uint_as_float(o[4 * v + 2]) * inv, __uint_as_float(o[4 * v + 3]) * inv);
          }
          __syncwarp();  // the tensor-memory loads are warp-wide: reconverge before the next one
        }
        if (write_row && (n_chunks > 1 || p.out_f32))
          p.part_lse[(size_t)slot_id * p.GQ + col] = l_run > 0.f ? m_ref + lg2(l_run) : -INFINITY;
        tc_fence_before_sync();  // the next unit's first P.V overwrites O: ordered behind these reads by q-ready
      }
    }
    if (!ok && lane == 0) atomicOr(&p.hdr->status, kStatusWaitTimeout);
  }
  // ---- common exit: release the tensor memory once every warp is done with it
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 5) tmem_dealloc(tmem, kTcTmemCols);
}

}  // namespace ooco
