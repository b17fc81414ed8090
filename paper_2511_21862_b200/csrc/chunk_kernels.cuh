// Paged attention of a prefill chunk for sm_100a: many query tokens per sequence (more than the 16
// score columns the decode kernel holds) over the paged cache, causal over the cache (Table "Operator
// Modeling", attention row with S_q > 1).
//
// The plan and the LSE merge are the decode path's (decode_kernels.cuh).  The score columns of a
// (sequence, kv head) pair -- column = query token * G + head of the group, G * q_len of them -- are cut
// into row tiles of 16 * NCW columns; a unit of work is (work item, row tile), where the item is the
// plan's (sequence, kv head, token chunk).  Here the roles of the two operands are the transpose of the
// decode kernel's: a consumer warp owns 16 score rows (query token x head) and walks over ALL tokens
// of a stage,
//   S[16 rows x 64 tok]  = Q (A, registers) x K_tile^T (B, ldmatrix)          mma.sync bf16
//   online softmax along the row (quad shuffles), P stays in registers as the next A operand
//   O[16 rows x D]      += P (A) x V_tile (B, ldmatrix.trans)                 mma.sync bf16
// so one CTA reads a K / V stage once for 16 * NCW rows.  A producer warp streams the stages through
// TMA (128-byte swizzle) exactly as in the decode kernel.  Tokens a row tile cannot see (causal limit)
// are never loaded; row tiles of one item run on neighbouring CTAs at about the same time, so the
// repeated K / V reads of the tiles hit L2.
#pragma once
#include "decode_kernels.cuh"

namespace ooco {

constexpr int kChunkStageTok = 64;  // tokens of K and of V per stage

template <int D>
struct ChunkSmem {
  static constexpr int kHalfBytes = kChunkStageTok * 128;          // [64 tok][64 dims] bf16
  static constexpr int kTileBytes = kHalfBytes * (D / 64);         // K (or V) of one stage: [D / 64][64][64]
  static constexpr int kStageBytes = 2 * kTileBytes;
  __host__ __device__ static size_t total(int nstages) {
    return 1024 + (size_t)nstages * (kStageBytes + 32 + 16) + 64;
  }
};

// One consumer warp on one stage.  kTail: some tokens of the stage are hidden from some of the warp's rows
// (causal limit, end of the chunk) or are not there at all (`ntok` < 64: rows beyond hold stale bytes).
//   e0 / e1   tokens [0, e) of the stage the lane's rows g / g + 8 may see
//   NTOK      tokens the call covers, starting at row 0 of `kst` / `vst`: a whole 64-token stage, or the
//             16-token slice of a warp that shares its rows with the other warps (row16_main_kernel)
template <int D, int NTOK, bool kTail>
__device__ __forceinline__ void chunk_consume(uint32_t kst, uint32_t vst, const uint32_t (&k_off)[2],
                                              const uint32_t (&v_off)[4], const uint32_t (&qf)[D / 16][4],
                                              float (&m_run)[2], float (&l_run)[2], float (&o_acc)[D / 8][4],
                                              float scale_log2e, int ntok, int e0, int e1, int t) {
  constexpr int KS = D / 16, NS = NTOK / 8, NO = D / 8;
  float s[NS][4];
#pragma unroll
  for (int j = 0; j < NS; ++j) s[j][0] = s[j][1] = s[j][2] = s[j][3] = 0.f;
  // ---- scores: two k-steps (32 dims) per ldmatrix
#pragma unroll
  for (int kp = 0; kp < KS / 2; ++kp) {
    const uint32_t ka = kst + (uint32_t)(kp >> 1) * ChunkSmem<D>::kHalfBytes + k_off[kp & 1];
#pragma unroll
    for (int j = 0; j < NS; j += 2) {  // two token tiles at a time: their MMAs do not depend on each other
      if (kTail && 8 * j >= ntok) continue;
      uint32_t b0, b1, b2, b3, c0, c1, c2, c3;
      ldmatrix_x4(ka + (uint32_t)j * 1024, b0, b1, b2, b3);
      ldmatrix_x4(ka + (uint32_t)(j + 1) * 1024, c0, c1, c2, c3);
      mma_bf16(s[j], qf[2 * kp][0], qf[2 * kp][1], qf[2 * kp][2], qf[2 * kp][3], b0, b1);
      mma_bf16(s[j + 1], qf[2 * kp][0], qf[2 * kp][1], qf[2 * kp][2], qf[2 * kp][3], c0, c1);
      mma_bf16(s[j], qf[2 * kp + 1][0], qf[2 * kp + 1][1], qf[2 * kp + 1][2], qf[2 * kp + 1][3], b2, b3);
      mma_bf16(s[j + 1], qf[2 * kp + 1][0], qf[2 * kp + 1][1], qf[2 * kp + 1][2], qf[2 * kp + 1][3], c2, c3);
    }
  }
  // ---- online softmax; lane (g, t) holds tokens 8j + 2t, + 1 of rows g (s[j][0..1]) and g + 8 (s[j][2..3])
  float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
  for (int j = 0; j < NS; ++j) {
#pragma unroll
    for (int e = 0; e < 4; ++e) s[j][e] *= scale_log2e;
    if (kTail) {
      const int c = 8 * j + 2 * t;
      if (c >= e0) s[j][0] = -INFINITY;
      if (c + 1 >= e0) s[j][1] = -INFINITY;
      if (c >= e1) s[j][2] = -INFINITY;
      if (c + 1 >= e1) s[j][3] = -INFINITY;
    }
    mx0 = fmaxf(mx0, fmaxf(s[j][0], s[j][1]));
    mx1 = fmaxf(mx1, fmaxf(s[j][2], s[j][3]));
  }
#pragma unroll
  for (int o = 1; o < 4; o <<= 1) {
    mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, o));
    mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, o));
  }
  const float mo0 = m_run[0], mo1 = m_run[1];
  float mn0 = fmaxf(mo0, mx0), mn1 = fmaxf(mo1, mx1);
  m_run[0] = mn0;
  m_run[1] = mn1;
  if (kTail) {  // a row that has seen nothing yet: keep the exponents finite
    mn0 = mn0 == -INFINITY ? 0.f : mn0;
    mn1 = mn1 == -INFINITY ? 0.f : mn1;
  }
  const float al0 = ex2(mo0 - mn0), al1 = ex2(mo1 - mn1);
  uint32_t pa[NS][2];
  float add0 = 0.f, add1 = 0.f;
#pragma unroll
  for (int j = 0; j < NS; ++j) {
    pa[j][0] = pack_bf16x2(ex2(s[j][0] - mn0), ex2(s[j][1] - mn0));
    pa[j][1] = pack_bf16x2(ex2(s[j][2] - mn1), ex2(s[j][3] - mn1));
    // sums use the rounded weights, so numerator and denominator agree exactly
    add0 += __uint_as_float(pa[j][0] << 16) + __uint_as_float(pa[j][0] & 0xffff0000u);
    add1 += __uint_as_float(pa[j][1] << 16) + __uint_as_float(pa[j][1] & 0xffff0000u);
  }
  l_run[0] = l_run[0] * al0 + add0;  // per lane: the quad's shares are added up in the epilogue
  l_run[1] = l_run[1] * al1 + add1;
  if (__any_sync(0xffffffffu, (al0 != 1.f) | (al1 != 1.f))) {
#pragma unroll
    for (int n = 0; n < NO; ++n) {
      o_acc[n][0] *= al0;
      o_acc[n][1] *= al0;
      o_acc[n][2] *= al1;
      o_acc[n][3] *= al1;
    }
  }
  // ---- values: 16 tokens per k-step, two 8-dim column tiles per ldmatrix
#pragma unroll
  for (int kk = 0; kk < NTOK / 16; ++kk) {
    if (kTail && 16 * kk >= ntok) continue;
    uint32_t mk01 = 0xffffffffu, mk23 = 0xffffffffu;
    if (kTail) {  // rows beyond the stage's tokens may hold anything (NaN included): clear them
      const int v = ntok - 16 * kk;
      mk01 = (2 * t < v ? 0x0000ffffu : 0u) | (2 * t + 1 < v ? 0xffff0000u : 0u);
      mk23 = (2 * t + 8 < v ? 0x0000ffffu : 0u) | (2 * t + 9 < v ? 0xffff0000u : 0u);
    }
    const uint32_t a0 = pa[2 * kk][0], a1 = pa[2 * kk][1], a2 = pa[2 * kk + 1][0], a3 = pa[2 * kk + 1][1];
#pragma unroll
    for (int np = 0; np < NO / 2; ++np) {
      uint32_t b0, b1, b2, b3;  // (tokens lo, dims 2np) (tokens hi, 2np) (tokens lo, 2np + 1) (tokens hi, 2np + 1)
      ldmatrix_x4_trans(vst + (uint32_t)(np >> 2) * ChunkSmem<D>::kHalfBytes + (uint32_t)kk * 2048 + v_off[np & 3], b0,
                        b1, b2, b3);
      if (kTail) {
        b0 &= mk01;
        b1 &= mk23;
        b2 &= mk01;
        b3 &= mk23;
      }
      mma_bf16(o_acc[2 * np], a0, a1, a2, a3, b0, b1);
      mma_bf16(o_acc[2 * np + 1], a0, a1, a2, a3, b2, b3);
    }
  }
}

// The producer warp of both kernels below: walks its units of work (item, row tile of RT score columns),
// streams the K / V stages of each through TMA and describes every stage in two int4 of `g_meta`:
//   {partial slot, sequence, kv head, tokens | first << 16 | last << 17}  {first token, T - S_q + 1, chunk end, row tile}
// KV8: the caches hold 8-bit codes; a stage is [64 tok][D bytes] of K, then of V (one 128-byte row per token at
// head_dim 128, one copy per box), for a consumer that widens it before use.
template <int D, bool KV8 = false>
__device__ __forceinline__ void chunk_produce(const CUtensorMap& tm_k, const CUtensorMap& tm_v, const DecodeParams& p,
                                              const int RT, const int nst, const uint32_t s_stage,
                                              const uint32_t s_full, const uint32_t s_empty, int4* g_meta,
                                              volatile int* s_abort, const int lane) {
  using L = ChunkSmem<D>;
  static_assert(!KV8 || D == 128, "the 8-bit stage layout is one 128-byte row per token");
  constexpr uint32_t kStageBytesP = KV8 ? 2u * kChunkStageTok * D : (uint32_t)L::kStageBytes;
  constexpr uint32_t kTileBytesP = KV8 ? (uint32_t)kChunkStageTok * D : (uint32_t)L::kTileBytes;
  constexpr uint32_t kCopiesPerBox = KV8 ? 1u : (uint32_t)(D / 64);
  const int nrt = (p.GQ + RT - 1) / RT;
  const long long n_units = (long long)p.hdr->n_items * nrt;
  // ================================================================= producer warp
  if (lane == 0) {
    prefetch_tmap(&tm_k);
    prefetch_tmap(&tm_v);
  }
  const int boxes_per_stage = kChunkStageTok / p.tile_rows;
  const uint32_t box_rows_bytes = (uint32_t)p.tile_rows * 128;  // one box of one 64-dim half
  const long long cap_tokens = (long long)p.MB * p.bs;
  int it = 0;
  bool ok = true;
  long long unit = blockIdx.x;
  // waits for stage `it`'s slot to be free; false when the wait gave up
  auto acquire = [&](int& slot) {
    slot = it % nst;
    return warp_wait(s_empty + 8 * slot, (((uint32_t)(it / nst)) & 1u) ^ 1u, s_abort);
  };
  // checked build: see the producer of decode_main_kernel
  auto table_entry = [&](const int32_t* e) {
    const int v = *e;
    return checked(chk_table_entry(v, p.NB), &p.hdr->status, kStatusBadTableEntry) ? v : p.NB;
  };
  bool violated = false;
  while (unit < n_units && ok) {
    int nxt = 0;
    if (lane == 0) nxt = atomicAdd(&p.hdr->next_item, 1);
    nxt = __shfl_sync(0xffffffffu, nxt, 0);
    // the last row tile of an item sees the most tokens: it goes first (longest work first)
    const int item = (int)(unit / nrt), rt = nrt - 1 - (int)(unit - (long long)item * nrt);
    const int4 d = p.items[item];
    if (!checked(chk_item(d.x, d.y, d.z, d.w, p.B, p.max_items, cap_tokens), &p.hdr->status, kStatusBadItem)) {
      *s_abort = 1;  // stop the CTA: the other warps leave through the abort flag
      violated = true;
      ok = false;
      break;
    }
    const int b = d.x, h = d.y % p.Hkv, t0 = d.z, t1 = d.w;
    long long T = p.context_lens[b];
    T = T < 0 ? 0 : (T > cap_tokens ? cap_tokens : T);
    const int lim_base = (int)T - p.Sq + 1;                       // tokens the first query token sees
    const int col_hi = min(p.GQ, (rt + 1) * RT) - 1;
    const int t1e = min(t1, lim_base + col_hi / p.G);              // nothing beyond is visible to this tile
    const int nstage = t1e > t0 ? (t1e - t0 + kChunkStageTok - 1) / kChunkStageTok : 0;
    const int32_t* row = p.block_table + (size_t)b * p.MB;
    int blk_cur = 0;
    {
      const int tb = t0 + lane * p.tile_rows;
      if (lane < boxes_per_stage && tb < t1e) blk_cur = table_entry(row + tb / p.bs);
    }
    if (nstage == 0) {  // the tile sees nothing of this chunk: one empty stage carries the bookkeeping
      int slot;
      if (!acquire(slot)) {
        ok = false;
        break;
      }
      if (lane == 0) {
        g_meta[2 * slot] = make_int4(d.y, b, h, 0 | (3 << 16));
        g_meta[2 * slot + 1] = make_int4(t0, lim_base, t1, rt);
        mbar_arrive(s_full + 8 * slot);
      }
      ++it;
    }
    for (int s = 0; s < nstage; ++s, ++it) {
      const int tok0 = t0 + s * kChunkStageTok;
      const int ntok = min(kChunkStageTok, t1e - tok0);
      const int nbox = (ntok + p.tile_rows - 1) / p.tile_rows;
      int blk_n = 0;  // table entries of the following stage, one stage ahead of their use
      {
        const int tb = tok0 + kChunkStageTok + lane * p.tile_rows;
        if (s + 1 < nstage && lane < boxes_per_stage && tb < t1e) blk_n = table_entry(row + tb / p.bs);
      }
      int slot;
      if (!acquire(slot)) {
        ok = false;
        break;
      }
      const uint32_t full = s_full + 8 * slot;
      if (lane == 0) {
        const int flags = (s == 0 ? 1 : 0) | (s == nstage - 1 ? 2 : 0);
        g_meta[2 * slot] = make_int4(d.y, b, h, ntok | (flags << 16));
        g_meta[2 * slot + 1] = make_int4(tok0, lim_base, t1, rt);
        mbar_arrive_expect_tx(full, 2u * (uint32_t)nbox * box_rows_bytes * kCopiesPerBox);
      }
      __syncwarp();
      bool span_ok = true;
      if (lane < nbox) {
        const int tb = tok0 + lane * p.tile_rows;
        const int c_tok = tb % p.bs;
        const uint32_t dk = s_stage + (uint32_t)slot * kStageBytesP + (uint32_t)lane * box_rows_bytes;
        const uint32_t dv = dk + kTileBytesP;
        // checked build: the box lands inside the first 64-dim half of the stage's K tile (the others follow it)
        span_ok = checked(chk_span(dk, box_rows_bytes, s_stage + (long long)slot * kStageBytesP,
                                   s_stage + (long long)slot * kStageBytesP + L::kHalfBytes) &&
                              chk_span(slot, 1, 0, nst),
                          &p.hdr->status, kStatusBadSmem);
        if (span_ok && KV8) {
          tma_load_4d(dk, &tm_k, full, 0, c_tok, h, blk_cur);
          tma_load_4d(dv, &tm_v, full, 0, c_tok, h, blk_cur);
        } else if (span_ok) {
#pragma unroll
          for (int j = 0; j < D / 64; ++j) {
            tma_load_4d(dk + j * L::kHalfBytes, &tm_k, full, 64 * j, c_tok, h, blk_cur);
            tma_load_4d(dv + j * L::kHalfBytes, &tm_v, full, 64 * j, c_tok, h, blk_cur);
          }
        }
      }
      if (kChecked && !__all_sync(0xffffffffu, span_ok)) {  // a skipped copy leaves the stage incomplete: stop
        *s_abort = 1;
        violated = true;
        ok = false;
        break;
      }
      blk_cur = blk_n;
    }
    unit = nxt;
  }
  if (ok) {  // end marker (one stage, seen by every consumer warp)
    int slot;
    if (acquire(slot)) {
      if (lane == 0) {
        g_meta[2 * slot] = make_int4(-1, 0, 0, 0);
        mbar_arrive(s_full + 8 * slot);
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
    const int pending = it < nst ? it : nst;
    for (int k = 0; k < pending; ++k) {
      const int j = it - 1 - k;
      mbar_wait_bounded(s_full + 8 * (j % nst), (uint32_t)(j / nst) & 1u, &dummy_abort, kWaitLimitNs / 8);
    }
  }
}

// NCW consumer warps (16 score rows each) + one producer warp.  p.grid_main is the number of CTAs the
// plan sized its chunks for (not this grid); the work counter starts at this grid's size.
template <int D, int NCW>
__global__ void __launch_bounds__((NCW + 1) * 32, NCW == 8 ? 1 : 2)
chunk_main_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                  const DecodeParams p) {
  using L = ChunkSmem<D>;
  constexpr int RT = 16 * NCW;  // score rows (columns of the decode kernel) per row tile
  constexpr int KS = D / 16, NO = D / 8;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* gen = smem_raw + (base - raw);
  const int nst = p.nstages;
  const uint32_t s_stage = base;
  const uint32_t s_meta = s_stage + (uint32_t)nst * L::kStageBytes;
  const uint32_t s_full = s_meta + (uint32_t)nst * 32;
  const uint32_t s_empty = s_full + (uint32_t)nst * 8;
  int4* g_meta = reinterpret_cast<int4*>(gen + (s_meta - base));
  volatile int* s_abort = reinterpret_cast<volatile int*>(gen + (s_empty + (uint32_t)nst * 8 - base));
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    *s_abort = 0;
    for (int i = 0; i < nst; ++i) {
      mbar_init(s_full + 8 * i, 1);
      mbar_init(s_empty + 8 * i, NCW);
    }
    fence_mbar_init();
  }
  __syncthreads();
  grid_dep_wait();    // the plan (and a fused append) must have completed
  grid_dep_launch();  // the merge kernel may queue up behind this grid

  if (warp == NCW) {
    chunk_produce<D>(tm_k, tm_v, p, RT, nst, s_stage, s_full, s_empty, g_meta, s_abort, lane);
    return;
  }

  // =================================================================== consumer warps
  const int g = lane >> 2, t = lane & 3;
  // per-lane ldmatrix offsets inside a stage's K / V tile ([half][64 tok][64 dims], 16-byte chunk ^= row & 7)
  const int lane_row = lane & 7, mi = lane >> 3;
  uint32_t k_off[2], v_off[4];
  {
    // K: matrix mi = 16-byte chunk 4 kp + mi of rows 8 j + lane_row (two k-steps of one 8-token tile)
    const uint32_t pat = (uint32_t)((mi ^ lane_row) << 4);
    k_off[0] = (uint32_t)lane_row * 128 + pat;
    k_off[1] = (uint32_t)lane_row * 128 + (pat ^ 64u);
    // V: matrices (tokens lo, chunk 2 np) (tokens hi, 2 np) (tokens lo, 2 np + 1) (tokens hi, 2 np + 1)
    const uint32_t vrow = (uint32_t)((mi & 1) * 8 + lane_row) * 128;
    const uint32_t vx = (uint32_t)(((mi >> 1) ^ lane_row) << 4);
#pragma unroll
    for (int i = 0; i < 4; ++i) v_off[i] = vrow + (((uint32_t)i * 32u) ^ vx);
  }
  float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
  float o_acc[NO][4];
  uint32_t qf[KS][4];
#pragma unroll
  for (int n = 0; n < NO; ++n) o_acc[n][0] = o_acc[n][1] = o_acc[n][2] = o_acc[n][3] = 0.f;
#pragma unroll
  for (int k = 0; k < KS; ++k) qf[k][0] = qf[k][1] = qf[k][2] = qf[k][3] = 0u;
  int lim_row0 = 0, lim_row1 = 0;  // tokens of the whole context the lane's two rows may see

  int slot = -1;
  uint32_t full_phase = 1u;
  for (;;) {
    if (++slot == nst) slot = 0;
    if (slot == 0) full_phase ^= 1u;
    if (!warp_wait(s_full + 8 * slot, full_phase, s_abort)) {
      if (lane == 0) atomicOr(&p.hdr->status, kStatusWaitTimeout);
      return;
    }
    const int4 meta = g_meta[2 * slot], meta2 = g_meta[2 * slot + 1];
    if (meta.x < 0) break;
    const int ntok = meta.w & 0xffff;
    const bool first = (meta.w >> 16) & 1, last = (meta.w >> 17) & 1;
    const int b = meta.y, h = meta.z, rt = meta2.w, lim_base = meta2.y;
    const int colw = rt * RT + 16 * warp;  // first score column of this warp
    const bool live = colw < p.GQ;          // a warp whose rows all lie beyond the last column idles
    if (first) {
      m_run[0] = m_run[1] = -INFINITY;
      l_run[0] = l_run[1] = 0.f;
#pragma unroll
      for (int n = 0; n < NO; ++n) o_acc[n][0] = o_acc[n][1] = o_acc[n][2] = o_acc[n][3] = 0.f;
      const int c0 = colw + g, c1 = c0 + 8;
      const int qi0 = c0 / p.G, qi1 = c1 / p.G;
      lim_row0 = lim_base + qi0;
      lim_row1 = lim_base + qi1;
      if (live) {
        const __nv_bfloat16* q0 = p.q + (((size_t)b * p.Sq + qi0) * p.Hq + (size_t)h * p.G + (c0 - qi0 * p.G)) * D;
        const __nv_bfloat16* q1 = p.q + (((size_t)b * p.Sq + qi1) * p.Hq + (size_t)h * p.G + (c1 - qi1 * p.G)) * D;
        const bool ok0 = c0 < p.GQ, ok1 = c1 < p.GQ;
#pragma unroll
        for (int k = 0; k < KS; ++k) {
          qf[k][0] = ok0 ? *reinterpret_cast<const uint32_t*>(q0 + 16 * k + 2 * t) : 0u;
          qf[k][1] = ok1 ? *reinterpret_cast<const uint32_t*>(q1 + 16 * k + 2 * t) : 0u;
          qf[k][2] = ok0 ? *reinterpret_cast<const uint32_t*>(q0 + 16 * k + 8 + 2 * t) : 0u;
          qf[k][3] = ok1 ? *reinterpret_cast<const uint32_t*>(q1 + 16 * k + 8 + 2 * t) : 0u;
        }
      }
    }
    if (live && ntok > 0) {
      const int tok0 = meta2.x, t1 = meta2.z;
      const int e0 = min(t1, lim_row0) - tok0, e1 = min(t1, lim_row1) - tok0;
      // warp-uniform bounds: the first row sees the fewest tokens, the last (real) row the most
      const int e_first = min(t1, lim_base + colw / p.G) - tok0;
      const int e_last = min(t1, lim_base + min(colw + 15, p.GQ - 1) / p.G) - tok0;
      if (e_last > 0) {
        const uint32_t kst = s_stage + (uint32_t)slot * L::kStageBytes;
        const uint32_t vst = kst + L::kTileBytes;
        if (e_first >= kChunkStageTok)
          chunk_consume<D, kChunkStageTok, false>(kst, vst, k_off, v_off, qf, m_run, l_run, o_acc, p.scale_log2e, ntok, e0, e1, t);
        else
          chunk_consume<D, kChunkStageTok, true>(kst, vst, k_off, v_off, qf, m_run, l_run, o_acc, p.scale_log2e, ntok, e0, e1, t);
      }
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(s_empty + 8 * slot);

    if (last && live) {
      // ---- the warp's 16 rows are complete for this item: normalise and write them
      const int slot_id = meta.x;
      const bool dst_ok = checked(chk_index(slot_id, p.max_items) && chk_index(b, p.B) && chk_index(h, p.Hkv),
                                  &p.hdr->status, kStatusBadIndex);
      const int n_chunks = dst_ok ? p.seq_first[b + 1] - p.seq_first[b] : 1;
      float l0 = l_run[0], l1 = l_run[1];
#pragma unroll
      for (int o = 1; o < 4; o <<= 1) {
        l0 += __shfl_xor_sync(0xffffffffu, l0, o);
        l1 += __shfl_xor_sync(0xffffffffu, l1, o);
      }
#pragma unroll
      for (int r = 0; r < 2; ++r) {
        const int col = colw + g + 8 * r;
        if (col >= p.GQ || (kChecked && !dst_ok)) continue;
        const float l = r ? l1 : l0, m = r ? m_run[1] : m_run[0];
        const float inv = l > 0.f ? 1.f / l : 0.f;  // l = 0: the row saw no token of this chunk
        if (n_chunks == 1 && !p.out_f32) {
          const int qi = col / p.G, head = col - qi * p.G;
          __nv_bfloat16* dst = p.out + (((size_t)b * p.Sq + qi) * p.Hq + (size_t)h * p.G + head) * D + 2 * t;
#pragma unroll
          for (int n = 0; n < NO; ++n)
            *reinterpret_cast<__nv_bfloat162*>(dst + 8 * n) =
                __floats2bfloat162_rn(o_acc[n][2 * r] * inv, o_acc[n][2 * r + 1] * inv);
        } else {
          float* dst = p.part_o + ((size_t)slot_id * p.GQ + col) * D + 2 * t;
#pragma unroll
          for (int n = 0; n < NO; ++n)
            *reinterpret_cast<float2*>(dst + 8 * n) = make_float2(o_acc[n][2 * r] * inv, o_acc[n][2 * r + 1] * inv);
          if (t == 0) p.part_lse[(size_t)slot_id * p.GQ + col] = l > 0.f ? m + lg2(l) : -INFINITY;
        }
      }
    }
  }
}

// ------------------------------------------------------------------------------------ 9 .. 16 score columns
// Up to 16 score columns (one 16-row tile), too few to give every warp rows of its own: the NCW consumer
// warps share the tile's rows and split the TOKENS of each 64-token stage, 16 per warp, in the row layout
// above (the decode kernel's column layout needs a second 8-column MMA tile and a transposition per tile
// for more than 8 columns).  Each warp keeps its own running maximum, sum and O[16 x D]; when an item ends
// the warps combine through shared memory and write the rows.  The scratch for that is the item's last
// stage itself: the K / V rows a warp alone reads (its 16-token slices) are exactly as large as its fp32
// O tile, so it overwrites them right after its last MMA, one mbarrier phase later every warp reads all
// four tiles, and only then is the stage handed back to the producer.
template <int NCW>
struct Row16Smem {
  static constexpr int kStatBytes = 2 * NCW * 16 * 2 * 4;  // running maximum and sum per (warp, row), two item parities
  template <int D>
  __host__ __device__ static size_t total(int nstages) {
    return 1024 + (size_t)nstages * (ChunkSmem<D>::kStageBytes + 32 + 16) + kStatBytes + 64;
  }
};

template <int D, int NCW>
__global__ void __launch_bounds__((NCW + 1) * 32, 2)
row16_main_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                  const DecodeParams p) {
  static_assert(NCW * 16 == kChunkStageTok, "one 16-token slice of a stage per consumer warp");
  using L = ChunkSmem<D>;
  using M = Row16Smem<NCW>;
  constexpr int KS = D / 16, NO = D / 8;
  constexpr int kRowBytes = D * 4;                // one fp32 row of a warp's O tile
  constexpr int kRowsPerPiece = 2048 / kRowBytes; // a warp's slice of one 64-dim half of K or V is 2 KiB
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* gen = smem_raw + (base - raw);
  const int nst = p.nstages;
  const uint32_t s_stage = base;
  const uint32_t s_merge = s_stage + (uint32_t)nst * L::kStageBytes;
  const uint32_t s_meta = s_merge + M::kStatBytes;
  const uint32_t s_full = s_meta + (uint32_t)nst * 32;
  const uint32_t s_empty = s_full + (uint32_t)nst * 8;
  const uint32_t s_mbar = s_empty + (uint32_t)nst * 8;
  float* g_stat = reinterpret_cast<float*>(gen + (s_merge - base));
  int4* g_meta = reinterpret_cast<int4*>(gen + (s_meta - base));
  volatile int* s_abort = reinterpret_cast<volatile int*>(gen + (s_mbar + 8 - base));
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    *s_abort = 0;
    for (int i = 0; i < nst; ++i) {
      mbar_init(s_full + 8 * i, 1);
      mbar_init(s_empty + 8 * i, NCW);
    }
    mbar_init(s_mbar, NCW * 32);
    fence_mbar_init();
  }
  __syncthreads();
  grid_dep_wait();    // the plan (and a fused append) must have completed
  grid_dep_launch();  // the merge kernel may queue up behind this grid

  if (warp == NCW) {
    chunk_produce<D>(tm_k, tm_v, p, 16, nst, s_stage, s_full, s_empty, g_meta, s_abort, lane);
    return;
  }

  // =================================================================== consumer warps
  const int g = lane >> 2, t = lane & 3;
  const int lane_row = lane & 7, mi = lane >> 3;
  uint32_t k_off[2], v_off[4];
  {
    const uint32_t pat = (uint32_t)((mi ^ lane_row) << 4);
    k_off[0] = (uint32_t)lane_row * 128 + pat;
    k_off[1] = (uint32_t)lane_row * 128 + (pat ^ 64u);
    const uint32_t vrow = (uint32_t)((mi & 1) * 8 + lane_row) * 128;
    const uint32_t vx = (uint32_t)(((mi >> 1) ^ lane_row) << 4);
#pragma unroll
    for (int i = 0; i < 4; ++i) v_off[i] = vrow + (((uint32_t)i * 32u) ^ vx);
  }
  const uint32_t slice = (uint32_t)warp * 16 * 128;  // this warp's 16 token rows inside a 64-dim half
  float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
  float o_acc[NO][4];
  uint32_t qf[KS][4];
#pragma unroll
  for (int n = 0; n < NO; ++n) o_acc[n][0] = o_acc[n][1] = o_acc[n][2] = o_acc[n][3] = 0.f;
#pragma unroll
  for (int k = 0; k < KS; ++k) qf[k][0] = qf[k][1] = qf[k][2] = qf[k][3] = 0u;
  int lim_row0 = 0, lim_row1 = 0;
  uint32_t mphase = 0;  // parity of the next combine-barrier phase to wait for = parity of the item count

  int slot = -1;
  uint32_t full_phase = 1u;
  for (;;) {
    if (++slot == nst) slot = 0;
    if (slot == 0) full_phase ^= 1u;
    if (!warp_wait(s_full + 8 * slot, full_phase, s_abort)) {
      if (lane == 0) atomicOr(&p.hdr->status, kStatusWaitTimeout);
      return;
    }
    const int4 meta = g_meta[2 * slot], meta2 = g_meta[2 * slot + 1];
    if (meta.x < 0) break;
    const int ntok = meta.w & 0xffff;
    const bool first = (meta.w >> 16) & 1, last = (meta.w >> 17) & 1;
    const int b = meta.y, h = meta.z, lim_base = meta2.y;
    if (first) {
      m_run[0] = m_run[1] = -INFINITY;
      l_run[0] = l_run[1] = 0.f;
#pragma unroll
      for (int n = 0; n < NO; ++n) o_acc[n][0] = o_acc[n][1] = o_acc[n][2] = o_acc[n][3] = 0.f;
      const int c0 = g, c1 = g + 8;
      const int qi0 = c0 / p.G, qi1 = c1 / p.G;
      lim_row0 = lim_base + qi0;
      lim_row1 = lim_base + qi1;
      const __nv_bfloat16* q0 = p.q + (((size_t)b * p.Sq + qi0) * p.Hq + (size_t)h * p.G + (c0 - qi0 * p.G)) * D;
      const __nv_bfloat16* q1 = p.q + (((size_t)b * p.Sq + qi1) * p.Hq + (size_t)h * p.G + (c1 - qi1 * p.G)) * D;
      const bool ok0 = c0 < p.GQ, ok1 = c1 < p.GQ;
#pragma unroll
      for (int k = 0; k < KS; ++k) {
        qf[k][0] = ok0 ? *reinterpret_cast<const uint32_t*>(q0 + 16 * k + 2 * t) : 0u;
        qf[k][1] = ok1 ? *reinterpret_cast<const uint32_t*>(q1 + 16 * k + 2 * t) : 0u;
        qf[k][2] = ok0 ? *reinterpret_cast<const uint32_t*>(q0 + 16 * k + 8 + 2 * t) : 0u;
        qf[k][3] = ok1 ? *reinterpret_cast<const uint32_t*>(q1 + 16 * k + 8 + 2 * t) : 0u;
      }
    }
    const int nslice = ntok - 16 * warp;  // tokens of this warp's slice that exist
    if (nslice > 0) {
      const int tokw = meta2.x + 16 * warp, t1 = meta2.z;
      const int e0 = min(t1, lim_row0) - tokw, e1 = min(t1, lim_row1) - tokw;
      const int e_first = min(t1, lim_base) - tokw;                       // row 0 sees the fewest tokens
      const int e_last = min(t1, lim_base + (p.GQ - 1) / p.G) - tokw;     // the last real row the most
      if (e_last > 0) {
        const uint32_t kst = s_stage + (uint32_t)slot * L::kStageBytes + slice;
        const uint32_t vst = kst + L::kTileBytes;
        if (e_first >= 16)
          chunk_consume<D, 16, false>(kst, vst, k_off, v_off, qf, m_run, l_run, o_acc, p.scale_log2e, nslice, e0, e1, t);
        else
          chunk_consume<D, 16, true>(kst, vst, k_off, v_off, qf, m_run, l_run, o_acc, p.scale_log2e, nslice, e0, e1, t);
      }
    }
    __syncwarp();
    if (!last) {
      if (lane == 0) mbar_arrive(s_empty + 8 * slot);
      continue;
    }
    // ---- the item is complete: combine the NCW warps' running states through this stage's memory
    {
      const int slot_id = meta.x;
      const bool dst_ok = checked(chk_index(slot_id, p.max_items) && chk_index(b, p.B) && chk_index(h, p.Hkv),
                                  &p.hdr->status, kStatusBadIndex);
      const int n_chunks = dst_ok ? p.seq_first[b + 1] - p.seq_first[b] : 1;
      float l0 = l_run[0], l1 = l_run[1];
#pragma unroll
      for (int o = 1; o < 4; o <<= 1) {
        l0 += __shfl_xor_sync(0xffffffffu, l0, o);
        l1 += __shfl_xor_sync(0xffffffffu, l1, o);
      }
      // O tile of warp w: row r lives in piece r / kRowsPerPiece (the warp's 2 KiB slices of K half 0, K half 1,
      // V half 0, V half 1, 8 KiB apart), 16-byte chunk c of a row at position c ^ (r & 7) (bank spreading)
      uint8_t* stage_gen = gen + (size_t)slot * L::kStageBytes;
      auto tile_row = [&](int w, int r) {
        return stage_gen + (size_t)(r / kRowsPerPiece) * L::kHalfBytes + (size_t)w * 2048 +
               (size_t)(r % kRowsPerPiece) * kRowBytes;
      };
      float* all_m = g_stat + (size_t)mphase * (NCW * 16 * 2);
      if (t == 0) {
        float* mm = all_m + ((size_t)warp * 16 + g) * 2;
        mm[0] = m_run[0];
        mm[1] = l0;
        mm[16] = m_run[1];
        mm[17] = l1;
      }
      {
        uint8_t* r0 = tile_row(warp, g);
        uint8_t* r1 = tile_row(warp, g + 8);
#pragma unroll
        for (int n = 0; n < NO; ++n) {
          const int off = (((2 * n + (t >> 1)) ^ g) << 4) + (t & 1) * 8;  // (g + 8) & 7 = g
          *reinterpret_cast<float2*>(r0 + off) = make_float2(o_acc[n][0], o_acc[n][1]);
          *reinterpret_cast<float2*>(r1 + off) = make_float2(o_acc[n][2], o_acc[n][3]);
        }
      }
      mbar_arrive(s_mbar);
      if (!warp_wait(s_mbar, mphase, s_abort)) {
        if (lane == 0) atomicOr(&p.hdr->status, kStatusWaitTimeout);
        return;
      }
      mphase ^= 1u;
      for (int idx = threadIdx.x; idx < p.GQ * (D / 4); idx += NCW * 32) {
        const int col = idx / (D / 4), c = idx % (D / 4);  // four dims 4c .. 4c + 3 of score column `col`
        float mx = -INFINITY;
#pragma unroll
        for (int w = 0; w < NCW; ++w) mx = fmaxf(mx, all_m[(w * 16 + col) * 2]);
        const float ms = mx == -INFINITY ? 0.f : mx;  // a row that saw nothing of this chunk (causal limit)
        float den = 0.f;
        float4 num = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int w = 0; w < NCW; ++w) {
          const float sw = ex2(all_m[(w * 16 + col) * 2] - ms);
          den += sw * all_m[(w * 16 + col) * 2 + 1];
          const float4 o = *reinterpret_cast<const float4*>(tile_row(w, col) + ((c ^ (col & 7)) << 4));
          num.x += sw * o.x;
          num.y += sw * o.y;
          num.z += sw * o.z;
          num.w += sw * o.w;
        }
        const float inv = den > 0.f ? 1.f / den : 0.f;
        if (kChecked && !dst_ok) continue;
        if (n_chunks == 1 && !p.out_f32) {
          const int qi = col / p.G, head = col - qi * p.G;
          __nv_bfloat16* dst = p.out + (((size_t)b * p.Sq + qi) * p.Hq + (size_t)h * p.G + head) * D + 4 * c;
          const __nv_bfloat162 lo = __floats2bfloat162_rn(num.x * inv, num.y * inv);
          const __nv_bfloat162 hi = __floats2bfloat162_rn(num.z * inv, num.w * inv);
          *reinterpret_cast<uint2*>(dst) =
              make_uint2(*reinterpret_cast<const uint32_t*>(&lo), *reinterpret_cast<const uint32_t*>(&hi));
        } else {
          *reinterpret_cast<float4*>(p.part_o + ((size_t)slot_id * p.GQ + col) * D + 4 * c) =
              make_float4(num.x * inv, num.y * inv, num.z * inv, num.w * inv);
          if (c == 0) p.part_lse[(size_t)slot_id * p.GQ + col] = den > 0.f ? mx + lg2(den) : -INFINITY;
        }
      }
      // the stage was written through the generic proxy; the producer refills it through the async proxy
      fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) mbar_arrive(s_empty + 8 * slot);
    }
  }
}

}  // namespace ooco
