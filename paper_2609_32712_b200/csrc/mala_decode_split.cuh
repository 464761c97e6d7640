// Split-KV decode, split kernel ("Fused decoding execution") for sm_100a, head size 128.
//
// A work item is one split of one (batch, KV head): the G = Hq/Hkv query heads that share the KV head
// are the rows of its tile (rows G..127 of the MMA tile read whatever follows the 16 loaded rows in
// shared memory and are ignored), L = Nk for every row, the tiles of the split are visited newest
// first with the item's own running (m, l), and the item ends with a normalised fp32 partial output
// and its log-normalizer per head.  The kernel is HBM-bound, so it is persistent: one CTA per SM walks
// over its items with the K (and, dense, V) rings, the score buffers and the two output accumulators
// running on across item boundaries; there is no per-item launch, TMEM allocation or pipeline drain.
//   warp 0  TMA producer: Q of the next item (16 rows), K ring; dense kernel: V ring one tile behind K
//   warp 1  UMMA issuer: S = Q K^T one tile ahead of the decision; MALA kernel: V loaded for retained tiles (and,
//           ahead of its vote, for the tile after a retained one); O[item parity] += P V
//   warp 4  softmax warp (TMEM lanes 0..31): row max, Eq. 3 vote, P, lazy rescale, partial output
// K is always streamed; a skipped tile issues no exp, no P and no PV, and reads no V unless its V copy had been
// issued ahead of the vote (only the tile right after a retained one can be in that case).
#pragma once
#include "sm100_ptx.cuh"

namespace mala {

struct DecParams {
  float* o_part;                 // [B, Hq, num_splits, 128] fp32, normalised per split
  float* lse_part;               // [B, Hq, num_splits] natural log; -inf for an empty split
  uint32_t* retained;            // [B, Hkv, num_splits] or null
  uint32_t* bitmask;             // [B, Hkv, num_splits, words] or null (zero-filled by the host)
  unsigned long long* totals;    // [2] or null
  int* status;
  int B, Hq, Hkv, Nk, tps, num_splits, words, n_items;
  float scale_log2, log2_tau;
};

struct DecCfg {
  static constexpr int kTileBytes = 128 * 128 * 2;
  static constexpr int kQBytes = 4096;                   // 16 rows x 128 columns, two 2 KB panels
  static constexpr int kKStages = 3, kVStages = 3;
  static constexpr int kSmemBytes = 2 * kQBytes + (kKStages + kVStages) * kTileBytes + 1024;
  static constexpr int kThreads = 160;
};

template <bool kDense>
__global__ void __launch_bounds__(160, 1)
mala_decode_split_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                         const __grid_constant__ CUtensorMap tmV, const DecParams p) {
  constexpr int KS = DecCfg::kKStages, VS = DecCfg::kVStages, TB = DecCfg::kTileBytes;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint8_t* sQ = smem;                      // [2] item parity
  uint8_t* sK = sQ + 2 * DecCfg::kQBytes;
  uint8_t* sV = sK + KS * TB;

  __shared__ uint64_t q_full[2], q_empty[2], k_full[KS], k_empty[KS], v_full[VS], v_empty[VS], s_full[2],
      vote_bar[2], p_full[2], o_done, item_done[2], o_free[2], fin_bar;
  __shared__ uint32_t tmem_base_s;
  __shared__ int flag[3];
  __shared__ int early_exit;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int G = p.Hq / p.Hkv;
  int* status = p.status;

  if (tid == 0) {
    early_exit = (*(volatile int*)status != 0);
    for (int s = 0; s < 2; ++s) {
      mbar_init(&q_full[s], 1); mbar_init(&q_empty[s], 1); mbar_init(&s_full[s], 1); mbar_init(&vote_bar[s], 1);
      mbar_init(&p_full[s], 1); mbar_init(&item_done[s], 1); mbar_init(&o_free[s], 1);
    }
    for (int s = 0; s < KS; ++s) { mbar_init(&k_full[s], 1); mbar_init(&k_empty[s], 1); }
    for (int s = 0; s < VS; ++s) { mbar_init(&v_full[s], 1); mbar_init(&v_empty[s], 1); }
    mbar_init(&o_done, 1);
    mbar_init(&fin_bar, 1);
    flag[0] = flag[1] = flag[2] = 0;
    mbar_fence_init();
  }
  __syncthreads();
  if (early_exit) return;
  if (warp == 0) { tmem_alloc(&tmem_base_s, 512); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tb = tmem_base_s;

  // geometry of work item `item`: batch, KV head, split, number of legal tiles, newest key block
  auto geometry = [&](int item, int& b, int& hkv, int& split, int& T, int& j0) {
    split = item % p.num_splits;
    const int bh = item / p.num_splits;
    hkv = bh % p.Hkv;
    b = bh / p.Hkv;
    const int lo = split * p.tps * 128;
    const int hi = min(p.Nk, lo + p.tps * 128);
    T = hi > lo ? (hi - lo + 127) / 128 : 0;
    j0 = lo / 128 + T - 1;
  };

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      tma_prefetch_desc(&tmQ); tma_prefetch_desc(&tmK); tma_prefetch_desc(&tmV);
      int ne = 0;                               // ordinal of the non-empty item
      int ks = 0, vs = 0;
      uint32_t kpar = 1, vpar = 1;              // "empty" parities (first pass: free)
      bool ok = true;
      for (int item = blockIdx.x; item < p.n_items && ok; item += gridDim.x) {
        int b, hkv, split, T, j0;
        geometry(item, b, hkv, split, T, j0);
        if (T == 0) continue;
        const int ip = ne & 1;
        ok = mbar_wait(&q_empty[ip], ((ne >> 1) & 1) ^ 1, status);
        if (!ok) break;
        mbar_arrive_expect_tx(&q_full[ip], DecCfg::kQBytes);
        tma_load_4d(sQ + ip * DecCfg::kQBytes, &tmQ, &q_full[ip], 0, hkv * G, 0, b);
        tma_load_4d(sQ + ip * DecCfg::kQBytes + 2048, &tmQ, &q_full[ip], 64, hkv * G, 0, b);
        for (int t = 0; t < T && ok; ++t) {
          ok = mbar_wait(&k_empty[ks], kpar, status);
          if (!ok) break;
          mbar_arrive_expect_tx(&k_full[ks], TB);
          tma_load_4d(sK + ks * TB, &tmK, &k_full[ks], 0, (j0 - t) * 128, hkv, b);
          tma_load_4d(sK + ks * TB + 16384, &tmK, &k_full[ks], 64, (j0 - t) * 128, hkv, b);
          if (++ks == KS) { ks = 0; kpar ^= 1; }
          if (kDense) {   // every tile is retained: V follows K
            ok = mbar_wait(&v_empty[vs], vpar, status);
            if (!ok) break;
            mbar_arrive_expect_tx(&v_full[vs], TB);
            tma_load_4d(sV + vs * TB, &tmV, &v_full[vs], 0, (j0 - t) * 128, hkv, b);
            tma_load_4d(sV + vs * TB + 16384, &tmV, &v_full[vs], 64, (j0 - t) * 128, hkv, b);
            if (++vs == VS) { vs = 0; vpar ^= 1; }
          }
        }
        ++ne;
      }
      // after an expired wait copies may still be in flight: give them time to land before the CTA exits
      if (!ok) { const long long t0 = clock64(); while (clock64() - t0 < 400000) {} }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ UMMA issuer (+ on-demand V loads)
    // All 32 lanes run this loop with identical values; MMAs, commits and TMA loads are issued by one elected lane.
    {
      const uint32_t leader = elect_one();
      constexpr uint32_t idesc_qk = make_idesc_bf16(128, 128, false, false);
      constexpr uint32_t idesc_pv = make_idesc_bf16(128, 128, false, true);
      const uint64_t dQ0 = make_smem_desc(smem_u32(sQ), 16, 1024);
      const uint64_t dK0 = make_smem_desc(smem_u32(sK), 16, 1024);
      const uint64_t dV0 = make_smem_desc(smem_u32(sV), 16384, 1024);
      bool ok = true;
      // cursor over (non-empty item, tile) in processing order, and a second one running one tile ahead
      struct Cur { int item, ne, t, T, b, hkv, split, j0; bool valid; };
      auto first_item = [&](Cur& c, int from, int ne) {
        c.valid = false;
        for (int item = from; item < p.n_items; item += gridDim.x) {
          int b, hkv, split, T, j0;
          geometry(item, b, hkv, split, T, j0);
          if (T > 0) { c = Cur{item, ne, 0, T, b, hkv, split, j0, true}; return; }
        }
      };
      auto advance = [&](Cur& c) {
        if (c.t + 1 < c.T) { ++c.t; return; }
        first_item(c, c.item + gridDim.x, c.ne + 1);
      };
      int g = 0;                                 // global tile counter (score buffer g & 1)
      int kc = 0; uint32_t kpar = 0;             // K ring consumer
      int vi = 0; uint32_t vipar = 1;            // V ring producer side (MALA: loads issued here)
      int vc = 0; uint32_t vcpar = 0;            // V ring consumer
      uint32_t ppar[2] = {0, 0};
      int q_seen = -1;                           // last non-empty item whose Q has been observed
      auto issue_qk = [&](const Cur& c, int gq) -> bool {
        const int ip = c.ne & 1;
        if (q_seen < c.ne) {
          if (!mbar_wait_warp(&q_full[ip], (c.ne >> 1) & 1, status)) return false;
          q_seen = c.ne;
        }
        if (!mbar_wait_warp(&k_full[kc], kpar, status)) return false;
        tc_fence_after();
        const uint32_t dS = tmem_addr(tb, 0, (gq & 1) * 128);
        const uint64_t dQ = desc_advance(dQ0, ip * DecCfg::kQBytes), dK = desc_advance(dK0, kc * TB);
#pragma unroll
        for (int k = 0; k < 8; ++k)   // Q panels lie 2 KB apart, K panels 16 KB
          mma_ss(dS, desc_advance(dQ, (k >> 2) * 2048 + (k & 3) * 32), desc_advance(dK, (k >> 2) * 16384 + (k & 3) * 32),
                 idesc_qk, k > 0, leader);
        if (leader) {
          tc_commit(&k_empty[kc]);
          tc_commit(&s_full[gq & 1]);
          if (c.t == c.T - 1) tc_commit(&q_empty[ip]);   // last QK of the item: its Q stage may be refilled
        }
        if (++kc == KS) { kc = 0; kpar ^= 1; }
        return true;
      };
      // MALA kernel: a V tile is needed only if its tile is retained, which is known after the vote -- too late to hide
      // an HBM round trip with one tile of look-ahead.  So the V copy of the next tile is issued ahead of its
      // votes while tiles are being retained (one tile ahead after a retained tile, and always for the first tile
      // of an item, which is retained by construction), as far as V stages are free.  A copy fetched for a tile
      // that is then skipped is handed back to the ring unused once it has landed: only then is a V tile read that
      // the method itself would not have read.
      auto load_v = [&](const Cur& c) {
        if (leader) {
          mbar_arrive_expect_tx(&v_full[vi], TB);
          tma_load_4d(sV + vi * TB, &tmV, &v_full[vi], 0, (c.j0 - c.t) * 128, c.hkv, c.b);
          tma_load_4d(sV + vi * TB + 16384, &tmV, &v_full[vi], 64, (c.j0 - c.t) * 128, c.hkv, c.b);
        }
        __syncwarp();
        if (++vi == VS) { vi = 0; vipar ^= 1; }
      };
      int v_upto = -1;                           // V copies have been issued for every retained tile <= v_upto and,
      Cur sp;                                    // ahead of their votes, for the tiles in (g, v_upto]; sp = tile v_upto + 1
      sp.valid = false;
      Cur cur, nxt;
      first_item(cur, blockIdx.x, 0);
      if (cur.valid) ok = issue_qk(cur, 0);
      int r_item = 0;
      while (cur.valid && ok) {
        nxt = cur;
        advance(nxt);
        if (nxt.valid) { ok = issue_qk(nxt, g + 1); if (!ok) break; }
        bool retain = true;
        if (!kDense) {
          ok = mbar_wait_warp(&vote_bar[g & 1], (g >> 1) & 1, status);
          if (!ok) break;
          retain = __shfl_sync(0xffffffffu, *(volatile int*)&flag[g % 3], 0) != 0;
          if (retain) {
            if (v_upto < g) {   // V of this tile, on demand
              ok = mbar_wait_warp(&v_empty[vi], vipar, status);
              if (!ok) break;
              load_v(cur);
            }
          } else if (v_upto >= g) {   // fetched ahead but not needed: back to the ring once it has landed
            ok = mbar_wait_warp(&v_full[vc], vcpar, status);
            if (!ok) break;
            if (leader) mbar_arrive(&v_empty[vc]);
            if (++vc == VS) { vc = 0; vcpar ^= 1; }
          }
          if (v_upto < g) { v_upto = g; sp = nxt; }
        }
        const int ip = cur.ne & 1;
        if (retain) {
          ok = mbar_wait_warp(&p_full[g & 1], ppar[g & 1], status);
          if (!ok) break;
          ppar[g & 1] ^= 1;
          ok = mbar_wait_warp(&v_full[vc], vcpar, status);
          if (!ok) break;
          if (r_item == 0 && cur.ne >= 2) {   // the softmax warp has read this accumulator's previous item
            ok = mbar_wait_warp(&o_free[ip], ((cur.ne >> 1) - 1) & 1, status);
            if (!ok) break;
          }
          tc_fence_after();
          const uint32_t aP = tmem_addr(tb, 0, (g & 1) * 128), dO = tmem_addr(tb, 0, 256 + ip * 128);
          const uint64_t dV = desc_advance(dV0, vc * TB);
          const uint32_t acc0 = r_item > 0 ? 1u : 0u;
#pragma unroll
          for (int k = 0; k < 8; ++k) mma_ts(dO, aP + k * 8, desc_advance(dV, k * 2048), idesc_pv, k > 0 ? 1u : acc0, leader);
          if (leader) { tc_commit(&v_empty[vc]); tc_commit(&o_done); }
          if (++vc == VS) { vc = 0; vcpar ^= 1; }
          ++r_item;
        }
        if (cur.t == cur.T - 1) { if (leader) tc_commit(&item_done[ip]); r_item = 0; }
        if (!kDense) {
          const int depth = (retain || (nxt.valid && nxt.t == 0)) ? 1 : 0;   // (two tiles ahead measured slower)
          while (v_upto < g + depth && sp.valid && __all_sync(0xffffffffu, mbar_try_wait(&v_empty[vi], vipar))) {
            load_v(sp);
            ++v_upto;
            advance(sp);
          }
        }
        cur = nxt;
        ++g;
      }
      __syncwarp();
      if (leader) tc_commit(&fin_bar);
      mbar_wait_warp(&fin_bar, 0, status);
      if (!ok) { const long long t0 = clock64(); while (clock64() - t0 < 400000) {} }
    }
  } else if (warp == 4) {
    // ------------------------------------------------------------------ softmax warp: lane = packed query head
    const int rl = lane;
    const bool valid = rl < G;
    const float c2 = p.scale_log2;
    const float theta = kDense ? -INFINITY : (p.log2_tau - log2f((float)p.Nk));
    int g = 0, ne = 0, rg = 0;      // global tile counter, non-empty item ordinal, PVs requested so far
    bool ok = true;
    for (int item = blockIdx.x; item < p.n_items && ok; item += gridDim.x) {
      int b, hkv, split, T, j0;
      geometry(item, b, hkv, split, T, j0);
      const size_t prow = ((size_t)b * p.Hq + hkv * G + rl) * p.num_splits + split;
      const size_t stat_row = (size_t)(b * p.Hkv + hkv) * p.num_splits + split;
      if (T == 0) {   // empty split: (0, -inf)
        if (valid) {
          float4* dst = reinterpret_cast<float4*>(p.o_part + prow * 128);
          for (int v = 0; v < 32; ++v) dst[v] = make_float4(0.f, 0.f, 0.f, 0.f);
          p.lse_part[prow] = -INFINITY;
        }
        if (lane == 0 && p.retained) p.retained[stat_row] = 0u;
        continue;
      }
      const int ip = ne & 1;
      const uint32_t colO = 256u + (uint32_t)ip * 128u;
      float m_ref = -INFINITY, l = 0.f;
      int r = 0;
      uint32_t bm_bits = 0;
      int bm_word = -1;
      uint32_t* bm_row = p.bitmask ? p.bitmask + stat_row * p.words : nullptr;
      for (int t = 0; t < T; ++t, ++g) {
        ok = mbar_wait(&s_full[g & 1], (g >> 1) & 1, status);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after();
        const uint32_t colS = (uint32_t)(g & 1) * 128u;
        uint32_t s0[32], s1[32], s2[32], s3[32];
        tmem_ld_x32(tmem_addr(tb, 0, colS + 0), s0);
        tmem_ld_x32(tmem_addr(tb, 0, colS + 32), s1);
        tmem_ld_x32(tmem_addr(tb, 0, colS + 64), s2);
        tmem_ld_x32(tmem_addr(tb, 0, colS + 96), s3);
        tmem_wait_ld();
        if (t == 0) {   // newest tile of the split: keys beyond the end of the cache
          const int lim = p.Nk - 1 - j0 * 128;
          const uint32_t ninf = 0xff800000u;
#pragma unroll
          for (int e = 0; e < 32; ++e) {
            if (e > lim) s0[e] = ninf;
            if (e + 32 > lim) s1[e] = ninf;
            if (e + 64 > lim) s2[e] = ninf;
            if (e + 96 > lim) s3[e] = ninf;
          }
        }
        float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
        for (int e = 0; e < 32; ++e) {
          mx0 = fmaxf(mx0, fmaxf(__uint_as_float(s0[e]), __uint_as_float(s1[e])));
          mx1 = fmaxf(mx1, fmaxf(__uint_as_float(s2[e]), __uint_as_float(s3[e])));
        }
        const float mt = fmaxf(mx0, mx1) * c2;
        bool retain = true;
        if (!kDense) {
          // Eq. 3 against the split's partial normalizer: skip iff rowmax - (m + log l) < log(tau / Nk) for all rows
          bool vote;
          if (l == 0.f) vote = valid;
          else vote = valid && !(((mt - (m_ref + log2f(l))) - theta) < 0.f);
          retain = __any_sync(0xffffffffu, vote);
          if (lane == 0) {
            *(volatile int*)&flag[g % 3] = retain ? 1 : 0;
            tc_fence_before();
            mbar_arrive(&vote_bar[g & 1]);
          }
        }
        if (!retain) continue;
        if (lane == 0 && bm_row) {
          const int bit = T - 1 - t;   // tile index inside the split
          if ((bit >> 5) != bm_word) {
            if (bm_word >= 0) bm_row[bm_word] = bm_bits;
            bm_word = bit >> 5;
            bm_bits = 0;
          }
          bm_bits |= 1u << (bit & 31);
        }
        if (r == 0) {
          m_ref = mt;
        } else {
          const bool need = mt > m_ref + 8.f;
          if (__any_sync(0xffffffffu, need)) {
            ok = mbar_wait(&o_done, (rg - 1) & 1, status);   // the previous PV has landed
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            const float m_new = fmaxf(m_ref, mt);
            const float alpha = fast_exp2(m_ref - m_new);
            l *= alpha;
            m_ref = m_new;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
              uint32_t o[32];
              tmem_ld_x32(tmem_addr(tb, 0, colO + c * 32), o);
              tmem_wait_ld();
#pragma unroll
              for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
              tmem_st_x32(tmem_addr(tb, 0, colO + c * 32), o);
            }
          }
        }
        const float nm = -m_ref;
        float sum0 = 0.f, sum1 = 0.f;
        uint32_t pk[16];
#define MALA_DEC_P(SRC, COL)                                                           \
        {                                                                              \
          _Pragma("unroll") for (int e = 0; e < 16; ++e) {                             \
            const float p0 = fast_exp2(fmaf(__uint_as_float(SRC[2 * e]), c2, nm));      \
            const float p1 = fast_exp2(fmaf(__uint_as_float(SRC[2 * e + 1]), c2, nm));  \
            sum0 += p0; sum1 += p1;                                                    \
            pk[e] = pack_bf16x2(p0, p1);                                               \
          }                                                                            \
          tmem_st_x16(tmem_addr(tb, 0, colS + (COL)), pk);                             \
        }
        MALA_DEC_P(s0, 0)
        MALA_DEC_P(s1, 16)
        MALA_DEC_P(s2, 32)
        MALA_DEC_P(s3, 48)
#undef MALA_DEC_P
        l += sum0 + sum1;
        tmem_wait_st();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&p_full[g & 1]);
        ++r;
        ++rg;
      }
      if (!ok) break;
      // partial output of this item once its last PV has retired: O / l in fp32 and the log-normalizer
      ok = mbar_wait(&item_done[ip], (ne >> 1) & 1, status);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      const float inv = 1.f / l;
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        uint32_t o[32];
        tmem_ld_x32(tmem_addr(tb, 0, colO + c * 32), o);
        tmem_wait_ld();
        if (c == 3) {
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(&o_free[ip]);   // the accumulator may take the item after next
        }
        if (valid) {
          float4* dst = reinterpret_cast<float4*>(p.o_part + prow * 128 + c * 32);
#pragma unroll
          for (int v = 0; v < 8; ++v)
            dst[v] = make_float4(__uint_as_float(o[4 * v]) * inv, __uint_as_float(o[4 * v + 1]) * inv,
                                 __uint_as_float(o[4 * v + 2]) * inv, __uint_as_float(o[4 * v + 3]) * inv);
        }
      }
      if (valid) p.lse_part[prow] = (m_ref + log2f(l)) * 0.6931471805599453f;
      if (lane == 0) {
        if (bm_row && bm_word >= 0) bm_row[bm_word] = bm_bits;
        if (p.retained) p.retained[stat_row] = (uint32_t)r;
        if (p.totals) {
          atomicAdd(&p.totals[0], (unsigned long long)r);
          atomicAdd(&p.totals[1], (unsigned long long)T);
        }
      }
      ++ne;
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tb, 512);
}

}  // namespace mala
