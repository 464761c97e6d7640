// MALA forward (Algorithm 1) and split-KV decode ("Fused decoding execution") for sm_100a.
//
// One CTA owns one 128-row query block of one (batch, query head) and walks its legal key blocks
// from the diagonal toward earlier keys.  Warp roles (192 threads):
//   warp 0      : TMA producer for Q (once) and the K ring
//   warp 1      : UMMA issuer.  S = Q K^T for EVERY tile into one of two TMEM score buffers; after the
//                 retention decision of a tile it issues the V load and, once P is ready, O += P V.
//                 A skipped tile issues no V load and no PV MMA.
//   warps 2..5  : softmax group, one thread per query row.  Reads S from TMEM, forms the row maximum,
//                 votes on retention (Eq. 3), and for retained tiles writes P (bf16) over S in TMEM
//                 and keeps the running (m, l); O is rescaled lazily in TMEM.
// All synchronisation is by mbarriers with bounded waits.
//
// Decode mode (kDecode): one CTA owns one split of one (batch, KV head).  The rows of its "query
// block" are the G = Hq/Hkv query heads that share the KV head (rows G..127 of the tile hold other
// heads or zeros and are ignored), L = Nk for every row, tiles of the split are visited newest
// first, and the CTA writes a normalised fp32 partial output and its log-normalizer per head.  Only
// one softmax warp (TMEM lanes 0..31) is active.
#pragma once
#include "sm100_ptx.cuh"

namespace mala {

struct FwdParams {
  __nv_bfloat16* o;
  int64_t o_sb, o_sn, o_sh;
  float* lse;                    // [B, Hq, N]
  uint32_t* retained;            // [B, Hq, Tr] or null
  uint32_t* bitmask;             // [B, Hq, Tr, words] or null (zero-filled by the host)
  unsigned long long* totals;    // [2] or null
  int* status;
  int B, Hq, Hkv, N, Tr, words, causal;
  // decode only
  float* o_part;                 // [B, Hq, num_splits, D] fp32, normalised per split
  float* lse_part;               // [B, Hq, num_splits] natural log; -inf for an empty split
  int tps, num_splits;           // tiles per split, number of splits (N is Nk)
  float scale_log2;              // scale * log2(e)
  float log2_tau;                // log2(tau); unused by the dense kernel
};

template <int D, bool kDense>
struct FwdCfg {
  static constexpr int kPanels = D / 64;                 // 64-column swizzle panels per tile
  static constexpr int kTileBytes = 128 * D * 2;
  static constexpr int kKStages = (D == 128) ? (kDense ? 3 : 4) : 4;
  static constexpr int kVStages = (D == 128) ? (kDense ? 3 : 2) : 3;
  static constexpr int kSmemBytes = (1 + kKStages + kVStages) * kTileBytes + 1024;
  static constexpr int kThreads = 192;
  static constexpr uint32_t kTmemCols = 512;
  static constexpr uint32_t kColS0 = 0, kColS1 = 128, kColO = 256;
};

template <int D, bool kDense, bool kDecode>
__global__ void __launch_bounds__(192, 1)
mala_fwd_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                const __grid_constant__ CUtensorMap tmV, const FwdParams p) {
  using Cfg = FwdCfg<D, kDense>;
  constexpr int KS = Cfg::kKStages, VS = Cfg::kVStages, PAN = Cfg::kPanels;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint8_t* sQ = smem;
  uint8_t* sK = sQ + Cfg::kTileBytes;
  uint8_t* sV = sK + KS * Cfg::kTileBytes;

  __shared__ uint64_t q_full, k_full[KS], k_empty[KS], s_full[2], vote_bar[2], p_full[2], v_full[VS], v_empty[VS],
      o_done, fin_bar;
  __shared__ uint32_t tmem_base_s;
  __shared__ int flag[3];
  __shared__ int early_exit;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int G = p.Hq / p.Hkv;
  const int b = blockIdx.z;
  int i, h, hkv, T, j0, q_row, q_head;
  if (kDecode) {
    const int split = blockIdx.x;
    hkv = blockIdx.y;
    h = hkv * G;
    i = split;
    const int lo = split * p.tps * 128;
    const int hi = min(p.N, lo + p.tps * 128);
    T = hi > lo ? (hi - lo + 127) / 128 : 0;   // legal tiles of this split
    j0 = lo / 128 + T - 1;                     // newest tile first
    q_row = hkv * G;                           // rows of the Q tile are query heads
    q_head = 0;
  } else {
    i = p.Tr - 1 - (int)blockIdx.x;            // longest blocks first
    h = blockIdx.y;
    hkv = h / G;
    T = p.causal ? (i + 1) : p.Tr;             // tiles to visit
    j0 = p.causal ? i : (p.Tr - 1);            // first visited key block
    q_row = i * 128;
    q_head = h;
  }
  constexpr int kSoftmaxWarps = kDecode ? 1 : 4;
  int* status = p.status;

  if (tid == 0) {
    early_exit = (*(volatile int*)status != 0);
    mbar_init(&q_full, 1);
    for (int s = 0; s < KS; ++s) { mbar_init(&k_full[s], 1); mbar_init(&k_empty[s], 1); }
    for (int s = 0; s < VS; ++s) { mbar_init(&v_full[s], 1); mbar_init(&v_empty[s], 1); }
    for (int s = 0; s < 2; ++s) {
      mbar_init(&s_full[s], 1); mbar_init(&vote_bar[s], kSoftmaxWarps); mbar_init(&p_full[s], kSoftmaxWarps);
    }
    mbar_init(&o_done, 1);
    mbar_init(&fin_bar, 1);
    flag[0] = flag[1] = flag[2] = 0;
    mbar_fence_init();
  }
  __syncthreads();
  if (early_exit) return;
  if (warp == 0) { tmem_alloc(&tmem_base_s, Cfg::kTmemCols); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tb = tmem_base_s;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer: Q, K ring
    if (lane == 0) {
      tma_prefetch_desc(&tmQ); tma_prefetch_desc(&tmK); tma_prefetch_desc(&tmV);
      mbar_arrive_expect_tx(&q_full, Cfg::kTileBytes);
      for (int pn = 0; pn < PAN; ++pn) tma_load_4d(sQ + pn * 16384, &tmQ, &q_full, pn * 64, q_row, q_head, b);
      int issued = 0;
      bool ok = true;
      for (int t = 0; t < T && ok; ++t) {
        const int s = t % KS;
        ok = mbar_wait(&k_empty[s], ((t / KS) & 1) ^ 1, status);
        if (!ok) break;
        mbar_arrive_expect_tx(&k_full[s], Cfg::kTileBytes);
        for (int pn = 0; pn < PAN; ++pn)
          tma_load_4d(sK + s * Cfg::kTileBytes + pn * 16384, &tmK, &k_full[s], pn * 64, (j0 - t) * 128, hkv, b);
        issued = t + 1;
      }
      if (!ok) {  // drain our own copies before leaving
        mbar_wait(&q_full, 0, status);
        for (int t = (issued > KS ? issued - KS : 0); t < issued; ++t) mbar_wait(&k_full[t % KS], (t / KS) & 1, status);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ UMMA issuer (+ V loads)
    if (lane == 0) {
      constexpr uint32_t idesc_qk = make_idesc_bf16(128, 128, false, false);
      constexpr uint32_t idesc_pv = make_idesc_bf16(128, D, false, true);
      // descriptors are built once; per MMA only the start-address field is advanced
      const uint64_t dQ = make_smem_desc(smem_u32(sQ), 16, 1024);
      const uint64_t dK0 = make_smem_desc(smem_u32(sK), 16, 1024);
      const uint64_t dV0 = make_smem_desc(smem_u32(sV), 16384, 1024);
      bool ok = mbar_wait(&q_full, 0, status);
      int v_issued = 0;   // V tiles requested so far
      int r = 0;          // PV MMAs issued so far (retained tiles)
      uint32_t pcount[2] = {0, 0};
      auto issue_qk = [&](int t) -> bool {
        const int s = t % KS;
        if (!mbar_wait(&k_full[s], (t / KS) & 1, status)) return false;
        tc_fence_after();
        const uint32_t dS = tmem_addr(tb, 0, (t & 1) ? Cfg::kColS1 : Cfg::kColS0);
        const uint64_t dK = desc_advance(dK0, s * Cfg::kTileBytes);
#pragma unroll
        for (int k = 0; k < D / 16; ++k) {
          const uint32_t off = (k >> 2) * 16384 + (k & 3) * 32;
          mma_ss(dS, desc_advance(dQ, off), desc_advance(dK, off), idesc_qk, k > 0);
        }
        tc_commit(&k_empty[s]);
        tc_commit(&s_full[t & 1]);
        return true;
      };
      auto issue_v = [&](int t) -> bool {   // V of visited tile t into stage v_issued % VS
        const int s = v_issued % VS;
        if (!mbar_wait(&v_empty[s], ((v_issued / VS) & 1) ^ 1, status)) return false;
        mbar_arrive_expect_tx(&v_full[s], Cfg::kTileBytes);
        for (int pn = 0; pn < PAN; ++pn)
          tma_load_4d(sV + s * Cfg::kTileBytes + pn * 16384, &tmV, &v_full[s], pn * 64, (j0 - t) * 128, hkv, b);
        ++v_issued;
        return true;
      };
      if (ok && T > 0) ok = issue_qk(0);
      if (kDense) {
        for (int t = 0; t < VS - 1 && t < T && ok; ++t) ok = issue_v(t);
      }
      for (int t = 0; t < T && ok; ++t) {
        if (t + 1 < T) { ok = issue_qk(t + 1); if (!ok) break; }
        bool retain = true;
        if (!kDense) {
          ok = mbar_wait(&vote_bar[t & 1], (t >> 1) & 1, status);
          if (!ok) break;
          retain = (*(volatile int*)&flag[t % 3]) != 0;
          if (retain) { ok = issue_v(t); if (!ok) break; }
        }
        if (retain) {
          const int s = r % VS;
          ok = mbar_wait(&p_full[t & 1], pcount[t & 1] & 1, status);
          if (!ok) break;
          ++pcount[t & 1];
          ok = mbar_wait(&v_full[s], (r / VS) & 1, status);
          if (!ok) break;
          tc_fence_after();
          const uint32_t aP = tmem_addr(tb, 0, (t & 1) ? Cfg::kColS1 : Cfg::kColS0);
          const uint32_t dO = tmem_addr(tb, 0, Cfg::kColO);
          const uint64_t dV = desc_advance(dV0, s * Cfg::kTileBytes);
          const uint32_t acc0 = r > 0 ? 1u : 0u;
#pragma unroll
          for (int k = 0; k < 8; ++k)
            mma_ts(dO, aP + k * 8, desc_advance(dV, k * 2048), idesc_pv, k > 0 ? 1u : acc0);
          tc_commit(&v_empty[s]);
          tc_commit(&o_done);
          ++r;
          if (kDense && t + VS - 1 < T) { ok = issue_v(t + VS - 1); if (!ok) break; }
        }
      }
      // all MMAs retired and all requested V copies landed before the CTA may exit
      tc_commit(&fin_bar);
      mbar_wait(&fin_bar, 0, status);
      if (!ok) {
        for (int u = (v_issued > VS ? v_issued - VS : 0); u < v_issued; ++u) mbar_wait(&v_full[u % VS], (u / VS) & 1, status);
      }
    }
  } else if (!kDecode || warp == 4) {
    // ------------------------------------------------------------------ softmax group: one thread per row
    const uint32_t lane_base = (uint32_t)(warp & 3) * 32u;
    const int rl = (int)lane_base + lane;            // row inside the block
    const int row = kDecode ? rl : i * 128 + rl;
    const bool valid = kDecode ? (rl < G) : (row < p.N);
    const float c2 = p.scale_log2;
    const float Lq = (p.causal && !kDecode) ? (float)(row + 1) : (float)p.N;
    const float theta = kDense ? -INFINITY : (p.log2_tau - log2f(Lq));
    float m_ref = -INFINITY, l = 0.f;
    int r = 0;                                       // retained tiles so far
    bool ok = true;
    uint32_t bm_bits = 0;
    int bm_word = -1;
    const bool stat_thread = (warp == (kDecode ? 4 : 2) && lane == 0);
    // telemetry row: (b, h, query block) in prefill, (b, hkv, split) in decode
    const size_t stat_row = kDecode ? ((size_t)(b * p.Hkv + hkv) * p.num_splits + i) : ((size_t)(b * p.Hq + h) * p.Tr + i);
    uint32_t* bm_row = p.bitmask ? p.bitmask + stat_row * p.words : nullptr;

    for (int t = 0; t < T; ++t) {
      const int j = j0 - t;
      ok = mbar_wait(&s_full[t & 1], (t >> 1) & 1, status);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      const uint32_t colS = (t & 1) ? Cfg::kColS1 : Cfg::kColS0;
      uint32_t s0[32], s1[32], s2[32], s3[32];
      tmem_ld_x32(tmem_addr(tb, lane_base, colS + 0), s0);
      tmem_ld_x32(tmem_addr(tb, lane_base, colS + 32), s1);
      tmem_ld_x32(tmem_addr(tb, lane_base, colS + 64), s2);
      tmem_ld_x32(tmem_addr(tb, lane_base, colS + 96), s3);
      tmem_wait_ld();
      if (t == 0) {
        // first visited tile: causal diagonal and / or the ragged end of the key range
        const int lim = (p.causal && !kDecode) ? rl : (p.N - 1 - j * 128);
        const uint32_t ninf = 0xff800000u;
#pragma unroll
        for (int e = 0; e < 32; ++e) {
          if (e > lim) s0[e] = ninf;
          if (e + 32 > lim) s1[e] = ninf;
          if (e + 64 > lim) s2[e] = ninf;
          if (e + 96 > lim) s3[e] = ninf;
        }
      }
      float mx = -INFINITY;
#pragma unroll
      for (int e = 0; e < 32; ++e) {
        mx = fmaxf(mx, fmaxf(fmaxf(__uint_as_float(s0[e]), __uint_as_float(s1[e])),
                             fmaxf(__uint_as_float(s2[e]), __uint_as_float(s3[e]))));
      }
      const float mt = mx * c2;   // row maximum of the scaled scores, log2 domain
      bool retain = true;
      if (!kDense) {
        // Eq. 3: skip iff rowmax - (m + log l) < log(tau / L) for every valid row
        bool vote;
        if (l == 0.f) vote = valid;   // nothing retained yet: the log-ratio is +inf
        else vote = valid && !(((mt - (m_ref + log2f(l))) - theta) < 0.f);
        const bool any = __any_sync(0xffffffffu, vote);
        if (lane == 0) {
          if (any) *(volatile int*)&flag[t % 3] = 1;
          if (warp == (kDecode ? 4 : 2)) *(volatile int*)&flag[(t + 1) % 3] = 0;
          tc_fence_before();
          mbar_arrive(&vote_bar[t & 1]);
        }
        ok = mbar_wait(&vote_bar[t & 1], (t >> 1) & 1, status);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        retain = (*(volatile int*)&flag[t % 3]) != 0;
      }
      if (!retain) continue;   // m, l, O unchanged; no exp, no P, no V load, no PV
      if (stat_thread && bm_row) {
        const int bit = kDecode ? (T - 1 - t) : j;   // decode: tile index inside the split
        if ((bit >> 5) != bm_word) {
          if (bm_word >= 0) bm_row[bm_word] = bm_bits;
          bm_word = bit >> 5;
          bm_bits = 0;
        }
        bm_bits |= 1u << (bit & 31);
      }
      // running maximum with lazy rescaling: the reference m_ref only moves when the row maximum
      // grew by more than 2^8, so P stays <= 256 and O is rarely touched
      if (r == 0) {
        m_ref = mt;
      } else {
        const bool need = mt > m_ref + 8.f;
        if (__any_sync(0xffffffffu, need)) {
          ok = mbar_wait(&o_done, (r - 1) & 1, status);   // PV of the previous retained tile has landed
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          tc_fence_after();
          const float m_new = fmaxf(m_ref, mt);
          const float alpha = fast_exp2(m_ref - m_new);
          l *= alpha;
          m_ref = m_new;
#pragma unroll
          for (int c = 0; c < D / 32; ++c) {
            uint32_t o[32];
            tmem_ld_x32(tmem_addr(tb, lane_base, Cfg::kColO + c * 32), o);
            tmem_wait_ld();
#pragma unroll
            for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
            tmem_st_x32(tmem_addr(tb, lane_base, Cfg::kColO + c * 32), o);
          }
        }
      }
      // P = exp2(s * c2 - m_ref), row sum in fp32 before the bf16 cast, P written over S
      const float nm = -m_ref;
      float sum = 0.f;
      uint32_t pk[16];
#define MALA_P_CHUNK(SRC, COL)                                                     \
      {                                                                            \
        _Pragma("unroll") for (int e = 0; e < 16; ++e) {                           \
          const float p0 = fast_exp2(fmaf(__uint_as_float(SRC[2 * e]), c2, nm));    \
          const float p1 = fast_exp2(fmaf(__uint_as_float(SRC[2 * e + 1]), c2, nm));\
          sum += p0 + p1;                                                          \
          pk[e] = pack_bf16x2(p0, p1);                                             \
        }                                                                          \
        tmem_st_x16(tmem_addr(tb, lane_base, colS + (COL)), pk);                   \
      }
      MALA_P_CHUNK(s0, 0)
      MALA_P_CHUNK(s1, 16)
      MALA_P_CHUNK(s2, 32)
      MALA_P_CHUNK(s3, 48)
#undef MALA_P_CHUNK
      l += sum;
      tmem_wait_st();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&p_full[t & 1]);
      ++r;
    }

    if (kDecode) {
      if (ok && T > 0) {
        // every PV has retired (o_done's parity alone cannot tell one pending PV from two)
        ok = mbar_wait(&fin_bar, 0, status);
        ok = __all_sync(0xffffffffu, ok);
      }
      if (ok) {
        // partial output of this split: O / l in fp32 and its log-normalizer (empty split: 0, -inf)
        tc_fence_after();
        const float inv = T > 0 ? 1.f / l : 0.f;
        const size_t prow = ((size_t)b * p.Hq + h + rl) * p.num_splits + i;
#pragma unroll
        for (int c = 0; c < D / 32; ++c) {
          uint32_t o[32];
          if (T > 0) {
            tmem_ld_x32(tmem_addr(tb, lane_base, Cfg::kColO + c * 32), o);
            tmem_wait_ld();
          } else {
#pragma unroll
            for (int e = 0; e < 32; ++e) o[e] = 0u;
          }
          if (valid) {
            float4* dst = reinterpret_cast<float4*>(p.o_part + prow * D + c * 32);
#pragma unroll
            for (int v = 0; v < 8; ++v)
              dst[v] = make_float4(__uint_as_float(o[4 * v]) * inv, __uint_as_float(o[4 * v + 1]) * inv,
                                   __uint_as_float(o[4 * v + 2]) * inv, __uint_as_float(o[4 * v + 3]) * inv);
          }
        }
        if (valid) p.lse_part[prow] = T > 0 ? (m_ref + log2f(l)) * 0.6931471805599453f : -INFINITY;
        if (stat_thread) {
          if (bm_row && bm_word >= 0) bm_row[bm_word] = bm_bits;
          if (p.retained) p.retained[stat_row] = (uint32_t)r;
          if (p.totals) {
            atomicAdd(&p.totals[0], (unsigned long long)r);
            atomicAdd(&p.totals[1], (unsigned long long)T);
          }
        }
      }
    } else {
    if (ok) {
      // finalize: O <- O / l, lse <- m + log l, once every PV has retired (the issuer commits fin_bar
      // after its last MMA; o_done's parity alone cannot tell one pending PV from two)
      ok = mbar_wait(&fin_bar, 0, status);
      ok = __all_sync(0xffffffffu, ok);
    }
    if (ok) {
      tc_fence_after();
      const float inv = 1.f / l;
      __nv_bfloat16* orow = p.o + (int64_t)b * p.o_sb + (int64_t)row * p.o_sn + (int64_t)h * p.o_sh;
#pragma unroll
      for (int c = 0; c < D / 32; ++c) {
        uint32_t o[32];
        tmem_ld_x32(tmem_addr(tb, lane_base, Cfg::kColO + c * 32), o);
        tmem_wait_ld();
        if (valid) {
#pragma unroll
          for (int v = 0; v < 4; ++v) {
            uint4 w;
            w.x = pack_bf16x2(__uint_as_float(o[8 * v + 0]) * inv, __uint_as_float(o[8 * v + 1]) * inv);
            w.y = pack_bf16x2(__uint_as_float(o[8 * v + 2]) * inv, __uint_as_float(o[8 * v + 3]) * inv);
            w.z = pack_bf16x2(__uint_as_float(o[8 * v + 4]) * inv, __uint_as_float(o[8 * v + 5]) * inv);
            w.w = pack_bf16x2(__uint_as_float(o[8 * v + 6]) * inv, __uint_as_float(o[8 * v + 7]) * inv);
            *reinterpret_cast<uint4*>(orow + c * 32 + v * 8) = w;
          }
        }
      }
      if (valid) p.lse[((size_t)b * p.Hq + h) * p.N + row] = (m_ref + log2f(l)) * 0.6931471805599453f;
      if (stat_thread) {
        if (bm_row && bm_word >= 0) bm_row[bm_word] = bm_bits;
        if (p.retained) p.retained[stat_row] = (uint32_t)r;
        if (p.totals) {
          atomicAdd(&p.totals[0], (unsigned long long)r);
          atomicAdd(&p.totals[1], (unsigned long long)T);
        }
      }
    }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tb, Cfg::kTmemCols);
}

}  // namespace mala
