// MALA forward (Algorithm 1) for sm_100a, prefill version: two query blocks per CTA (one with a head size above 128).
//
// One CTA owns the two consecutive 128-row query blocks A = 2c and B = 2c+1 of one (batch, query
// head).  They share the K tiles; each block has its own UMMA-issuing warp, softmax warpgroup,
// score buffer, V stage and output accumulator (TMEM: S_A, S_B, O_A, O_B = 512 columns).  Per block the
// chain S = QK^T -> row max -> exp -> O += PV -> next QK is strictly serial (P overwrites S: there is no
// TMEM left for a second score buffer), so one block's rows are in the softmax path while the tensor
// pipe works for the other block, and the two softmax groups take turns in the exponential phase.
// Each block keeps the semantics of Algorithm 1 on its own: its tiles are visited from ITS diagonal
// toward earlier keys, the test for a tile uses the state left by that block's previous retained tile,
// and a skipped tile issues no exp, no P, no V load and no PV.
//
// Warp roles (384 threads):
//   warp 0       TMA producer: Q_A, Q_B once, K ring (a K stage is released when both issuers are done)
//   warp 1, 2    UMMA issuers of block A and B: S_X = Q_X K^T for every tile, then (after the vote) the V
//                load of that block and O_X += P_X V; the next QK of X follows its PV in program order, so
//                the single score buffer of X is reused in tensor-pipe order without a barrier
//   warps 4-7    softmax group of block A, warps 8-11 of block B (one thread per query row)
// All synchronisation is by mbarriers with bounded waits.
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
  int B, Hq, Hkv, N, Tr, words, causal;   // N, Tr: query rows and query blocks
  int Nk, Tk, koff;              // keys, key blocks; causal: the queries are the last N positions, koff = (Nk - N) / 128
  int qshift;                    // causal: (Nk - N) % 128.  The query blocks follow the key positions: block i holds
                                 // the rows q with 128 i <= q + qshift < 128 (i + 1), Tr = ceil((N + qshift) / 128),
                                 // and its newest legal key block is i + koff
  // Packed sequences of different lengths (null: B sequences of N rows each): sequence b holds rows
  // cu[b] .. cu[b+1]-1 of q, k, v, o (which are then [1, total, H, d] tensors); lse is [Hq, total]; N, Tr, Nk, Tk
  // above describe the longest sequence (grid, telemetry strides)
  const int* cu;
  int total;
  // Keys and values in pages (null: not paged): k, v are [num_pages, page_size, Hkv, D] with page_size a multiple of
  // 128; keys 128 x .. of sequence b lie in page block_table[b * bt_stride + x / tpp]; it has seqlens_k[b] keys and
  // its queries (packed, cu) are its last positions
  const int* block_table;
  const int* seqlens_k;
  int bt_stride, tpp;
  // Pages smaller than a tile (8, 16, 32 or 64 keys): ppt = 128 / page_size copies of prows = page_size rows make
  // up a tile, copy c of key block x from page block_table[b * bt_stride + x * ppt + c] (tpp = 1 then; a table
  // entry past the row's end reads as "no page": zeros).  ppt = 1 otherwise.
  int ppt, prows;
  const int* cu_k;               // packed sequences whose keys are longer than their queries (a cached prefix): the keys
                                 // of sequence b are rows cu_k[b] .. cu_k[b+1]-1 of k, v; its queries are the last
                                 // positions (null: keys as queries)
  // Key range cut into num_splits ranges of tps key blocks (num_splits > 1): grid z = b * num_splits + split; a CTA
  // runs its blocks on the key blocks of its range only and writes the normalised fp32 result and the
  // log-normalizer of the range; a merge kernel combines the ranges.
  int num_splits, tps;
  float* o_part;                 // [B, Hq, num_splits, N, D]
  int d;                         // head size of the tensors (<= D; the columns d .. D-1 are zeros and never stored)
  float* lse_part;               // [B, Hq, num_splits, N] natural log
  float scale_log2;              // scale * log2(e)
  float log2_tau;                // log2(tau); unused by the dense kernel
};

template <int D, bool kDense>
struct FwdCfg {
  static constexpr int kPanels = D / 64;
  static constexpr int kTileBytes = 128 * D * 2;
  // Head sizes above 128: a tile is 64 KB, so a CTA owns ONE query block (block A; the warps of block B find no
  // block) with one Q tile, one K stage and one V stage, and its accumulators S (128 columns) and O (256) fill the
  // tensor memory that two blocks of 128 columns fill otherwise.
  static constexpr bool kOne = D > 128;
  static constexpr int kKStages = kOne ? 1 : 3;
  static constexpr int kBlocks = kOne ? 1 : 2;     // Q tiles and V stages
  // Q_A, Q_B, K ring, V_A, V_B
  static constexpr int kSmemBytes = (kBlocks + kKStages + kBlocks) * kTileBytes + 1024;
  static constexpr int kThreads = 384;
  static constexpr uint32_t kTmemCols = 512;
};

// kSmall: the keys and values lie in pages smaller than a tile (a kernel of its own, so that the copy loop with its
// table lookups costs the other layouts nothing).
template <int D, bool kDense, bool kSmall = false>
__global__ void __launch_bounds__(384, 1)
mala_fwd_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                 const __grid_constant__ CUtensorMap tmV, const FwdParams p) {
  using Cfg = FwdCfg<D, kDense>;
  constexpr int KS = Cfg::kKStages, PAN = Cfg::kPanels, VS = Cfg::kBlocks;
  constexpr bool kOne = Cfg::kOne;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint8_t* sQ = smem;                               // [2] blocks A, B
  uint8_t* sK = sQ + Cfg::kBlocks * Cfg::kTileBytes;
  uint8_t* sV = sK + KS * Cfg::kTileBytes;          // [2] blocks A, B

  __shared__ uint64_t q_full, k_full[KS], k_empty[KS], v_full[2], v_empty[2], s_full[2], vote_bar[2], p_full[2][2],
      fin_bar, turn_bar[2];
  __shared__ uint32_t tmem_base_s;
  __shared__ int flag[2][3];
  __shared__ int early_exit;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int G = p.Hq / p.Hkv;
  const int sp = p.num_splits > 1 ? (int)blockIdx.z % p.num_splits : 0;
  const int b = p.num_splits > 1 ? (int)blockIdx.z / p.num_splits : (int)blockIdx.z;
  const int h = blockIdx.y, hkv = h / G;
  // this sequence: first rows in the tensors, rows, keys, blocks
  const int row0 = p.cu ? __ldg(p.cu + b) : 0;
  const int Nq = p.cu ? __ldg(p.cu + b + 1) - row0 : p.N;
  const bool own_keys = p.cu_k || p.block_table;      // the sequence's key count differs from its query count
  const int krow0 = p.cu_k ? __ldg(p.cu_k + b) : row0;
  // (paged: a length beyond what the block table's row can map is clamped, so no lookup ever leaves the row)
  const int Nkeys = p.block_table ? min(__ldg(p.seqlens_k + b), p.bt_stride * (p.ppt > 1 ? p.prows : p.tpp * 128))
                                  : (p.cu_k ? __ldg(p.cu_k + b + 1) - krow0 : (p.cu ? Nq : p.Nk));
  if (own_keys && (Nkeys <= 0 || (p.causal && Nkeys < Nq))) return;   // (not defined: no keys, more queries than keys)
  const int koff = own_keys ? (p.causal ? (Nkeys - Nq) / 128 : 0) : p.koff;
  const int qshift = own_keys ? (p.causal ? (Nkeys - Nq) % 128 : 0) : p.qshift;
  // TMA coordinates (key row, outermost index) of key block jt
  auto key_coord = [&](int jt, int& row, int& outer) {
    if (p.block_table) {
      const int pg = jt / p.tpp;
      outer = __ldg(p.block_table + (size_t)b * p.bt_stride + pg);
      row = (jt - pg * p.tpp) * 128;
    } else {
      outer = p.cu ? 0 : b;
      row = krow0 + jt * 128;
    }
  };
  auto load_tile_small = [&](uint8_t* dst, const CUtensorMap* tm, uint64_t* bar, int jt) {
    for (int c = 0; c < p.ppt; ++c) {
      const int pg = jt * p.ppt + c;
      const int outer = pg < p.bt_stride ? __ldg(p.block_table + (size_t)b * p.bt_stride + pg) : -1;
#pragma unroll
      for (int pn = 0; pn < D / 64; ++pn) tma_load_4d(dst + pn * 16384 + c * p.prows * 128, tm, bar, pn * 64, 0, hkv, outer);
    }
  };
  constexpr bool small_pages = kSmall;
  const int Tr = p.cu ? (Nq + qshift + 127) / 128 : p.Tr;
  const int Tk = p.cu ? (Nkeys + 127) / 128 : p.Tk;
  const int bz = p.cu ? 0 : b;                        // outermost TMA coordinate
  const int npairs = kOne ? Tr : (Tr + 1) / 2;
  if ((int)blockIdx.x >= npairs) return;             // (a sequence shorter than the longest one)
  const int c = npairs - 1 - (int)blockIdx.x;        // longest pairs first
  int iA = kOne ? c : 2 * c, iB = kOne ? c : 2 * c + 1;
  bool hasB = !kOne && iB < Tr;
  int dA = p.causal ? iA + koff : Tk - 1;            // newest key block with a legal key, per block
  const int dB = p.causal ? iB + koff : Tk - 1;
  int jlo = 0, jhi = Tk - 1;                         // key blocks of this CTA
  if (p.num_splits > 1) {
    jlo = sp * p.tps;
    jhi = min(Tk, jlo + p.tps) - 1;
    if (jlo > dA) {                                  // the range holds no legal key of block A
      if (!hasB || jlo > dB) return;                 // ... nor of block B: nothing to do (the merge knows)
      iA = iB; dA = dB; hasB = false;                // only B's diagonal block: run B alone
    }
  }
  // key steps u = 0 .. U-1 visit key block j0 - u; block X takes part from step first[X] on
  const int hA = min(dA, jhi), hB = min(dB, jhi);    // first key block each block visits
  const int j0 = hasB ? hB : hA;
  const int U = j0 - jlo + 1;
  const int firstA = hasB ? hB - hA : 0;             // 1 when B's diagonal key block, not legal for A, is in the range
  int* status = p.status;

  if (tid == 0) {
    early_exit = (*(volatile int*)status != 0);
    mbar_init(&q_full, 1);
    for (int s = 0; s < KS; ++s) { mbar_init(&k_full[s], 1); mbar_init(&k_empty[s], 2); }
    for (int x = 0; x < 2; ++x) {
      mbar_init(&v_full[x], 1); mbar_init(&v_empty[x], kDense ? 2 : 1);
      mbar_init(&s_full[x], 1); mbar_init(&vote_bar[x], 4); mbar_init(&p_full[x][0], 4); mbar_init(&p_full[x][1], 4);
      flag[x][0] = flag[x][1] = flag[x][2] = 0;
    }
    mbar_init(&fin_bar, 2);
    mbar_init(&turn_bar[0], 4); mbar_init(&turn_bar[1], 4);
    mbar_fence_init();
  }
  __syncthreads();
  if (early_exit) return;
  if (warp == 0) { tmem_alloc(&tmem_base_s, Cfg::kTmemCols); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tb = tmem_base_s;
  if (warp < 4) {
  // warps 0-3 (producer, issuers) need few registers; the two softmax warpgroups take the rest
  reg_dealloc<72>();
  if (warp == 0 && kSmall) {
    // ------------------------------------------------------------------ TMA producer, pages smaller than a tile:
    // the loop of the producer below run by all 32 lanes (waits and counters warp-uniform); lane x issues copy
    // x / PAN of panel x % PAN of a tile, so the table lookups are one coalesced load and the copies are issued side
    // by side instead of one after the other
    auto load_tile_small_warp = [&](uint8_t* dst, const CUtensorMap* tm, uint64_t* bar, int jt) {
      const int pn = lane % PAN;
      // (up to 16 copies of PAN panels: one per lane with up to two panels, two rounds with four)
      for (int c = lane / PAN; c < p.ppt; c += 32 / PAN) {
        const int pg = jt * p.ppt + c;
        const int outer = pg < p.bt_stride ? __ldg(p.block_table + (size_t)b * p.bt_stride + pg) : -1;
        tma_load_4d(dst + pn * 16384 + c * p.prows * 128, tm, bar, pn * 64, 0, hkv, outer);
      }
    };
    if (lane == 0) {
      tma_prefetch_desc(&tmQ); tma_prefetch_desc(&tmK); tma_prefetch_desc(&tmV);
      mbar_arrive_expect_tx(&q_full, (hasB ? 2 : 1) * Cfg::kTileBytes);
      for (int pn = 0; pn < PAN; ++pn) {
        tma_load_4d(sQ + pn * 16384, &tmQ, &q_full, pn * 64, row0 + iA * 128 - qshift, h, bz);
        if (hasB)
          tma_load_4d(sQ + Cfg::kTileBytes + pn * 16384, &tmQ, &q_full, pn * 64, row0 + iB * 128 - qshift, h, bz);
      }
    }
    int issued = 0, v_issued = 0, s = 0;
    uint32_t par = 1;
    bool ok = true;
    for (int u = 0; u < U && ok; ++u) {
      ok = mbar_wait_warp(&k_empty[s], par, status);
      if (!ok) break;
      if (lane == 0) mbar_arrive_expect_tx(&k_full[s], Cfg::kTileBytes);
      __syncwarp();
      load_tile_small_warp(sK + s * Cfg::kTileBytes, &tmK, &k_full[s], j0 - u);
      issued = u + 1;
      if (++s == KS) { s = 0; par ^= 1; }
      if (kDense) {
        ok = mbar_wait_warp(&v_empty[u % VS], ((u / VS) & 1) ^ 1, status);
        if (!ok) break;
        if (lane == 0) mbar_arrive_expect_tx(&v_full[u % VS], Cfg::kTileBytes);
        __syncwarp();
        load_tile_small_warp(sV + (u % VS) * Cfg::kTileBytes, &tmV, &v_full[u % VS], j0 - u);
        v_issued = u + 1;
      }
    }
    if (!ok && lane == 0) {
      mbar_wait(&q_full, 0, status);
      for (int u = (issued > KS ? issued - KS : 0); u < issued; ++u) mbar_wait(&k_full[u % KS], (u / KS) & 1, status);
      for (int u = (v_issued > VS ? v_issued - VS : 0); u < v_issued; ++u) mbar_wait(&v_full[u % VS], (u / VS) & 1, status);
    }
  } else if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer: Q_A, Q_B, K ring
    if (lane == 0) {
      tma_prefetch_desc(&tmQ); tma_prefetch_desc(&tmK); tma_prefetch_desc(&tmV);
      mbar_arrive_expect_tx(&q_full, (hasB ? 2 : 1) * Cfg::kTileBytes);
      for (int pn = 0; pn < PAN; ++pn) {
        // (the first block of a chunk that starts inside a tile begins before row 0: those rows read as zeros)
        tma_load_4d(sQ + pn * 16384, &tmQ, &q_full, pn * 64, row0 + iA * 128 - qshift, h, bz);
        if (hasB)
          tma_load_4d(sQ + Cfg::kTileBytes + pn * 16384, &tmQ, &q_full, pn * 64, row0 + iB * 128 - qshift, h, bz);
      }
      int issued = 0, v_issued = 0, s = 0;
      uint32_t par = 1;                 // parity of the "empty" phase to wait for (first pass: free)
      bool ok = true;
      for (int u = 0; u < U && ok; ++u) {
        int krow, kouter;
        key_coord(j0 - u, krow, kouter);   // (a page lookup is in flight while the stage is waited for)
        ok = mbar_wait(&k_empty[s], par, status);
        if (!ok) break;
        mbar_arrive_expect_tx(&k_full[s], Cfg::kTileBytes);
        for (int pn = 0; pn < PAN; ++pn)
          tma_load_4d(sK + s * Cfg::kTileBytes + pn * 16384, &tmK, &k_full[s], pn * 64, krow, hkv, kouter);
        issued = u + 1;
        if (++s == KS) { s = 0; par ^= 1; }
        if (kDense) {   // dense: every tile is retained, so V(u) is prefetched into the shared 2-stage ring
          ok = mbar_wait(&v_empty[u % VS], ((u / VS) & 1) ^ 1, status);
          if (!ok) break;
          mbar_arrive_expect_tx(&v_full[u % VS], Cfg::kTileBytes);
          for (int pn = 0; pn < PAN; ++pn)
            tma_load_4d(sV + (u % VS) * Cfg::kTileBytes + pn * 16384, &tmV, &v_full[u % VS], pn * 64, krow, hkv, kouter);
          v_issued = u + 1;
        }
      }
      if (!ok) {
        mbar_wait(&q_full, 0, status);
        for (int u = (issued > KS ? issued - KS : 0); u < issued; ++u) mbar_wait(&k_full[u % KS], (u / KS) & 1, status);
        for (int u = (v_issued > VS ? v_issued - VS : 0); u < v_issued; ++u) mbar_wait(&v_full[u % VS], (u / VS) & 1, status);
      }
    }
  } else if (warp == 1 || warp == 2) {
    // ------------------------------------------------------------------ UMMA issuer of block x (+ its V loads)
    // All 32 lanes run this loop with identical values; MMAs, commits, arrivals and TMA loads are issued by
    // one elected lane.
    const int x = warp - 1;
    {
      const uint32_t leader = elect_one();
      constexpr uint32_t idesc_qk = make_idesc_bf16(128, 128, false, false);
      constexpr uint32_t idesc_pv = make_idesc_bf16(128, D, false, true);
      const bool present_x = (x == 0) || hasB;
      const int first = (x == 0) ? firstA : 0;
      const uint64_t dQ = make_smem_desc(smem_u32(sQ + x * Cfg::kTileBytes), 16, 1024);
      const uint64_t dK0 = make_smem_desc(smem_u32(sK), 16, 1024);
      const uint64_t dV0 = make_smem_desc(smem_u32(sV), 16384, 1024);
      const uint32_t tS = tmem_addr(tb, 0, x * 128), tO = tmem_addr(tb, 0, 256 + x * 128);
      bool ok = mbar_wait_warp(&q_full, 0, status);
      int r = 0;                       // PVs issued (retained tiles); also counts this block's V loads
      int s = 0;                       // K stage of the next step to be scored
      uint32_t kpar = 0;               // parity of k_full[s] for that step
      // S = Q K^T of the step whose K sits in stage s (k_full already observed)
      auto issue_qk = [&]() {
        tc_fence_after();
        const uint64_t dK = desc_advance(dK0, s * Cfg::kTileBytes);
#pragma unroll
        for (int k = 0; k < D / 16; ++k) {
          const uint32_t off = (k >> 2) * 16384 + (k & 3) * 32;
          mma_ss(tS, desc_advance(dQ, off), desc_advance(dK, off), idesc_qk, k > 0, leader);
        }
        if (leader) { tc_commit(&k_empty[s]); tc_commit(&s_full[x]); }
        if (++s == KS) { s = 0; kpar ^= 1; }
      };
      // steps at which this block has no tile (all of them for an absent block): only release the stages
      int u = 0;
      for (; u < U && ok && (!present_x || u < first); ++u) {
        ok = mbar_wait_warp(&k_full[s], kpar, status);
        if (!ok) break;
        if (leader) mbar_arrive(&k_empty[s]);
        if (kDense) {                  // release the shared V stage too, paced by its arrival
          ok = mbar_wait_warp(&v_full[u % VS], (u / VS) & 1, status);
          if (!ok) break;
          if (leader) mbar_arrive(&v_empty[u % VS]);
        }
        if (++s == KS) { s = 0; kpar ^= 1; }
      }
      if (ok && u < U) {
        ok = mbar_wait_warp(&k_full[s], kpar, status);
        if (ok) issue_qk();
      }
      // Per tile: everything that does not depend on P (the next step's K, whose copy landed long ago) is observed
      // before the wait for P, so that between the second half of P and the next S = Q K^T only the PV and QK
      // issue themselves remain -- this warp runs a serial instruction stream, and every instruction on the path from
      // "P is there" to "the next scores are there" lengthens the block's per-tile chain.
      for (; u < U && ok; ++u) {
        const int t = u - first;       // tile index of this block
        const bool has_next = (u + 1 < U);
        if (has_next) {
          ok = mbar_wait_warp(&k_full[s], kpar, status);
          if (!ok) break;
        }
        bool retain = true;
        if (!kDense) {
          ok = mbar_wait_warp(&vote_bar[x], t & 1, status);
          if (!ok) break;
          retain = __shfl_sync(0xffffffffu, *(volatile int*)&flag[x][t % 3], 0) != 0;
        }
        if (retain) {
          // MALA: V is loaded on demand into this block's own stage (free once its previous PV retired);
          // dense: V(u) sits in the shared ring stage u & 1
          const int vs = kDense ? (u % VS) : x;
          const uint32_t vpar = kDense ? ((u / VS) & 1) : (r & 1);
          if (!kDense) {
            ok = mbar_wait_warp(&v_empty[x], (r & 1) ^ 1, status);
            if (!ok) break;
            if (leader) {
              mbar_arrive_expect_tx(&v_full[x], Cfg::kTileBytes);
              if (small_pages) {
                load_tile_small(sV + x * Cfg::kTileBytes, &tmV, &v_full[x], j0 - u);
              } else {
                int vrow, vouter;
                key_coord(j0 - u, vrow, vouter);
                for (int pn = 0; pn < PAN; ++pn)
                  tma_load_4d(sV + x * Cfg::kTileBytes + pn * 16384, &tmV, &v_full[x], pn * 64, vrow, hkv, vouter);
              }
            }
            __syncwarp();
          }
          const uint32_t acc0 = r > 0 ? 1u : 0u;
          const uint64_t dVs = desc_advance(dV0, vs * Cfg::kTileBytes);
          // P arrives in two halves of 64 keys: the first four k-steps of O += P V run while the second half
          // of the exponentials is still being computed
          ok = mbar_wait_warp(&v_full[vs], vpar, status);
          if (ok) ok = mbar_wait_warp(&p_full[x][0], r & 1, status);
          if (!ok) break;
          tc_fence_after();
#pragma unroll
          for (int k = 0; k < 4; ++k)
            mma_ts(tO, tS + k * 8, desc_advance(dVs, k * 2048), idesc_pv, k > 0 ? 1u : acc0, leader);
          ok = mbar_wait_warp(&p_full[x][1], r & 1, status);
          if (!ok) break;
          tc_fence_after();
#pragma unroll
          for (int k = 4; k < 8; ++k)
            mma_ts(tO, tS + k * 8, desc_advance(dVs, k * 2048), idesc_pv, 1u, leader);
          if (leader) tc_commit(&v_empty[vs]);
          ++r;
        }
        if (has_next) issue_qk();      // in tensor-pipe order after this tile's PV: the score buffer is reused
      }
      // every MMA of this block has retired (and every V copy landed) before the CTA may exit
      __syncwarp();
      if (leader) tc_commit(&fin_bar);
      mbar_wait_warp(&fin_bar, 0, status);
      if (!kDense && !ok && r > 0) mbar_wait_warp(&v_full[x], (r - 1) & 1, status);
    }
  }
  } else {
    reg_alloc<208>();
    // ------------------------------------------------------------------ softmax groups: one thread per row
    const int x = (warp - 4) >> 2;                   // 0 = block A, 1 = block B
    const int i = x ? iB : iA;
    const bool present_x = (x == 0) || hasB;
    const uint32_t lane_base = (uint32_t)(warp & 3) * 32u;
    const int rl = (int)lane_base + lane;
    const int prow_ = i * 128 + rl;                   // row counted in whole blocks from the first block's start
    const int row = prow_ - qshift;                   // row of q, o, lse
    const bool valid = row >= 0 && row < Nq;
    const float c2 = p.scale_log2;
    const float Lq = p.causal ? (float)(prow_ + 1 + koff * 128) : (float)Nkeys;   // visible keys
    const float theta = kDense ? -INFINITY : (p.log2_tau - log2f(Lq));
    const uint32_t colS = (uint32_t)x * 128u, colO = 256u + (uint32_t)x * 128u;
    const int first = (x == 0) ? firstA : 0;
    const int T = present_x ? (U - first) : 0;       // tiles of this block
    const bool mask_first = x ? (hB == dB) : (hA == dA);
    float m_ref = -INFINITY, l = 0.f;
    int r = 0;
    bool ok = true;
    uint32_t bm_bits = 0;
    int bm_word = -1;
    const bool stat_thread = ((warp & 3) == 0 && lane == 0);
    const size_t stat_row = (size_t)(b * p.Hq + h) * p.Tr + i;
    uint32_t* bm_row = (p.bitmask && present_x) ? p.bitmask + stat_row * p.words : nullptr;

    for (int t = 0; t < T; ++t) {
      const int j = j0 - first - t;
      ok = mbar_wait(&s_full[x], t & 1, status);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      uint32_t s0[32], s1[32], s2[32], s3[32];
      tmem_ld_x32(tmem_addr(tb, lane_base, colS + 0), s0);
      tmem_ld_x32(tmem_addr(tb, lane_base, colS + 32), s1);
      tmem_ld_x32(tmem_addr(tb, lane_base, colS + 64), s2);
      tmem_ld_x32(tmem_addr(tb, lane_base, colS + 96), s3);
      tmem_wait_ld();
      if (t == 0 && mask_first) {
        // first visited tile, when it is the block's newest legal one: causal diagonal and / or the ragged end of
        // the keys
        const int lim = p.causal ? rl : (Nkeys - 1 - j * 128);
        const uint32_t ninf = 0xff800000u;
#pragma unroll
        for (int e = 0; e < 32; ++e) {
          if (e > lim) s0[e] = ninf;
          if (e + 32 > lim) s1[e] = ninf;
          if (e + 64 > lim) s2[e] = ninf;
          if (e + 96 > lim) s3[e] = ninf;
        }
      }
      // row maximum of the 128 scores: four chains of three-input maxima (half the instructions of pairwise maxima)
      float mx[4];
      mx[0] = __uint_as_float(s0[0]); mx[1] = __uint_as_float(s1[0]); mx[2] = __uint_as_float(s2[0]); mx[3] = __uint_as_float(s3[0]);
#pragma unroll
      for (int e = 1; e < 31; e += 2) {
        mx[0] = max3(mx[0], __uint_as_float(s0[e]), __uint_as_float(s0[e + 1]));
        mx[1] = max3(mx[1], __uint_as_float(s1[e]), __uint_as_float(s1[e + 1]));
        mx[2] = max3(mx[2], __uint_as_float(s2[e]), __uint_as_float(s2[e + 1]));
        mx[3] = max3(mx[3], __uint_as_float(s3[e]), __uint_as_float(s3[e + 1]));
      }
      // row maximum of the scaled scores, log2 domain
      const float mt = fmaxf(max3(mx[0], mx[1], __uint_as_float(s0[31])), max3(mx[2], mx[3], fmaxf(fmaxf(__uint_as_float(s1[31]), __uint_as_float(s2[31])), __uint_as_float(s3[31])))) * c2;
      bool retain = true;
      if (!kDense) {
        // Eq. 3: skip iff rowmax - (m + log l) < log(tau / L) for every valid row
        bool vote;
        if (l == 0.f) vote = valid;   // nothing retained yet: the log-ratio is +inf
        else vote = valid && !(((mt - (m_ref + __log2f(l))) - theta) < 0.f);
        const bool any = __any_sync(0xffffffffu, vote);
        if (lane == 0) {
          if (any) *(volatile int*)&flag[x][t % 3] = 1;
          if ((warp & 3) == 0) *(volatile int*)&flag[x][(t + 1) % 3] = 0;
          tc_fence_before();
          mbar_arrive(&vote_bar[x]);
        }
        // A warp that found a retaining row knows the outcome (the vote is an OR) and goes straight on; only a warp
        // without one has to wait for the other three.
        if (!any) {
          ok = mbar_wait(&vote_bar[x], t & 1, status);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          retain = (*(volatile int*)&flag[x][t % 3]) != 0;
        }
      }
      if (!kDense) retain = __all_sync(0xffffffffu, retain);   // same value in every lane: the branch below is uniform
      if (!retain) {   // m, l, O unchanged; no exp, no P, no PV: take the turn (see below) and pass it on at once
        if (!kDense && hasB) {
          const int idx = (x == 0) ? t : (t - 1 - firstA);
          if (idx >= 0) {
            ok = mbar_wait(&turn_bar[x], idx & 1, status);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
          }
          __syncwarp();
          if (lane == 0 && (x == 0 || t >= firstA)) mbar_arrive(&turn_bar[1 - x]);
        }
        continue;
      }
      if (stat_thread && bm_row) {
        if ((j >> 5) != bm_word) {
          if (bm_word >= 0) {
            if (p.num_splits > 1) atomicOr(&bm_row[bm_word], bm_bits);   // (ranges share words of the row)
            else bm_row[bm_word] = bm_bits;
          }
          bm_word = j >> 5;
          bm_bits = 0;
        }
        bm_bits |= 1u << (j & 31);
      }
      // Lazy rescaling: the reference maximum only moves when the row maximum grew by more than 2^8.
      // The scores of this tile were produced after every earlier PV of this block (same tensor pipe,
      // program order), so O may be touched here without a further wait.
      // (warp votes stay out of conditional code: there the compiler has to re-converge the warp around each of them)
      const bool need_any = __any_sync(0xffffffffu, r > 0 && mt > m_ref + 8.f);
      if (r == 0) {
        m_ref = mt;
      } else {
        if (need_any) {
          const float m_new = fmaxf(m_ref, mt);
          const float alpha = fast_exp2(m_ref - m_new);
          l *= alpha;
          m_ref = m_new;
#pragma unroll
          for (int cc = 0; cc < D / 32; ++cc) {
            uint32_t o[32];
            tmem_ld_x32(tmem_addr(tb, lane_base, colO + cc * 32), o);
            tmem_wait_ld();
#pragma unroll
            for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
            tmem_st_x32(tmem_addr(tb, lane_base, colO + cc * 32), o);
          }
        }
      }
      // The two softmax groups take turns in the exponential phase (B(0), A(0), B(1), A(1), ...; a skipped tile
      // takes its turn and passes it on at once)
      // so that one block's exponentials run while the tensor pipe works for the other block, instead of
      // both groups contending for the MUFU at the same time and then for the tensor pipe at the same time.
      // A's tile t follows B's tile of the same key step (t + firstA); B's tile t follows A's tile of the previous
      // step (t - 1 - firstA).  turn_bar[0] counts B's finished exp phases from tile firstA on, turn_bar[1] A's, so
      // every waiter sees the phases in sequence.
      {
        const int idx = (x == 0) ? t : (t - 1 - firstA);
        bool okw = true;
        if (hasB && idx >= 0) okw = mbar_wait(&turn_bar[x], idx & 1, status);
        ok = __all_sync(0xffffffffu, okw);
        if (!ok) break;
      }
      // P = exp2(s * c2 - m_ref), row sum in fp32 before the bf16 cast, P written over S
      const float nm = -m_ref;
      float sum0 = 0.f, sum1 = 0.f, sum2 = 0.f, sum3 = 0.f;
      uint32_t pk[16];
#define MALA_P_CHUNK(SRC, COL)                                                         \
      {                                                                                \
        _Pragma("unroll") for (int e = 0; e < 8; ++e) {                                \
          const float p0 = fast_exp2(fmaf(__uint_as_float(SRC[4 * e]), c2, nm));        \
          const float p1 = fast_exp2(fmaf(__uint_as_float(SRC[4 * e + 1]), c2, nm));    \
          const float p2 = fast_exp2(fmaf(__uint_as_float(SRC[4 * e + 2]), c2, nm));    \
          const float p3 = fast_exp2(fmaf(__uint_as_float(SRC[4 * e + 3]), c2, nm));    \
          sum0 += p0; sum1 += p1; sum2 += p2; sum3 += p3;                              \
          pk[2 * e] = pack_bf16x2(p0, p1);                                             \
          pk[2 * e + 1] = pack_bf16x2(p2, p3);                                         \
        }                                                                              \
        tmem_st_x16(tmem_addr(tb, lane_base, colS + (COL)), pk);                       \
      }
      MALA_P_CHUNK(s0, 0)
      MALA_P_CHUNK(s1, 16)
      tmem_wait_st();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&p_full[x][0]);   // keys 0..63 of P are in place
      MALA_P_CHUNK(s2, 32)
      // hand the exponential phase over a little before it ends: the other group needs a few hundred cycles
      // to notice, and the MUFU would idle meanwhile
      __syncwarp();
      if (lane == 0 && hasB && (x == 0 || t >= firstA)) mbar_arrive(&turn_bar[1 - x]);
      MALA_P_CHUNK(s3, 48)
#undef MALA_P_CHUNK
      l += (sum0 + sum1) + (sum2 + sum3);
      tmem_wait_st();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&p_full[x][1]);
      ++r;
    }

    if (ok && present_x) {
      // finalize once every PV has retired: O <- O / l, lse <- m + log l
      ok = mbar_wait(&fin_bar, 0, status);
      ok = __all_sync(0xffffffffu, ok);
    }
    if (ok && present_x && p.num_splits > 1) {
      // one range of the keys: normalised fp32 partial and the range's log-normalizer
      tc_fence_after();
      const float inv = 1.f / l;
      const size_t prow = (((size_t)b * p.Hq + h) * p.num_splits + sp) * p.N + row;
#pragma unroll
      for (int cc = 0; cc < D / 32; ++cc) {
        uint32_t o[32];
        tmem_ld_x32(tmem_addr(tb, lane_base, colO + cc * 32), o);
        tmem_wait_ld();
        if (valid) {
#pragma unroll
          for (int v = 0; v < 8; ++v)
            if (cc * 32 + v * 4 < p.d)
              *reinterpret_cast<float4*>(p.o_part + prow * D + cc * 32 + v * 4) =
                make_float4(__uint_as_float(o[4 * v]) * inv, __uint_as_float(o[4 * v + 1]) * inv,
                            __uint_as_float(o[4 * v + 2]) * inv, __uint_as_float(o[4 * v + 3]) * inv);
        }
      }
      if (valid) p.lse_part[prow] = (m_ref + log2f(l)) * 0.6931471805599453f;
      if (stat_thread) {   // several ranges add to the same telemetry rows
        if (bm_row && bm_word >= 0) atomicOr(&bm_row[bm_word], bm_bits);
        if (p.retained) atomicAdd(&p.retained[stat_row], (uint32_t)r);
        if (p.totals) {
          atomicAdd(&p.totals[0], (unsigned long long)r);
          atomicAdd(&p.totals[1], (unsigned long long)T);
        }
      }
    } else if (ok && present_x) {
      tc_fence_after();
      const float inv = 1.f / l;
      __nv_bfloat16* orow = p.o + (int64_t)bz * p.o_sb + (int64_t)(row0 + row) * p.o_sn + (int64_t)h * p.o_sh;
#pragma unroll
      for (int cc = 0; cc < D / 32; ++cc) {
        uint32_t o[32];
        tmem_ld_x32(tmem_addr(tb, lane_base, colO + cc * 32), o);
        tmem_wait_ld();
        if (valid) {
#pragma unroll
          for (int v = 0; v < 4; ++v) {
            uint4 w;
            w.x = pack_bf16x2(__uint_as_float(o[8 * v + 0]) * inv, __uint_as_float(o[8 * v + 1]) * inv);
            w.y = pack_bf16x2(__uint_as_float(o[8 * v + 2]) * inv, __uint_as_float(o[8 * v + 3]) * inv);
            w.z = pack_bf16x2(__uint_as_float(o[8 * v + 4]) * inv, __uint_as_float(o[8 * v + 5]) * inv);
            w.w = pack_bf16x2(__uint_as_float(o[8 * v + 6]) * inv, __uint_as_float(o[8 * v + 7]) * inv);
            if (cc * 32 + v * 8 < p.d) *reinterpret_cast<uint4*>(orow + cc * 32 + v * 8) = w;
          }
        }
      }
      if (valid)
        p.lse[p.cu ? (size_t)h * p.total + row0 + row : ((size_t)b * p.Hq + h) * p.N + row] =
            (m_ref + log2f(l)) * 0.6931471805599453f;
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

  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tb, Cfg::kTmemCols);
}

// Merge of the key ranges of the split forward: lse = log sum_s exp(lse_s), o = sum_s exp(lse_s - lse) o_s over the
// ranges that hold a legal key of the row's block (range s does iff s * tps <= the block's newest legal key block).
// One block of D threads per (b, head, row).
template <int D>
__global__ void __launch_bounds__(D)
fwd_merge_splits_kernel(const float* __restrict__ o_part, const float* __restrict__ lse_part,
                        __nv_bfloat16* __restrict__ o, int64_t o_sb, int64_t o_sn, int64_t o_sh,
                        float* __restrict__ lse, int Hq, int N, int num_splits, int tps, int Tk, int koff, int qshift,
                        int causal, int d) {
  const long long idx = blockIdx.x;
  const int row = (int)(idx % N), h = (int)((idx / N) % Hq), b = (int)(idx / ((long long)N * Hq)), c = threadIdx.x;
  const int newest = causal ? (row + qshift) / 128 + koff : Tk - 1;
  const int ns = min(num_splits, newest / tps + 1);
  const size_t base = ((size_t)b * Hq + h) * num_splits;
  float mx = -INFINITY;
  for (int s = 0; s < ns; ++s) mx = fmaxf(mx, lse_part[(base + s) * N + row]);
  float Z = 0.f, acc = 0.f;
  for (int s = 0; s < ns; ++s) {
    const float w = exp2f((lse_part[(base + s) * N + row] - mx) * 1.4426950408889634f);
    Z += w;
    if (c < d) acc += w * o_part[((base + s) * N + row) * D + c];
  }
  if (c < d) o[b * o_sb + (int64_t)row * o_sn + h * o_sh + c] = __float2bfloat16(acc / Z);
  if (c == 0) lse[((size_t)b * Hq + h) * N + row] = mx + logf(Z);
}

inline size_t fwd_split_workspace_bytes(int B, int Hq, int N, int D, int S) {   // D: padded head size
  const int d = D;
  auto align256 = [](size_t x) { return (x + 255) & ~(size_t)255; };
  return align256((size_t)B * Hq * S * N * d * sizeof(float)) + align256((size_t)B * Hq * S * N * sizeof(float));
}

}  // namespace mala
