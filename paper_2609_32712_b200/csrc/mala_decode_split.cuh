// Split-KV decode, split kernel ("Fused decoding execution") for sm_100a, head size 64, 128 or 256.
//
// A work item is one split of one (batch, KV head): the G = Hq/Hkv <= 16 query heads that share the KV head
// are processed together, L = Nk for every head, the tiles of the split are visited newest first with the
// item's own running (m, l), and the item ends with a normalised fp32 partial output and its log-normalizer
// per head.  The kernel is HBM-bound, so it is persistent: one CTA per SM walks over its items with the K / V
// rings and the score buffers running on across item boundaries.
//
// The problem is held transposed, keys (and output channels) in the TMEM lanes and the packed query heads as the
// N = 16 columns of the MMAs:
//     S^T [128 keys x 16]  = K_tile [128 x d] . Q^T [d x 16]        (A = K tile, B = Q tile, both K-major)
//     O^T [d x 16]        += V_tile^T [d x 128 keys] . P^T [128 x 16]  (A = V tile read MN-major, B = P^T from smem)
// so that all 128 softmax threads share a tile's work (16 scores each instead of one lane per head with 128), a
// score buffer takes 16 TMEM columns (ring of four) and P^T is a 4 KB shared-memory tile (ring of four).
//   warp 0     TMA producer: Q of the next item (16 rows), K ring; dense kernel: V ring one tile behind K
//   warp 1     UMMA warp, event driven.  Three cursors walk over the tiles in order: S^T (as soon as a score
//              buffer and the K tile are there), the vote (MALA kernel: the V copy of a retained tile is issued
//              the moment its vote is known) and O^T += V^T P^T (as soon as P^T and V are there).  No step waits
//              for another one's data, so the HBM latency of a V copy that can only be requested after the vote
//              is hidden behind the tiles that follow.
//   warps 4-7  softmax group, thread = key of the tile: per-row maxima and sums by warp shuffles and one small
//              exchange per tile between the four warps, Eq. 3, P^T -> smem; lazy rescale of O^T
//   warps 8-11 second softmax group when the item has eight or more rows: each group takes half of the rows (its
//              own score columns, P^T rows and O^T columns of the same TMEM lanes); the tile is retained if either
//              group's rows need it
// K is always streamed; a skipped tile issues no exp, no P, no V load and no PV.
// The cache may be held in pages (pages of whole tiles, looked up in a block table by the producer, which hands
// the V tile's coordinates to the UMMA warp) and every sequence may have its own length (which then takes the
// place of Nk in the item geometry, in L and in the mask of the newest tile).
#pragma once
#include "sm100_ptx.cuh"

namespace mala {

struct DecParams {
  float* o_part;                 // [B, Sq, Hq, num_splits, 128] fp32, normalised per split
  float* lse_part;               // [B, Sq, Hq, num_splits] natural log; -inf for an empty split
  uint32_t* retained;            // [B, Hkv, num_splits] or null
  uint32_t* bitmask;             // [B, Hkv, num_splits, words] or null (zero-filled by the host)
  unsigned long long* totals;    // [2] or null
  int* status;
  // Paged / variable-length caches (both null for one contiguous cache of Nk keys per sequence):
  const int* seqlens;            // [B] keys held by sequence b (<= Nk); L = seqlens[b] for its rows
  const int* block_table;        // [B, bt_stride] page of the tpp consecutive tiles number x*tpp .. x*tpp + tpp - 1
  int bt_stride, tpp;            // tpp: tiles per page (page size / 128; 1 for smaller pages)
  int ppt, prows;                // pages per tile and keys per page when a page is smaller than a tile (else 1, 128):
                                 // a tile is then fetched as ppt copies of prows rows, block_table holds one entry
                                 // per page
  int Sq;                        // new tokens per sequence (the last Sq positions of the cache); rows = Sq * Hq/Hkv
  int B, Hq, Hkv, Nk, tps, num_splits, words, n_items;   // Nk: longest cache the splits are laid out for
  float scale_log2, log2_tau;
};

// D: columns of the kernel (64, 128 or 256).  With 256 a K / V tile is 64 KB (four panels), the rings hold two K
// tiles and one V tile in the 192 KB that otherwise hold three and three, and O^T has a second pair of accumulators
// for the channels 128 .. 255.
template <int D>
struct DecCfgT {
  static constexpr int kTileBytes = D > 128 ? 128 * 256 * 2 : 128 * 128 * 2;
  static constexpr int kQBytes = D > 128 ? 8192 : 4096;  // 16 rows x 128 (256) columns, 2 KB panels
  static constexpr int kPBytes = 4096;                   // P^T: 16 rows (heads) x 128 keys, two 2 KB panels
  static constexpr int kKStages = D > 128 ? 2 : 3, kVStages = D > 128 ? 1 : 3, kPStages = 4, kSStages = 4;
  static constexpr int kSmemBytes = 2 * kQBytes + (kKStages + kVStages) * kTileBytes + kPStages * kPBytes + 1024;
  static constexpr int kThreads = 384;                   // producer, UMMA warp, two idle warps, up to two softmax groups
  static constexpr uint32_t kTmemCols = 128;             // S^T ring 4 x 16, O^T 2 x 16 (item parity), O^T of channels 128.. 2 x 16
  static constexpr uint32_t kColO = 64, kColOHi = 96;
};
using DecCfg = DecCfgT<128>;

// Warp-wide reduction of N independent values per lane (N a power of two <= 16) in N-ish shuffles instead of 5 N:
// while more than one value is left, a lane hands the half of its values that its partner (lane ^ OFF) keeps to that
// partner and folds the partner's half into the half it keeps; the remaining offsets are plain butterfly steps.
// Afterwards v[0] holds, in every lane, the reduction over the warp of value number lane >> (5 - log2 N).
template <int N, int OFF, bool kMax>
struct RowReduce {
  static __device__ __forceinline__ void run(float* v, int lane) {
    if constexpr (OFF > 0) {
      if constexpr (N > 1) {
        constexpr int H = N / 2;
        const bool up = (lane & OFF) != 0;
#pragma unroll
        for (int i = 0; i < H; ++i) {
          const float send = up ? v[i] : v[i + H];
          const float keep = up ? v[i + H] : v[i];
          const float recv = __shfl_xor_sync(0xffffffffu, send, OFF);
          v[i] = kMax ? fmaxf(keep, recv) : keep + recv;
        }
        RowReduce<H, OFF / 2, kMax>::run(v, lane);
      } else {
        const float recv = __shfl_xor_sync(0xffffffffu, v[0], OFF);
        v[0] = kMax ? fmaxf(v[0], recv) : v[0] + recv;
        RowReduce<1, OFF / 2, kMax>::run(v, lane);
      }
    }
  }
};

// N consecutive floats from shared memory (16-byte aligned), as 128-bit loads where N allows
template <int N>
__device__ __forceinline__ void lds_row(const float* src, float (&dst)[N]) {
  if constexpr (N >= 4) {
#pragma unroll
    for (int i = 0; i < N; i += 4) {
      const float4 t = *reinterpret_cast<const float4*>(src + i);
      dst[i] = t.x; dst[i + 1] = t.y; dst[i + 2] = t.z; dst[i + 3] = t.w;
    }
  } else {
#pragma unroll
    for (int i = 0; i < N; ++i) dst[i] = src[i];
  }
}

// GP: the number of packed rows rounded up to a power of two (compile-time, so that the per-row loops of the
// softmax group unroll without branches).  kMulti: several new tokens per sequence, i.e. rows that see
// different numbers of keys (one token: every row sees all keys, and the per-row limits fold into scalars).
// D: head size, 64, 128 or 256.  The shared-memory stages keep their 128-wide size for D = 64 and only their first
// 64-column panel is filled; O^T is then still accumulated as a 128-row MMA whose rows 64.. (fed from the unfilled
// half of the V stage) are never read.  With D = 256 O^T is two 128-row MMAs per key step, on the tile's panels 0-1
// and 2-3, into two accumulators; a softmax thread then owns the output channels kt and 128 + kt.
template <bool kDense, int GP, bool kMulti, int D>
__global__ void __launch_bounds__(384, 1)
mala_decode_split_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                         const __grid_constant__ CUtensorMap tmV, const DecParams p) {
  using DecCfg = DecCfgT<D>;
  constexpr int KS = DecCfg::kKStages, VS = DecCfg::kVStages, TB = DecCfg::kTileBytes;
  constexpr int PAN = D / 64;                    // 64-column panels of a K / V / Q tile
  constexpr uint32_t kTileTx = 128u * D * 2u;    // bytes one K or V tile copy delivers
  constexpr int NG = GP >= 8 ? 2 : 1;      // softmax groups (four warps each)
  constexpr bool kInOrder = !kDense && NG == 1 && !kMulti;   // separate in-order issuing warps (see there)
  constexpr int GH = GP / NG;              // rows per group
  constexpr int LDN = NG == 1 ? 16 : GH;   // TMEM columns a softmax thread reads at a time
  // The dense kernel at sixteen rows (bound by its softmax groups' instruction streams, not by HBM) sums a tile's
  // probabilities per thread and crosses the group once per item: no test needs the normalizer earlier.  (The variants
  // with fewer rows are bound by HBM and keep the per-tile sums, whose exchange rides with the maxima's.)
  constexpr bool kLocalSums = kDense && GP >= 16;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint8_t* sQ = smem;                      // [2] item parity
  uint8_t* sK = sQ + 2 * DecCfg::kQBytes;
  uint8_t* sV = sK + KS * TB;
  uint8_t* sP = sV + VS * TB;              // [4] P^T ring

  __shared__ uint64_t q_full[2], q_empty[2], k_full[KS], k_empty[KS], v_full[VS], v_empty[VS], s_full[4], s_free[4],
      vote_bar[4], vote_read[4], ret_full[8], ret_free[8], p_full[4], p_free[4], item_done[2], o_free[2], fin_bar, grp_a[2];
  __shared__ uint32_t tmem_base_s;
  __shared__ int flag[2][4];               // [softmax group][vote ring]
  __shared__ int ret_ring[8];              // decision of tile g at g & 7 (vote warp -> accumulating warp)
  __shared__ int v_row[8], v_outer[8];     // TMA coordinates of the V tile of tile g (ring; written by the producer;
                                           // pages smaller than a tile: sequence and key block instead)
  __shared__ __align__(16) float xch_max[2][2][4][8], xch_sum[2][2][4][8];   // [buffer][group][warp][row]: per-tile exchange
  __shared__ int early_exit;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int G = p.Hq / p.Hkv;
  const int R = kMulti ? G * p.Sq : G;     // rows of a work item: row s * G + g = token s, head g of the group
  int* status = p.status;

  // the Q tile of an item has R <= 16 rows; the other rows of the two stages are never written: clear them once
  for (int i = tid; i < 2 * DecCfg::kQBytes / 16; i += DecCfg::kThreads) reinterpret_cast<uint4*>(sQ)[i] = make_uint4(0u, 0u, 0u, 0u);
  // likewise the rows R..15 of the P^T ring, so that those columns of O^T stay finite
  for (int i = tid; i < DecCfg::kPStages * DecCfg::kPBytes / 16; i += DecCfg::kThreads) reinterpret_cast<uint4*>(sP)[i] = make_uint4(0u, 0u, 0u, 0u);
  fence_proxy_async_smem();
  if (tid == 0) {
    early_exit = (*(volatile int*)status != 0);
    for (int s = 0; s < 2; ++s) {
      mbar_init(&q_full[s], 1); mbar_init(&q_empty[s], 1); mbar_init(&item_done[s], 1); mbar_init(&o_free[s], 4 * NG);
      mbar_init(&grp_a[s], 4);
    }
    for (int s = 0; s < KS; ++s) { mbar_init(&k_full[s], 1); mbar_init(&k_empty[s], 1); }
    for (int s = 0; s < VS; ++s) { mbar_init(&v_full[s], 1); mbar_init(&v_empty[s], 1); }
    for (int s = 0; s < 4; ++s) {
      mbar_init(&s_full[s], 1); mbar_init(&s_free[s], 4 * NG); mbar_init(&vote_bar[s], NG); mbar_init(&vote_read[s], 1);
      mbar_init(&p_full[s], 4 * NG); mbar_init(&p_free[s], 1);
      flag[0][s] = flag[1][s] = 0;
    }
    for (int s = 0; s < 8; ++s) { mbar_init(&ret_full[s], 1); mbar_init(&ret_free[s], 1); }
    mbar_init(&fin_bar, 1);
    mbar_fence_init();
  }
  __syncthreads();
  if (early_exit) return;
  if (warp == 0) { tmem_alloc(&tmem_base_s, DecCfg::kTmemCols); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tb = tmem_base_s;

  // geometry of work item `item`: batch, KV head, split, number of legal tiles, newest key block, keys of the
  // sequence
  auto geometry = [&](int item, int& b, int& hkv, int& split, int& T, int& j0, int& nk) {
    split = item % p.num_splits;
    const int bh = item / p.num_splits;
    hkv = bh % p.Hkv;
    b = bh / p.Hkv;
    nk = p.seqlens ? min(p.Nk, max(0, __ldg(p.seqlens + b))) : p.Nk;
    const int lo = split * p.tps * 128;
    const int hi = min(nk, lo + p.tps * 128);
    T = hi > lo ? (hi - lo + 127) / 128 : 0;
    j0 = lo / 128 + T - 1;
  };
  // TMA coordinates (key row, outermost index) of key block jt of sequence b, one copy per tile
  auto tile_coord = [&](int b, int jt, int& row, int& outer) {
    if (p.block_table) {
      const int pg = jt / p.tpp;
      outer = __ldg(p.block_table + (size_t)b * p.bt_stride + pg);
      row = (jt - pg * p.tpp) * 128;
    } else {
      outer = b;
      row = jt * 128;
    }
  };
  // Pages smaller than a tile (ppt > 1): the tile is put together from ppt copies of prows rows, copy c from page
  // jt * ppt + c of the sequence (a table entry past the last page reads as "no page": zeros).
  auto small_page = [&](int b, int jt, int c) -> int {
    const int pg = jt * p.ppt + c;
    return pg < p.bt_stride ? __ldg(p.block_table + (size_t)b * p.bt_stride + pg) : -1;
  };

  // The copies of a tile are issued by a whole converged warp: lane x issues copy x / PAN of panel x % PAN, so the
  // table lookups are one coalesced load and the copies are issued side by side (one lane alone cannot issue 16 to 32 copies per tile in a
  // tile's HBM time).  The barrier's expect_tx has been posted by then.
  auto load_tile_small_warp = [&](uint8_t* dst, const CUtensorMap* tm, uint64_t* bar, int b, int jt, int hkv) {
    const int pn = lane % PAN;
    if constexpr (PAN <= 2) {   // up to 16 copies of up to two panels: one per lane
      const int c = lane / PAN;
      if (c < p.ppt) tma_load_4d(dst + pn * 16384 + c * p.prows * 128, tm, bar, pn * 64, 0, hkv, small_page(b, jt, c));
    } else {
      for (int c = lane / PAN; c < p.ppt; c += 32 / PAN)
        tma_load_4d(dst + pn * 16384 + c * p.prows * 128, tm, bar, pn * 64, 0, hkv, small_page(b, jt, c));
    }
  };

  if (warp == 0 && p.ppt > 1) {
    // ------------------------------------------------------------------ TMA producer, pages smaller than a tile:
    // the loop of the producer below, run by all 32 lanes (waits and counters warp-uniform)
    if (lane == 0) { tma_prefetch_desc(&tmQ); tma_prefetch_desc(&tmK); tma_prefetch_desc(&tmV); }
    int ne = 0, g = 0, ks = 0, vs = 0;
    uint32_t kpar = 1, vpar = 1;
    bool ok = true;
    for (int item = blockIdx.x; item < p.n_items && ok; item += gridDim.x) {
      int b, hkv, split, T, j0, nk;
      geometry(item, b, hkv, split, T, j0, nk);
      if (T == 0) continue;
      const int ip = ne & 1;
      ok = mbar_wait_warp(&q_empty[ip], ((ne >> 1) & 1) ^ 1, status);
      if (!ok) break;
      if (lane == 0) {
        mbar_arrive_expect_tx(&q_full[ip], (uint32_t)R * 128u * PAN);
#pragma unroll
        for (int pn = 0; pn < PAN; ++pn)
          tma_load_4d(sQ + ip * DecCfg::kQBytes + pn * 2048, &tmQ, &q_full[ip], pn * 64, hkv * G, 0, b);
      }
      for (int t = 0; t < T && ok; ++t, ++g) {
        ok = mbar_wait_warp(&k_empty[ks], kpar, status);
        if (!ok) break;
        if (lane == 0) {
          if (!kDense) { v_row[g & 7] = j0 - t; v_outer[g & 7] = b; }
          mbar_arrive_expect_tx(&k_full[ks], kTileTx);
        }
        __syncwarp();
        load_tile_small_warp(sK + ks * TB, &tmK, &k_full[ks], b, j0 - t, hkv);
        if (++ks == KS) { ks = 0; kpar ^= 1; }
        if (kDense) {   // every tile is retained: V follows K
          ok = mbar_wait_warp(&v_empty[vs], vpar, status);
          if (!ok) break;
          if (lane == 0) mbar_arrive_expect_tx(&v_full[vs], kTileTx);
          __syncwarp();
          load_tile_small_warp(sV + vs * TB, &tmV, &v_full[vs], b, j0 - t, hkv);
          if (++vs == VS) { vs = 0; vpar ^= 1; }
        }
      }
      ++ne;
    }
    if (!ok) { const long long t0 = clock64(); while (clock64() - t0 < 400000) {} }
  } else if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      tma_prefetch_desc(&tmQ); tma_prefetch_desc(&tmK); tma_prefetch_desc(&tmV);
      int ne = 0;                               // ordinal of the non-empty item
      int g = 0;                                // global tile counter
      int ks = 0, vs = 0;
      uint32_t kpar = 1, vpar = 1;              // "empty" parities (first pass: free)
      bool ok = true;
      for (int item = blockIdx.x; item < p.n_items && ok; item += gridDim.x) {
        int b, hkv, split, T, j0, nk;
        geometry(item, b, hkv, split, T, j0, nk);
        if (T == 0) continue;
        const int ip = ne & 1;
        ok = mbar_wait(&q_empty[ip], ((ne >> 1) & 1) ^ 1, status);
        if (!ok) break;
        mbar_arrive_expect_tx(&q_full[ip], (uint32_t)R * 128u * PAN);   // panels of R rows x 128 bytes
#pragma unroll
        for (int pn = 0; pn < PAN; ++pn)
          tma_load_4d(sQ + ip * DecCfg::kQBytes + pn * 2048, &tmQ, &q_full[ip], pn * 64, hkv * G, 0, b);
        for (int t = 0; t < T && ok; ++t, ++g) {
          int row, outer;
          tile_coord(b, j0 - t, row, outer);     // (a page lookup is in flight while the slot is waited for)
          ok = mbar_wait(&k_empty[ks], kpar, status);
          if (!ok) break;
          // The UMMA warp requests V of tile g from these coordinates after the vote.  It cannot be more than six
          // tiles behind this one (K ring of three behind the S^T cursor, vote cursor at most four behind that),
          // and it sees the two stores through the K tile's barrier.
          if (!kDense) { v_row[g & 7] = row; v_outer[g & 7] = outer; }
          mbar_arrive_expect_tx(&k_full[ks], kTileTx);
#pragma unroll
          for (int pn = 0; pn < PAN; ++pn)
            tma_load_4d(sK + ks * TB + pn * 16384, &tmK, &k_full[ks], pn * 64, row, hkv, outer);
          if (++ks == KS) { ks = 0; kpar ^= 1; }
          if (kDense) {   // every tile is retained: V follows K
            ok = mbar_wait(&v_empty[vs], vpar, status);
            if (!ok) break;
            mbar_arrive_expect_tx(&v_full[vs], kTileTx);
#pragma unroll
            for (int pn = 0; pn < PAN; ++pn)
              tma_load_4d(sV + vs * TB + pn * 16384, &tmV, &v_full[vs], pn * 64, row, hkv, outer);
            if (++vs == VS) { vs = 0; vpar ^= 1; }
          }
        }
        ++ne;
      }
      // after an expired wait copies may still be in flight: give them time to land before the CTA exits
      if (!ok) { const long long t0 = clock64(); while (clock64() - t0 < 400000) {} }
    }
  } else if (kInOrder && warp <= 3) {
    // ------------------------------------------------------------------ the three issuing warps
    // (MALA kernel, one softmax group, one token per step.)  Each has one job, walks the CTA's tiles in order and
    // blocks on exactly what its next instruction needs, so that the V copy of a retained tile is requested as soon as
    // its vote is in: 6 % faster on the gated inputs than the one polling warp of the other variants below, which
    // reacts to each event a loop iteration late.  (For the dense kernel and for sixteen rows the polling warp is the
    // faster one -- 670 against 700 us dense, 900 against 1135 us with four tokens per step -- and stays.)  All 32 lanes
    // run these loops with identical values; MMAs, commits and TMA loads are issued by one elected lane.
    const uint32_t leader = elect_one();
    // cursor over (non-empty item, tile) in processing order; g = global tile number
    struct Cur { int item, ne, t, T, b, hkv, j0, g; bool valid; };
    auto first_item = [&](Cur& c, int from, int ne, int g) {
      c.valid = false;
      c.g = g;
      for (int item = from; item < p.n_items; item += gridDim.x) {
        int b, hkv, split, T, j0, nk;
        geometry(item, b, hkv, split, T, j0, nk);
        if (T > 0) { c.item = item; c.ne = ne; c.t = 0; c.T = T; c.b = b; c.hkv = hkv; c.j0 = j0; c.valid = true; return; }
      }
    };
    auto advance = [&](Cur& c) {
      if (c.t + 1 < c.T) { ++c.t; ++c.g; return; }
      first_item(c, c.item + gridDim.x, c.ne + 1, c.g + 1);
    };
    Cur c;
    first_item(c, blockIdx.x, 0, 0);
    bool ok = true;
    if (warp == 1) {
      // ---- S^T = K Q^T of every tile: its score buffer (g & 3) is free once the softmax group has read tile g - 4
      //      and (MALA) the vote of that tile has been read, so that its flag may be overwritten
      constexpr uint32_t idesc_qk = make_idesc_bf16(128, 16, false, false);
      const uint64_t dQ0 = make_smem_desc(smem_u32(sQ), 16, 1024);
      const uint64_t dK0 = make_smem_desc(smem_u32(sK), 16, 1024);
      int kc = 0; uint32_t kpar = 0;             // K ring consumer
      for (; c.valid && ok; advance(c)) {
        const int ip = c.ne & 1, sb = c.g & 3;
        if (c.g >= 4) {
          ok = mbar_wait_warp_idle(&s_free[sb], (uint32_t)(((c.g >> 2) - 1) & 1), status);
          if (!kDense && ok) ok = mbar_wait_warp_idle(&vote_read[sb], (uint32_t)(((c.g >> 2) - 1) & 1), status);
        }
        if (ok && c.t == 0) ok = mbar_wait_warp_idle(&q_full[ip], (uint32_t)((c.ne >> 1) & 1), status);
        if (ok) ok = mbar_wait_warp_idle(&k_full[kc], kpar, status);
        if (!ok) break;
        tc_fence_after();
        const uint32_t dS = tmem_addr(tb, 0, (uint32_t)sb * 16u);
        const uint64_t dQ = desc_advance(dQ0, ip * DecCfg::kQBytes), dK = desc_advance(dK0, kc * TB);
#pragma unroll
        for (int k = 0; k < D / 16; ++k)   // K panels lie 16 KB apart, Q panels 2 KB
          mma_ss(dS, desc_advance(dK, (k >> 2) * 16384 + (k & 3) * 32), desc_advance(dQ, (k >> 2) * 2048 + (k & 3) * 32),
                 idesc_qk, k > 0, leader);
        if (leader) {
          tc_commit(&k_empty[kc]);
          tc_commit(&s_full[sb]);
          if (c.t == c.T - 1) tc_commit(&q_empty[ip]);   // last S^T of the item: its Q stage may be refilled
        }
        __syncwarp();
        if (++kc == KS) { kc = 0; kpar ^= 1; }
      }
    } else if (warp == 2) {
      // ---- the votes (MALA kernel): V of a retained tile is requested the moment its vote is known, and the
      //      decision is passed on to the accumulating warp
      if (!kDense) {
        int vi = 0; uint32_t vipar = 1;          // V ring producer side
        for (; c.valid && ok; advance(c)) {
          const int g = c.g;
          ok = mbar_wait_warp_idle(&vote_bar[g & 3], (uint32_t)((g >> 2) & 1), status);
          if (ok && g >= 8) ok = mbar_wait_warp_idle(&ret_free[g & 7], (uint32_t)(((g >> 3) - 1) & 1), status);
          if (!ok) break;
          const bool retain = __shfl_sync(0xffffffffu, *(volatile int*)&flag[0][g & 3] |
                                                                (NG > 1 ? *(volatile int*)&flag[1][g & 3] : 0), 0) != 0;
          __syncwarp();
          if (leader) mbar_arrive(&vote_read[g & 3]);
          if (retain) {
            ok = mbar_wait_warp_idle(&v_empty[vi], vipar, status);
            if (!ok) break;
            if (leader) {
              const int row = *(volatile int*)&v_row[g & 7], outer = *(volatile int*)&v_outer[g & 7];
              mbar_arrive_expect_tx(&v_full[vi], kTileTx);
              if (p.ppt > 1) {   // (one lane, copy after copy)
                for (int cc = 0; cc < p.ppt; ++cc) {
                  const int pgid = small_page(outer, row, cc);
#pragma unroll
                  for (int pn = 0; pn < PAN; ++pn)
                    tma_load_4d(sV + vi * TB + pn * 16384 + cc * p.prows * 128, &tmV, &v_full[vi], pn * 64, 0, c.hkv, pgid);
                }
              } else {
#pragma unroll
                for (int pn = 0; pn < PAN; ++pn)
                  tma_load_4d(sV + vi * TB + pn * 16384, &tmV, &v_full[vi], pn * 64, row, c.hkv, outer);
              }
            }
            __syncwarp();
            if (++vi == VS) { vi = 0; vipar ^= 1; }
          }
          if (leader) {
            *(volatile int*)&ret_ring[g & 7] = retain ? 1 : 0;
            mbar_arrive(&ret_full[g & 7]);
          }
          __syncwarp();
        }
      }
    } else if (warp == 3) {
      // ---- O^T += V^T P^T of every retained tile
      constexpr uint32_t idesc_pv = make_idesc_bf16(128, 16, true, true);
      const uint64_t dV0 = make_smem_desc(smem_u32(sV), 16384, 1024);   // V tile read MN-major (M = channel)
      // P^T is read MN-major without swizzle: per key the 16 rows as two 16-byte halves, each half of the tile a plane
      // of 8-key core matrices 128 bytes apart (so that a softmax thread writes its key's values as one vector store)
      const uint64_t dP0 = make_smem_desc(smem_u32(sP), 128, 2048) & ~((uint64_t)7 << 61);
      int vc = 0; uint32_t vcpar = 0;            // V ring consumer
      int npv = 0;                               // PVs issued so far (P^T ring slot npv & 3)
      int r_item = 0;                            // PVs of the current item so far
      for (; c.valid && ok; advance(c)) {
        const int g = c.g, ip = c.ne & 1;
        bool retain = true;
        if (!kDense) {
          ok = mbar_wait_warp_idle(&ret_full[g & 7], (uint32_t)((g >> 3) & 1), status);
          if (!ok) break;
          retain = __shfl_sync(0xffffffffu, *(volatile int*)&ret_ring[g & 7], 0) != 0;
          __syncwarp();
          if (leader) mbar_arrive(&ret_free[g & 7]);
        }
        if (retain) {
          const int ps = npv & 3;
          ok = mbar_wait_warp_idle(&p_full[ps], (uint32_t)((npv >> 2) & 1), status);
          if (ok) ok = mbar_wait_warp_idle(&v_full[vc], vcpar, status);
          // (first PV of an item: the softmax group has read this accumulator's previous item)
          if (ok && r_item == 0 && c.ne >= 2) ok = mbar_wait_warp_idle(&o_free[ip], (uint32_t)(((c.ne >> 1) - 1) & 1), status);
          if (!ok) break;
          tc_fence_after();
          const uint32_t dO = tmem_addr(tb, 0, DecCfg::kColO + (uint32_t)ip * 16u);
          const uint64_t dV = desc_advance(dV0, vc * TB), dP = desc_advance(dP0, ps * DecCfg::kPBytes);
          const uint32_t acc0 = r_item > 0 ? 1u : 0u;
#pragma unroll
          for (int k = 0; k < 8; ++k)   // k-step = 16 keys: 2 KB further on in the V tile, two core matrices of P^T
            mma_ss(dO, desc_advance(dV, k * 2048), desc_advance(dP, k * 256), idesc_pv, k > 0 ? 1u : acc0, leader);
          if constexpr (D > 128) {      // channels 128 .. 255: the tile's panels 2 and 3, the second accumulator
#pragma unroll
            for (int k = 0; k < 8; ++k)
              mma_ss(dO + (DecCfg::kColOHi - DecCfg::kColO), desc_advance(dV, 32768 + k * 2048), desc_advance(dP, k * 256),
                     idesc_pv, k > 0 ? 1u : acc0, leader);
          }
          if (leader) { tc_commit(&v_empty[vc]); tc_commit(&p_free[ps]); }
          if (++vc == VS) { vc = 0; vcpar ^= 1; }
          ++npv;
          ++r_item;
        }
        if (c.t == c.T - 1) { if (leader) tc_commit(&item_done[ip]); r_item = 0; }
        __syncwarp();
      }
      __syncwarp();
      if (leader) tc_commit(&fin_bar);
      mbar_wait_warp(&fin_bar, 0, status);
    }
    if (!ok) { const long long t0 = clock64(); while (clock64() - t0 < 400000) {} }
  } else if (!kInOrder && warp == 1) {
    // ------------------------------------------------------------------ UMMA warp (+ on-demand V loads)
    // All 32 lanes run this loop with identical values; MMAs, commits and TMA loads are issued by one elected lane.
    {
      const uint32_t leader = elect_one();
      constexpr uint32_t idesc_qk = make_idesc_bf16(128, 16, false, false);
      constexpr uint32_t idesc_pv = make_idesc_bf16(128, 16, true, true);
      const uint64_t dQ0 = make_smem_desc(smem_u32(sQ), 16, 1024);
      const uint64_t dK0 = make_smem_desc(smem_u32(sK), 16, 1024);
      const uint64_t dV0 = make_smem_desc(smem_u32(sV), 16384, 1024);   // V tile read MN-major (M = channel)
      // P^T is read MN-major without swizzle: per key the 16 rows as two 16-byte halves, each half of the tile a plane
      // of 8-key core matrices 128 bytes apart (so that a softmax thread writes its key's values as one vector store)
      const uint64_t dP0 = make_smem_desc(smem_u32(sP), 128, 2048) & ~((uint64_t)7 << 61);
      // cursor over (non-empty item, tile) in processing order; g = global tile number
      struct Cur { int item, ne, t, T, b, hkv, j0, g; bool valid; };
      auto first_item = [&](Cur& c, int from, int ne, int g) {
        c.valid = false;
        c.g = g;
        for (int item = from; item < p.n_items; item += gridDim.x) {
          int b, hkv, split, T, j0, nk;
          geometry(item, b, hkv, split, T, j0, nk);
          if (T > 0) { c.item = item; c.ne = ne; c.t = 0; c.T = T; c.b = b; c.hkv = hkv; c.j0 = j0; c.valid = true; return; }
        }
      };
      auto advance = [&](Cur& c) {
        if (c.t + 1 < c.T) { ++c.t; ++c.g; return; }
        first_item(c, c.item + gridDim.x, c.ne + 1, c.g + 1);
      };
      auto ready = [&](uint64_t* bar, uint32_t parity) -> bool { return __all_sync(0xffffffffu, mbar_test_wait(bar, parity)); };
      Cur cq, cv, cp;                            // next tile to score, to take the vote of, to accumulate
      first_item(cq, blockIdx.x, 0, 0);
      cv = cq; cp = cq;
      int kc = 0; uint32_t kpar = 0;             // K ring consumer
      int vi = 0; uint32_t vipar = 1;            // V ring producer side (MALA: copies issued here)
      int vc = 0; uint32_t vcpar = 0;            // V ring consumer
      uint32_t ret_bits = 0;                     // bit (g & 3): tile g was retained
      int npv = 0;                               // PVs issued so far (P^T ring slot npv & 3)
      int r_item = 0;                            // PVs of the accumulating cursor's item so far
      bool ok = true;
      long long t_progress = clock64();
      uint32_t idle = 0;
      while (cp.valid && ok) {
        bool progress = false;
        // ---- S^T of tile cq.g: its score buffer (g & 3) is free once the softmax group has read tile g - 4, and
        //      at most four votes are outstanding (the size of their ring)
        if (cq.valid && cq.g - cv.g < 4) {
          const int ip = cq.ne & 1, sb = cq.g & 3;
          if ((cq.g < 4 || ready(&s_free[sb], (uint32_t)(((cq.g >> 2) - 1) & 1))) &&
              (cq.t > 0 || ready(&q_full[ip], (cq.ne >> 1) & 1)) && ready(&k_full[kc], kpar)) {
            tc_fence_after();
            const uint32_t dS = tmem_addr(tb, 0, (uint32_t)sb * 16u);
            const uint64_t dQ = desc_advance(dQ0, ip * DecCfg::kQBytes), dK = desc_advance(dK0, kc * TB);
#pragma unroll
            for (int k = 0; k < D / 16; ++k)   // K panels lie 16 KB apart, Q panels 2 KB
              mma_ss(dS, desc_advance(dK, (k >> 2) * 16384 + (k & 3) * 32), desc_advance(dQ, (k >> 2) * 2048 + (k & 3) * 32),
                     idesc_qk, k > 0, leader);
            if (leader) {
              tc_commit(&k_empty[kc]);
              tc_commit(&s_full[sb]);
              if (cq.t == cq.T - 1) tc_commit(&q_empty[ip]);   // last S^T of the item: its Q stage may be refilled
            }
            if (++kc == KS) { kc = 0; kpar ^= 1; }
            advance(cq);
            progress = true;
          }
        }
        // ---- vote of tile cv.g (dense: every tile is retained and V comes from the producer)
        if (cv.valid && (!cq.valid || cv.g < cq.g) && cv.g - cp.g < 4) {   // (four tiles: the size of ret_bits)
          if (kDense) {
            ret_bits |= 1u << (cv.g & 3);
            advance(cv);
            progress = true;
          } else if (ready(&vote_bar[cv.g & 3], (cv.g >> 2) & 1)) {
            const bool retain = __shfl_sync(0xffffffffu, *(volatile int*)&flag[0][cv.g & 3] |
                                                                  (NG > 1 ? *(volatile int*)&flag[1][cv.g & 3] : 0), 0) != 0;
            if (!retain) {
              ret_bits &= ~(1u << (cv.g & 3));
              advance(cv);
              progress = true;
            } else if (ready(&v_empty[vi], vipar)) {   // V of this tile, on demand
              if (leader) {
                const int row = *(volatile int*)&v_row[cv.g & 7], outer = *(volatile int*)&v_outer[cv.g & 7];
                mbar_arrive_expect_tx(&v_full[vi], kTileTx);
                if (p.ppt > 1) {   // (one lane, copy after copy: this warp's time belongs to the MMAs)
                  for (int c = 0; c < p.ppt; ++c) {
                    const int pgid = small_page(outer, row, c);
#pragma unroll
                    for (int pn = 0; pn < PAN; ++pn)
                      tma_load_4d(sV + vi * TB + pn * 16384 + c * p.prows * 128, &tmV, &v_full[vi], pn * 64, 0, cv.hkv, pgid);
                  }
                } else {
#pragma unroll
                  for (int pn = 0; pn < PAN; ++pn)
                    tma_load_4d(sV + vi * TB + pn * 16384, &tmV, &v_full[vi], pn * 64, row, cv.hkv, outer);
                }
              }
              __syncwarp();
              if (++vi == VS) { vi = 0; vipar ^= 1; }
              ret_bits |= 1u << (cv.g & 3);
              advance(cv);
              progress = true;
            }
          }
        }
        // ---- O^T += V^T P^T of tile cp.g (or nothing, if it was skipped)
        if (!cv.valid || cp.g < cv.g) {
          const bool retain = (ret_bits >> (cp.g & 3)) & 1u;
          bool done = !retain;
          const int ip = cp.ne & 1, ps = npv & 3;
          if (retain && ready(&p_full[ps], (uint32_t)((npv >> 2) & 1)) && ready(&v_full[vc], vcpar) &&
              (r_item > 0 || cp.ne < 2 || ready(&o_free[ip], (uint32_t)(((cp.ne >> 1) - 1) & 1)))) {
            // (first PV of an item: the softmax group has read this accumulator's previous item)
            tc_fence_after();
            const uint32_t dO = tmem_addr(tb, 0, DecCfg::kColO + (uint32_t)ip * 16u);
            const uint64_t dV = desc_advance(dV0, vc * TB), dP = desc_advance(dP0, ps * DecCfg::kPBytes);
            const uint32_t acc0 = r_item > 0 ? 1u : 0u;
#pragma unroll
            for (int k = 0; k < 8; ++k)   // k-step = 16 keys: 2 KB further on in the V tile, 32 B in a P^T panel
              mma_ss(dO, desc_advance(dV, k * 2048), desc_advance(dP, k * 256), idesc_pv,
                     k > 0 ? 1u : acc0, leader);
            if constexpr (D > 128) {      // channels 128 .. 255: the tile's panels 2 and 3, the second accumulator
#pragma unroll
              for (int k = 0; k < 8; ++k)
                mma_ss(dO + (DecCfg::kColOHi - DecCfg::kColO), desc_advance(dV, 32768 + k * 2048), desc_advance(dP, k * 256),
                       idesc_pv, k > 0 ? 1u : acc0, leader);
            }
            if (leader) { tc_commit(&v_empty[vc]); tc_commit(&p_free[ps]); }
            if (++vc == VS) { vc = 0; vcpar ^= 1; }
            ++npv;
            ++r_item;
            done = true;
          }
          if (done) {
            if (cp.t == cp.T - 1) { if (leader) tc_commit(&item_done[ip]); r_item = 0; }
            advance(cp);
            progress = true;
          }
        }
        if (progress) {
          t_progress = clock64();
          idle = 0;
        } else {
          // nothing could be done: back off (a warp that spins here takes issue slots from the softmax warp on
          // its scheduler, and the whole group waits for that one at its barriers); bounded like every other wait
          __nanosleep(100);
          if (((++idle) & 0x3f) == 0) {
            if (*(volatile int*)status != 0) ok = false;
            else if (clock64() - t_progress > kWaitLimitCycles) { atomicCAS(status, 0, kDevTimeout); ok = false; }
            ok = __all_sync(0xffffffffu, ok);
          }
        }
      }
      __syncwarp();
      if (leader) tc_commit(&fin_bar);
      mbar_wait_warp(&fin_bar, 0, status);
      if (!ok) { const long long t0 = clock64(); while (clock64() - t0 < 400000) {} }
    }
  } else if (warp >= 4 && ((warp - 4) >> 2) < NG) {
    // ------------------------------------------------------------------ softmax groups: thread = key of the tile
    // A group of four warps handles GH rows (all of them, or half of them each when there are eight or more: the
    // rows are independent of one another except for the tile's vote).  One exchange per tile between the four
    // warps of a group: every warp publishes the per-row maxima of its 32 keys of this tile together with its
    // per-row sums of P of the previous retained tile; after one group barrier every thread holds the tile's row
    // maxima and the up-to-date normalizers and evaluates Eq. 3 for the group's rows itself.
    const int w = warp & 3;
    const int grp = (warp - 4) >> 2;               // softmax group
    const int rb = grp * GH;                       // its first row
    const uint32_t lane_base = (uint32_t)w * 32u;
    const int kt = (int)lane_base + lane;          // key inside the tile; output channel in the epilogue
    const float c2 = p.scale_log2;
    const bool ghead = (kt == 0);                  // the thread that casts the group's vote
    const bool head = ghead && grp == 0;           // the thread that keeps the telemetry
    // The reference of the exponentials follows the scores only when they exceed it by 2^60: fp32 sums and bf16 P
    // have the exponent range for it, and moving the reference means waiting until every PV issued so far has
    // retired (their V copies included), which would stall this group for a whole HBM round trip.
    constexpr float kRescaleGap = 60.f;
    // row q = token tok[q] of the Sq new ones (the last positions of the cache), head q - tok[q] * G of the group:
    // it sees the keys before position nk - back[q] and its partials lie rowoff[q] rows after the item's first
    constexpr int kLanesPerRow = 32 / GH;              // after RowReduce, row r sits in lanes r * kLanesPerRow ..
    const int pub_row = lane / kLanesPerRow;
    const bool publisher = (lane % kLanesPerRow) == 0;
    int back[GH];
    size_t rowoff[GH];
#pragma unroll
    for (int q = 0; q < GH; ++q) {
      const int qa = rb + q;                       // row number in the item
      const int tok = (kMulti && qa < R) ? qa / G : 0;
      back[q] = p.Sq - 1 - tok;
      rowoff[q] = kMulti ? ((size_t)tok * p.Hq + (size_t)(qa - tok * G)) * p.num_splits : (size_t)qa * p.num_splits;
    }
    int g = 0, ne = 0, rg = 0;                     // global tile counter, non-empty item ordinal, retained tiles so far
    uint32_t xc = 0;                               // exchanges so far (buffer xc & 1, barrier phase xc & 1)
    bool ok = true;
    // The partial output of an item needs its last PV, which trails this group by the V copies still in flight; it
    // is therefore written two tiles into the NEXT item (or at that item's end), not where the item ends: the
    // group never drains the pipeline at an item boundary.  Only O / l is deferred; everything else is known.
    bool pend = false;
    int pend_ip = 0, pend_ne = 0;
    size_t pend_prow0 = 0;
    float pend_l[GH];
#pragma unroll
    for (int q = 0; q < GH; ++q) pend_l[q] = 1.f;
    auto flush = [&]() -> bool {
      bool k = mbar_wait(&item_done[pend_ip], (uint32_t)((pend_ne >> 1) & 1), status);
      k = __all_sync(0xffffffffu, k);
      if (!k) return false;
      tc_fence_after();
      uint32_t o[LDN], o2[D > 128 ? LDN : 1];
      tmem_ld_cols<LDN>(tmem_addr(tb, lane_base, DecCfg::kColO + (uint32_t)pend_ip * 16u + (uint32_t)rb), o);
      if constexpr (D > 128) tmem_ld_cols<LDN>(tmem_addr(tb, lane_base, DecCfg::kColOHi + (uint32_t)pend_ip * 16u + (uint32_t)rb), o2);
      tmem_wait_ld();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&o_free[pend_ip]);   // the accumulator may take the item after next
#pragma unroll
      for (int q = 0; q < GH; ++q)
        if (rb + q < R && kt < D) {   // (a row that saw no key of the split: (0, -inf))
          p.o_part[(pend_prow0 + rowoff[q]) * D + kt] =
              (!kMulti || pend_l[q] > 0.f) ? __uint_as_float(o[q]) / pend_l[q] : 0.f;
          if constexpr (D > 128)
            p.o_part[(pend_prow0 + rowoff[q]) * D + 128 + kt] =
                (!kMulti || pend_l[q] > 0.f) ? __uint_as_float(o2[q]) / pend_l[q] : 0.f;
        }
      pend = false;
      return true;
    };
    for (int item = blockIdx.x; item < p.n_items && ok; item += gridDim.x) {
      int b, hkv, split, T, j0, nk;
      geometry(item, b, hkv, split, T, j0, nk);
      // L of a row = the keys it sees: all nk of the sequence for the newest token, one less per token before it
      int lim[GH];
      float theta[GH];
#pragma unroll
      for (int q = 0; q < GH; ++q) {
        lim[q] = kMulti ? nk - back[q] : nk;
        theta[q] = kDense ? -INFINITY : (p.log2_tau - log2f((float)max(lim[q], 1)));
      }
      const size_t prow0 = ((size_t)b * p.Sq * p.Hq + hkv * G) * p.num_splits + split;   // row q: + rowoff[q]
      const size_t stat_row = (size_t)(b * p.Hkv + hkv) * p.num_splits + split;
      if (T == 0) {   // empty split: (0, -inf)
#pragma unroll
        for (int q = 0; q < GH; ++q)
          if (rb + q < R) {
            if (kt < D) p.o_part[(prow0 + rowoff[q]) * D + kt] = 0.f;
            if constexpr (D > 128) p.o_part[(prow0 + rowoff[q]) * D + 128 + kt] = 0.f;
            if (kt == q) p.lse_part[prow0 + rowoff[q]] = -INFINITY;
          }
        if (head && p.retained) p.retained[stat_row] = 0u;
        continue;
      }
      const int ip = ne & 1;
      const uint32_t colO = DecCfg::kColO + (uint32_t)ip * 16u;
      float m_ref[GH], l[GH], lgl[GH];
      float psum = 0.f;   // this warp's sum of P of the last retained tile, for the row this lane publishes
#pragma unroll
      for (int q = 0; q < GH; ++q) { m_ref[q] = -INFINITY; l[q] = 0.f; lgl[q] = -INFINITY; }
      float lacc[kLocalSums ? GH : 1];   // this thread's share of the row sums
#pragma unroll
      for (int q = 0; q < (kLocalSums ? GH : 1); ++q) lacc[q] = 0.f;
      int r = 0;
      bool pending_sum = false;
      uint32_t bm_bits = 0;
      int bm_word = -1;
      uint32_t* bm_row = p.bitmask ? p.bitmask + stat_row * p.words : nullptr;
      // publishes this warp's (maximum, sum) of row pub_row -- each row by the first lane that holds it after the
      // warp reduction --, waits for the group, returns the combined maxima in tmax and adds the combined sums to l
      auto exchange = [&](float mx_row, float (&tmax)[GH]) -> bool {
        const int xb = xc & 1;
        if (publisher) { xch_max[xb][grp][w][pub_row] = mx_row; xch_sum[xb][grp][w][pub_row] = psum; }
        __syncwarp();
        if (lane == 0) mbar_arrive(&grp_a[grp]);
        bool k = mbar_wait(&grp_a[grp], xc & 1, status);
        k = __all_sync(0xffffffffu, k);
        ++xc;
        if (!k) return false;
        float a0[GH], a1[GH], a2[GH], a3[GH];
        lds_row<GH>(xch_max[xb][grp][0], a0); lds_row<GH>(xch_max[xb][grp][1], a1);
        lds_row<GH>(xch_max[xb][grp][2], a2); lds_row<GH>(xch_max[xb][grp][3], a3);
#pragma unroll
        for (int q = 0; q < GH; ++q) tmax[q] = fmaxf(fmaxf(a0[q], a1[q]), fmaxf(a2[q], a3[q]));
        if (pending_sum) {
          lds_row<GH>(xch_sum[xb][grp][0], a0); lds_row<GH>(xch_sum[xb][grp][1], a1);
          lds_row<GH>(xch_sum[xb][grp][2], a2); lds_row<GH>(xch_sum[xb][grp][3], a3);
#pragma unroll
          for (int q = 0; q < GH; ++q) {
            l[q] += (a0[q] + a1[q]) + (a2[q] + a3[q]);
            lgl[q] = __log2f(l[q]);
          }
        }
        pending_sum = false;
        return true;
      };
      for (int t = 0; t < T; ++t, ++g) {
        if (pend && t == 2) { ok = flush(); if (!ok) break; }
        const int sb = g & 3;
        ok = mbar_wait(&s_full[sb], (uint32_t)((g >> 2) & 1), status);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after();
        uint32_t sr[LDN];
        tmem_ld_cols<LDN>(tmem_addr(tb, lane_base, (uint32_t)sb * 16u + (uint32_t)rb), sr);
        tmem_wait_ld();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&s_free[sb]);     // the scores are in registers
        const int kpos = (j0 - t) * 128 + kt;   // only the newest tile of the sequence has keys that a row does not see
        float x[GH], mx[GH], tmax[GH];
#pragma unroll
        for (int q = 0; q < GH; ++q) { x[q] = (kpos < lim[q] && rb + q < R) ? __uint_as_float(sr[q]) * c2 : -INFINITY; mx[q] = x[q]; }
        RowReduce<GH, 16, true>::run(mx, lane);   // mx[0]: the warp's maximum of row pub_row
        ok = exchange(mx[0], tmax);
        if (!ok) break;
        // Eq. 3 against the split's partial normalizer: skip iff rowmax - (m + log l) < log(tau / Nk) for every head
        bool retain = true;
        if (!kDense && r > 0) {
          retain = false;
#pragma unroll
          for (int q = 0; q < GH; ++q)   // (a row without a visible key in the tile does not constrain it)
            retain = retain || (rb + q < R && (!kMulti || tmax[q] > -INFINITY) &&
                                !(((tmax[q] - (m_ref[q] + lgl[q])) - theta[q]) < 0.f));
        }
        if (!kDense && ghead) {
          *(volatile int*)&flag[grp][g & 3] = retain ? 1 : 0;
          mbar_arrive(&vote_bar[g & 3]);
        }
        if (!kDense && NG > 1) {   // the tile is retained if a row of either group needs it
          ok = mbar_wait(&vote_bar[g & 3], (uint32_t)((g >> 2) & 1), status);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          retain = (*(volatile int*)&flag[0][g & 3] | *(volatile int*)&flag[1][g & 3]) != 0;
          retain = __all_sync(0xffffffffu, retain);
        }
        if (!retain) continue;
        if (head && bm_row) {
          const int bit = T - 1 - t;   // tile index inside the split
          if ((bit >> 5) != bm_word) {
            if (bm_word >= 0) bm_row[bm_word] = bm_bits;
            bm_word = bit >> 5;
            bm_bits = 0;
          }
          bm_bits |= 1u << (bit & 31);
        }
        if (r == 0) {
#pragma unroll
          for (int q = 0; q < GH; ++q) m_ref[q] = kMulti ? fmaxf(tmax[q], -1e30f) : tmax[q];   // (finite also for a row that sees no key yet)
        } else {
          float alpha[GH];
          bool resc = false;
#pragma unroll
          for (int q = 0; q < GH; ++q) {
            alpha[q] = 1.f;
            if (rb + q < R && tmax[q] > m_ref[q] + kRescaleGap) {   // lazy rescaling: the reference only moves when it has to
              alpha[q] = fast_exp2(m_ref[q] - tmax[q]);
              l[q] *= alpha[q];
              if constexpr (kLocalSums) lacc[q] *= alpha[q];
              lgl[q] = __log2f(l[q]);
              m_ref[q] = tmax[q];
              resc = true;
            }
          }
          if (resc) {   // (the same decision in every thread: it only depends on exchanged values)
            // every PV so far has landed: the latest one (number rg - 1) releases its P^T slot last.  (A parity wait
            // must be neither ahead of nor two phases behind its barrier; per slot this one is exactly in step.)
            ok = mbar_wait(&p_free[(rg - 1) & 3], (uint32_t)(((rg - 1) >> 2) & 1), status);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            uint32_t o[LDN];
            tmem_ld_cols<LDN>(tmem_addr(tb, lane_base, colO + (uint32_t)rb), o);
            tmem_wait_ld();
#pragma unroll
            for (int q = 0; q < GH; ++q) o[q] = __float_as_uint(__uint_as_float(o[q]) * alpha[q]);
            tmem_st_cols<LDN>(tmem_addr(tb, lane_base, colO + (uint32_t)rb), o);
            if constexpr (D > 128) {
              constexpr uint32_t hi = DecCfg::kColOHi - DecCfg::kColO;
              tmem_ld_cols<LDN>(tmem_addr(tb, lane_base, colO + hi + (uint32_t)rb), o);
              tmem_wait_ld();
#pragma unroll
              for (int q = 0; q < GH; ++q) o[q] = __float_as_uint(__uint_as_float(o[q]) * alpha[q]);
              tmem_st_cols<LDN>(tmem_addr(tb, lane_base, colO + hi + (uint32_t)rb), o);
            }
            tmem_wait_st();
            tc_fence_before();
          }
        }
        // P^T into slot rg & 3 of its ring, free once the PV that last read it has retired
        const int ps = rg & 3;
        if (rg >= 4) {
          ok = mbar_wait(&p_free[ps], (uint32_t)(((rg >> 2) - 1) & 1), status);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
        }
        {
          // the key's GH values of this group: rows rb .. rb + GH - 1 of the 16, i.e. GH * 2 bytes of half rb / 8
          uint8_t* dst = sP + ps * DecCfg::kPBytes + (rb >> 3) * 2048 + (kt >> 3) * 128 + (kt & 7) * 16 + (rb & 7) * 2;
#pragma unroll
          for (int q = 0; q < GH; ++q) x[q] = (rb + q < R) ? fast_exp2(x[q] - m_ref[q]) : 0.f;
          if constexpr (GH == 1) {
            *reinterpret_cast<__nv_bfloat16*>(dst) = __float2bfloat16_rn(x[0]);
          } else {
            uint32_t pk[GH / 2];
#pragma unroll
            for (int q = 0; q < GH; q += 2) pk[q / 2] = pack_bf16x2(x[q], x[q + 1]);
            if constexpr (GH == 2) *reinterpret_cast<uint32_t*>(dst) = pk[0];
            else if constexpr (GH == 4) *reinterpret_cast<uint2*>(dst) = make_uint2(pk[0], pk[1]);
            else *reinterpret_cast<uint4*>(dst) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
          }
        }
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(&p_full[ps]);
        if constexpr (kLocalSums) {
#pragma unroll
          for (int q = 0; q < GH; ++q) lacc[q] += x[q];
        } else {
          // this warp's per-row sums of the tile (fp32, before the bf16 cast); they travel with the next exchange
          RowReduce<GH, 16, false>::run(x, lane);
          psum = x[0];
          pending_sum = true;
        }
        ++r;
        ++rg;
      }
      if (!ok) break;
      if constexpr (kLocalSums) {
        RowReduce<GH, 16, false>::run(lacc, lane);
        psum = lacc[0];
        pending_sum = true;
      }
      if (pending_sum) {   // the sums of the last retained tile
        float dummy[GH];
        ok = exchange(-INFINITY, dummy);
        if (!ok) break;
      }
      // the log-normalizer and the telemetry now; O / l (see above) once the item's last PV has retired
      if (pend) { ok = flush(); if (!ok) break; }   // (a short item: the previous one is still pending)
      pend = true;
      pend_ip = ip;
      pend_ne = ne;
      pend_prow0 = prow0;
#pragma unroll
      for (int q = 0; q < GH; ++q) pend_l[q] = l[q];
#pragma unroll
      for (int q = 0; q < GH; ++q)
        if (rb + q < R && kt == q)
          p.lse_part[prow0 + rowoff[q]] = (!kMulti || l[q] > 0.f) ? (m_ref[q] + lgl[q]) * 0.6931471805599453f : -INFINITY;
      if (head) {
        if (bm_row && bm_word >= 0) bm_row[bm_word] = bm_bits;
        if (p.retained) p.retained[stat_row] = (uint32_t)r;
        if (p.totals) {
          atomicAdd(&p.totals[0], (unsigned long long)r);
          atomicAdd(&p.totals[1], (unsigned long long)T);
        }
      }
      ++ne;
    }
    if (ok && pend) flush();
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tb, DecCfg::kTmemCols);
}

}  // namespace mala
