// MALA backward (Algorithm 2) for sm_100a.
//
//   bwd_preprocess_kernel : D = rowsum(O o dO), lse in the log2 domain and the per-query test offset
//                           lse2 + log2(tau / L_q), all padded to whole tiles (HBM-bound).
//   mala_bwd_kernel       : one CTA per (key block j, KV head, batch).  K_j, V_j stay in shared memory;
//                           for every query head of the group and every query block i >= j (ascending)
//                           S^T = K_j Q_i^T is recomputed on tensor cores and tested against the saved
//                           lse (Eq. 4).  Only retained tiles run dP^T = V dO^T, P^T,
//                           dS^T = P^T o (dP^T - D), dV += P^T dO, dK += dS^T Q, dQ_i += dS K_j
//                           (dO is fetched ahead for every tile: the vote comes too late to hide the copy).
//                           dK, dV accumulate in TMEM; dQ tiles are added to an fp32 accumulator in
//                           global memory, one half of the columns by vector reductions from registers
//                           (red.global.add.v4.f32), the other half by TMA reduce-add from shared memory.
//                           Either path alone is slower: an SM sustains about 25 B/clk of reductions, the
//                           TMA path is starved of shared-memory bandwidth while SS MMAs run, and its source
//                           buffer (32 KB, the tile's dS^T stage) is held until the reduction has read it.
//                           Accumulator layout, per 128 x D tile (b, head, query block), D / 2 = h:
//                             columns 0..h-1  : float (c / 4) * 512 + r * 4 + c % 4  (the 32 rows of a warp
//                                               are 512 contiguous bytes of one column group)
//                             columns h..D-1  : row-major [128][h] after those 128 * h floats
//   bwd_convert_dq_kernel : dq = bf16(scale * accumulator), back in row-major order.
//
// Warp roles of the main kernel (768 threads; registers are re-split between the warpgroups):
//   warp 0       TMA producer (K_j, V_j once; Q ring; dO ring)
//   warp 1       UMMA warp (all 32 lanes run the issue loop, one elected lane issues); warps 2-3 idle
//   warps 4-19   score group, four threads per key row (32 query columns each): reads S^T once, applies
//                Eq. 4 and votes; retained tiles: P^T -> TMEM (A operand of dV), then, with P^T still in
//                registers, dS^T = P^T o (dP^T - D) -> TMEM (A operand of dK) and shared memory (operand of dQ)
//   warps 20-23  dQ group, one thread per query row: takes the whole dQ tile out of TMEM at once (so that
//                the next dP^T can be issued) and adds it to the global accumulator
// Registers released by warps 0-19 (setmaxnreg) go to the dQ group, which holds a 128-column row.
// The warps run serial instruction streams at one dependent instruction per few cycles, so whatever a warp
// executes between the barrier it waited on and the barrier it arrives on (or the MMA it issues) is on the
// per-tile critical path: tile coordinates are kept by increments (no integer division per tile), waits whose
// data arrived long ago come before the wait for fresh data, and a warp with a positive vote does not wait
// for the group's vote.
#pragma once
#include <cuda_runtime.h>

#include "../../include/mala.h"
#include "sm100_ptx.cuh"
#include "tensor_map.h"

#ifndef MALA_BWD_TWO_PASS
#define MALA_BWD_TWO_PASS 1
#endif
#ifndef MALA_BWD_SAMPLE
#define MALA_BWD_SAMPLE 1
#endif

namespace mala {

struct BwdParams {
  const float* lse2;    // [B,Hq,Np] lse * log2(e); +inf on padding rows
  const float* bq;      // [B,Hq,Np] lse2 + log2(tau / L_q); +inf on padding rows
  const float* Dq;      // [B,Hq,Np] rowsum(O o dO); 0 on padding rows
  float* dq_acc;        // [B,Hq,Np,D] fp32
  __nv_bfloat16* dk; int64_t dk_sb, dk_sn, dk_sh;
  __nv_bfloat16* dv; int64_t dv_sb, dv_sn, dv_sh;
  uint32_t* retained;   // [B,Hq,Tc] or null
  uint32_t* bitmask;    // [B,Hq,Tc,words] or null (zero-filled by the host)
  unsigned long long* totals;
  int* status;
  int B, Hq, Hkv, N, Np, T, words, causal;   // N, Np, T: query rows, padded query rows, query blocks
  int Nk, Tk, koff;     // keys, key blocks; causal: the queries are the last N positions, koff = (Nk - N) / 128
  // Causal with (Nk - N) % 128 = qshift != 0: the query blocks follow the positions, block i = the rows q with
  // 128 i <= q + qshift < 128 (i + 1); T and Np count those blocks, and the per-query vectors and the dQ
  // accumulator are indexed by q + qshift.  The first block's missing rows load as zeros (rows before the tensor)
  // and carry lse = +inf like the rows past the end, so they neither vote nor contribute.
  int qshift;
  int d;                // head size of the tensors (<= D; columns d .. D-1 are zeros and never stored)
  // Packed sequences of different lengths (null: B sequences of N rows each): sequence b holds rows cu[b] ..
  // cu[b+1]-1 of the [1, total, H, d] tensors.  N, T, Nk, Tk then describe the longest sequence (grid, telemetry
  // strides); the per-query vectors are [Hq, Np] and the dQ accumulator [Hq, Np, D] with Np >= total + 128 B, where
  // sequence b owns the rows from (cu[b] + 128 b) / 128 * 128 on (tile-aligned, never overlapping the next one's).
  const int* cu;
  // Packed sequences with more keys than queries (null: keys packed like the queries): sequence b's keys are rows
  // cu_k[b] .. cu_k[b+1]-1 of k, v, dk, dv; koff and qshift are then derived per sequence, and sequence b owns the
  // padded rows from (cu[b] + 384 b) / 128 * 128 on (a short first block and a ragged last one each need a tile more).
  const int* cu_k;
  // List mode (second pass behind mala_bwd_scout_kernel): the masks of the retained tiles, rows padded to wpad words
  const uint32_t* list_mask;   // [B,Hq,Tk,wpad]
  int wpad;
  // One-pass kernel behind the first pass: only the heads whose row count is kScoutDirectRow are handled, and dK, dV
  // are added to what the list-mode launch stored
  const uint32_t* sel_rows;    // [B,Hq,Tk] or null (all heads)
  int accum_dkv;
  float scale, scale_log2;
};

template <int D>
struct BwdCfg {
  static constexpr int kPanels = D / 64;
  static constexpr int kTileBytes = 128 * D * 2;
  static constexpr int kDsBytes = 128 * 128 * 2;
  // K, V, Q x2, dO x2.  dS^T (32 KB) of a retained tile overwrites that tile's dO stage once dP and dV
  // have consumed it (D = 128); for D = 64 a dO stage is too small, so two separate dS stages follow.
  static constexpr int kSmemBytes = 6 * kTileBytes + (D == 128 ? 0 : 2 * kDsBytes) + 1024;
  static constexpr int kThreads = 768;
  static constexpr uint32_t kColS = 0, kColDP = 128, kColDV = 256, kColDK = 384;
};

// Walks the set bits of the G mask rows of a CTA (query heads of the group, then query blocks, ascending): the tile
// sequence of the list mode.  Every role keeps its own copy and advances it in step with its tile counter.
struct ListIter {
  const uint32_t* m;
  int wpad, G, h, w;
  uint32_t bits;
  __device__ __forceinline__ void init(const uint32_t* mask, int wpad_, int G_) {
    m = mask; wpad = wpad_; G = G_; h = 0; w = 0; bits = mask[0];
  }
  __device__ __forceinline__ bool next(int& h_out, int& i_out) {
    while (bits == 0u) {
      if (++w == wpad) { w = 0; if (++h == G) return false; }
      bits = m[h * wpad + w];
    }
    i_out = w * 32 + __ffs(bits) - 1;
    bits &= bits - 1u;
    h_out = h;
    return true;
  }
};

constexpr int kBwdListWords = 4096;   // mask words of one CTA's G rows held in shared memory (list mode)

// kList (with kDense): the tiles are those of the mask rows in p.list_mask, all of them retained: no test, no votes,
// the dense tile pipeline on a sparse tile sequence.
template <int D, bool kDense, bool kList = false>
__global__ void __launch_bounds__(768, 1)
mala_bwd_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmDO,
                const __grid_constant__ CUtensorMap tmAcc, const BwdParams p) {
  using Cfg = BwdCfg<D>;
  constexpr int PAN = Cfg::kPanels;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint8_t* sK = smem;
  uint8_t* sV = sK + Cfg::kTileBytes;
  uint8_t* sQ = sV + Cfg::kTileBytes;          // 2 stages
  uint8_t* sDO = sQ + 2 * Cfg::kTileBytes;     // 2 stages
  // dS^T stages, [2 halves][128 key rows][64 q] bf16, 128B swizzle
  uint8_t* sDS = (D == 128) ? sDO : sDO + 2 * Cfg::kTileBytes;

  __shared__ uint64_t kv_full, q_full[2], q_empty[2], do_full[2], do_empty[2], s_full, vote_bar[2], p_full, dp_full,
      ds_full, dst_full, dv_done, dq_full, dq_empty, dq_info_bar, grp_bar, fin_bar, stg_full, ds_free;
  __shared__ __align__(16) float vec[3][3][128];   // [slot][lse2 | bq | Dq][query column]
  __shared__ uint32_t tmem_base_s;
  __shared__ int flag[3];
  __shared__ int dq_info;
  __shared__ int early_exit;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int j = blockIdx.x, hkv = blockIdx.y, b = blockIdx.z;
  const int G = p.Hq / p.Hkv;
  // this sequence: first row in the tensors, rows, blocks, first row in the padded per-head arrays
  const int row0 = p.cu ? __ldg(p.cu + b) : 0;
  const int Nq = p.cu ? __ldg(p.cu + b + 1) - row0 : p.N;
  const int krow0 = p.cu_k ? __ldg(p.cu_k + b) : row0;
  const int Nkeys = p.cu_k ? __ldg(p.cu_k + b + 1) - krow0 : (p.cu ? Nq : p.Nk);
  const int koff = p.cu_k ? (p.causal ? (Nkeys - Nq) / 128 : 0) : p.koff;
  const int qshift = p.cu_k ? (p.causal ? (Nkeys - Nq) % 128 : 0) : p.qshift;
  const int T = p.cu ? (Nq + qshift + 127) / 128 : p.T;
  const int bz = p.cu ? 0 : b;                         // outermost TMA coordinate
  const int prow0 = p.cu ? ((row0 + (p.cu_k ? 384 : 128) * b) / 128) * 128 : 0;
  if (p.cu && j >= (Nkeys + 127) / 128) return;        // (a sequence shorter than the longest one)
  if (p.cu_k && (Nq <= 0 || (p.causal && Nkeys < Nq))) {
    // keys without queries (or lengths the call does not allow): their gradients are zero
    for (int x = threadIdx.x; x < 128 * (p.d / 8); x += blockDim.x) {
      const int key = j * 128 + x / (p.d / 8), c = (x % (p.d / 8)) * 8;
      if (key < Nkeys) {
        *reinterpret_cast<uint4*>(p.dk + (int64_t)(krow0 + key) * p.dk_sn + (int64_t)hkv * p.dk_sh + c) = make_uint4(0, 0, 0, 0);
        *reinterpret_cast<uint4*>(p.dv + (int64_t)(krow0 + key) * p.dv_sn + (int64_t)hkv * p.dv_sh + c) = make_uint4(0, 0, 0, 0);
      }
    }
    return;
  }
  static_assert(!kList || kDense, "the list mode runs the dense tile pipeline");
  __shared__ uint32_t lmask[kList ? kBwdListWords : 1];
  __shared__ int list_total;
  const int i0 = p.causal ? max(j - koff, 0) : 0;      // first query block that sees key block j
  const int ni = T - i0;
  int n_tot = G * ni;
  int* status = p.status;
  if (kList) {
    // the masks of this CTA's G rows into shared memory, and the number of tiles they hold
    if (tid == 0) list_total = 0;
    __syncthreads();
    int cnt = 0;
    for (int x = tid; x < G * p.wpad; x += blockDim.x) {
      const uint32_t wv = __ldg(p.list_mask + (((size_t)b * p.Hq + (size_t)hkv * G + x / p.wpad) * p.Tk + j) * p.wpad + x % p.wpad);
      lmask[x] = wv;
      cnt += __popc(wv);
    }
    for (int sft = 16; sft > 0; sft >>= 1) cnt += __shfl_xor_sync(0xffffffffu, cnt, sft);
    if (lane == 0 && cnt) atomicAdd(&list_total, cnt);
    __syncthreads();
    n_tot = list_total;
    if (n_tot == 0) {   // nothing retained in this key block: zero gradients
      for (int x = threadIdx.x; x < 128 * (p.d / 8); x += blockDim.x) {
        const int key = j * 128 + x / (p.d / 8), c = (x % (p.d / 8)) * 8;
        if (key < Nkeys) {
          *reinterpret_cast<uint4*>(p.dk + (int64_t)bz * p.dk_sb + (int64_t)(krow0 + key) * p.dk_sn + (int64_t)hkv * p.dk_sh + c) = make_uint4(0, 0, 0, 0);
          *reinterpret_cast<uint4*>(p.dv + (int64_t)bz * p.dv_sb + (int64_t)(krow0 + key) * p.dv_sn + (int64_t)hkv * p.dv_sh + c) = make_uint4(0, 0, 0, 0);
        }
      }
      return;
    }
  }

  // the query heads of the group this CTA handles: all of them, or (one-pass kernel behind the first pass) those whose
  // rows the first pass left alone
  __shared__ int hsel[16];
  __shared__ int nsel_s;
  if (warp == 0) {   // (one row flag per lane)
    bool mine = lane < G && lane < 16;
    if (!kList && !kDense && p.sel_rows)
      mine = mine && __ldg(p.sel_rows + ((size_t)b * p.Hq + (size_t)hkv * G + lane) * p.Tk + j) == 0xffffffffu;
    const uint32_t m = __ballot_sync(0xffffffffu, mine);
    if (mine) hsel[__popc(m & ((1u << lane) - 1u))] = lane;
    if (lane == 0) nsel_s = __popc(m);
  }
  if (tid == 0) {
    early_exit = (*(volatile int*)status != 0);
    mbar_init(&kv_full, 1);
    for (int s = 0; s < 2; ++s) {
      mbar_init(&q_full[s], 1); mbar_init(&q_empty[s], 1);
      mbar_init(&do_full[s], 1); mbar_init(&do_empty[s], 1);
      mbar_init(&vote_bar[s], 16);
    }
    mbar_init(&s_full, 1); mbar_init(&p_full, 16); mbar_init(&dp_full, 1); mbar_init(&ds_full, 16); mbar_init(&dst_full, 16);
    mbar_init(&dv_done, 1); mbar_init(&grp_bar, 16); mbar_init(&dq_full, 1); mbar_init(&dq_empty, 4); mbar_init(&dq_info_bar, 1);
    mbar_init(&fin_bar, 1);
    mbar_init(&stg_full, 4); mbar_init(&ds_free, 1);
    flag[0] = flag[1] = flag[2] = 0;
    dq_info = -1;
    mbar_fence_init();
  }
  __syncthreads();
  if (early_exit || nsel_s == 0) return;
  if (!kList && !kDense) n_tot = nsel_s * ni;
  if (warp == 0) { tmem_alloc(&tmem_base_s, 512); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tb = tmem_base_s;

  if (warp < 4) {
  reg_dealloc<40>();
  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      tma_prefetch_desc(&tmQ); tma_prefetch_desc(&tmK); tma_prefetch_desc(&tmV); tma_prefetch_desc(&tmDO);
      mbar_arrive_expect_tx(&kv_full, 2 * Cfg::kTileBytes);
      for (int pn = 0; pn < PAN; ++pn) {
        tma_load_4d(sK + pn * 16384, &tmK, &kv_full, pn * 64, krow0 + j * 128, hkv, bz);
        tma_load_4d(sV + pn * 16384, &tmV, &kv_full, pn * 64, krow0 + j * 128, hkv, bz);
      }
      bool ok = true;
      int issued = 0;
      int hk = 0, i = i0;   // tile n = (hk-th handled query head, query block), kept by increments: no division per tile
      ListIter it;
      if (kList) it.init(lmask, p.wpad, G);
      for (int n = 0; n < n_tot && ok; ++n, ++i) {
        if (kList) it.next(hk, i);
        else if (i == T) { i = i0; ++hk; }
        const int hq = hkv * G + (kList ? hk : hsel[hk]);
        const int s = n & 1;
        ok = mbar_wait(&q_empty[s], ((n >> 1) & 1) ^ 1, status);
        if (!ok) break;
        mbar_arrive_expect_tx(&q_full[s], Cfg::kTileBytes);
        for (int pn = 0; pn < PAN; ++pn)
          tma_load_4d(sQ + s * Cfg::kTileBytes + pn * 16384, &tmQ, &q_full[s], pn * 64, row0 + i * 128 - qshift, hq, bz);
        // dO of every tile is fetched ahead, retained or not (the vote comes too late to hide the copy behind it);
        // a skipped tile's stage is handed straight back by the issuer
        ok = mbar_wait(&do_empty[s], ((n >> 1) & 1) ^ 1, status);
        if (!ok) { mbar_wait(&q_full[s], (n >> 1) & 1, status); break; }
        mbar_arrive_expect_tx(&do_full[s], Cfg::kTileBytes);
        for (int pn = 0; pn < PAN; ++pn)
          tma_load_4d(sDO + s * Cfg::kTileBytes + pn * 16384, &tmDO, &do_full[s], pn * 64, row0 + i * 128 - qshift, hq, bz);
        issued = n + 1;
      }
      if (!ok) {
        mbar_wait(&kv_full, 0, status);
        for (int n = (issued > 2 ? issued - 2 : 0); n < issued; ++n) {
          mbar_wait(&q_full[n & 1], (n >> 1) & 1, status);
          mbar_wait(&do_full[n & 1], (n >> 1) & 1, status);
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ UMMA issuer
    // All 32 lanes run this loop with identical values; MMAs, commits, arrivals and TMA loads are issued by
    // one elected lane.
    {
      const uint32_t leader = elect_one();
      constexpr uint32_t idesc_s = make_idesc_bf16(128, 128, false, false);    // S^T, dP^T
      constexpr uint32_t idesc_dv = make_idesc_bf16(128, D, false, true);      // dV (A in TMEM), dK
      constexpr uint32_t idesc_dq = make_idesc_bf16(128, D, true, true);       // dQ
      // descriptors are built once; per MMA only the start-address field is advanced
      const uint64_t dKk = make_smem_desc(smem_u32(sK), 16, 1024);        // K_j as K-major A (S^T)
      const uint64_t dKm = make_smem_desc(smem_u32(sK), 16384, 1024);     // K_j as MN-major B (dQ)
      const uint64_t dVk = make_smem_desc(smem_u32(sV), 16, 1024);        // V_j as K-major A (dP^T)
      const uint64_t dQk0 = make_smem_desc(smem_u32(sQ), 16, 1024);       // Q stage 0 as K-major B (S^T)
      const uint64_t dQm0 = make_smem_desc(smem_u32(sQ), 16384, 1024);    // Q stage 0 as MN-major B (dK)
      const uint64_t dDOk0 = make_smem_desc(smem_u32(sDO), 16, 1024);     // dO stage 0 as K-major B (dP^T)
      const uint64_t dDOm0 = make_smem_desc(smem_u32(sDO), 16384, 1024);  // dO stage 0 as MN-major B (dV)
      const uint64_t dDSm0 = make_smem_desc(smem_u32(sDS), 16384, 1024);  // dS^T stage 0 as MN-major A (dQ)
      bool ok = mbar_wait_warp(&kv_full, 0, status);
      int r = 0;   // retained tiles so far
      auto issue_qk = [&](int n) -> bool {
        const int s = n & 1;
        if (!mbar_wait_warp(&q_full[s], (n >> 1) & 1, status)) return false;
        tc_fence_after();
        const uint64_t dQk = desc_advance(dQk0, s * Cfg::kTileBytes);
#pragma unroll
        for (int k = 0; k < D / 16; ++k) {
          const uint32_t off = (k >> 2) * 16384 + (k & 3) * 32;
          mma_ss(tmem_addr(tb, 0, Cfg::kColS), desc_advance(dKk, off), desc_advance(dQk, off), idesc_s, k > 0, leader);
        }
        if (leader) tc_commit(&s_full);
        return true;
      };
      if (ok) ok = issue_qk(0);
      for (int n = 0; n < n_tot && ok; ++n) {
        const int s = n & 1;
        bool retain = true;
        if (!kDense) {
          ok = mbar_wait_warp(&vote_bar[n & 1], (n >> 1) & 1, status);
          if (!ok) break;
          retain = __shfl_sync(0xffffffffu, *(volatile int*)&flag[n % 3], 0) != 0;
        }
        const int ds = s;       // dO stage (the dS^T / dQ staging of the tile reuses it)
        if (retain) {
          if (r > 0) {   // the dQ tile of the previous retained tile (aliased with dP) has been read out
            ok = mbar_wait_warp(&dq_empty, (r - 1) & 1, status);
            if (!ok) break;
          }
          ok = mbar_wait_warp(&do_full[ds], (n >> 1) & 1, status);
          if (!ok) break;
          tc_fence_after();
          const uint64_t dDOk = desc_advance(dDOk0, ds * Cfg::kTileBytes);
          const uint64_t dDOm = desc_advance(dDOm0, ds * Cfg::kTileBytes);
          const uint32_t acc0 = r > 0 ? 1u : 0u;
#pragma unroll
          for (int k = 0; k < D / 16; ++k) {   // dP^T = V dO^T
            const uint32_t off = (k >> 2) * 16384 + (k & 3) * 32;
            mma_ss(tmem_addr(tb, 0, Cfg::kColDP), desc_advance(dVk, off), desc_advance(dDOk, off), idesc_s, k > 0, leader);
          }
          if (leader) tc_commit(&dp_full);
          ok = mbar_wait_warp(&p_full, r & 1, status);
          if (!ok) break;
          tc_fence_after();
#pragma unroll
          for (int k = 0; k < 8; ++k)   // dV += P^T dO
            mma_ts(tmem_addr(tb, 0, Cfg::kColDV), tmem_addr(tb, 0, Cfg::kColS + (k >> 1) * 32 + (k & 1) * 8),
                   desc_advance(dDOm, k * 2048), idesc_dv, k > 0 ? 1u : acc0, leader);
          if (leader) tc_commit(&dv_done);
        }
        // the score buffer is free once dV has been issued (the score group keeps P^T in registers):
        // recompute the next tile's scores while dS is being formed
        if (n + 1 < n_tot) { ok = issue_qk(n + 1); if (!ok) break; }
        if (retain) {
          ok = mbar_wait_warp(&dst_full, r & 1, status);
          if (!ok) break;
          tc_fence_after();
          const uint64_t dDSm = desc_advance(dDSm0, ds * Cfg::kDsBytes);
          const uint64_t dQm = desc_advance(dQm0, s * Cfg::kTileBytes);
          const uint32_t acc1 = r > 0 ? 1u : 0u;
#pragma unroll
          for (int k = 0; k < 8; ++k)     // dK += dS^T Q, dS^T read from TMEM (the dP columns)
            mma_ts(tmem_addr(tb, 0, Cfg::kColDK), tmem_addr(tb, 0, Cfg::kColDP + (k >> 1) * 32 + (k & 1) * 8),
                   desc_advance(dQm, k * 2048), idesc_dv, k > 0 ? 1u : acc1, leader);
          if (leader) tc_commit(&q_empty[s]);
          ok = mbar_wait_warp(&ds_full, r & 1, status);   // the shared-memory copy of dS^T
          if (!ok) break;
          tc_fence_after();
#pragma unroll
          for (int k = 0; k < 8; ++k)     // dQ_i tile = dS K_j, into the dP columns (after dK has read dS^T from them)
            mma_ss(tmem_addr(tb, 0, Cfg::kColDP), desc_advance(dDSm, k * 2048), desc_advance(dKm, k * 2048), idesc_dq,
                   k > 0, leader);
          if (leader) {
            *(volatile int*)&dq_info = n * 2 + ds;
            mbar_arrive(&dq_info_bar);
            tc_commit(&dq_full);
            tc_commit(&ds_free);   // dS^T has been consumed: the dQ group may stage the dQ tile in that stage
          }
          ++r;
        } else {
          // skipped tile: Q and the dO fetched ahead (once it has landed) go back to their rings
          ok = mbar_wait_warp(&do_full[ds], (n >> 1) & 1, status);
          if (!ok) break;
          if (leader) { mbar_arrive(&q_empty[s]); mbar_arrive(&do_empty[ds]); }
        }
      }
      // tell the dQ group that nothing more will come, then wait for every MMA to retire
      __syncwarp();
      bool ok2 = true;
      if (r > 0) ok2 = mbar_wait_warp(&dq_empty, (r - 1) & 1, status);
      if (leader) {
        if (ok2) { *(volatile int*)&dq_info = -1; mbar_arrive(&dq_info_bar); }
        tc_commit(&fin_bar);
      }
      mbar_wait_warp(&fin_bar, 0, status);
    }
  }
  } else if (warp < 20) {
    // ------------------------------------------------------------------ score group
    // Four threads per key row: warps 4-7 own query columns 0..31 of the transposed tile, warps 8-11
    // columns 32..63, and so on (the four warps of a row reach the same TMEM lane quadrant).  A thread
    // reads its 32 score columns once; P^T (bf16, 16 packed columns) overwrites the first half of the
    // thread's own score columns, so no thread ever touches a column another thread still has to read.
    reg_dealloc<72>();
    const uint32_t lane_base = (uint32_t)(warp & 3) * 32u;
    const int rl = (int)lane_base + lane;
    const int qt = (warp - 4) >> 2;                 // column quarter
    const bool valid_key = (j * 128 + rl) < Nkeys;
    const float c2 = p.scale_log2;
    const bool stat_thread = (warp == 4 && lane == 0);
    bool ok = true;
    int r = 0;
    int r_head = 0;
    uint32_t bm_bits = 0;
    int bm_word = -1;

    auto vec_index = [&](int hq_local, int i) -> size_t {
      return ((size_t)bz * p.Hq + hkv * G + hq_local) * p.Np + (size_t)prow0 + (size_t)i * 128 + rl;
    };
    // (list mode: the tile sequence comes from the masks; one tile of look-ahead for the vectors' prefetch)
    ListIter it;
    int h_nx = 0, i_nx = i0;
    bool have_nx = true;
    if (kList) { it.init(lmask, p.wpad, G); have_nx = it.next(h_nx, i_nx); }
    // per-query vectors of tile 0 into slot 0 (published by the first column quarter), then a group sync
    if (qt == 0) {
      const size_t x = vec_index(kList ? h_nx : hsel[0], kList ? i_nx : i0);
      vec[0][0][rl] = p.lse2[x];
      vec[0][1][rl] = p.bq[x];
      vec[0][2][rl] = p.Dq[x];
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(&grp_bar);
    ok = mbar_wait(&grp_bar, 0, status);
    ok = __all_sync(0xffffffffu, ok);

    // tile n = (query head hq_n of the group, query block i): kept by increments, no division per tile
    int hq_n = 0, i = i0, slot = 0;   // (hq_n: index into the handled heads; list mode: the head itself)
    for (int n = 0; n < n_tot && ok; ++n, ++i, slot = (slot == 2 ? 0 : slot + 1)) {
      if (kList) { hq_n = h_nx; i = i_nx; have_nx = it.next(h_nx, i_nx); }
      else if (i == T) { i = i0; ++hq_n; }
      const bool first_of_head = !kList && (i == i0), last_of_head = !kList && (i == T - 1);
      // prefetch the per-query vectors of the next tile
      float nx0 = 0.f, nx1 = 0.f, nx2 = 0.f;
      if (qt == 0 && n + 1 < n_tot) {
        const size_t x = kList ? vec_index(h_nx, i_nx) : (last_of_head ? vec_index(hsel[hq_n + 1], i0) : vec_index(hsel[hq_n], i + 1));
        nx0 = p.lse2[x]; nx1 = p.bq[x]; nx2 = p.Dq[x];
      }
      ok = mbar_wait(&s_full, n & 1, status);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      uint32_t sc[32];
      tmem_ld_x32(tmem_addr(tb, lane_base, Cfg::kColS + qt * 32), sc);
      tmem_wait_ld();
      if (p.cu && !valid_key) {   // packed sequences: a row past this sequence's end holds the next one's key
        const uint32_t ninf = 0xff800000u;
#pragma unroll
        for (int e = 0; e < 32; ++e) sc[e] = ninf;
      }
      if (p.causal && i + koff == j) {   // diagonal tile: entry (key rl, query col) is legal iff rl <= col
        const uint32_t ninf = 0xff800000u;
        const int c0 = qt * 32;
#pragma unroll
        for (int e = 0; e < 32; ++e)
          if (c0 + e < rl) sc[e] = ninf;
      }
      // Eq. 4 (MALA only): skip iff s - lse_q < log(tau / L_q) on every valid entry
      float crit = -INFINITY;
      if (!kDense) {
        const float4* bb = reinterpret_cast<const float4*>(vec[slot][1]) + qt * 8;
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          const float4 x0 = bb[e];
          crit = fmaxf(crit, fmaxf(fmaxf(fmaf(__uint_as_float(sc[4 * e + 0]), c2, -x0.x), fmaf(__uint_as_float(sc[4 * e + 1]), c2, -x0.y)),
                                   fmaxf(fmaf(__uint_as_float(sc[4 * e + 2]), c2, -x0.z), fmaf(__uint_as_float(sc[4 * e + 3]), c2, -x0.w))));
        }
      }
      // publish the next tile's vectors.  Slot (n+1) % 3 was last read in tile n-2, which every warp has left:
      // the scores of tile n only exist because all 16 warps delivered P^T of tile n-1, after their tile n-2.
      // The readers in tile n+1 see the values through the chain arrive (P^T / vote) -> UMMA warp -> scores.
      if (qt == 0) {
        const int ns = (slot == 2 ? 0 : slot + 1);
        vec[ns][0][rl] = nx0; vec[ns][1][rl] = nx1; vec[ns][2][rl] = nx2;
      }
      bool retain = true;
      if (!kDense) {
        const bool vote = valid_key && !(crit < 0.f);
        const bool any = __any_sync(0xffffffffu, vote);
        if (lane == 0) {
          if (any) *(volatile int*)&flag[slot] = 1;
          if (warp == 4) *(volatile int*)&flag[slot == 2 ? 0 : slot + 1] = 0;
          tc_fence_before();
          mbar_arrive(&vote_bar[n & 1]);
        }
        // A warp that found a retained entry knows the outcome (the vote is an OR) and goes straight on; a warp
        // without one waits for the others.
        if (!any) {
          ok = mbar_wait(&vote_bar[n & 1], (n >> 1) & 1, status);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          retain = (*(volatile int*)&flag[slot]) != 0;
        }
      }
      if (!kDense) retain = __all_sync(0xffffffffu, retain);   // same value in every lane: the branch below is uniform
      if (stat_thread && first_of_head) { r_head = 0; bm_bits = 0; bm_word = -1; }
      if (retain) {
        if (stat_thread) {
          ++r_head;
          if (p.bitmask) {
            uint32_t* bm_row = p.bitmask + ((size_t)(b * p.Hq + hkv * G + hsel[hq_n]) * p.Tk + j) * p.words;
            if ((i >> 5) != bm_word) {
              if (bm_word >= 0) bm_row[bm_word] = bm_bits;
              bm_word = i >> 5;
              bm_bits = 0;
            }
            bm_bits |= 1u << (i & 31);
          }
        }
        // P^T = exp2(s * c2 - lse2_q) (bf16), written over S^T in TMEM as the A operand of dV
        uint32_t pk[16];
        {
          const float4* ll = reinterpret_cast<const float4*>(vec[slot][0]) + qt * 8;
#pragma unroll
          for (int e = 0; e < 8; ++e) {
            const float4 x = ll[e];
            const float p0 = fast_exp2(fmaf(__uint_as_float(sc[4 * e + 0]), c2, -x.x));
            const float p1 = fast_exp2(fmaf(__uint_as_float(sc[4 * e + 1]), c2, -x.y));
            const float p2 = fast_exp2(fmaf(__uint_as_float(sc[4 * e + 2]), c2, -x.z));
            const float p3 = fast_exp2(fmaf(__uint_as_float(sc[4 * e + 3]), c2, -x.w));
            pk[2 * e] = pack_bf16x2(p0, p1);
            pk[2 * e + 1] = pack_bf16x2(p2, p3);
          }
        }
        tmem_st_x16(tmem_addr(tb, lane_base, Cfg::kColS + qt * 32), pk);
        tmem_wait_st();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&p_full);
        // dS^T = P^T o (dP^T - D_q): values first, then, once dV has also finished reading the dO stage that
        // dS^T overwrites (D = 128), into shared memory for the dQ and dK MMAs
        ok = mbar_wait(&dp_full, r & 1, status);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after();
        uint32_t w[16];
        {
          uint32_t dp[32];
          tmem_ld_x32(tmem_addr(tb, lane_base, Cfg::kColDP + qt * 32), dp);
          tmem_wait_ld();
          const float4* dd = reinterpret_cast<const float4*>(vec[slot][2]) + qt * 8;
#pragma unroll
          for (int e = 0; e < 8; ++e) {
            const float4 x = dd[e];
            const uint32_t pa = pk[2 * e], pb = pk[2 * e + 1];
            const float p0 = __uint_as_float(pa << 16), p1 = __uint_as_float(pa & 0xffff0000u);
            const float p2 = __uint_as_float(pb << 16), p3 = __uint_as_float(pb & 0xffff0000u);
            w[2 * e] = pack_bf16x2(p0 * (__uint_as_float(dp[4 * e + 0]) - x.x), p1 * (__uint_as_float(dp[4 * e + 1]) - x.y));
            w[2 * e + 1] = pack_bf16x2(p2 * (__uint_as_float(dp[4 * e + 2]) - x.z), p3 * (__uint_as_float(dp[4 * e + 3]) - x.w));
          }
        }
        // dS^T also goes to TMEM, over this thread's own (already consumed) dP^T columns: A operand of dK
        tmem_st_x16(tmem_addr(tb, lane_base, Cfg::kColDP + qt * 32), w);
        tmem_wait_st();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&dst_full);       // dK may start while the shared-memory copy is written
        ok = mbar_wait(&dv_done, r & 1, status);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        {
          uint8_t* dst = sDS + (n & 1) * Cfg::kDsBytes + (qt >> 1) * 16384;
#pragma unroll
          for (int v = 0; v < 4; ++v)
            *reinterpret_cast<uint4*>(dst + sw128_offset((uint32_t)rl, (uint32_t)((qt & 1) * 32 + v * 8))) =
                make_uint4(w[4 * v], w[4 * v + 1], w[4 * v + 2], w[4 * v + 3]);
        }
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(&ds_full);
        ++r;
      }
      if (stat_thread && last_of_head) {   // last tile of this query head
        const size_t row = (size_t)(b * p.Hq + hkv * G + hsel[hq_n]) * p.Tk + j;
        if (p.bitmask && bm_word >= 0) p.bitmask[row * p.words + bm_word] = bm_bits;
        if (p.retained) p.retained[row] = (uint32_t)r_head;
        if (p.totals) {
          atomicAdd(&p.totals[0], (unsigned long long)r_head);
          atomicAdd(&p.totals[1], (unsigned long long)ni);
        }
      }
    }

    // epilogue: dK_j (x scale), dV_j -> global; the four threads of a row store a quarter of its columns each
    if (ok) {
      ok = mbar_wait(&fin_bar, 0, status);
      ok = __all_sync(0xffffffffu, ok);
    }
    if (ok) {
      tc_fence_after();
      const int key = j * 128 + rl;
      __nv_bfloat16* dvrow = p.dv + (int64_t)bz * p.dv_sb + (int64_t)(krow0 + key) * p.dv_sn + (int64_t)hkv * p.dv_sh;
      __nv_bfloat16* dkrow = p.dk + (int64_t)bz * p.dk_sb + (int64_t)(krow0 + key) * p.dk_sn + (int64_t)hkv * p.dk_sh;
#pragma unroll
      for (int which = 0; which < 2; ++which) {
        __nv_bfloat16* out = which ? dkrow : dvrow;
        const float f = which ? p.scale : 1.f;
        const uint32_t col0 = which ? Cfg::kColDK : Cfg::kColDV;
        if (qt < D / 32) {   // warp-uniform: D = 64 has two 32-column chunks, taken by the first two quarters
          const int c = qt;
          uint32_t o[32];
          if (r > 0) {
            tmem_ld_x32(tmem_addr(tb, lane_base, col0 + c * 32), o);
            tmem_wait_ld();
          } else {
#pragma unroll
            for (int e = 0; e < 32; ++e) o[e] = 0u;
          }
          if (valid_key) {
#pragma unroll
            for (int v = 0; v < 4; ++v) {
              uint4 w;
              w.x = pack_bf16x2(__uint_as_float(o[8 * v + 0]) * f, __uint_as_float(o[8 * v + 1]) * f);
              w.y = pack_bf16x2(__uint_as_float(o[8 * v + 2]) * f, __uint_as_float(o[8 * v + 3]) * f);
              w.z = pack_bf16x2(__uint_as_float(o[8 * v + 4]) * f, __uint_as_float(o[8 * v + 5]) * f);
              w.w = pack_bf16x2(__uint_as_float(o[8 * v + 6]) * f, __uint_as_float(o[8 * v + 7]) * f);
              if (!kDense && p.accum_dkv && c * 32 + v * 8 < p.d) {   // add to what the list-mode launch stored for the other heads
                const uint4 pv = *reinterpret_cast<const uint4*>(out + c * 32 + v * 8);
                const uint32_t pr[4] = {pv.x, pv.y, pv.z, pv.w};
                uint32_t nw[4];
#pragma unroll
                for (int e = 0; e < 4; ++e)
                  nw[e] = pack_bf16x2(__uint_as_float(o[8 * v + 2 * e]) * f + __uint_as_float(pr[e] << 16),
                                      __uint_as_float(o[8 * v + 2 * e + 1]) * f + __uint_as_float(pr[e] & 0xffff0000u));
                w = make_uint4(nw[0], nw[1], nw[2], nw[3]);
              }
              if (c * 32 + v * 8 < p.d) *reinterpret_cast<uint4*>(out + c * 32 + v * 8) = w;
            }
          }
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ dQ group: thread = query row
    // Each retained tile's dQ (fp32, 128 x D) is taken out of TMEM in one go and the dP / dQ columns are
    // released at once.  The first D / 2 columns go to the global accumulator by vector reductions from
    // registers; the others are staged as 32-column swizzled panels in the tile's dS^T stage -- free once
    // dQ has retired -- and added by TMA reduce-add; the stage goes back to the dO ring when the TMA has
    // read it.
    reg_alloc<152>();
    const uint32_t lane_base = (uint32_t)(warp & 3) * 32u;
    const int rl = (int)lane_base + lane;
    const bool elected = (warp == 20 && lane == 0);
    if (elected) tma_prefetch_desc(&tmAcc);
    ListIter it;
    if (kList) it.init(lmask, p.wpad, G);
    for (int k = 0;; ++k) {
      bool ok = mbar_wait(&dq_info_bar, k & 1, status);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      const int info = *(volatile int*)&dq_info;
      if (info < 0) break;
      const int n = info >> 1, ds = info & 1;
      // (the tile's coordinates while the dQ MMAs are still running: the announcement precedes their completion)
      int hq = hkv * G + hsel[n / ni], i = i0 + n % ni;
      if (kList) { int hl; it.next(hl, i); hq = hkv * G + hl; }   // (every tile of the list is announced, in order)
      const int tile = p.cu ? (int)((size_t)hq * (p.Np / 128) + (size_t)(prow0 / 128 + i))
                            : (int)(((size_t)b * p.Hq + hq) * p.T + (size_t)i);
      uint8_t* stg = sDS + ds * Cfg::kDsBytes;     // D / 64 panels of 16 KB
      float* const acc_tile = p.dq_acc + (size_t)tile * (128 * D) + rl * 4;
      asm volatile("" :: "l"(acc_tile), "l"(stg) : "memory");   // keep the address arithmetic ahead of the wait
      ok = mbar_wait(&dq_full, k & 1, status);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      uint32_t a[D / 32][32];
#pragma unroll
      for (int c = 0; c < D / 32; ++c) tmem_ld_x32(tmem_addr(tb, lane_base, Cfg::kColDP + c * 32), a[c]);
      tmem_wait_ld();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&dq_empty);       // TMEM columns may be reused by the next dP
      {
        float* acc = acc_tile;
#pragma unroll
        for (int c = 0; c < D / 64; ++c)
#pragma unroll
          for (int v = 0; v < 8; ++v)
            red_add_v4(acc + (c * 8 + v) * 512, a[c][4 * v], a[c][4 * v + 1], a[c][4 * v + 2], a[c][4 * v + 3]);
      }
      ok = mbar_wait(&ds_free, k & 1, status);     // dQ and dK have consumed dS^T: its stage may be overwritten
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
#pragma unroll
      for (int c = D / 64; c < D / 32; ++c) {
        uint8_t* pan = stg + (c - D / 64) * 16384;
#pragma unroll
        for (int v = 0; v < 8; ++v)
          *reinterpret_cast<uint4*>(pan + rl * 128 + ((v ^ (rl & 7)) << 4)) =
              make_uint4(a[c][4 * v], a[c][4 * v + 1], a[c][4 * v + 2], a[c][4 * v + 3]);
      }
      fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) mbar_arrive(&stg_full);
      if (elected) {
        ok = mbar_wait(&stg_full, k & 1, status);
        if (ok) {
#pragma unroll
          for (int c = 0; c < D / 64; ++c) tma_reduce_add_3d(&tmAcc, stg + c * 16384, c * 32, 0, tile);
          bulk_commit_group();
          bulk_wait_read_all();
        }
        mbar_arrive(&do_empty[ds]);                // stage back to the dO ring
      }
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
    }
    if (elected) bulk_wait_all();
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tb, 512);
}

// D = rowsum(O o dO), lse2 = lse * log2(e), bq = lse2 + log2(tau / L_q); one warp per (b, h, row) with row below
// Npg, the padded length of the (longest) sequence; entry `row` describes query row - qshift (qshift != 0 only
// without cu).  Packed sequences (cu != null): the vectors are [Hq, Np] with
// sequence b's rows from (cu[b] + 128 b) / 128 * 128 on, lse is [Hq, total].
__global__ void bwd_preprocess_kernel(const __nv_bfloat16* __restrict__ o, int64_t o_sb, int64_t o_sn, int64_t o_sh,
                                      const __nv_bfloat16* __restrict__ dout, int64_t d_sb, int64_t d_sn, int64_t d_sh,
                                      const float* __restrict__ lse, float* __restrict__ lse2, float* __restrict__ bq,
                                      float* __restrict__ Dq, int B, int Hq, int N, int Np, int Nk, int d, int causal,
                                      float log2_tau, const int* __restrict__ cu, int total_rows, int Npg, int qshift,
                                      const int* __restrict__ cu_k) {
  const int warps_per_block = blockDim.x >> 5;
  const long long wi = (long long)blockIdx.x * warps_per_block + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  const long long total = (long long)B * Hq * Npg;
  if (wi >= total) return;
  int row = (int)(wi % Npg);
  const int h = (int)((wi / Npg) % Hq);
  int b = (int)(wi / ((long long)Npg * Hq));
  long long w = wi;                                  // index into the vectors
  int row0 = 0;
  if (cu) {
    row0 = cu[b];
    N = cu[b + 1] - row0;
    Nk = cu_k ? cu_k[b + 1] - cu_k[b] : N;
    if (cu_k) qshift = (causal && Nk >= N) ? (Nk - N) % 128 : 0;   // (per sequence)
    if (row >= ((N + qshift + 127) / 128) * 128) return;           // beyond this sequence's padded rows
    w = (long long)h * Np + ((row0 + (cu_k ? 384 : 128) * b) / 128) * 128 + row;
    b = 0;
  }
  row -= qshift;                                     // the query this entry describes
  if (row < 0 || row >= N) {
    if (lane == 0) { lse2[w] = INFINITY; bq[w] = INFINITY; Dq[w] = 0.f; }
    return;
  }
  const __nv_bfloat16* op = o + b * o_sb + (int64_t)(row0 + row) * o_sn + h * o_sh;
  const __nv_bfloat16* dp = dout + b * d_sb + (int64_t)(row0 + row) * d_sn + h * d_sh;
  float acc = 0.f;
  for (int c = lane * 2; c < d; c += 64) {
    const __nv_bfloat162 a = *reinterpret_cast<const __nv_bfloat162*>(op + c);
    const __nv_bfloat162 g = *reinterpret_cast<const __nv_bfloat162*>(dp + c);
    acc += __bfloat162float(a.x) * __bfloat162float(g.x) + __bfloat162float(a.y) * __bfloat162float(g.y);
  }
#pragma unroll
  for (int s = 16; s > 0; s >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, s);
  if (lane == 0) {
    const float l2 = lse[cu ? (size_t)h * total_rows + row0 + row : ((size_t)b * Hq + h) * N + row] * 1.4426950408889634f;
    const float L = causal ? (float)(row + 1 + (Nk - N)) : (float)Nk;   // visible keys
    lse2[w] = l2;
    bq[w] = l2 + (log2_tau - log2f(L));
    Dq[w] = acc;
  }
}

// dq = bf16(scale * acc); one thread per 8 output elements.  The accumulator is tiled (see the file header):
// consecutive threads take consecutive rows of a tile.
// (Packed sequences, cu != null: the index runs over (b, h, block i of the longest sequence); the accumulator is
// [Hq, Np, d] with sequence b's tiles from (cu[b] + 128 b) / 128 on.)
__global__ void bwd_convert_dq_kernel(const float* __restrict__ acc, __nv_bfloat16* __restrict__ dq, int64_t sb,
                                      int64_t sn, int64_t sh, int B, int Hq, int N, int Np, int d, float scale,
                                      const int* __restrict__ cu, int Npg, int qshift, int d_out,
                                      const int* __restrict__ cu_k, int causal) {
  // d: columns of the accumulator (the padded head size); d_out <= d: columns of dq
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const int per_row = d / 8;
  const long long total = (long long)B * Hq * Npg * per_row;
  if (idx >= total) return;
  const int r = (int)(idx % 128);
  const int cg = (int)((idx / 128) % per_row);             // columns 8 cg .. 8 cg + 7
  long long tile = idx / (128LL * per_row);                // (b * Hq + h) * (Npg / 128) + i
  const int T = Npg / 128;
  const int i = (int)(tile % T);
  const int h = (int)((tile / T) % Hq);
  int b = (int)(tile / ((long long)T * Hq));
  int row = i * 128 + r;
  if (cu) {
    const int row0 = cu[b];
    N = cu[b + 1] - row0;
    if (cu_k) {
      const int Nk = cu_k[b + 1] - cu_k[b];
      qshift = (causal && Nk >= N) ? (Nk - N) % 128 : 0;   // (per sequence)
    }
  }
  row -= qshift;
  if (cu) {
    const int row0 = cu[b];
    if (row < 0 || row >= N) return;
    tile = (long long)h * (Np / 128) + (row0 + (cu_k ? 384 : 128) * b) / 128 + i;
    row += row0;
    N += row0;
    b = 0;
  }
  if (row < 0 || row >= N || cg * 8 >= d_out) return;
  const int half = d / 2;
  const float* base = acc + (size_t)tile * 128 * d;
  float4 x, y;
  if (cg * 8 < half) {
    const float* src = base + (size_t)(2 * cg) * 512 + r * 4;
    x = *reinterpret_cast<const float4*>(src);
    y = *reinterpret_cast<const float4*>(src + 512);
  } else {
    const float* src = base + (size_t)128 * half + (size_t)r * half + (cg * 8 - half);
    x = *reinterpret_cast<const float4*>(src);
    y = *reinterpret_cast<const float4*>(src + 4);
  }
  uint4 w;
  w.x = pack_bf16x2(x.x * scale, x.y * scale);
  w.y = pack_bf16x2(x.z * scale, x.w * scale);
  w.z = pack_bf16x2(y.x * scale, y.y * scale);
  w.w = pack_bf16x2(y.z * scale, y.w * scale);
  *reinterpret_cast<uint4*>(dq + b * sb + row * sn + h * sh + cg * 8) = w;
}

}  // namespace mala
#include "mala_bwd_scout.cuh"
namespace mala {

inline size_t bwd_align256(size_t x) { return (x + 255) & ~(size_t)255; }

// Two-pass backward (tau > 0): words per mask row (padded to four) and bytes of the masks + row counts of a call with
// T query blocks and Tk key blocks
inline int bwd_mask_wpad(int T) { return (((T + 31) / 32) + 3) & ~3; }
inline size_t bwd_list_bytes(int B, int Hq, int T, int Tk) {
  return bwd_align256((size_t)B * Hq * Tk * bwd_mask_wpad(T) * sizeof(uint32_t)) + bwd_align256((size_t)B * Hq * Tk * sizeof(uint32_t));
}

// (Packed sequences: B = 1 and N = total rows + 128 x number of sequences.)
inline size_t bwd_base_workspace_bytes(int B, int Hq, int N, int d) {   // d: the padded head size
  const size_t Np = (size_t)((N + 127) / 128) * 128;
  return bwd_align256((size_t)B * Hq * Np * d * sizeof(float)) + 3 * bwd_align256((size_t)B * Hq * Np * sizeof(float));
}
// What mala_workspace_bytes reports: the base scratch plus the masks of the two-pass path for as many key blocks as
// query blocks (a call with more key blocks than that takes the two-pass path only if it is given room for them).
inline size_t bwd_workspace_bytes(int B, int Hq, int N, int d) {
  const int T = (N + 127) / 128;
  return bwd_base_workspace_bytes(B, Hq, N, d) + bwd_list_bytes(B, Hq, T, T);
}

inline bool bwd_set_attributes() {
  bool ok = true;
  ok = ok && cudaFuncSetAttribute(mala_bwd_kernel<128, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, BwdCfg<128>::kSmemBytes) == cudaSuccess;
  ok = ok && cudaFuncSetAttribute(mala_bwd_kernel<128, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, BwdCfg<128>::kSmemBytes) == cudaSuccess;
  ok = ok && cudaFuncSetAttribute(mala_bwd_kernel<64, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, BwdCfg<64>::kSmemBytes) == cudaSuccess;
  ok = ok && cudaFuncSetAttribute(mala_bwd_kernel<64, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, BwdCfg<64>::kSmemBytes) == cudaSuccess;
  ok = ok && cudaFuncSetAttribute(mala_bwd_kernel<128, true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, BwdCfg<128>::kSmemBytes) == cudaSuccess;
  ok = ok && cudaFuncSetAttribute(mala_bwd_kernel<64, true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, BwdCfg<64>::kSmemBytes) == cudaSuccess;
  ok = ok && cudaFuncSetAttribute(mala_bwd_scout_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, ScoutCfg<128>::kSmemBytes) == cudaSuccess;
  ok = ok && cudaFuncSetAttribute(mala_bwd_scout_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, ScoutCfg<64>::kSmemBytes) == cudaSuccess;
  return ok;
}

template <int D, bool kDense, bool kList = false>
inline int bwd_launch_main(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv, const CUtensorMap& tdo,
                           const CUtensorMap& tacc, const BwdParams& p, cudaStream_t stream) {
  dim3 grid(p.Tk, p.Hkv, p.B);
  mala_bwd_kernel<D, kDense, kList><<<grid, BwdCfg<D>::kThreads, BwdCfg<D>::kSmemBytes, stream>>>(tq, tk, tv, tdo, tacc, p);
  return cudaGetLastError() == cudaSuccess ? MALA_OK : MALA_ERR_CUDA;
}

template <int D>
inline int bwd_launch_scout(const CUtensorMap& tq, const CUtensorMap& tk, const ScoutParams& sp, cudaStream_t stream) {
  dim3 grid((sp.Tk + 1) / 2, sp.Hkv, sp.B);
  mala_bwd_scout_kernel<D><<<grid, ScoutCfg<D>::kThreads, ScoutCfg<D>::kSmemBytes, stream>>>(tq, tk, sp);
  return cudaGetLastError() == cudaSuccess ? MALA_OK : MALA_ERR_CUDA;
}

inline int bwd_launch(mala_tin q, mala_tin k, mala_tin v, mala_tin o, mala_tin dout, const float* lse, mala_tout dq,
                      mala_tout dk, mala_tout dv, const mala_stats* st, int B, int Hq, int Hkv, int N, int Nk, int d,
                      int causal, float scale, float tau, void* ws, size_t ws_bytes, int* status, cudaStream_t stream,
                      const int* cu = nullptr, int total = 0, const int* cu_k = nullptr, int total_k = 0) {
  // Packed sequences (cu): N = Nk = the longest sequence; the tensors are [1, total, H, d]; the per-query vectors and
  // the dQ accumulator are laid out per head over Np = total + 128 B rows (rounded up to a tile).
  const int D = padded_head_size(d);         // columns of the kernels and of the dQ accumulator
  const int qshift = (causal && !cu) ? (Nk - N) % 128 : 0;
  // (cu_k: every sequence has its own shift below 128, so the longest one may span a block more than its rows fill)
  const int T = (N + (cu_k ? 127 : qshift) + 127) / 128, Npg = T * 128, Tk = (Nk + 127) / 128;
  const int Np = cu ? ((total + (cu_k ? 384 : 128) * B + 127) / 128) * 128 : Npg;
  const int Bl = cu ? 1 : B;                 // batch extent of the tensors and of the workspace arrays
  const int Nt = cu ? total : N, Nkt = cu ? (cu_k ? total_k : total) : Nk;   // row extents of the tensors
  uint8_t* w = (uint8_t*)ws;
  float* acc = (float*)w;
  w += bwd_align256((size_t)Bl * Hq * Np * D * sizeof(float));
  const size_t vbytes = bwd_align256((size_t)Bl * Hq * Np * sizeof(float));
  float* lse2 = (float*)w;
  float* bq = (float*)(w + vbytes);
  float* Dq = (float*)(w + 2 * vbytes);

  CUtensorMap tq, tk, tv, tdo, tacc;
  if (!make_tensor_map_f32_tiles(&tacc, acc + 64 * D, (uint64_t)Bl * Hq * (Np / 128), D / 2,
                                 (uint64_t)128 * D * sizeof(float)) ||
      !make_tensor_map_bnhd(&tq, q.p, Bl, Nt, Hq, d, q.sb, q.sn, q.sh, 128) ||
      !make_tensor_map_bnhd(&tk, k.p, Bl, Nkt, Hkv, d, k.sb, k.sn, k.sh, 128) ||
      !make_tensor_map_bnhd(&tv, v.p, Bl, Nkt, Hkv, d, v.sb, v.sn, v.sh, 128) ||
      !make_tensor_map_bnhd(&tdo, dout.p, Bl, Nt, Hq, d, dout.sb, dout.sn, dout.sh, 128))
    return MALA_ERR_TENSOR_MAP;

  if (cudaMemsetAsync(acc, 0, (size_t)Bl * Hq * Np * D * sizeof(float), stream) != cudaSuccess) return MALA_ERR_CUDA;
  BwdParams p;
  p.lse2 = lse2; p.bq = bq; p.Dq = Dq; p.dq_acc = acc;
  p.dk = (__nv_bfloat16*)dk.p; p.dk_sb = dk.sb; p.dk_sn = dk.sn; p.dk_sh = dk.sh;
  p.dv = (__nv_bfloat16*)dv.p; p.dv_sb = dv.sb; p.dv_sn = dv.sn; p.dv_sh = dv.sh;
  p.retained = st ? st->retained_per_block : nullptr;
  p.bitmask = st ? st->tile_bitmask : nullptr;
  p.totals = st ? (unsigned long long*)st->totals : nullptr;
  p.status = status;
  p.B = B; p.Hq = Hq; p.Hkv = Hkv; p.N = N; p.Np = Np; p.T = T; p.words = (T + 31) / 32; p.causal = causal;
  p.Nk = Nk; p.Tk = Tk; p.koff = causal ? (Nk - N) / 128 : 0; p.qshift = qshift;
  p.cu = cu; p.cu_k = cu_k; p.d = d;
  if (cu_k) { p.koff = 0; p.qshift = 0; }    // per sequence, on the device
  p.scale = scale; p.scale_log2 = scale * 1.4426950408889634f;
  p.list_mask = nullptr; p.wpad = 0; p.sel_rows = nullptr; p.accum_dkv = 0;
  if (p.bitmask &&
      cudaMemsetAsync(p.bitmask, 0, (size_t)B * Hq * Tk * p.words * sizeof(uint32_t), stream) != cudaSuccess)
    return MALA_ERR_CUDA;

  {
    const long long rows = (long long)B * Hq * Npg;
    const int wpb = 8;
    const unsigned blocks = (unsigned)((rows + wpb - 1) / wpb);
    bwd_preprocess_kernel<<<blocks, wpb * 32, 0, stream>>>((const __nv_bfloat16*)o.p, o.sb, o.sn, o.sh,
                                                          (const __nv_bfloat16*)dout.p, dout.sb, dout.sn, dout.sh, lse,
                                                          lse2, bq, Dq, B, Hq, N, Np, Nk, d, causal,
                                                          tau > 0.f ? log2f(tau) : -INFINITY, cu, total, Npg, qshift, cu_k);
    if (cudaGetLastError() != cudaSuccess) return MALA_ERR_CUDA;
  }
  const bool dense = (tau == 0.f);
  // tau > 0: two passes where their limits hold and the workspace has room for the masks -- the test of every legal
  // tile first (mala_bwd_scout_kernel), then the dense tile pipeline on the retained tiles only; otherwise the one-pass
  // kernel that tests and works tile by tile.
  const int wpad = bwd_mask_wpad(T);
  const size_t base_bytes = bwd_align256((size_t)Bl * Hq * Np * D * sizeof(float)) + 3 * vbytes;
  const bool two_pass = !dense && MALA_BWD_TWO_PASS && (Hq / Hkv) * 2 * wpad <= kScoutMaskWords && (Hq / Hkv) <= 16 &&
                        ws_bytes >= base_bytes + bwd_list_bytes(B, Hq, T, Tk);
  int rc;
  if (two_pass) {
    uint8_t* lw = (uint8_t*)ws + base_bytes;
    ScoutParams sp;
    sp.bq = bq;
    sp.mask = (uint32_t*)lw;
    sp.row_count = (uint32_t*)(lw + bwd_align256((size_t)B * Hq * Tk * wpad * sizeof(uint32_t)));
    sp.tel_retained = p.retained; sp.tel_bitmask = p.bitmask; sp.totals = p.totals;
    sp.status = status;
    sp.B = B; sp.Hq = Hq; sp.Hkv = Hkv; sp.N = N; sp.Np = Np; sp.T = T; sp.words = p.words; sp.wpad = wpad; sp.causal = causal;
    sp.Nk = Nk; sp.Tk = Tk; sp.koff = p.koff; sp.qshift = p.qshift; sp.cu = cu; sp.cu_k = cu_k;
    sp.scale_log2 = p.scale_log2;
    sp.sample = MALA_BWD_SAMPLE;
    CUtensorMap tq2;   // the queries again, in boxes of two tiles
    if (!make_tensor_map_bnhd(&tq2, q.p, Bl, Nt, Hq, d, q.sb, q.sn, q.sh, 256)) return MALA_ERR_TENSOR_MAP;
    rc = (D == 128) ? bwd_launch_scout<128>(tq2, tk, sp, stream) : bwd_launch_scout<64>(tq2, tk, sp, stream);
    if (rc != MALA_OK) return rc;
    BwdParams pl = p;
    pl.retained = nullptr; pl.bitmask = nullptr; pl.totals = nullptr;   // (the first pass wrote the telemetry of these rows)
    pl.list_mask = sp.mask; pl.wpad = wpad;
    rc = (D == 128) ? bwd_launch_main<128, true, true>(tq, tk, tv, tdo, tacc, pl, stream)
                    : bwd_launch_main<64, true, true>(tq, tk, tv, tdo, tacc, pl, stream);
    if (rc != MALA_OK) return rc;
    if (sp.sample) {   // the rows the first pass left alone: tested and worked tile by tile, added to the stored dK, dV
      BwdParams pd = p;
      pd.sel_rows = sp.row_count; pd.accum_dkv = 1;
      rc = (D == 128) ? bwd_launch_main<128, false>(tq, tk, tv, tdo, tacc, pd, stream)
                      : bwd_launch_main<64, false>(tq, tk, tv, tdo, tacc, pd, stream);
    }
  } else if (D == 128) {
    rc = dense ? bwd_launch_main<128, true>(tq, tk, tv, tdo, tacc, p, stream) : bwd_launch_main<128, false>(tq, tk, tv, tdo, tacc, p, stream);
  } else {
    rc = dense ? bwd_launch_main<64, true>(tq, tk, tv, tdo, tacc, p, stream) : bwd_launch_main<64, false>(tq, tk, tv, tdo, tacc, p, stream);
  }
  if (rc != MALA_OK) return rc;
  {
    const long long n_out = (long long)B * Hq * Npg * (D / 8);
    const unsigned blocks = (unsigned)((n_out + 255) / 256);
    bwd_convert_dq_kernel<<<blocks, 256, 0, stream>>>(acc, (__nv_bfloat16*)dq.p, dq.sb, dq.sn, dq.sh, B, Hq, N, Np, D,
                                                      scale, cu, Npg, qshift, d, cu_k, causal);
    if (cudaGetLastError() != cudaSuccess) return MALA_ERR_CUDA;
  }
  return MALA_OK;
}

}  // namespace mala
