// First pass of the MALA backward (Algorithm 2): the offline test of Eq. 4 for every legal tile, and nothing else.
//
// The backward test of a tile depends only on its scores and on the saved log-normalizers, not on any other tile, so
// the retained support of a key block can be found before any gradient work starts.  This kernel does that at the rate
// the tensor pipe forms the scores: one CTA per (pair of key blocks, KV head, batch) keeps both K tiles in shared
// memory and streams the Q tiles of the group's query heads, two at a time, through a ring of two 256-row stages; a
// pair of Q tiles feeds two MMA batches S^T = K_j [Q_i; Q_i+1]^T of shape 128 x 256, one per key block, into two TMEM
// buffers of 256 columns, and four warpgroups -- one per 128-column half of a buffer -- read and test their score tile
// while the other buffer is being formed.  (Why this shape: with one key block per CTA the kernel was bound by the
// delivery of the Q tiles, 32 KB per score tile from L2; with 128 x 128 MMAs it was bound by shared-memory bandwidth,
// which an SS MMA of that shape takes whole, leaving none for the copies that refill the ring; a 128 x 256 MMA reads
// 12 KB per 128 clk and leaves a quarter of it.)  Nothing waits for a vote: a warp that finds a retained entry sets the tile's bit in a shared-memory copy of
// the row's mask, and the row is written out when the head's last tile has been tested.  The second pass
// (mala_bwd_kernel in its list mode) then visits the retained tiles only and runs the dense tile pipeline on them.
//
// Rows that retain everything gain nothing from a first pass (their scores would be formed twice), so the rows of a
// CTA are sampled first: every eighth tile of every head.  A head whose sampled tiles are all retained, for both key
// blocks of the pair, is left to the one-pass kernel (mala_bwd_kernel without the list, restricted to such heads), which
// tests and works tile by tile; only the other heads are tested in full here.
//
// Output, per (batch, query head, key block j): the row's mask (bit i set iff tile (j, i) is retained; rows padded to
// a multiple of four words) and its number of set bits, or an empty mask and the count kScoutDirectRow for a row that
// is left to the one-pass kernel.
//
// Warp roles (640 threads): warp 0 TMA producer (K_j once, Q ring), warp 1 UMMA issuer, warp 2 per-query test offsets
// (bq = lse2 + log2(tau / L_q) of the tile's 128 queries into a ring of four shared-memory slots, with the minimum of
// each 32-column chunk), warps 4-19 the four test groups (thread = key row).
#pragma once
#include <cuda_runtime.h>

#include "../../include/mala.h"
#include "sm100_ptx.cuh"
#include "tensor_map.h"

namespace mala {

constexpr uint32_t kScoutDirectRow = 0xffffffffu;   // row_count of a row left to the one-pass kernel
constexpr int kScoutMaskWords = 4096;               // mask words of one CTA (G heads x 2 key blocks x wpad) in shared memory
constexpr int kScoutSampleStride = 16;              // one pair of every sixteen tiles of a row is sampled first ...
constexpr int kScoutSampleMinTiles = 32;            // ... in rows of at least this many tiles

struct ScoutParams {
  const float* bq;            // [B,Hq,Np] lse2 + log2(tau / L_q); +inf on padding rows
  uint32_t* mask;             // [B,Hq,Tk,wpad] (packed sequences: B entries as well)
  uint32_t* row_count;        // [B,Hq,Tk]
  uint32_t* tel_retained;     // telemetry (may be null): [B,Hq,Tk]
  uint32_t* tel_bitmask;      // telemetry (may be null): [B,Hq,Tk,words], zero-filled by the host
  unsigned long long* totals; // telemetry (may be null)
  int* status;
  int B, Hq, Hkv, N, Np, T, words, wpad, causal;
  int Nk, Tk, koff, qshift;
  const int* cu;
  const int* cu_k;
  int sample;                 // sample the rows first and leave the ones that retain everything to the one-pass kernel
  float scale_log2;
};

template <int D>
struct ScoutCfg {
  static constexpr int kPanels = D / 64;
  static constexpr int kTileBytes = 128 * D * 2;
  static constexpr int kPairBytes = 2 * kTileBytes;                      // two Q tiles: panels of 256 rows
  static constexpr int kSmemBytes = 2 * kTileBytes + 2 * kPairBytes + 1024;   // K of two key blocks, ring of two Q pairs
  static constexpr int kThreads = 640;
};

// The sequence of Q-tile pairs of a CTA, the same for every role: the sampled pairs of all heads, then -- once the
// sampled votes have decided which heads are left to the one-pass kernel (`sync` returns after dflag[] has been
// written) -- the other pairs of the other heads.  body(h, i) handles the Q tiles i, i + 1 of head h (i + 1 may lie
// beyond the last tile); both return false to stop.
template <class Body, class Sync>
__device__ __forceinline__ bool scout_for_each_pair(int G, int i0a, int T, bool sampling, const volatile int* dflag,
                                                    Body body, Sync sync) {
  if (sampling) {
    for (int h = 0; h < G; ++h)
      for (int i = i0a; i < T; i += kScoutSampleStride)
        if (!body(h, i)) return false;
    if (!sync()) return false;
  }
  for (int h = 0; h < G; ++h) {
    if (sampling && dflag[h]) continue;
    for (int i = i0a; i < T; i += 2) {
      if (sampling && ((i - i0a) % kScoutSampleStride) == 0) continue;
      if (!body(h, i)) return false;
    }
  }
  return true;
}

template <int D>
__global__ void __launch_bounds__(640, 1)
mala_bwd_scout_kernel(const __grid_constant__ CUtensorMap tmQ2, const __grid_constant__ CUtensorMap tmK,
                      const ScoutParams p) {
  using Cfg = ScoutCfg<D>;
  constexpr int PAN = Cfg::kPanels;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint8_t* sK = smem;                          // key blocks ja, jb
  uint8_t* sQ = sK + 2 * Cfg::kTileBytes;      // 2 stages of two Q tiles each ([panel][256 rows][128 B])

  __shared__ uint64_t k_full, q_full[2], q_empty[2], s_full[2], s_empty[2], vec_full[2], vec_empty[2], fin_bar, phase_bar;
  __shared__ __align__(16) float vec[2][256];  // [batch & 1][query column of the pair]: bq
  __shared__ float vmin[2][8];                 // [batch & 1][32-column chunk]: smallest bq of the chunk
  __shared__ uint32_t rowmask[kScoutMaskWords];   // [head][key block of the pair][wpad]
  __shared__ int dflag[16];                    // head is left to the one-pass kernel
  __shared__ uint32_t tmem_base_s;
  __shared__ int early_exit;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int ja = 2 * (int)blockIdx.x, jb = ja + 1, hkv = blockIdx.y, b = blockIdx.z;
  const int G = p.Hq / p.Hkv;
  // this sequence (the geometry of mala_bwd_kernel)
  const int row0 = p.cu ? __ldg(p.cu + b) : 0;
  const int Nq = p.cu ? __ldg(p.cu + b + 1) - row0 : p.N;
  const int krow0 = p.cu_k ? __ldg(p.cu_k + b) : row0;
  const int Nkeys = p.cu_k ? __ldg(p.cu_k + b + 1) - krow0 : (p.cu ? Nq : p.Nk);
  const int koff = p.cu_k ? (p.causal ? (Nkeys - Nq) / 128 : 0) : p.koff;
  const int qshift = p.cu_k ? (p.causal ? (Nkeys - Nq) % 128 : 0) : p.qshift;
  const int T = p.cu ? (Nq + qshift + 127) / 128 : p.T;
  const int bz = p.cu ? 0 : b;
  const int prow0 = p.cu ? ((row0 + (p.cu_k ? 384 : 128) * b) / 128) * 128 : 0;
  const int Tk_seq = p.cu ? (Nkeys + 127) / 128 : p.Tk;                      // key blocks of this sequence
  const bool none = p.cu_k && (Nq <= 0 || (p.causal && Nkeys < Nq));         // (no defined tile at all)
  const bool has_a = !none && ja < Tk_seq, has_b = !none && jb < Tk_seq;
  // Q tiles i0a .. T-1 of every head; the second key block's tile exists from i0b on
  const int i0a = p.causal ? max(ja - koff, 0) : 0;
  const int i0b = has_b ? (p.causal ? max(jb - koff, 0) : 0) : T;
  const int ni = has_a ? T - i0a : 0;
  const bool sampling = p.sample && ni >= kScoutSampleMinTiles;
  const size_t out_row0 = ((size_t)b * p.Hq + (size_t)hkv * G) * p.Tk;        // + h * Tk + j
  const int wpad = p.wpad;
  int* status = p.status;
  if (ni <= 0) {   // key blocks without queries: empty rows
    for (int kb = 0; kb < 2; ++kb) {
      const int j = ja + kb;
      if (j >= p.Tk) continue;
      for (int x = tid; x < G * wpad; x += blockDim.x)
        p.mask[(out_row0 + (size_t)(x / wpad) * p.Tk + j) * wpad + x % wpad] = 0u;
      if (tid < G) {
        p.row_count[out_row0 + (size_t)tid * p.Tk + j] = 0u;
        if (p.tel_retained) p.tel_retained[out_row0 + (size_t)tid * p.Tk + j] = 0u;
      }
    }
    return;
  }

  if (tid == 0) {
    early_exit = (*(volatile int*)status != 0);
    mbar_init(&k_full, 1);
    for (int s = 0; s < 2; ++s) {
      mbar_init(&q_full[s], 1); mbar_init(&q_empty[s], 1); mbar_init(&s_full[s], 1); mbar_init(&s_empty[s], 8);
      mbar_init(&vec_full[s], 1); mbar_init(&vec_empty[s], 8);
    }
    mbar_init(&fin_bar, 1); mbar_init(&phase_bar, 1);
    mbar_fence_init();
  }
  for (int x = tid; x < G * 2 * wpad; x += blockDim.x) rowmask[x] = 0u;
  if (tid < 16) dflag[tid] = 0;
  __syncthreads();
  if (early_exit) return;
  if (warp == 0) { tmem_alloc(&tmem_base_s, 512); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tb = tmem_base_s;
  // An MMA batch per key block of the pair and Q pair: batch A always, batch B where the second key block has a legal
  // tile in the pair.  Batch m goes to TMEM buffer m & 1.
  auto batches = [&](int i) -> int { return (has_b && i + 1 >= i0b) ? 2 : 1; };

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      tma_prefetch_desc(&tmQ2); tma_prefetch_desc(&tmK);
      mbar_arrive_expect_tx(&k_full, (has_b ? 2 : 1) * Cfg::kTileBytes);
      for (int pn = 0; pn < PAN; ++pn) {
        tma_load_4d(sK + pn * 16384, &tmK, &k_full, pn * 64, krow0 + ja * 128, hkv, bz);
        if (has_b) tma_load_4d(sK + Cfg::kTileBytes + pn * 16384, &tmK, &k_full, pn * 64, krow0 + jb * 128, hkv, bz);
      }
      int n = 0;
      scout_for_each_pair(G, i0a, T, sampling, dflag, [&](int h, int i) -> bool {
        const int s = n & 1;
        if (!mbar_wait(&q_empty[s], ((n >> 1) & 1) ^ 1, status)) return false;
        mbar_arrive_expect_tx(&q_full[s], Cfg::kPairBytes);
        for (int pn = 0; pn < PAN; ++pn)   // (rows past the tensor read as zeros; a second tile past the head's last one is ignored)
          tma_load_4d(sQ + s * Cfg::kPairBytes + pn * 32768, &tmQ2, &q_full[s], pn * 64, row0 + i * 128 - qshift, hkv * G + h, bz);
        ++n;
        return true;
      }, [&]() -> bool { return mbar_wait(&phase_bar, 0, status); });
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ UMMA issuer (warp-uniform issue loop)
    const uint32_t leader = elect_one();
    constexpr uint32_t idesc = make_idesc_bf16(128, 256, false, false);
    const uint64_t dKa = make_smem_desc(smem_u32(sK), 16, 1024);
    const uint64_t dKb = make_smem_desc(smem_u32(sK + Cfg::kTileBytes), 16, 1024);
    const uint64_t dQ0 = make_smem_desc(smem_u32(sQ), 16, 1024);
    bool ok = mbar_wait_warp(&k_full, 0, status);
    int n = 0, m = 0;
    if (ok) scout_for_each_pair(G, i0a, T, sampling, dflag, [&](int h, int i) -> bool {
      const int s = n & 1;
      if (!mbar_wait_warp(&q_full[s], (n >> 1) & 1, status)) return false;
      const uint64_t dQ = desc_advance(dQ0, s * Cfg::kPairBytes);
      const int nb = batches(i);
      for (int kb = 0; kb < nb; ++kb, ++m) {
        const int buf = m & 1;
        if (!mbar_wait_warp(&s_empty[buf], ((m >> 1) & 1) ^ 1, status)) return false;   // the buffer's previous batch has been read
        tc_fence_after();
        const uint64_t dK = kb ? dKb : dKa;
#pragma unroll
        for (int k = 0; k < D / 16; ++k)
          mma_ss(tmem_addr(tb, 0, buf * 256), desc_advance(dK, (k >> 2) * 16384 + (k & 3) * 32),
                 desc_advance(dQ, (k >> 2) * 32768 + (k & 3) * 32), idesc, k > 0, leader);
        if (leader) tc_commit(&s_full[buf]);
      }
      if (leader) tc_commit(&q_empty[s]);
      ++n;
      return true;
    }, [&]() -> bool { return mbar_wait_warp(&phase_bar, 0, status); });
    __syncwarp();
    if (leader) tc_commit(&fin_bar);
    mbar_wait_warp(&fin_bar, 0, status);
  } else if (warp == 2) {
    // ------------------------------------------------------------------ test offsets of every batch's 256 queries
    int m = 0;
    scout_for_each_pair(G, i0a, T, sampling, dflag, [&](int h, int i) -> bool {
      // lane l carries queries 8 l .. 8 l + 7 of the pair (a second tile past the head's last one reads what follows
      // in the padded vector or +inf beyond it: never used)
      const size_t x = ((size_t)bz * p.Hq + hkv * G + h) * p.Np + (size_t)prow0 + (size_t)i * 128 + lane * 8;
      const bool in = (i + 1 < T) || lane < 16;
      const float4 inf4 = make_float4(INFINITY, INFINITY, INFINITY, INFINITY);
      const float4 v0 = in ? *reinterpret_cast<const float4*>(p.bq + x) : inf4;
      const float4 v1 = in ? *reinterpret_cast<const float4*>(p.bq + x + 4) : inf4;
      float mn = fminf(fminf(fminf(v0.x, v0.y), fminf(v0.z, v0.w)), fminf(fminf(v1.x, v1.y), fminf(v1.z, v1.w)));
      mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, 1));
      mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, 2));
      const int nb = batches(i);
      for (int kb = 0; kb < nb; ++kb, ++m) {   // (one slot per batch: both key blocks get their copy)
        const int s = m & 1;
        if (!mbar_wait_warp(&vec_empty[s], ((m >> 1) & 1) ^ 1, status)) return false;
        *reinterpret_cast<float4*>(&vec[s][lane * 8]) = v0;
        *reinterpret_cast<float4*>(&vec[s][lane * 8 + 4]) = v1;
        if ((lane & 3) == 0) vmin[s][lane >> 2] = mn;
        __syncwarp();
        if (lane == 0) mbar_arrive(&vec_full[s]);
      }
      return true;
    }, [&]() -> bool { return mbar_wait_warp(&phase_bar, 0, status); });
  } else if (warp >= 4) {
    // ------------------------------------------------------------------ test groups: group g takes the 128-column half g & 1
    // (the Q tile i + (g & 1) of the pair) of the batches in buffer g >> 1
    const int g = (warp - 4) >> 2, buf = g >> 1, hf = g & 1;
    const uint32_t lane_base = (uint32_t)(warp & 3) * 32u;
    const int rl = (int)lane_base + lane;
    const float c2 = p.scale_log2;
    const int st = tid - 128;                      // 0 .. 511 among the test threads
    bool ok = true;                                // (a warp whose wait failed goes on through the barriers below)
    int use = 0;                                   // batches this group's buffer has held (parity of its barriers)
    int m = 0;
    scout_for_each_pair(G, i0a, T, sampling, dflag, [&](int h, int i0p) -> bool {
      const int nb = batches(i0p);
      for (int kb = 0; kb < nb; ++kb, ++m) {
        if ((m & 1) != buf || !ok) continue;
        const int j = ja + kb, i = i0p + hf;
        const bool legal = i < T && i >= (kb ? i0b : i0a);     // (the other half of the pair / the first key block only)
        const bool valid_key = (j * 128 + rl) < Nkeys;
        ok = mbar_wait(&s_full[buf], use & 1, status);
        if (ok) ok = mbar_wait(&vec_full[buf], use & 1, status);
        ok = __all_sync(0xffffffffu, ok);
        ++use;
        if (!ok) continue;
        tc_fence_after();
        const bool diag = p.causal && (i + koff == j);
        bool vote = false;
        if (legal) {
#pragma unroll 1
          for (int c = 0; c < 4; ++c) {
            uint32_t sc[32];
            tmem_ld_x32(tmem_addr(tb, lane_base, buf * 256 + hf * 128 + c * 32), sc);
            tmem_wait_ld();
            if (diag) {   // entry (key rl, query col) is legal iff rl <= col
              const uint32_t ninf = 0xff800000u;
#pragma unroll
              for (int e = 0; e < 32; ++e)
                if (c * 32 + e < rl) sc[e] = ninf;
            }
            // bound first: max_e (s_e c2 - bq_e) <= (max_e s_e) c2 - min_e bq_e (c2 > 0; fma is monotone in each argument)
            float m0 = __uint_as_float(sc[0]), m1 = __uint_as_float(sc[1]);
#pragma unroll
            for (int e = 0; e < 7; ++e) {
              m0 = max3(m0, __uint_as_float(sc[2 + 4 * e]), __uint_as_float(sc[3 + 4 * e]));
              m1 = max3(m1, __uint_as_float(sc[4 + 4 * e]), __uint_as_float(sc[5 + 4 * e]));
            }
            const float mx = max3(m0, m1, fmaxf(__uint_as_float(sc[30]), __uint_as_float(sc[31])));
            const bool cand = valid_key && !(fmaf(mx, c2, -vmin[buf][hf * 4 + c]) < 0.f);
            if (__any_sync(0xffffffffu, cand)) {
              const float4* bb = reinterpret_cast<const float4*>(vec[buf] + hf * 128) + c * 8;
              float c0 = -INFINITY, c1 = -INFINITY;
#pragma unroll
              for (int e = 0; e < 8; ++e) {
                const float4 x0 = bb[e];
                c0 = max3(c0, fmaf(__uint_as_float(sc[4 * e + 0]), c2, -x0.x), fmaf(__uint_as_float(sc[4 * e + 1]), c2, -x0.y));
                c1 = max3(c1, fmaf(__uint_as_float(sc[4 * e + 2]), c2, -x0.z), fmaf(__uint_as_float(sc[4 * e + 3]), c2, -x0.w));
              }
              vote = vote || (valid_key && !(fmaxf(c0, c1) < 0.f));
            }
            // (one retaining entry decides the tile: the other chunks need not be read)
            if (__any_sync(0xffffffffu, vote)) break;
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) {
          mbar_arrive(&s_empty[buf]);
          mbar_arrive(&vec_empty[buf]);
        }
        if (__any_sync(0xffffffffu, vote) && lane == 0) atomicOr(&rowmask[(h * 2 + kb) * wpad + (i >> 5)], 1u << (i & 31));
      }
      return true;
    }, [&]() -> bool {
      // all sampled tiles have been tested once the sixteen warps meet here: a head whose samples are all retained,
      // for both key blocks, is left to the one-pass kernel
      asm volatile("bar.sync 1, 512;" ::: "memory");
      if (st < G) {
        int got = 0;
        for (int x = 0; x < 2 * wpad; ++x) got += __popc(rowmask[st * 2 * wpad + x]);
        int want = 0;
        for (int i = i0a; i < T; i += kScoutSampleStride)
          for (int e = 0; e < 2; ++e)
            if (i + e < T) want += (i + e >= i0b) ? 2 : 1;
        dflag[st] = (got == want);
      }
      asm volatile("bar.sync 1, 512;" ::: "memory");
      if (st == 0) mbar_arrive(&phase_bar);
      return true;
    });
    // every tile has been tested once the sixteen warps meet here: the rows go out
    asm volatile("bar.sync 1, 512;" ::: "memory");
    for (int r = (st >> 5); r < G * 2; r += 16) {           // one warp per row
      const int h = r >> 1, kb = r & 1, j = ja + kb;
      if (j >= p.Tk) continue;
      const bool direct = sampling && dflag[h] != 0;
      const size_t orow = out_row0 + (size_t)h * p.Tk + j;
      uint32_t pop = 0;
      for (int x = lane; x < wpad; x += 32) {
        const uint32_t wv = direct ? 0u : rowmask[r * wpad + x];
        p.mask[orow * wpad + x] = wv;
        if (!direct && p.tel_bitmask && x < p.words) p.tel_bitmask[orow * p.words + x] = wv;
        pop += __popc(wv);
      }
      for (int sft = 16; sft > 0; sft >>= 1) pop += __shfl_xor_sync(0xffffffffu, pop, sft);
      if (lane == 0) {
        p.row_count[orow] = direct ? kScoutDirectRow : pop;
        const bool present = kb ? has_b : true;
        if (!direct) {
          if (p.tel_retained) p.tel_retained[orow] = pop;
          if (p.totals && present) {
            atomicAdd(&p.totals[0], (unsigned long long)pop);
            atomicAdd(&p.totals[1], (unsigned long long)(kb ? max(T - i0b, 0) : ni));
          }
        }
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tb, 512);
}

}  // namespace mala
