// Split-KV decode over an 8-bit (e4m3) KV cache ("Fused decoding execution"; the cache itself is untouched, only its
// storage type differs).  The decode step is bound by the bytes of K and V it streams, so an 8-bit cache halves its
// time.  Keys and values are stored as e4m3 with one fp32 scale per (sequence, KV head, 128-key tile):
//     k = kscale[b, h_kv, tile] * e4m3(k8),   v = vscale[b, h_kv, tile] * e4m3(v8)
// and the kernel computes exactly the operator of mala_decode on those dequantised values.
//
// The structure is that of mala_decode_split_kernel (transposed problem, keys in the TMEM lanes, packed query heads as
// the N = 16 columns, persistent CTAs, event-driven UMMA warp, V of a retained tile requested after its vote), with the
// 8-bit tiles handled as follows.
//   K  The raw e4m3 tile is an MMA operand as it lands (tcgen05 kind::f8f6f4, 128 bytes of K per row = the whole head
//      size in one swizzle panel): no conversion, no second copy in shared memory.  The other operand has to be 8-bit
//      too, so each query row is written as the sum of two e4m3 rows: with 2^k the power of two that brings the row's
//      largest magnitude into [128, 256), q1 = e4m3(q 2^k) and q2 = e4m3(16 (q 2^k - q1)).  A bf16 significand has 8
//      bits and q1 takes the leading 4, so q 2^k = q1 + q2 / 16 exactly, up to entries 2^-17 below the row's largest
//      (e4m3's subnormal floor).  The two rows are columns h and 4 + h of the MMA (hence at most four heads per KV
//      head), products of e4m3 values are exact in the fp32 accumulator, and the softmax thread forms
//      (S[h] + S[4 + h] / 16) * scale * kscale / 2^k.
//   V  The converter group widens each raw tile to fp16 -- exact: every e4m3 value is an fp16 value -- and applies the
//      tile's scale as two fp16 multiplications (the scale's significand rounded to fp16, then its power of two), so
//      the fp16 V the MMA reads is scale * e4m3(code) to a relative 2^-11.  (Folding the scale into the probabilities
//      instead would push most of them into fp16's subnormal range whenever the scale is small.)  P^T is written as
//      fp16 and O^T += V^T P^T runs as kind::f16.
// fp16 has a narrower range than the bf16 of the other kernels: the running reference maximum may lag the true one by
// at most 2^12 (P^T <= 4096) before O^T is rescaled, and |v| is expected inside fp16's range (|v| <= 65504; values
// below 6e-5 lose precision).
//   warp 0      TMA producer (Q, raw K ring of four; dense kernel: raw V ring of four)
//   warp 1      UMMA warp (and the on-demand raw V copies of the MALA kernel)
//   warps 4-7   softmax group (thread = key of the tile), up to four packed query heads
//   warps 8-11  converter group: Q bf16 -> two e4m3 rows per head (warp = head), raw V -> fp16 stage (thread = key row)
#pragma once
#include <cuda_fp16.h>

#include "mala_decode_split.cuh"
#include "sm100_ptx.cuh"

namespace mala {

#ifdef MALA_F8_TRACE
__device__ long long f8_trace[64 * 16];
#define F8TR(slot, g) do { if (blockIdx.x == 0 && (g) >= 64 && (g) < 128 && (threadIdx.x & 31) == 0) f8_trace[((g) - 64) * 16 + (slot)] = clock64(); } while (0)
#else
#define F8TR(slot, g) do {} while (0)
#endif

struct DecF8Params {
  float* o_part;                 // [B, Hq, num_splits, 128] fp32, normalised per split
  float* lse_part;               // [B, Hq, num_splits] natural log; -inf for an empty split
  uint32_t* retained;            // [B, Hkv, num_splits] or null
  uint32_t* bitmask;             // [B, Hkv, num_splits, words] or null (zero-filled by the host)
  unsigned long long* totals;    // [2] or null
  int* status;
  const float* kscale;           // [B, Hkv, nt]
  const float* vscale;           // [B, Hkv, nt]
  int B, Hq, Hkv, Nk, tps, num_splits, words, n_items, nt;
  float scale_log2, log2_tau;
};

struct DecF8Cfg {
  static constexpr int kRawBytes = 128 * 128;            // one e4m3 tile
  static constexpr int kTileBytes = 128 * 128 * 2;       // one fp16 tile
  static constexpr int kQBytes = 4096, kPBytes = 4096;
  static constexpr int kPStages = 4;
  static constexpr int kQ8Bytes = 2048;                  // 16 rows x 128 e4m3
  static constexpr int kRawStages = 4;                   // raw K ring, raw V ring
  static constexpr int kSmemBytes = 2 * kQBytes + 2 * kQ8Bytes + 2 * kRawStages * kRawBytes + 2 * kTileBytes + kPStages * kPBytes + 1024;
  static constexpr int kThreads = 384;
  static constexpr uint32_t kTmemCols = 128;             // S^T ring 4 x 16, O^T 2 x 16 (item parity)
  static constexpr uint32_t kColO = 64;
};

// Instruction descriptor of tcgen05.mma kind::f16 with fp16 A and B, fp32 accumulate
__host__ __device__ constexpr uint32_t make_idesc_f16(int M, int N, bool a_mn_major, bool b_mn_major) {
  return (1u << 4) | ((a_mn_major ? 1u : 0u) << 15) | ((b_mn_major ? 1u : 0u) << 16) | ((uint32_t)(N >> 3) << 17) |
         ((uint32_t)(M >> 4) << 24);
}

// Instruction descriptor of tcgen05.mma kind::f8f6f4 with e4m3 A and B (format 0), both K-major, fp32 accumulate
__host__ __device__ constexpr uint32_t make_idesc_e4m3(int M, int N) {
  return (1u << 4) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

// two floats -> two e4m3 values (a in the low byte), round to nearest, saturating
__device__ __forceinline__ uint32_t f32x2_to_e4m3x2(float a, float b) {
  uint16_t r;
  asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(b), "f"(a));
  return (uint32_t)r;
}

// two e4m3 values (low byte first) -> two fp16 values
__device__ __forceinline__ uint32_t e4m3x2_to_f16x2(uint32_t two) {
  uint32_t r;
  const uint16_t h = (uint16_t)two;
  asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(r) : "h"(h));
  return r;
}

template <bool kDense, int GP>
__global__ void __launch_bounds__(384, 1)
mala_decode_fp8_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                       const __grid_constant__ CUtensorMap tmV, const DecF8Params p) {
  using Cfg = DecF8Cfg;
  constexpr int RB = Cfg::kRawBytes, TB = Cfg::kTileBytes;
  constexpr int GH = GP;                   // rows of the (single) softmax group
  constexpr int LDN = 16;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  constexpr int RS = Cfg::kRawStages;
  uint8_t* sQ = smem;                      // [2] item parity, bf16 as copied
  uint8_t* sKr = sQ + 2 * Cfg::kQBytes;    // [4] raw K
  uint8_t* sVr = sKr + RS * RB;            // [4] raw V
  uint8_t* sV = sVr + RS * RB;             // [2] fp16 V
  uint8_t* sP = sV + 2 * TB;               // [4] P^T ring
  uint8_t* sQ8 = sP + Cfg::kPStages * Cfg::kPBytes;   // [2] item parity: rows h = q1, 4 + h = q2 (e4m3), rest zero

  __shared__ uint64_t qr_full[2], q_full[2], q_empty[2], kr_full[4], kr_empty[4], vr_full[4], vr_empty[4], v_full[2],
      v_empty[2], s_full[4], s_free[4], vote_bar[4], p_full[4], p_free[4], item_done[2], o_free[2], fin_bar, grp_a;
  __shared__ uint32_t tmem_base_s;
  __shared__ int flag[4];
  __shared__ int v_row[8], v_outer[8];
  __shared__ int v_total_s;                // V tiles requested in all (known when the vote cursor has finished)
  __shared__ int v_sidx[8];                // index of the scale of requested V tile number n, at n & 7
  __shared__ float q_inv[8][4];            // 2^-k of the rows of non-empty item number n, at n & 7
  __shared__ int v_req_s;                  // V tiles requested so far (written after v_sidx, before the copy is issued)
  __shared__ __align__(16) float xch_max[2][4][8], xch_sum[2][4][8];
  __shared__ int early_exit;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int G = p.Hq / p.Hkv;
  const int R = G;
  int* status = p.status;

  for (int i = tid; i < 2 * Cfg::kQ8Bytes / 16; i += Cfg::kThreads) reinterpret_cast<uint4*>(sQ8)[i] = make_uint4(0u, 0u, 0u, 0u);
  for (int i = tid; i < Cfg::kPStages * Cfg::kPBytes / 16; i += Cfg::kThreads) reinterpret_cast<uint4*>(sP)[i] = make_uint4(0u, 0u, 0u, 0u);
  fence_proxy_async_smem();
  if (tid == 0) {
    early_exit = (*(volatile int*)status != 0);
    for (int s = 0; s < 2; ++s) {
      mbar_init(&qr_full[s], 1); mbar_init(&q_full[s], 4); mbar_init(&q_empty[s], 1); mbar_init(&item_done[s], 1);
      mbar_init(&o_free[s], 4);
      mbar_init(&v_full[s], 4); mbar_init(&v_empty[s], 1);
    }
    for (int s = 0; s < 4; ++s) {
      mbar_init(&kr_full[s], 1); mbar_init(&kr_empty[s], 1);
      mbar_init(&vr_full[s], 1); mbar_init(&vr_empty[s], 4);
      mbar_init(&s_full[s], 1); mbar_init(&s_free[s], 4); mbar_init(&vote_bar[s], 1);
      mbar_init(&p_full[s], 4); mbar_init(&p_free[s], 1);
      flag[s] = 0;
    }
    mbar_init(&fin_bar, 1); mbar_init(&grp_a, 4);
    v_total_s = -1;
    v_req_s = 0;
    mbar_fence_init();
  }
  __syncthreads();
  if (early_exit) return;
  if (warp == 0) { tmem_alloc(&tmem_base_s, Cfg::kTmemCols); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tb = tmem_base_s;

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
  auto ready = [&](uint64_t* bar, uint32_t parity) -> bool { return __all_sync(0xffffffffu, mbar_test_wait(bar, parity)); };
  auto scale_index = [&](int b, int hkv, int jt) -> int { return (b * p.Hkv + hkv) * p.nt + jt; };

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      tma_prefetch_desc(&tmQ); tma_prefetch_desc(&tmK); tma_prefetch_desc(&tmV);
      int ne = 0, g = 0;
      bool ok = true;
      for (int item = blockIdx.x; item < p.n_items && ok; item += gridDim.x) {
        int b, hkv, split, T, j0;
        geometry(item, b, hkv, split, T, j0);
        if (T == 0) continue;
        const int ip = ne & 1;
        ok = mbar_wait(&q_empty[ip], ((ne >> 1) & 1) ^ 1, status);
        if (!ok) break;
        mbar_arrive_expect_tx(&qr_full[ip], (uint32_t)R * 128u * 2u);   // two panels of R rows x 128 bytes
        for (int pn = 0; pn < 2; ++pn)
          tma_load_4d(sQ + ip * Cfg::kQBytes + pn * 2048, &tmQ, &qr_full[ip], pn * 64, hkv * G, 0, b);
        for (int t = 0; t < T && ok; ++t, ++g) {
          const int s = g & 3;
          ok = mbar_wait(&kr_empty[s], ((g >> 2) & 1) ^ 1, status);
          if (!ok) break;
          if (!kDense) { v_row[g & 7] = (j0 - t) * 128; v_outer[g & 7] = b; }
          F8TR(0, g);
          mbar_arrive_expect_tx(&kr_full[s], RB);
          tma_load_4d(sKr + s * RB, &tmK, &kr_full[s], 0, (j0 - t) * 128, hkv, b);
          if (kDense) {   // every tile is retained: V follows K
            ok = mbar_wait(&vr_empty[s], ((g >> 2) & 1) ^ 1, status);
            if (!ok) break;
            *(volatile int*)&v_sidx[g & 7] = scale_index(b, hkv, j0 - t);
            __threadfence_block();
            *(volatile int*)&v_req_s = g + 1;
            mbar_arrive_expect_tx(&vr_full[s], RB);
            tma_load_4d(sVr + s * RB, &tmV, &vr_full[s], 0, (j0 - t) * 128, hkv, b);
          }
        }
        ++ne;
      }
      if (!ok) { const long long t0 = clock64(); while (clock64() - t0 < 400000) {} }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ UMMA warp (+ on-demand raw V copies)
    const uint32_t leader = elect_one();
    constexpr uint32_t idesc_qk = make_idesc_e4m3(128, 16);
    constexpr uint32_t idesc_pv = make_idesc_f16(128, 16, true, false);
    const uint64_t dQ0 = make_smem_desc(smem_u32(sQ8), 16, 1024);
    const uint64_t dK0 = make_smem_desc(smem_u32(sKr), 16, 1024);
    const uint64_t dV0 = make_smem_desc(smem_u32(sV), 16384, 1024);   // V tile read MN-major (M = channel)
    const uint64_t dP0 = make_smem_desc(smem_u32(sP), 16, 1024);
    struct Cur { int item, ne, t, T, b, hkv, j0, g; bool valid; };
    auto first_item = [&](Cur& c, int from, int ne, int g) {
      c.valid = false;
      c.g = g;
      for (int item = from; item < p.n_items; item += gridDim.x) {
        int b, hkv, split, T, j0;
        geometry(item, b, hkv, split, T, j0);
        if (T > 0) { c.item = item; c.ne = ne; c.t = 0; c.T = T; c.b = b; c.hkv = hkv; c.j0 = j0; c.valid = true; return; }
      }
    };
    auto advance = [&](Cur& c) {
      if (c.t + 1 < c.T) { ++c.t; ++c.g; return; }
      first_item(c, c.item + gridDim.x, c.ne + 1, c.g + 1);
    };
    Cur cq, cv, cp;                            // next tile to score, to take the vote of, to accumulate
    first_item(cq, blockIdx.x, 0, 0);
    cv = cq; cp = cq;
    int nv = 0;                                // raw V copies requested (MALA) -- ring slot nv & 1
    int npv = 0;                               // PVs issued so far: V stage npv & 1, P^T slot npv & 3
    uint32_t ret_bits = 0;
    int r_item = 0;
    bool ok = true;
    bool told = false;
    long long t_progress = clock64();
    uint32_t idle = 0;
    while (cp.valid && ok) {
      bool progress = false;
      if (!told && !cv.valid) {   // every vote is in: the converter group learns how many V tiles there are
        if (leader) *(volatile int*)&v_total_s = kDense ? cq.g : nv;
        told = true;
      }
      // ---- S^T of tile cq.g
      if (cq.valid && cq.g - cv.g < 4) {
        const int ip = cq.ne & 1, sb = cq.g & 3, kc = cq.g & 3;
        if ((cq.g < 4 || ready(&s_free[sb], (uint32_t)(((cq.g >> 2) - 1) & 1))) &&
            (cq.t > 0 || ready(&q_full[ip], (cq.ne >> 1) & 1)) && ready(&kr_full[kc], (cq.g >> 2) & 1)) {
          tc_fence_after();
          F8TR(1, cq.g);
          const uint32_t dS = tmem_addr(tb, 0, (uint32_t)sb * 16u);
          const uint64_t dQ = desc_advance(dQ0, ip * Cfg::kQ8Bytes), dK = desc_advance(dK0, kc * RB);
#pragma unroll
          for (int k = 0; k < 4; ++k)     // 32 e4m3 elements of the head size per instruction
            mma_ss_f8(dS, desc_advance(dK, k * 32), desc_advance(dQ, k * 32), idesc_qk, k > 0, leader);
          if (leader) {
            tc_commit(&kr_empty[kc]);
            tc_commit(&s_full[sb]);
            if (cq.t == cq.T - 1) tc_commit(&q_empty[ip]);
          }
          advance(cq);
          progress = true;
        }
      }
      // ---- vote of tile cv.g
      if (cv.valid && (!cq.valid || cv.g < cq.g) && cv.g - cp.g < 4) {
        if (kDense) {
          ret_bits |= 1u << (cv.g & 3);
          advance(cv);
          progress = true;
        } else if (ready(&vote_bar[cv.g & 3], (cv.g >> 2) & 1)) {
          const bool retain = __shfl_sync(0xffffffffu, *(volatile int*)&flag[cv.g & 3], 0) != 0;
          if (!retain) {
            ret_bits &= ~(1u << (cv.g & 3));
            advance(cv);
            progress = true;
          } else if (nv < 4 || ready(&vr_empty[nv & 3], (uint32_t)(((nv >> 2) - 1) & 1))) {   // raw V of this tile, on demand
            if (leader) {
              const int row = *(volatile int*)&v_row[cv.g & 7], outer = *(volatile int*)&v_outer[cv.g & 7];
              *(volatile int*)&v_sidx[nv & 7] = scale_index(outer, cv.hkv, row >> 7);
              __threadfence_block();
              *(volatile int*)&v_req_s = nv + 1;
              mbar_arrive_expect_tx(&vr_full[nv & 3], RB);
              tma_load_4d(sVr + (nv & 3) * RB, &tmV, &vr_full[nv & 3], 0, row, cv.hkv, outer);
            }
            __syncwarp();
            ++nv;
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
        const int ip = cp.ne & 1, ps = npv & 3, vc = npv & 1;
        if (retain && ready(&p_full[ps], (uint32_t)((npv >> 2) & 1)) && ready(&v_full[vc], (uint32_t)((npv >> 1) & 1)) &&
            (r_item > 0 || cp.ne < 2 || ready(&o_free[ip], (uint32_t)(((cp.ne >> 1) - 1) & 1)))) {
          tc_fence_after();
          F8TR(2, cp.g);
          const uint32_t dO = tmem_addr(tb, 0, Cfg::kColO + (uint32_t)ip * 16u);
          const uint64_t dV = desc_advance(dV0, vc * TB), dP = desc_advance(dP0, ps * Cfg::kPBytes);
          const uint32_t acc0 = r_item > 0 ? 1u : 0u;
#pragma unroll
          for (int k = 0; k < 8; ++k)
            mma_ss(dO, desc_advance(dV, k * 2048), desc_advance(dP, (k >> 2) * 2048 + (k & 3) * 32), idesc_pv,
                   k > 0 ? 1u : acc0, leader);
          if (leader) { tc_commit(&v_empty[vc]); tc_commit(&p_free[ps]); }
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
        __nanosleep(100);
        if (((++idle) & 0x3f) == 0) {
          if (*(volatile int*)status != 0) ok = false;
          else if (clock64() - t_progress > kWaitLimitCycles) { atomicCAS(status, 0, kDevTimeout); ok = false; }
          ok = __all_sync(0xffffffffu, ok);
        }
      }
    }
    if (!told && leader) *(volatile int*)&v_total_s = kDense ? cq.g : nv;
    __syncwarp();
    if (leader) tc_commit(&fin_bar);
    mbar_wait_warp(&fin_bar, 0, status);
    if (!ok) { const long long t0 = clock64(); while (clock64() - t0 < 400000) {} }
  } else if (warp >= 8) {
    // ------------------------------------------------------------------ converter group
    const int row = (warp - 8) * 32 + lane;    // V: thread = key row of the tile
    const int qh = warp - 8;                   // Q: warp = head of the group
    int nI = 0;                                // non-empty items of this CTA
    for (int item = blockIdx.x; item < p.n_items; item += gridDim.x) {
      int b, hkv, split, T, j0;
      geometry(item, b, hkv, split, T, j0);
      if (T > 0) ++nI;
    }
    // raw row `row`: eight 16-byte chunks, chunk c stored at position c ^ (row & 7); its 16 values become fp16 chunks
    // 2 (c % 4), 2 (c % 4) + 1 of panel c / 4 of the fp16 stage (same swizzle), times the tile's scale
    auto convert_tile = [&](const uint8_t* raw, uint8_t* dst, float sc) {
      const uint8_t* src = raw + row * 128;
      // sc = significand in [1, 2) x power of two, both as fp16 pairs (the power clamped to fp16's range)
      const float sig = __uint_as_float((__float_as_uint(sc) & 0x007fffffu) | 0x3f800000u);
      const int ex = min(max((int)((__float_as_uint(sc) >> 23) & 0xffu) - 127, -24), 15);
      const __half2 sig2 = __float2half2_rn(sig);
      const __half2 pow2 = __float2half2_rn(__uint_as_float((uint32_t)(ex + 127) << 23));
#pragma unroll
      for (int c = 0; c < 8; ++c) {
        const uint4 v = *reinterpret_cast<const uint4*>(src + ((c ^ (row & 7)) << 4));
        const uint32_t w4[4] = {v.x, v.y, v.z, v.w};
        uint32_t h[8];
#pragma unroll
        for (int e = 0; e < 4; ++e) { h[2 * e] = e4m3x2_to_f16x2(w4[e] & 0xffffu); h[2 * e + 1] = e4m3x2_to_f16x2(w4[e] >> 16); }
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          const __half2 t = __hmul2(__hmul2(*reinterpret_cast<const __half2*>(&h[e]), sig2), pow2);
          h[e] = *reinterpret_cast<const uint32_t*>(&t);
        }
        uint8_t* drow = dst + (c >> 2) * 16384 + row * 128;
        const int c0 = 2 * (c & 3);
        *reinterpret_cast<uint4*>(drow + (((c0) ^ (row & 7)) << 4)) = make_uint4(h[0], h[1], h[2], h[3]);
        *reinterpret_cast<uint4*>(drow + (((c0 + 1) ^ (row & 7)) << 4)) = make_uint4(h[4], h[5], h[6], h[7]);
      }
    };
    // Q row qh of an item (128 bf16 in two 64-column panels, lane = four consecutive columns) -> rows qh and 4 + qh
    // of the e4m3 operand
    auto convert_q = [&](const uint8_t* qraw, uint8_t* q8, float* inv) {
      if (qh < R) {
        const int e0 = lane * 4;               // first column of this lane
        const uint8_t* src = qraw + (e0 >> 6) * 2048 + qh * 128 + (((((e0 & 63) >> 3)) ^ (qh & 7)) << 4) + (e0 & 7) * 2;
        const uint2 w = *reinterpret_cast<const uint2*>(src);
        float a[4] = {__uint_as_float(w.x << 16), __uint_as_float(w.x & 0xffff0000u), __uint_as_float(w.y << 16),
                      __uint_as_float(w.y & 0xffff0000u)};
        float mx = fmaxf(fmaxf(fabsf(a[0]), fabsf(a[1])), fmaxf(fabsf(a[2]), fabsf(a[3])));
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        // 2^k brings the row's largest magnitude into [128, 256)  (k = 0 for a zero row; k kept inside fp32's exponents)
        const int ef = (int)((__float_as_uint(mx) >> 23) & 0xffu);
        const int k = ef == 0 ? 0 : min(max(134 - ef, -100), 100);
        const float up = __uint_as_float((uint32_t)(k + 127) << 23), down = __uint_as_float((uint32_t)(127 - k) << 23);
#pragma unroll
        for (int i = 0; i < 4; ++i) a[i] *= up;
        const uint32_t c1 = f32x2_to_e4m3x2(a[0], a[1]) | (f32x2_to_e4m3x2(a[2], a[3]) << 16);
        const uint32_t u01 = e4m3x2_to_f16x2(c1 & 0xffffu), u23 = e4m3x2_to_f16x2(c1 >> 16);   // q1 as rounded
        const float2 f01 = __half22float2(*reinterpret_cast<const __half2*>(&u01));
        const float2 f23 = __half22float2(*reinterpret_cast<const __half2*>(&u23));
        const uint32_t c2 = f32x2_to_e4m3x2((a[0] - f01.x) * 16.f, (a[1] - f01.y) * 16.f) |
                            (f32x2_to_e4m3x2((a[2] - f23.x) * 16.f, (a[3] - f23.y) * 16.f) << 16);
        const int r2 = 4 + qh;
        *reinterpret_cast<uint32_t*>(q8 + qh * 128 + (((e0 >> 4) ^ (qh & 7)) << 4) + (e0 & 15)) = c1;
        *reinterpret_cast<uint32_t*>(q8 + r2 * 128 + (((e0 >> 4) ^ (r2 & 7)) << 4) + (e0 & 15)) = c2;
        if (lane == 0) inv[qh] = down;
      }
    };
    int vq = 0, qq = 0;
    int vpf = 0;                               // V scales requested from memory so far (at most two ahead of vq)
    float vsc0 = 1.f, vsc1 = 1.f;              // scale of V tile number n at n & 1
    bool ok = true;
    long long t_progress = clock64();
    uint32_t idle = 0;
    while (ok) {
      const int v_total = *(volatile int*)&v_total_s;
      if (qq == nI && v_total >= 0 && vq == v_total) break;
      bool progress = false;
      if (vpf - vq < 2 && vpf < *(volatile int*)&v_req_s) {   // the scale of a requested V tile, ahead of its arrival
        const float sc = __ldg(p.vscale + *(volatile int*)&v_sidx[vpf & 7]);
        if (vpf & 1) vsc1 = sc; else vsc0 = sc;
        ++vpf;
      }
      if (qq < nI && ready(&qr_full[qq & 1], (qq >> 1) & 1)) {
        convert_q(sQ + (qq & 1) * Cfg::kQBytes, sQ8 + (qq & 1) * Cfg::kQ8Bytes, q_inv[qq & 7]);
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(&q_full[qq & 1]);
        ++qq;
        progress = true;
      }
      if ((v_total < 0 || vq < v_total) && ready(&vr_full[vq & 3], (vq >> 2) & 1) &&
          (vq < 2 || ready(&v_empty[vq & 1], (uint32_t)(((vq >> 1) - 1) & 1)))) {
        if (vpf == vq) {   // (the request was published before the copy was issued, so it is visible by now)
          const float sc = __ldg(p.vscale + *(volatile int*)&v_sidx[vpf & 7]);
          if (vpf & 1) vsc1 = sc; else vsc0 = sc;
          ++vpf;
        }
        if (warp == 8) F8TR(7, vq);
        convert_tile(sVr + (vq & 3) * RB, sV + (vq & 1) * TB, (vq & 1) ? vsc1 : vsc0);
        fence_proxy_async_smem();
        __syncwarp();
        if (warp == 8) F8TR(8, vq);
        if (lane == 0) { mbar_arrive(&v_full[vq & 1]); mbar_arrive(&vr_empty[vq & 3]); }
        ++vq;
        progress = true;
      }
      if (progress) {
        t_progress = clock64();
        idle = 0;
      } else {
        __nanosleep(64);
        if (((++idle) & 0x3f) == 0) {
          if (*(volatile int*)status != 0) ok = false;
          else if (clock64() - t_progress > kWaitLimitCycles) { atomicCAS(status, 0, kDevTimeout); ok = false; }
          ok = __all_sync(0xffffffffu, ok);
        }
      }
    }
  } else if (warp >= 4) {
    // ------------------------------------------------------------------ softmax group: thread = key of the tile
    const int w = warp & 3;
    const uint32_t lane_base = (uint32_t)w * 32u;
    const int kt = (int)lane_base + lane;
    const float c2 = p.scale_log2;
    const bool head = (kt == 0);
    constexpr float kRescaleGap = 12.f;          // P^T is fp16: exp2(12) is as large as a probability may get
    constexpr int kLanesPerRow = 32 / GH;
    const int pub_row = lane / kLanesPerRow;
    const bool publisher = (lane % kLanesPerRow) == 0;
    int g = 0, ne = 0, rg = 0;
    uint32_t xc = 0;
    bool ok = true;
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
      uint32_t o[LDN];
      tmem_ld_cols<LDN>(tmem_addr(tb, lane_base, Cfg::kColO + (uint32_t)pend_ip * 16u), o);
      tmem_wait_ld();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&o_free[pend_ip]);
#pragma unroll
      for (int q = 0; q < GH; ++q)
        if (q < R) p.o_part[(pend_prow0 + (size_t)q * p.num_splits) * 128 + kt] = __uint_as_float(o[q]) / pend_l[q];
      pend = false;
      return true;
    };
    // the K scale of the tile after this one (in processing order) is requested a tile ahead
    float ks_nx = 1.f;
    bool first = true;
    for (int item = blockIdx.x; item < p.n_items && ok; item += gridDim.x) {
      int b, hkv, split, T, j0;
      geometry(item, b, hkv, split, T, j0);
      const float theta = kDense ? -INFINITY : (p.log2_tau - log2f((float)max(p.Nk, 1)));
      const size_t prow0 = ((size_t)b * p.Hq + hkv * G) * p.num_splits + split;
      const size_t stat_row = (size_t)(b * p.Hkv + hkv) * p.num_splits + split;
      if (T == 0) {
#pragma unroll
        for (int q = 0; q < GH; ++q)
          if (q < R) {
            p.o_part[(prow0 + (size_t)q * p.num_splits) * 128 + kt] = 0.f;
            if (kt == q) p.lse_part[prow0 + (size_t)q * p.num_splits] = -INFINITY;
          }
        if (head && p.retained) p.retained[stat_row] = 0u;
        continue;
      }
      if (first) { ks_nx = __ldg(p.kscale + scale_index(b, hkv, j0)); first = false; }
      // the first tile of the next non-empty item (for the look-ahead at this item's last tile)
      int nb = -1, nh = 0, nj = 0;
      for (int it2 = item + gridDim.x; it2 < p.n_items; it2 += gridDim.x) {
        int b2, h2, s2, T2, j2;
        geometry(it2, b2, h2, s2, T2, j2);
        if (T2 > 0) { nb = b2; nh = h2; nj = j2; break; }
      }
      const int ip = ne & 1;
      const uint32_t colO = Cfg::kColO + (uint32_t)ip * 16u;
      float m_ref[GH], l[GH], lgl[GH], c2q[GH];
      float psum = 0.f;
#pragma unroll
      for (int q = 0; q < GH; ++q) c2q[q] = c2;
#pragma unroll
      for (int q = 0; q < GH; ++q) { m_ref[q] = -INFINITY; l[q] = 0.f; lgl[q] = -INFINITY; }
      int r = 0;
      bool pending_sum = false;
      uint32_t bm_bits = 0;
      int bm_word = -1;
      uint32_t* bm_row = p.bitmask ? p.bitmask + stat_row * p.words : nullptr;
      auto exchange = [&](float mx_row, float (&tmax)[GH]) -> bool {
        const int xb = xc & 1;
        if (publisher) { xch_max[xb][w][pub_row] = mx_row; xch_sum[xb][w][pub_row] = psum; }
        __syncwarp();
        if (lane == 0) mbar_arrive(&grp_a);
        bool k = mbar_wait(&grp_a, xc & 1, status);
        k = __all_sync(0xffffffffu, k);
        ++xc;
        if (!k) return false;
        float a0[GH], a1[GH], a2[GH], a3[GH];
        lds_row<GH>(xch_max[xb][0], a0); lds_row<GH>(xch_max[xb][1], a1);
        lds_row<GH>(xch_max[xb][2], a2); lds_row<GH>(xch_max[xb][3], a3);
#pragma unroll
        for (int q = 0; q < GH; ++q) tmax[q] = fmaxf(fmaxf(a0[q], a1[q]), fmaxf(a2[q], a3[q]));
        if (pending_sum) {
          lds_row<GH>(xch_sum[xb][0], a0); lds_row<GH>(xch_sum[xb][1], a1);
          lds_row<GH>(xch_sum[xb][2], a2); lds_row<GH>(xch_sum[xb][3], a3);
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
        const float ks = ks_nx;
        if (t + 1 < T) ks_nx = __ldg(p.kscale + scale_index(b, hkv, j0 - t - 1));
        else if (nb >= 0) ks_nx = __ldg(p.kscale + scale_index(nb, nh, nj));
        const int sb = g & 3;
        ok = mbar_wait(&s_full[sb], (uint32_t)((g >> 2) & 1), status);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        if (w == 0) F8TR(3, g);
        tc_fence_after();
        uint32_t sr[LDN];
        tmem_ld_cols<LDN>(tmem_addr(tb, lane_base, (uint32_t)sb * 16u), sr);
        tmem_wait_ld();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&s_free[sb]);
        if (t == 0) {
#pragma unroll
          for (int q = 0; q < GH; ++q) c2q[q] = c2 * *(volatile float*)&q_inv[ne & 7][q];
        }
        const int kpos = (j0 - t) * 128 + kt;
        float x[GH], mx[GH], tmax[GH];
#pragma unroll
        for (int q = 0; q < GH; ++q) {   // the two e4m3 rows of the head, the row's 2^-k and the K tile's scale
          x[q] = (kpos < p.Nk && q < R) ? fmaf(__uint_as_float(sr[4 + q]), 0.0625f, __uint_as_float(sr[q])) * (c2q[q] * ks) : -INFINITY;
          mx[q] = x[q];
        }
        RowReduce<GH, 16, true>::run(mx, lane);
        ok = exchange(mx[0], tmax);
        if (!ok) break;
        if (w == 0) F8TR(4, g);
        bool retain = true;
        if (!kDense && r > 0) {
          retain = false;
#pragma unroll
          for (int q = 0; q < GH; ++q)
            retain = retain || (q < R && !(((tmax[q] - (m_ref[q] + lgl[q])) - theta) < 0.f));
        }
        if (!kDense && head) {
          *(volatile int*)&flag[g & 3] = retain ? 1 : 0;
          mbar_arrive(&vote_bar[g & 3]);
        }
        if (!retain) continue;
        if (head && bm_row) {
          const int bit = T - 1 - t;
          if ((bit >> 5) != bm_word) {
            if (bm_word >= 0) bm_row[bm_word] = bm_bits;
            bm_word = bit >> 5;
            bm_bits = 0;
          }
          bm_bits |= 1u << (bit & 31);
        }
        if (r == 0) {
#pragma unroll
          for (int q = 0; q < GH; ++q) m_ref[q] = tmax[q];
        } else {
          float alpha[GH];
          bool resc = false;
#pragma unroll
          for (int q = 0; q < GH; ++q) {
            alpha[q] = 1.f;
            if (q < R && tmax[q] > m_ref[q] + kRescaleGap) {
              alpha[q] = fast_exp2(m_ref[q] - tmax[q]);
              l[q] *= alpha[q];
              lgl[q] = __log2f(l[q]);
              m_ref[q] = tmax[q];
              resc = true;
            }
          }
          if (resc) {
            ok = mbar_wait(&p_free[(rg - 1) & 3], (uint32_t)(((rg - 1) >> 2) & 1), status);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            uint32_t o[LDN];
            tmem_ld_cols<LDN>(tmem_addr(tb, lane_base, colO), o);
            tmem_wait_ld();
#pragma unroll
            for (int q = 0; q < GH; ++q) o[q] = __float_as_uint(__uint_as_float(o[q]) * alpha[q]);
            tmem_st_cols<LDN>(tmem_addr(tb, lane_base, colO), o);
            tmem_wait_st();
            tc_fence_before();
          }
        }
        const int ps = rg & 3;
        if (rg >= 4) {
          ok = mbar_wait(&p_free[ps], (uint32_t)(((rg >> 2) - 1) & 1), status);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
        }
        {
          uint8_t* dst = sP + ps * Cfg::kPBytes + (kt >> 6) * 2048;
          const uint32_t col = (uint32_t)(kt & 63);
#pragma unroll
          for (int q = 0; q < GH; ++q) {
            x[q] = (q < R) ? fast_exp2(x[q] - m_ref[q]) : 0.f;
            *reinterpret_cast<__half*>(dst + sw128_offset((uint32_t)q, col)) = __float2half_rn(x[q]);
          }
        }
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(&p_full[ps]);
        if (w == 0) F8TR(5, g);
        RowReduce<GH, 16, false>::run(x, lane);
        psum = x[0];
        if (w == 0) F8TR(6, g);
        pending_sum = true;
        ++r;
        ++rg;
      }
      if (!ok) break;
      if (pending_sum) {
        float dummy[GH];
        ok = exchange(-INFINITY, dummy);
        if (!ok) break;
      }
      if (pend) { ok = flush(); if (!ok) break; }
      pend = true;
      pend_ip = ip;
      pend_ne = ne;
      pend_prow0 = prow0;
#pragma unroll
      for (int q = 0; q < GH; ++q) pend_l[q] = l[q];
#pragma unroll
      for (int q = 0; q < GH; ++q)
        if (q < R && kt == q) p.lse_part[prow0 + (size_t)q * p.num_splits] = (m_ref[q] + lgl[q]) * 0.6931471805599453f;
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
  if (warp == 0) tmem_dealloc(tb, Cfg::kTmemCols);
}

}  // namespace mala
