// Split-KV decode over an 8-bit (e4m3) KV cache ("Fused decoding execution"; the cache itself is untouched, only its
// storage type differs).  The decode step is bound by the bytes of K and V it streams, so an 8-bit cache halves its
// time.  Keys and values are stored as e4m3 with one fp32 scale per (sequence, KV head, 128-key tile):
//     k = kscale[b, h_kv, tile] * e4m3(k8),   v = vscale[b, h_kv, tile] * e4m3(v8)
// and the kernel computes the operator of mala_decode on those dequantised values.
//
// The problem is laid out as in mala_decode_split_kernel (transposed: keys in the TMEM lanes, the packed query heads
// as the N = 16 columns, persistent CTAs over (sequence, KV head, split) work items, V of a retained tile requested
// after its vote).  What differs is that the raw 8-bit tiles are MMA operands as they land (tcgen05 kind::f8f6f4):
// nothing is widened, nothing is copied a second time in shared memory, and a tile costs the shared-memory bandwidth
// of one write and one read of 16 KB.  The other operand of such an MMA has to be 8-bit too, and e4m3 keeps only four
// significant bits, so it is written as the sum of two e4m3 rows, a leading part and sixteen times the remainder:
//   S^T = K8 Q8^T   each query row q becomes q1 = e4m3(q 2^k) and q2 = e4m3(16 (q 2^k - q1)), 2^k the power of two
//                   that brings the row's largest magnitude into [128, 256).  A bf16 significand has 8 bits and q1
//                   takes the leading 4, so q 2^k = q1 + q2 / 16 exactly, up to entries 2^-17 below the row's largest
//                   (e4m3's subnormal floor).  The two rows are columns h and 4 + h of the MMA (hence at most four
//                   heads per KV head), products of e4m3 values are exact in the fp32 accumulator, and a softmax
//                   thread forms (S[h] + S[4 + h] / 16) * scale * kscale / 2^k.
//   O^T += V8^T P8^T  V8 is read MN-major.  A probability enters as P' = 64 exp2(y - yref) with y = x + log2(vscale)
//                   the score of the key weighted by its V tile's scale and yref a running reference of the stream
//                   (so the tile's scale rides on P', inside e4m3's narrow range whatever its magnitude), split as
//                   p1 = e4m3(P'), p2 = e4m3(16 (P' - p1)): relative error 2^-9 for P' >= 2^-6, absolute 2^-14 below
//                   (2^-20 of the largest probability).  yref is raised, and O^T rescaled, whenever a tile's largest
//                   P' would pass e4m3's 448, i.e. when y exceeds yref by more than log2(448 / 64).  The normalizer
//                   is summed in fp32 from the unrounded exp2(x - m), with its own reference m.
//
// At one byte per element a tile arrives twice as fast as in the bf16 kernels, faster than one softmax group can
// take tiles one after the other (its per-tile chain of TMEM load, two cross-warp reductions, exponentials and the
// P^T store is latency, not throughput).  Two softmax groups therefore take alternate tiles (by the CTA's running tile
// count, so that a group's consecutive tiles are never further apart than the rings of four are deep), each with its
// own references, normalizer, P^T slots and O^T accumulator: two online-softmax streams per work item, merged when
// the item is written out.  Everything a tile needs is computed without the item's state -- its row maxima, its
// probabilities against the group's own references, their sums -- except the skip test of Eq. 3, which needs the
// normalizer after the tile before it.  That test is the "turn" of a tile, and turns are taken in tile order (a ring
// of barriers): one thread of the group waits for the turn before, combines its stream's log-sum-exp with the other
// group's published one (all that the test needs), decides, publishes and hands the turn on -- a few dozen
// instructions of one thread -- and the rest of the group picks the decision up behind it.  The probabilities of a
// tile that turns out to be skipped were computed for nothing (a few exponentials per thread); its P^T slot is
// simply reused.  A tile that needs a reference raised takes the slow order instead (decision first, then the
// rescaling, then the probabilities, the turn held meanwhile).  The dense kernel (tau = 0) has no decision to take
// and its groups run unordered.
//
// Every warp that issues asynchronous work walks the CTA's tiles in order and blocks on exactly what its next
// instruction needs (a warp that polls the barriers of several jobs in one loop, sleeping in between, reacts to each
// event a loop iteration late, which at this rate is slower than the tiles arrive):
//   warp 0       TMA producer (Q, raw K ring of six; dense kernel: raw V ring of six)
//   warp 1       converts an item's queries, issues S^T of every tile
//   warp 2       MALA kernel: takes the votes in tile order, requests the raw V copy of a retained tile
//   warp 3       issues O^T += V8^T P8^T of every retained tile
//   warps 4-7    softmax group 0 (thread = key of the tile), up to four packed query heads
//   warps 8-11   softmax group 1
//   warps 12-15  epilogue group (thread = output channel): merges the streams of a finished item, writes its partial
//                output and log-sum-exp, hands the item's state slot and accumulators back
#pragma once
#include <cuda_fp16.h>

#include "mala_decode_split.cuh"
#include "sm100_ptx.cuh"

namespace mala {

// Division of a 32-bit number by a divisor known at launch, as a multiplication and shifts (every thread of the
// softmax groups works out which sequence, KV head and split a work item is; hardware has no integer divide, and the
// few dozen dependent instructions of an emulated one sit on the per-tile chain of those threads).
struct FastDiv {
  uint32_t d, mul, sh;
  __host__ void set(uint32_t divisor) {
    d = divisor;
    uint32_t l = 0;
    while ((1ull << l) < divisor) ++l;
    sh = l;
    mul = (uint32_t)(((1ull << 32) * ((1ull << l) - divisor)) / divisor + 1);
  }
  __device__ __forceinline__ uint32_t div(uint32_t n) const {
    if (d == 1u) return n;
    const uint32_t t = __umulhi(mul, n);
    return (t + ((n - t) >> 1)) >> (sh - 1u);
  }
};

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
  FastDiv by_splits, by_hkv;
};

// NG_: softmax groups -- two for the MALA kernel (their turns couple them; a third only adds to the chain), three for
// the dense kernel (unordered groups; at most three: the rings of four)
template <int NG_>
struct DecF8Cfg {
  static constexpr int kRawBytes = 128 * 128;            // one e4m3 tile
  static constexpr int kStages = 6;                      // raw K ring, raw V ring
  static constexpr int kQBytes = 4096;                   // 16 rows x 128 bf16, as copied
  static constexpr int kQ8Bytes = 2048;                  // 16 rows x 128 e4m3
  static constexpr int kP8Bytes = 2048;                  // 16 rows x 128 e4m3
  static constexpr int kGroups = NG_;
  static constexpr int kPPerGroup = kGroups == 2 ? 4 : 2;                   // P8^T slots of a group: how far it may run ahead of its PVs
  static constexpr int kPSlots = kPPerGroup * kGroups;
  static constexpr int kSmemBytes = 2 * kStages * kRawBytes + 2 * kQBytes + 2 * kQ8Bytes + kPSlots * kP8Bytes + 1024;
  static constexpr int kThreads = 128 * (2 + kGroups);   // issuing warps, softmax groups, epilogue group
  static constexpr uint32_t kColO = 64;                  // S^T ring 4 x 16, then O^T 2 x kGroups x 16 (item parity, group)
  static constexpr uint32_t kTmemCols = (kColO + 2 * kGroups * 16) <= 128 ? 128 : 256;
};

// Instruction descriptor of tcgen05.mma kind::f8f6f4 with e4m3 A and B (format 0), fp32 accumulate
__host__ __device__ constexpr uint32_t make_idesc_e4m3(int M, int N, bool a_mn_major, bool b_mn_major) {
  return (1u << 4) | ((a_mn_major ? 1u : 0u) << 15) | ((b_mn_major ? 1u : 0u) << 16) | ((uint32_t)(N >> 3) << 17) |
         ((uint32_t)(M >> 4) << 24);
}

// two floats -> two e4m3 values (a in the low byte), round to nearest, saturating
__device__ __forceinline__ uint32_t f32x2_to_e4m3x2(float a, float b) {
  uint16_t r;
  asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(b), "f"(a));
  return (uint32_t)r;
}

// two e4m3 values (low byte first) -> two floats (exact)
__device__ __forceinline__ float2 e4m3x2_to_f32x2(uint32_t two) {
  uint32_t r;
  const uint16_t h = (uint16_t)two;
  asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(r) : "h"(h));
  return __half22float2(*reinterpret_cast<const __half2*>(&r));
}

// a and b as e4m3 leading parts (low two bytes of .x) and e4m3 parts of sixteen times the remainders (.y)
__device__ __forceinline__ uint2 split_e4m3x2(float a, float b) {
  const uint32_t lead = f32x2_to_e4m3x2(a, b);
  const float2 back = e4m3x2_to_f32x2(lead);
  return make_uint2(lead, f32x2_to_e4m3x2((a - back.x) * 16.f, (b - back.y) * 16.f));
}

template <bool kDense, int GP, int NG_ = (kDense ? 3 : 2)>
__global__ void __launch_bounds__(DecF8Cfg<NG_>::kThreads, 1)
mala_decode_fp8_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                       const __grid_constant__ CUtensorMap tmV, const DecF8Params p) {
  using Cfg = DecF8Cfg<NG_>;
  constexpr int RB = Cfg::kRawBytes, NS = Cfg::kStages, NG = Cfg::kGroups, PP = Cfg::kPPerGroup;
  constexpr int GH = GP;                   // rows of a softmax group
  constexpr int LDN = 16;
  constexpr float kPScale = 64.f;          // P' of the key that sets the reference
  constexpr float kPGap = 2.8f;            // log2(448 / 64), rounded down: how far y may pass yref
  constexpr float kMGap = 60.f;            // ... and x the normalizer's reference (fp32)
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint8_t* sKr = smem;                     // [6] raw K
  uint8_t* sVr = sKr + NS * RB;            // [6] raw V
  uint8_t* sQ = sVr + NS * RB;             // [2] item parity, bf16 as copied
  uint8_t* sQ8 = sQ + 2 * Cfg::kQBytes;    // [2] item parity: rows h = q1, 4 + h = q2, rest zero
  uint8_t* sP = sQ8 + 2 * Cfg::kQ8Bytes;   // [4 NG] P8^T slots (4 group + n % 4): rows h = p1, 4 + h = p2, rest zero

  __shared__ uint64_t qr_full[2], q_empty[2], kr_full[NS], kr_empty[NS], v_full[NS], v_empty[NS], s_full[4], s_free[4],
      vote_bar[4], vote_read[4], turn_done[4], p_full[PP * NG], p_free[PP * NG], item_done[2], o_free[2], fin_bar,
      grp_bar[NG], dec_bar[NG], ret_full[8], ret_free[8];
  __shared__ uint32_t tmem_base_s;
  __shared__ int flag[4];
  __shared__ int ret_ring[8];              // decision of tile g at g & 7 (vote warp -> PV warp)
  __shared__ float q_inv[8][4];            // 2^-k of the rows of non-empty item number n, at n & 7
  __shared__ __align__(16) float xch[NG][2][4][8];         // [group][buffer][warp][row]
  __shared__ __align__(16) float st_m[2][NG][4], st_l[2][NG][4], st_y[2][NG][4];   // [item parity][group][row]: (m, l, yref)
  __shared__ __align__(16) float st_a[2][NG][4];           // ... and m + log2 l, all that the other groups' turns need
  __shared__ int st_r[2][NG];                              // ... and retained tiles of the group in the item
  __shared__ int early_exit;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int G = p.Hq / p.Hkv;
  const int R = G;
  int* status = p.status;

  for (int i = tid; i < (2 * Cfg::kQ8Bytes + Cfg::kPSlots * Cfg::kP8Bytes) / 16; i += Cfg::kThreads)
    reinterpret_cast<uint4*>(sQ8)[i] = make_uint4(0u, 0u, 0u, 0u);
  fence_proxy_async_smem();
  if (tid == 0) {
    early_exit = (*(volatile int*)status != 0);
    for (int s = 0; s < 2; ++s) {
      mbar_init(&qr_full[s], 1); mbar_init(&q_empty[s], 1); mbar_init(&item_done[s], 1); mbar_init(&o_free[s], 4);
    }
    for (int s = 0; s < NG; ++s) { mbar_init(&grp_bar[s], 4); mbar_init(&dec_bar[s], 1); }
    for (int s = 0; s < PP * NG; ++s) { mbar_init(&p_full[s], 4); mbar_init(&p_free[s], 1); }
    for (int s = 0; s < NS; ++s) {
      mbar_init(&kr_full[s], 1); mbar_init(&kr_empty[s], 1); mbar_init(&v_full[s], 1); mbar_init(&v_empty[s], 1);
    }
    for (int s = 0; s < 4; ++s) {
      mbar_init(&s_full[s], 1); mbar_init(&s_free[s], 4); mbar_init(&vote_bar[s], 1); mbar_init(&vote_read[s], 1);
      mbar_init(&turn_done[s], 1);
      flag[s] = 0;
    }
    for (int s = 0; s < 8; ++s) { mbar_init(&ret_full[s], 1); mbar_init(&ret_free[s], 1); }
    mbar_init(&fin_bar, 1);
    for (int i = 0; i < 2 * NG * 4; ++i) {
      (&st_l[0][0][0])[i] = 0.f; (&st_m[0][0][0])[i] = -INFINITY; (&st_y[0][0][0])[i] = 0.f; (&st_a[0][0][0])[i] = -INFINITY;
    }
    for (int i = 0; i < 2 * NG; ++i) (&st_r[0][0])[i] = 0;
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
    const int bh = (int)p.by_splits.div((uint32_t)item);
    split = item - bh * p.num_splits;
    b = (int)p.by_hkv.div((uint32_t)bh);
    hkv = bh - b * p.Hkv;
    const int lo = split * p.tps * 128;
    const int hi = min(p.Nk, lo + p.tps * 128);
    T = hi > lo ? (hi - lo + 127) / 128 : 0;
    j0 = lo / 128 + T - 1;
  };
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
          const int s = g % NS;
          const uint32_t ph = (uint32_t)((g / NS) & 1);
          ok = mbar_wait(&kr_empty[s], ph ^ 1u, status);
          if (!ok) break;
          mbar_arrive_expect_tx(&kr_full[s], RB);
          tma_load_4d(sKr + s * RB, &tmK, &kr_full[s], 0, (j0 - t) * 128, hkv, b);
          if (kDense) {   // every tile is retained: V follows K
            ok = mbar_wait(&v_empty[s], ph ^ 1u, status);
            if (!ok) break;
            mbar_arrive_expect_tx(&v_full[s], RB);
            tma_load_4d(sVr + s * RB, &tmV, &v_full[s], 0, (j0 - t) * 128, hkv, b);
          }
        }
        ++ne;
      }
      if (!ok) { const long long t0 = clock64(); while (clock64() - t0 < 400000) {} }
    }
  } else if (warp <= 3) {
    // ------------------------------------------------------------------ the three issuing warps
    const uint32_t leader = elect_one();
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
    Cur c;
    first_item(c, blockIdx.x, 0, 0);
    bool ok = true;
    if (warp == 1) {
      // ---- Q of an item -> two e4m3 rows per head; S^T = K8 Q8^T of every tile
      constexpr uint32_t idesc_qk = make_idesc_e4m3(128, 16, false, false);
      const uint64_t dQ0 = make_smem_desc(smem_u32(sQ8), 16, 1024);
      const uint64_t dK0 = make_smem_desc(smem_u32(sKr), 16, 1024);
      for (; c.valid && ok; advance(c)) {
        const int ip = c.ne & 1, sb = c.g & 3, kc = c.g % NS;
        if (c.g >= 4) {
          ok = mbar_wait_warp(&s_free[sb], (uint32_t)(((c.g >> 2) - 1) & 1), status);
          // (the vote of the tile that had this slot has been read: its flag may be overwritten)
          if (!kDense && ok) ok = mbar_wait_warp(&vote_read[sb], (uint32_t)(((c.g >> 2) - 1) & 1), status);
        }
        if (ok && c.t == 0) {
          // the item's queries have landed (which the producer requested once the MMAs of the item two before had
          // read this slot): row qh (128 bf16 in two 64-column panels, lane = four consecutive columns) becomes
          // rows qh and 4 + qh of the e4m3 operand
          ok = mbar_wait_warp(&qr_full[ip], (uint32_t)((c.ne >> 1) & 1), status);
          if (!ok) break;
          const uint8_t* qraw = sQ + ip * Cfg::kQBytes;
          uint8_t* q8 = sQ8 + ip * Cfg::kQ8Bytes;
          for (int qh = 0; qh < R; ++qh) {
            const int e0 = lane * 4;
            const uint8_t* src = qraw + (e0 >> 6) * 2048 + qh * 128 + (((((e0 & 63) >> 3)) ^ (qh & 7)) << 4) + (e0 & 7) * 2;
            const uint2 w2 = *reinterpret_cast<const uint2*>(src);
            float a[4] = {__uint_as_float(w2.x << 16), __uint_as_float(w2.x & 0xffff0000u), __uint_as_float(w2.y << 16),
                          __uint_as_float(w2.y & 0xffff0000u)};
            float mx = fmaxf(fmaxf(fabsf(a[0]), fabsf(a[1])), fmaxf(fabsf(a[2]), fabsf(a[3])));
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
            // 2^k brings the row's largest magnitude into [128, 256)  (k = 0 for a zero row; kept inside fp32's exponents)
            const int ef = (int)((__float_as_uint(mx) >> 23) & 0xffu);
            const int k = ef == 0 ? 0 : min(max(134 - ef, -100), 100);
            const float up = __uint_as_float((uint32_t)(k + 127) << 23), down = __uint_as_float((uint32_t)(127 - k) << 23);
            const uint2 s01 = split_e4m3x2(a[0] * up, a[1] * up), s23 = split_e4m3x2(a[2] * up, a[3] * up);
            const int r2 = 4 + qh;
            *reinterpret_cast<uint32_t*>(q8 + qh * 128 + (((e0 >> 4) ^ (qh & 7)) << 4) + (e0 & 15)) = s01.x | (s23.x << 16);
            *reinterpret_cast<uint32_t*>(q8 + r2 * 128 + (((e0 >> 4) ^ (r2 & 7)) << 4) + (e0 & 15)) = s01.y | (s23.y << 16);
            if (lane == 0) q_inv[c.ne & 7][qh] = down;
          }
          fence_proxy_async_smem();
          __syncwarp();
        }
        if (ok) ok = mbar_wait_warp(&kr_full[kc], (uint32_t)((c.g / NS) & 1), status);
        if (!ok) break;
        tc_fence_after();
        const uint32_t dS = tmem_addr(tb, 0, (uint32_t)sb * 16u);
        const uint64_t dQ = desc_advance(dQ0, ip * Cfg::kQ8Bytes), dK = desc_advance(dK0, kc * RB);
#pragma unroll
        for (int k = 0; k < 4; ++k)     // 32 e4m3 elements of the head size per instruction
          mma_ss_f8(dS, desc_advance(dK, k * 32), desc_advance(dQ, k * 32), idesc_qk, k > 0, leader);
        if (leader) {
          tc_commit(&kr_empty[kc]);
          tc_commit(&s_full[sb]);
          if (c.t == c.T - 1) tc_commit(&q_empty[ip]);
        }
        __syncwarp();
      }
    } else if (warp == 2) {
      // ---- the votes (MALA kernel): a retained tile's raw V copy is requested, the decision is passed on
      if (!kDense) {
        int nv = 0;                              // raw V copies requested -- ring slot nv % 6
        for (; c.valid && ok; advance(c)) {
          ok = mbar_wait_warp(&vote_bar[c.g & 3], (uint32_t)((c.g >> 2) & 1), status);
          if (ok && c.g >= 8) ok = mbar_wait_warp(&ret_free[c.g & 7], (uint32_t)(((c.g >> 3) - 1) & 1), status);
          if (!ok) break;
          const bool retain = __shfl_sync(0xffffffffu, *(volatile int*)&flag[c.g & 3], 0) != 0;
          __syncwarp();
          if (leader) mbar_arrive(&vote_read[c.g & 3]);
          if (retain) {
            const int vs = nv % NS;
            if (nv >= NS) ok = mbar_wait_warp(&v_empty[vs], (uint32_t)(((nv / NS) - 1) & 1), status);
            if (!ok) break;
            if (leader) {
              mbar_arrive_expect_tx(&v_full[vs], RB);
              tma_load_4d(sVr + vs * RB, &tmV, &v_full[vs], 0, (c.j0 - c.t) * 128, c.hkv, c.b);
            }
            ++nv;
          }
          if (leader) {
            *(volatile int*)&ret_ring[c.g & 7] = retain ? 1 : 0;
            mbar_arrive(&ret_full[c.g & 7]);
          }
          __syncwarp();
        }
      }
    } else {
      // ---- O^T += V8^T P8^T of every retained tile, into the accumulator of the tile's softmax group
      constexpr uint32_t idesc_pv = make_idesc_e4m3(128, 16, true, false);
      const uint64_t dV0 = make_smem_desc(smem_u32(sVr), 16384, 1024);   // V tile read MN-major (M = channel)
      const uint64_t dP0 = make_smem_desc(smem_u32(sP), 16, 1024);
      int npv = 0;                               // PVs issued so far: raw V stage npv % 6
      int npv_g[NG], r_item_g[NG];               // ... per softmax group (P8^T slot 4 group + n % 4), and of the current item
#pragma unroll
      for (int i = 0; i < NG; ++i) { npv_g[i] = 0; r_item_g[i] = 0; }
      int r_item = 0;
      for (; c.valid && ok; advance(c)) {
        bool retain = true;
        if (!kDense) {
          ok = mbar_wait_warp(&ret_full[c.g & 7], (uint32_t)((c.g >> 3) & 1), status);
          if (!ok) break;
          retain = __shfl_sync(0xffffffffu, *(volatile int*)&ret_ring[c.g & 7], 0) != 0;
          __syncwarp();
          if (leader) mbar_arrive(&ret_free[c.g & 7]);
        }
        const int ip = c.ne & 1;
        if (retain) {
          const int gp = c.g % NG;               // the softmax group of this tile
          int n_g = 0, ri_g = 0;
#pragma unroll
          for (int i = 0; i < NG; ++i) if (i == gp) { n_g = npv_g[i]; ri_g = r_item_g[i]; }
          const int ps = PP * gp + (n_g % PP), vc = npv % NS;
          ok = mbar_wait_warp(&p_full[ps], (uint32_t)((n_g / PP) & 1), status);
          if (ok) ok = mbar_wait_warp(&v_full[vc], (uint32_t)((npv / NS) & 1), status);
          if (ok && r_item == 0 && c.ne >= 2)
            ok = mbar_wait_warp(&o_free[ip], (uint32_t)(((c.ne >> 1) - 1) & 1), status);
          if (!ok) break;
          tc_fence_after();
          const uint32_t dO = tmem_addr(tb, 0, Cfg::kColO + (uint32_t)(ip * NG + gp) * 16u);
          const uint64_t dV = desc_advance(dV0, vc * RB), dP = desc_advance(dP0, ps * Cfg::kP8Bytes);
          const uint32_t acc0 = ri_g > 0 ? 1u : 0u;
#pragma unroll
          for (int k = 0; k < 4; ++k)     // 32 keys per instruction: 32 rows of the V tile, 32 bytes of a P8^T row
            mma_ss_f8(dO, desc_advance(dV, k * 4096), desc_advance(dP, k * 32), idesc_pv, k > 0 ? 1u : acc0, leader);
          if (leader) { tc_commit(&v_empty[vc]); tc_commit(&p_free[ps]); }
          ++npv;
          ++r_item;
#pragma unroll
          for (int i = 0; i < NG; ++i) if (i == gp) { ++npv_g[i]; ++r_item_g[i]; }
        }
        if (c.t == c.T - 1) {
          if (leader) tc_commit(&item_done[ip]);
          r_item = 0;
#pragma unroll
          for (int i = 0; i < NG; ++i) r_item_g[i] = 0;
        }
        __syncwarp();
      }
      if (leader) tc_commit(&fin_bar);
      __syncwarp();
      mbar_wait_warp(&fin_bar, 0, status);
    }
    if (!ok) { const long long t0 = clock64(); while (clock64() - t0 < 400000) {} }
  } else if (warp >= 4 + 4 * NG) {
    // ------------------------------------------------------------------ epilogue group: thread = output channel
    // An item is written out when its last PV has completed: the groups' streams (m, l, yref, O^T) are merged, the
    // split's partial output and log-sum-exp stored, and the item's state slot and accumulators handed back.
    const int w = warp & 3;
    const uint32_t lane_base = (uint32_t)w * 32u;
    const int kt = (int)lane_base + lane;
    const bool head = (kt == 0);
    int ne = 0;
    bool ok = true;
    for (int item = blockIdx.x; item < p.n_items && ok; item += gridDim.x) {
      int b, hkv, split, T, j0;
      geometry(item, b, hkv, split, T, j0);
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
      const int ip = ne & 1;
      ok = mbar_wait(&item_done[ip], (uint32_t)((ne >> 1) & 1), status);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      float M[GH], L[GH], num[GH];
#pragma unroll
      for (int q = 0; q < GH; ++q) { M[q] = -INFINITY; L[q] = 0.f; num[q] = 0.f; }
      int r_all = 0;
#pragma unroll
      for (int s2 = 0; s2 < NG; ++s2) {
        float ms[GH], ls[GH];
        lds_row<GH>(st_m[ip][s2], ms);
        lds_row<GH>(st_l[ip][s2], ls);
#pragma unroll
        for (int q = 0; q < GH; ++q) M[q] = fmaxf(M[q], ls[q] > 0.f ? ms[q] : -INFINITY);
        r_all += *(volatile int*)&st_r[ip][s2];
      }
#pragma unroll
      for (int s2 = 0; s2 < NG; ++s2) {
        float ms[GH], ls[GH], ys[GH];
        lds_row<GH>(st_m[ip][s2], ms);
        lds_row<GH>(st_l[ip][s2], ls);
        lds_row<GH>(st_y[ip][s2], ys);
        uint32_t o[LDN];
        tmem_ld_cols<LDN>(tmem_addr(tb, lane_base, Cfg::kColO + (uint32_t)(ip * NG + s2) * 16u), o);
        tmem_wait_ld();
#pragma unroll
        for (int q = 0; q < GH; ++q)
          if (ls[q] > 0.f) {   // (the accumulator of a group that retained nothing was never written)
            L[q] += ls[q] * fast_exp2(ms[q] - M[q]);
            num[q] += fmaf(__uint_as_float(o[4 + q]), 0.0625f, __uint_as_float(o[q])) * fast_exp2(ys[q] - M[q]);
          }
      }
      tc_fence_before();
      asm volatile("bar.sync 1, 128;" ::: "memory");   // every thread of the group has read the item's state
      if (head) {     // the slot starts the item after next empty
#pragma unroll
        for (int s2 = 0; s2 < NG; ++s2) {
#pragma unroll
          for (int q = 0; q < GH; ++q) { st_l[ip][s2][q] = 0.f; st_a[ip][s2][q] = -INFINITY; }
          *(volatile int*)&st_r[ip][s2] = 0;
        }
      }
      if (lane == 0) mbar_arrive(&o_free[ip]);
#pragma unroll
      for (int q = 0; q < GH; ++q)
        if (q < R) {
          p.o_part[(prow0 + (size_t)q * p.num_splits) * 128 + kt] = num[q] / (L[q] * kPScale);
          if (kt == q) p.lse_part[prow0 + (size_t)q * p.num_splits] = (M[q] + __log2f(L[q])) * 0.6931471805599453f;
        }
      if (head) {
        if (p.retained) p.retained[stat_row] = (uint32_t)r_all;
        if (p.totals) {
          atomicAdd(&p.totals[0], (unsigned long long)r_all);
          atomicAdd(&p.totals[1], (unsigned long long)T);
        }
      }
      ++ne;
    }
  } else {
    // ------------------------------------------------------------------ softmax groups: thread = key of the tile
    // Group n takes the CTA's tiles n, n + NG, .. (counted through all its items, so that a group's consecutive
    // tiles are never further apart than the rings of four are deep).
    const int grp = (warp - 4) >> 2;
    const int w = warp & 3;
    const uint32_t lane_base = (uint32_t)w * 32u;
    const int kt = (int)lane_base + lane;
    const float c2 = p.scale_log2;
    const bool head = (kt == 0);
    constexpr int kLanesPerRow = 32 / GH;
    const int pub_row = lane / kLanesPerRow;
    const bool publisher = (lane % kLanesPerRow) == 0;
    const float theta = kDense ? -INFINITY : (p.log2_tau - log2f((float)max(p.Nk, 1)));
    int ne = 0, g0 = 0;                          // non-empty items so far, tiles of those items
    int rg = 0;                                  // retained tiles of this group so far: P8^T slot 4 grp + rg % 4
    int nt_own = 0;                              // tiles of this group so far (phase of its decision barrier)
    uint32_t xc = 0;                             // exchanges of this group so far (buffer and barrier phase xc & 1)
    bool ok = true;
    // one value per (warp, row) to all threads of the group
    auto exchange = [&](float mine, float (&a0)[GH], float (&a1)[GH], float (&a2)[GH], float (&a3)[GH]) -> bool {
      const int xb = xc & 1;
      if (publisher) xch[grp][xb][w][pub_row] = mine;
      __syncwarp();
      if (lane == 0) mbar_arrive(&grp_bar[grp]);
      bool k = mbar_wait(&grp_bar[grp], xc & 1, status);
      k = __all_sync(0xffffffffu, k);
      ++xc;
      if (!k) return false;
      lds_row<GH>(xch[grp][xb][0], a0); lds_row<GH>(xch[grp][xb][1], a1);
      lds_row<GH>(xch[grp][xb][2], a2); lds_row<GH>(xch[grp][xb][3], a3);
      return true;
    };
    // scales of the tile this group takes next (requested while the one before it is processed; loaded straight
    // into the registers they are used from)
    auto ld_scale = [&](const float* base, int idx) -> float {
      float v;
      asm volatile("ld.global.nc.f32 %0, [%1];" : "=f"(v) : "l"(base + idx));
      return v;
    };
    float ks_nx = 1.f, vs_nx = 1.f;
    bool first = true;
    for (int item = blockIdx.x; item < p.n_items && ok; item += gridDim.x) {
      int b, hkv, split, T, j0;
      geometry(item, b, hkv, split, T, j0);
      const size_t stat_row = (size_t)(b * p.Hkv + hkv) * p.num_splits + split;
      if (T == 0) continue;
      const int ip = ne & 1;
      const uint32_t colO = Cfg::kColO + (uint32_t)(ip * NG + grp) * 16u;
      uint32_t* bm_row = p.bitmask ? p.bitmask + stat_row * p.words : nullptr;
      float m_ref[GH], l[GH], yref[GH], c2q[GH], a_own[GH];
#pragma unroll
      for (int q = 0; q < GH; ++q) { m_ref[q] = -INFINITY; l[q] = 0.f; yref[q] = 0.f; c2q[q] = c2; a_own[q] = -INFINITY; }
      int r = 0;                                 // tiles of the item this group has retained
      bool have_q = false, have_slot = false;
      for (int t = (grp + NG - g0 % NG) % NG; t < T; t += NG) {
        const int g = g0 + t;
        if (first) {
          ks_nx = ld_scale(p.kscale, scale_index(b, hkv, j0 - t));
          vs_nx = ld_scale(p.vscale, scale_index(b, hkv, j0 - t));
          first = false;
        }
        const float ks = ks_nx, lv = __log2f(vs_nx);
        if (t + NG < T) {
          ks_nx = ld_scale(p.kscale, scale_index(b, hkv, j0 - t - NG));
          vs_nx = ld_scale(p.vscale, scale_index(b, hkv, j0 - t - NG));
        } else {   // the group's first tile in the next item that has one
          int g0n = g0 + T;
          for (int it2 = item + gridDim.x; it2 < p.n_items; it2 += gridDim.x) {
            int b2, h2, s2, T2, j2;
            geometry(it2, b2, h2, s2, T2, j2);
            const int t2 = (grp + NG - g0n % NG) % NG;
            if (t2 < T2) {
              ks_nx = ld_scale(p.kscale, scale_index(b2, h2, j2 - t2));
              vs_nx = ld_scale(p.vscale, scale_index(b2, h2, j2 - t2));
              break;
            }
            g0n += T2;
          }
        }
        const int sb = g & 3;
        ok = mbar_wait(&s_full[sb], (uint32_t)((g >> 2) & 1), status);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after();
        uint32_t sr[LDN];
        tmem_ld_cols<LDN>(tmem_addr(tb, lane_base, (uint32_t)sb * 16u), sr);
        tmem_wait_ld();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&s_free[sb]);
        if (!have_q) {
#pragma unroll
          for (int q = 0; q < GH; ++q) c2q[q] = c2 * *(volatile float*)&q_inv[ne & 7][q];
          have_q = true;
        }
        const int kpos = (j0 - t) * 128 + kt;
        float x[GH], tmax[GH], psum[GH];
#pragma unroll
        for (int q = 0; q < GH; ++q) {   // the two e4m3 rows of the head, the row's 2^-k and the K tile's scale
          x[q] = (kpos < p.Nk && q < R) ? fmaf(__uint_as_float(sr[4 + q]), 0.0625f, __uint_as_float(sr[q])) * (c2q[q] * ks) : -INFINITY;
          psum[q] = 0.f;
        }
        const int ps = PP * grp + (rg % PP);
        // P8^T of this tile into slot ps against the group's references; e[] = the unrounded exp2(x - m)
        auto store_p = [&](float (&e)[GH]) -> bool {
          if (rg >= PP) {
            bool k = mbar_wait(&p_free[ps], (uint32_t)(((rg / PP) - 1) & 1), status);
            k = __all_sync(0xffffffffu, k);
            if (!k) return false;
          }
          float pp[GH];
#pragma unroll
          for (int q = 0; q < GH; ++q) {
            e[q] = (q < R) ? fast_exp2(x[q] - m_ref[q]) : 0.f;
            // P' = 64 exp2(x + lv - yref) = e * 64 exp2(m + lv - yref): the tile's V scale rides on the probability
            pp[q] = (q < R) ? e[q] * (kPScale * fast_exp2((m_ref[q] + lv) - yref[q])) : 0.f;
          }
          uint8_t* dst = sP + ps * Cfg::kP8Bytes;
          const uint32_t chunk = (uint32_t)kt >> 4, within = (uint32_t)kt & 15u;
          if constexpr (GH == 1) {
            const uint2 s0 = split_e4m3x2(pp[0], 0.f);
            dst[0 * 128 + ((chunk ^ 0u) << 4) + within] = (uint8_t)s0.x;
            dst[4 * 128 + ((chunk ^ 4u) << 4) + within] = (uint8_t)s0.y;
          } else {
#pragma unroll
            for (int q = 0; q < GH; q += 2) {
              const uint2 s01 = split_e4m3x2(pp[q], pp[q + 1]);
              dst[(q + 0) * 128 + ((chunk ^ (uint32_t)(q + 0)) << 4) + within] = (uint8_t)s01.x;
              dst[(q + 1) * 128 + ((chunk ^ (uint32_t)(q + 1)) << 4) + within] = (uint8_t)(s01.x >> 8);
              dst[(q + 4) * 128 + ((chunk ^ (uint32_t)(q + 4)) << 4) + within] = (uint8_t)s01.y;
              dst[(q + 5) * 128 + ((chunk ^ (uint32_t)(q + 5)) << 4) + within] = (uint8_t)(s01.y >> 8);
            }
          }
          fence_proxy_async_smem();
          return true;
        };
        // ... and its row sums over the group
        auto probabilities = [&]() -> bool {
          float e[GH], a0[GH], a1[GH], a2[GH], a3[GH];
          if (!store_p(e)) return false;
          RowReduce<GH, 16, false>::run(e, lane);
          if (!exchange(e[0], a0, a1, a2, a3)) return false;
#pragma unroll
          for (int q = 0; q < GH; ++q) psum[q] = (a0[q] + a1[q]) + (a2[q] + a3[q]);
          return true;
        };
        // The row maxima first; then the probabilities against the group's references, ahead of the decision, unless
        // a maximum is too far above a reference (they are then formed on the slow path, after the decision).
        bool fast = true;
        {
          float mx[GH], a0[GH], a1[GH], a2[GH], a3[GH];
#pragma unroll
          for (int q = 0; q < GH; ++q) mx[q] = x[q];
          RowReduce<GH, 16, true>::run(mx, lane);
          ok = exchange(mx[0], a0, a1, a2, a3);
          if (!ok) break;
#pragma unroll
          for (int q = 0; q < GH; ++q) tmax[q] = fmaxf(fmaxf(a0[q], a1[q]), fmaxf(a2[q], a3[q]));
        }
        if (r == 0) {
#pragma unroll
          for (int q = 0; q < GH; ++q) { m_ref[q] = tmax[q]; yref[q] = tmax[q] + lv; }   // (nothing accumulated yet)
        } else {
#pragma unroll
          for (int q = 0; q < GH; ++q)
            fast = fast && !(q < R && (tmax[q] + lv > yref[q] + kPGap || tmax[q] > m_ref[q] + kMGap));
        }
        if (fast) { ok = probabilities(); if (!ok) break; }
        // ---- the turn of tile g.  Eq. 3 needs the normalizer after tile g - 1: the streams of all groups as published
        // at their last turns.  One thread of the group (its head) takes the turn -- waits for the turn before, decides,
        // publishes the group's new state and hands the turn on -- so that the chain from tile to tile is a few dozen
        // instructions of one thread; the others pick the decision up behind it.
        if (!have_slot) {   // the item's state slot is that of the item two before, which has to have been written out
          if (ne >= 2) {
            ok = mbar_wait(&o_free[ip], (uint32_t)(((ne >> 1) - 1) & 1), status);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
          }
          have_slot = true;
        }
        // raises the references to this tile's maxima: l follows here, this group's O^T (whose earlier PVs have to be
        // complete) in TMEM; then the probabilities against the new references
        auto slow_probabilities = [&]() -> bool {
          float alpha[GH];
          bool touch = false;
#pragma unroll
          for (int q = 0; q < GH; ++q) {
            alpha[q] = 1.f;
            if (q < R) {
              const float mn = fmaxf(m_ref[q], tmax[q]), yn = fmaxf(yref[q], tmax[q] + lv);
              l[q] *= fast_exp2(m_ref[q] - mn);
              alpha[q] = fast_exp2(yref[q] - yn);
              touch = touch || yn > yref[q];
              m_ref[q] = mn;
              yref[q] = yn;
            }
          }
          if (touch) {
            bool k = mbar_wait(&p_free[PP * grp + ((rg - 1) % PP)], (uint32_t)(((rg - 1) / PP) & 1), status);
            k = __all_sync(0xffffffffu, k);
            if (!k) return false;
            tc_fence_after();
            uint32_t o[LDN];
            tmem_ld_cols<LDN>(tmem_addr(tb, lane_base, colO), o);
            tmem_wait_ld();
#pragma unroll
            for (int q = 0; q < GH; ++q) {
              o[q] = __float_as_uint(__uint_as_float(o[q]) * alpha[q]);
              o[4 + q] = __float_as_uint(__uint_as_float(o[4 + q]) * alpha[q]);
            }
            tmem_st_cols<LDN>(tmem_addr(tb, lane_base, colO), o);
            tmem_wait_st();
            tc_fence_before();
          }
          return probabilities();
        };
        // the group's state after this tile, for the other groups' turns and the write-out
        auto publish = [&](int r_new) {
#pragma unroll
          for (int q = 0; q < GH; ++q) { st_m[ip][grp][q] = m_ref[q]; st_l[ip][grp][q] = l[q]; st_y[ip][grp][q] = yref[q]; }
          *(volatile int*)&st_r[ip][grp] = r_new;
        };
        bool retain = true;
        if (kDense) {
          // no decision to take, hence no order between the groups: the state only serves the write-out
          if (!fast) { ok = slow_probabilities(); if (!ok) break; }
#pragma unroll
          for (int q = 0; q < GH; ++q) l[q] += psum[q];
          ++r;
          if (head) publish(r);
        } else {
          bool handed_on = false;
          if (head) {
            // everything that does not need the other groups is ready before the wait: this stream's log-sum-exp
            // before the tile (a_own) and after it, should it be retained (psum is known on the fast path)
            float a_ret[GH];
#pragma unroll
            for (int q = 0; q < GH; ++q) a_ret[q] = m_ref[q] + __log2f(l[q] + psum[q]);
            if (g > 0) ok = mbar_wait(&turn_done[(g - 1) & 3], (uint32_t)(((g - 1) >> 2) & 1), status);
            if (ok) {
              if (t > 0) {
                float lse[GH];
#pragma unroll
                for (int q = 0; q < GH; ++q) lse[q] = a_own[q];
#pragma unroll
                for (int o2 = 1; o2 < NG; ++o2) {
                  float ao[GH];
                  lds_row<GH>(st_a[ip][(grp + o2) % NG], ao);
#pragma unroll
                  for (int q = 0; q < GH; ++q) {   // log2(2^lse + 2^ao); a stream without a tile is at -inf
                    const float M = fmaxf(lse[q], ao[q]), d = fminf(lse[q], ao[q]) - M;
                    lse[q] = M + __log2f(1.f + fast_exp2(d));
                  }
                }
                retain = false;
#pragma unroll
                for (int q = 0; q < GH; ++q) retain = retain || (q < R && !(((tmax[q] - lse[q]) - theta) < 0.f));
              }
              *(volatile int*)&flag[g & 3] = retain ? 1 : 0;
              if (fast || !retain) {   // the stream's new log-sum-exp is known: the turn is handed on at once
#pragma unroll
                for (int q = 0; q < GH; ++q) st_a[ip][grp][q] = retain ? a_ret[q] : a_own[q];
                mbar_arrive(&turn_done[g & 3]);
                if (retain) {
#pragma unroll
                  for (int q = 0; q < GH; ++q) l[q] += psum[q];
                }
                publish(r + (retain ? 1 : 0));
                mbar_arrive(&vote_bar[g & 3]);
                handed_on = true;
              }
              mbar_arrive(&dec_bar[grp]);
            }
          }
          ok = __all_sync(0xffffffffu, ok);
          if (ok && !head) ok = mbar_wait(&dec_bar[grp], (uint32_t)(nt_own & 1), status);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          retain = *(volatile int*)&flag[g & 3] != 0;
          if (retain && !fast) {   // (every thread of the group; the head keeps the turn until the state is known)
            ok = slow_probabilities();
            if (!ok) break;
          }
          if (retain) {
            if (!(head && handed_on)) {
#pragma unroll
              for (int q = 0; q < GH; ++q) l[q] += psum[q];
            }
            ++r;
          }
          // this stream's log-sum-exp after the tile (all threads keep it; the head's copy is the one that is used)
          if (retain) {
#pragma unroll
            for (int q = 0; q < GH; ++q) a_own[q] = m_ref[q] + __log2f(l[q]);
          }
          if (head && !handed_on) {
#pragma unroll
            for (int q = 0; q < GH; ++q) st_a[ip][grp][q] = a_own[q];
            mbar_arrive(&turn_done[g & 3]);
            publish(r);
            mbar_arrive(&vote_bar[g & 3]);
          }
        }
        ++nt_own;
        if (head && retain && bm_row) atomicOr(bm_row + ((T - 1 - t) >> 5), 1u << ((T - 1 - t) & 31));
        // (the state was published before the tile's P8^T is handed on: the PV, the item's completion and its write-out
        // follow from the arrivals below)
        __syncwarp();
        if (retain) {
          ++rg;
          if (lane == 0) mbar_arrive(&p_full[ps]);
        }
      }
      if (!ok) break;
      ++ne;
      g0 += T;
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tb, Cfg::kTmemCols);
}

}  // namespace mala
