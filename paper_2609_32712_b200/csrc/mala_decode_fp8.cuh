// Split-KV decode over an 8-bit (e4m3) KV cache ("Fused decoding execution"; the cache itself is untouched, only its
// storage type differs).  The decode step is bound by the bytes of K and V it streams, so an 8-bit cache halves its
// time.  Keys and values are stored as e4m3 with one fp32 scale per (sequence, KV head, 128-key tile):
//     k = kscale[b, h_kv, tile] * e4m3(k8),   v = vscale[b, h_kv, tile] * e4m3(v8)
// (paged caches: per tile of a page, or per page where a page is smaller than a tile) and the kernel computes the
// operator of mala_decode on those dequantised values.
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
//                   (e4m3's subnormal floor).  The two rows are columns h and HALF + h of the MMA, HALF = 4 with up to
//                   four heads per KV head and 8 with five to eight (hence at most eight heads), products of e4m3
//                   values are exact in the fp32 accumulator, and a softmax thread forms
//                   (S[h] + S[HALF + h] / 16) * scale * kscale / 2^k.
//   O^T += V8^T P8^T  V8 is read MN-major.  A probability enters as P' = 64 exp2(y - yref) with y = x + log2(vscale)
//                   the score of the key weighted by its V tile's scale and yref a running reference of the item
//                   (so the tile's scale rides on P', inside e4m3's narrow range whatever its magnitude), split as
//                   p1 = e4m3(P'), p2 = e4m3(16 (P' - p1)): relative error 2^-9 for P' >= 2^-6, absolute 2^-14 below
//                   (2^-20 of the largest probability).  yref is raised, and O^T rescaled, whenever a tile's largest
//                   P' would pass e4m3's 448, i.e. when y exceeds yref by more than log2(448 / 64).  The normalizer
//                   is summed in fp32 from the unrounded exp2(x - m), with its own reference m.
//
// At one byte per element a tile arrives twice as fast as in the bf16 kernels, faster than one softmax group can
// take tiles one after the other: its per-tile chain (TMEM load, a cross-warp maximum, the Eq. 3 test, exponentials,
// the P^T store, a cross-warp sum) is latency, not throughput, and Eq. 3 makes it sequential within a work item.  So
// a CTA runs NG independent pipelines ("streams") side by side, each the whole of what the bf16 kernel's CTA is: its
// own rings of raw K and V tiles, S^T ring, P^T slots, accumulators, its own issuing warps and its own softmax group
// walking one work item at a time, tile by tile, with the item's state in registers.  The CTA's work items go to
// the streams in turn.  Nothing is shared between the streams but the SM, so none ever waits for another.  An item's
// partial output is written by an epilogue group once its last PV has completed, so that no softmax group stalls at
// an item boundary.
//
// Every warp that issues asynchronous work has one job, walks its stream's tiles in order and blocks on exactly what
// its next instruction needs (a warp that polls the barriers of several jobs in one loop, sleeping in between,
// reacts to each event a loop iteration late, which at this rate is slower than the tiles arrive).  Per stream k:
//   warp k            TMA producer (Q, raw K ring; dense kernel: raw V ring)
//   warp NG + k       converts an item's queries, issues S^T of every tile
//   warp 2NG + k      MALA kernel: takes the votes in order, requests the raw V copy of a retained tile
//   warp 3NG + k      issues O^T += V8^T P8^T of every retained tile
//   warps 4NG + 4k .. softmax group (thread = key of the tile), up to four packed query heads; with five to eight heads
//                     the group is eight warps, warps 4NG + 8k .., two threads per key with four heads each
// and for all streams
//   last four warps   epilogue group (thread = output channel)
#pragma once
#include <cuda_fp16.h>

#include "mala_decode_split.cuh"
#include "sm100_ptx.cuh"

namespace mala {

// Division of a 32-bit number by a divisor known at launch, as a multiplication and shifts (every role works out for
// itself which sequence, KV head and split a work item is; hardware has no integer divide, and the few dozen
// dependent instructions of an emulated one would sit on the per-tile chain of the softmax threads).
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
  // paged cache (block_table != null): K / V are [num_pages, page_size, Hkv, d], the scales [num_pages, Hkv, tpp];
  // Nk = max_pages * page_size lays out the splits, a sequence holds seqlens[b] keys (null: Nk)
  const int32_t* block_table;    // [B, max_pages]
  const int32_t* seqlens;        // [B] or null
  int num_pages, max_pages, tpp; // tpp = tiles (128 keys) per page
  FastDiv by_tpp;
  // pages smaller than a tile (16, 32 or 64 keys; kSmall kernels): a tile is put together from ppt = 128 / page_size
  // copies of prows = page_size rows, copy c of key block x from page block_table[b][x * ppt + c]; the scales are
  // [num_pages, Hkv], one per (page, KV head)
  int ppt, prows;
  // several new tokens per sequence (kMulti kernels): q, o are [B, Sq, Hq, d], the partials [B, Sq, Hq, splits, ..];
  // row t * G + g of a work item is token t (0 = oldest, at position nk - Sq + t), head g of the group
  int Sq;
};

// NG_: streams (two: a third, with the registers moved from the issuing warps to the softmax groups and rings of two
// stages, gained the MALA kernel 4% and the dense kernel nothing).  kDense_: the dense kernel requests V with K and splits a stream's six stages evenly; the MALA kernel
// requests V only after a tile's vote, a memory latency before its PV, and gives the V ring the larger share.
// kSplit_: five to eight query heads per KV head.  A stream's softmax group is then eight warps, two threads per key:
// warps 0-3 carry the heads 0-3 through the chain and warps 4-7 the heads 4-7 (both read the same TMEM lanes, their
// own columns), so that a thread's chain is as long as with four heads; the two halves only meet in the tile's vote.
template <int NG_, bool kDense_, bool kSplit_ = false>
struct DecF8Cfg {
  static constexpr int kRawBytes = 128 * 128;            // one e4m3 tile
  static constexpr int kGroups = NG_;
  static constexpr int kKStages = kDense_ ? 3 : 2;       // raw K ring of a stream
  static constexpr int kVStages = kDense_ ? 3 : 4;       // raw V ring
  static constexpr int kQBytes = 2048;                   // landing buffer of an item's queries as copied: up to 8 rows x 128 bf16
  static constexpr int kQ8Bytes = 2048;                  // 16 rows x 128 e4m3, one per item parity
  static constexpr int kP8Bytes = 2048;                  // 16 rows x 128 e4m3
  static constexpr int kPPerGroup = 4;                   // P8^T slots of a stream: how far its softmax group may run ahead of its PVs
  static constexpr int kStreamBytes = (kKStages + kVStages) * kRawBytes + kQBytes + 2 * kQ8Bytes + kPPerGroup * kP8Bytes;
  static constexpr int kSmemBytes = kGroups * kStreamBytes + 1024;
  static constexpr int kHalves = kSplit_ ? 2 : 1;        // warpgroups of a stream's softmax group
  static constexpr int kThreads = 32 * (4 * kGroups) + 128 * kGroups * kHalves + 128;   // issuing warps, softmax groups, epilogue group
  static constexpr uint32_t kColsPerStream = 96;         // S^T ring 4 x 16, O^T 2 x 16 (item parity)
  static constexpr uint32_t kTmemCols = kGroups * kColsPerStream <= 128 ? 128 : 256;
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

// The CTA's tile sequence.  Its non-empty work items (blockIdx.x, + gridDim.x, ..) are handed to the NG streams in
// order, each stream taking the next one when it has finished its own; the tiles of the streams' current items are
// interleaved round-robin.  pos counts the tiles of the sequence (ring slots are pos % depth).  The state is a few
// integers and depends on tile counts only, so every role keeps its own copy in step.
// kPaged: the cache lies in pages (block table, one length per sequence).  In either layout the producer works out
// where a tile lies (a page lookup if paged) and publishes its TMA coordinates and the index of its scales in a small
// ring; the vote warp takes the V copy's coordinates from there, and the S warp loads the tile's two scales and hands
// them to the softmax group with the scores, so that the softmax chain carries no address arithmetic and no loads
// (with the softmax group requesting the next tile's scales itself, a tile ahead, the contiguous step was 6 % slower).
// kSmall (with kPaged): pages smaller than a tile.  The producer and the vote warp issue a tile's copies from as many
// lanes as it has pages, a key's scales are those of its page (a softmax thread is a key, so it reads its own), and
// the reference of the 8-bit probabilities is kept against the largest V scale of the tile.
// kMulti: Sq > 1 new tokens per sequence, rows = Sq * G <= 8.  A row then sees the keys up to its own position,
// has its own L (Section 2.1) and threshold, and a row that sees no key of a tile does not constrain the tile.
template <bool kDense, int GP, bool kPaged = false, int NG_ = 2, bool kSmall = false, bool kMulti = false>
__global__ void __launch_bounds__(DecF8Cfg<NG_, kDense, (GP > 4)>::kThreads, 1)
mala_decode_fp8_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                       const __grid_constant__ CUtensorMap tmV, const DecF8Params p) {
  using Cfg = DecF8Cfg<NG_, kDense, (GP > 4)>;
  constexpr int RB = Cfg::kRawBytes, NK = Cfg::kKStages, NV = Cfg::kVStages, NG = Cfg::kGroups, PP = Cfg::kPPerGroup;
  constexpr bool kSplit = GP > 4;          // two threads per key, four heads each
  constexpr int HS = Cfg::kHalves;
  constexpr int GS = kSplit ? 4 : GP;      // heads a softmax thread carries
  // The dense kernel with two threads per key sums a tile's probabilities per thread and crosses the group once per
  // item (no test needs the normalizer earlier): 5 % off its per-tile chain, which bounds it.  (With one thread per key
  // the dense kernel is bound by HBM, and the same change made it 3 % slower: 378 against 365 us at cfg5.)
  constexpr bool kLocalSums = kDense && kSplit;
  static_assert(!kDense || NK == NV, "the dense producer walks both rings with one index");
  constexpr int GH = GP;                   // rows of a softmax group
  constexpr int HALF = GP > 4 ? 8 : 4;     // rows (MMA columns) of the leading parts; the remainders follow them
  constexpr int LDN = 2 * HALF;            // S^T / O^T columns a thread reads
  constexpr float kPScale = 64.f;          // P' of the key that sets the reference
  constexpr float kPGap = 2.8f;            // log2(448 / 64), rounded down: how far y may pass yref
  constexpr float kMGap = 60.f;            // ... and x the normalizer's reference (fp32)
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);

  // per stream
  __shared__ uint64_t qr_full[NG], qr_free[NG], q8_free[NG][2], kr_full[NG][NK], kr_empty[NG][NK], v_full[NG][NV],
      v_empty[NG][NV], s_full[NG][4], s_free[NG][4], vote_bar[NG][4], vote_read[NG][4], p_full[NG][PP], p_free[NG][PP],
      item_done[NG][2], st_full[NG][2], o_free[NG][2], grp_bar[NG][2], ret_full[NG][8], ret_free[NG][8], fin_bar[NG];
  __shared__ uint32_t tmem_base_s;
  __shared__ int flag[NG][2][8];           // [stream][half of the softmax group][tile g & 7]: that half's vote
  __shared__ int ret_ring[NG][8];          // decision of the stream's tile g at g & 7 (vote warp -> PV warp)
  static_assert(!kSmall || kPaged, "small pages are pages");
  __shared__ int t_row[NG][8], t_outer[NG][8], t_sidx[NG][8];   // TMA coordinates and scale index of tile g (producer ->)
  __shared__ int t_page[NG][8][8];                              // small pages: the up to eight pages of tile g
  // the scales of the tile in S^T slot g & 3 (S warp -> softmax); small pages: one per page, and the largest V scale
  __shared__ float sc_k[NG][4][8], sc_v[NG][4][8], sc_vmax[NG][4];
  __shared__ float q_inv[NG][2][8];        // 2^-k of the query rows of a stream's item
  __shared__ __align__(16) float xch[NG][2][2][4][16];     // [stream][half][buffer][warp][row maxima 0..7, row sums 8..15]
  __shared__ __align__(16) float st_m[NG][2][8], st_l[NG][2][8], st_y[NG][2][8];   // a finished item's (m, l, yref)
  __shared__ int st_r[NG][2];                              // ... and its retained tiles
  __shared__ int early_exit;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int G = p.Hq / p.Hkv;
  const int R = kMulti ? G * p.Sq : G;     // rows of a work item
  int* status = p.status;

  // the stream's part of shared memory
  auto stream_base = [&](int k) -> uint8_t* { return smem + k * Cfg::kStreamBytes; };
  // [NK] raw K | [NV] raw V | [2] Q8 (item parity) | [PP] P8^T | [2] Q landing buffers
  auto sKr_of = [&](int k) -> uint8_t* { return stream_base(k); };
  auto sVr_of = [&](int k) -> uint8_t* { return stream_base(k) + NK * RB; };
  auto sQ8_of = [&](int k) -> uint8_t* { return stream_base(k) + (NK + NV) * RB; };
  auto sP_of = [&](int k) -> uint8_t* { return stream_base(k) + (NK + NV) * RB + 2 * Cfg::kQ8Bytes; };
  auto sQ_of = [&](int k) -> uint8_t* { return stream_base(k) + (NK + NV) * RB + 2 * Cfg::kQ8Bytes + PP * Cfg::kP8Bytes; };

  for (int k = 0; k < NG; ++k)   // Q8 and P8^T rows that are never written stay zero
    for (int i = tid; i < (2 * Cfg::kQ8Bytes + PP * Cfg::kP8Bytes) / 16; i += Cfg::kThreads)
      reinterpret_cast<uint4*>(sQ8_of(k))[i] = make_uint4(0u, 0u, 0u, 0u);
  fence_proxy_async_smem();
  if (tid == 0) {
    early_exit = (*(volatile int*)status != 0);
    for (int k = 0; k < NG; ++k) {
      mbar_init(&grp_bar[k][0], 4); mbar_init(&grp_bar[k][1], 4);
      mbar_init(&fin_bar[k], 1); mbar_init(&qr_full[k], 1); mbar_init(&qr_free[k], 1);
      for (int i = 0; i < 2; ++i) {
        mbar_init(&q8_free[k][i], 1);
        mbar_init(&item_done[k][i], 1); mbar_init(&st_full[k][i], HS); mbar_init(&o_free[k][i], 4);
      }
      for (int s = 0; s < PP; ++s) { mbar_init(&p_full[k][s], 4 * HS); mbar_init(&p_free[k][s], 1); }
      for (int s = 0; s < NK; ++s) { mbar_init(&kr_full[k][s], 1); mbar_init(&kr_empty[k][s], 1); }
      for (int s = 0; s < NV; ++s) { mbar_init(&v_full[k][s], 1); mbar_init(&v_empty[k][s], 1); }
      for (int s = 0; s < 4; ++s) {
        mbar_init(&s_full[k][s], 1); mbar_init(&s_free[k][s], 4 * HS); mbar_init(&vote_bar[k][s], HS); mbar_init(&vote_read[k][s], 1);
      }
      for (int s = 0; s < 8; ++s) {
        mbar_init(&ret_full[k][s], 1); mbar_init(&ret_free[k][s], 1);
        flag[k][0][s] = flag[k][1][s] = 0;
      }
    }
    mbar_fence_init();
  }
  __syncthreads();
  if (early_exit) return;
  if (warp == 0) { tmem_alloc(&tmem_base_s, Cfg::kTmemCols); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tb = tmem_base_s;

  // Tiles, sequence, KV head, split and newest tile of a work item.  The KV head is the fastest index of an item's
  // number: the CTAs that run side by side then read the same keys of a key-major cache, each its own head's 128
  // bytes of every key's row, and the row is fetched from memory once, not once per head.
  auto keys_of = [&](int b) -> int {   // keys the sequence holds
    return (kPaged && p.seqlens) ? min(p.Nk, max(0, __ldg(p.seqlens + b))) : p.Nk;
  };
  auto tiles_of = [&](int item) -> int {
    const int bs = (int)p.by_hkv.div((uint32_t)item);
    const int b = (int)p.by_splits.div((uint32_t)bs);
    const int split = bs - b * p.num_splits;
    const int lo = split * p.tps * 128;
    const int hi = min(keys_of(b), lo + p.tps * 128);
    return hi > lo ? (hi - lo + 127) >> 7 : 0;
  };
  // where key block jt of sequence b lies: TMA row and outer coordinate, index of its scales (-1: no such page)
  auto tile_coord = [&](int b, int hkv, int jt, int& row, int& outer, int& sidx) {
    if (kPaged) {
      const int x = (int)p.by_tpp.div((uint32_t)jt);
      const int pg = __ldg(p.block_table + (size_t)b * p.max_pages + x);
      const int in_page = jt - x * p.tpp;
      row = in_page * 128;
      outer = pg;
      sidx = (pg >= 0 && pg < p.num_pages) ? (pg * p.Hkv + hkv) * p.tpp + in_page : -1;
    } else {
      row = jt * 128;
      outer = b;
      sidx = (b * p.Hkv + hkv) * p.nt + jt;
    }
  };
  auto geometry = [&](int item, int& b, int& hkv, int& split, int& j0, int T) {
    const int bs = (int)p.by_hkv.div((uint32_t)item);
    hkv = item - bs * p.Hkv;
    b = (int)p.by_splits.div((uint32_t)bs);
    split = bs - b * p.num_splits;
    j0 = split * p.tps + T - 1;
  };
  // the CTA's work items are blockIdx.x, + gridDim.x, ..; stream k takes the k-th, (k + NG)-th, .. of them
  const int item_step = NG * (int)gridDim.x;

  if (warp < 4 * NG) {
    // ------------------------------------------------------------------ the issuing warps of stream k
    const int job = warp / NG, k = warp - job * NG;
    const int item0 = (int)blockIdx.x + k * (int)gridDim.x;
    uint8_t* sKr = sKr_of(k);
    uint8_t* sVr = sVr_of(k);
    uint8_t* sQ8 = sQ8_of(k);
    uint8_t* sP = sP_of(k);
    uint8_t* sQ = sQ_of(k);
    const uint32_t tS = tmem_addr(tb, 0, (uint32_t)k * Cfg::kColsPerStream);          // S^T ring of the stream
    const uint32_t tO = tmem_addr(tb, 0, (uint32_t)k * Cfg::kColsPerStream + 64u);    // its two accumulators
    const uint32_t leader = elect_one();
    bool ok = true;
    if (job == 0 && kSmall) {
      // ---- TMA producer, pages smaller than a tile: the loop below run by all 32 lanes (waits and counters
      //      warp-uniform); lane c looks up the page of copy c and issues that copy
      if (lane == 0) { tma_prefetch_desc(&tmQ); tma_prefetch_desc(&tmK); tma_prefetch_desc(&tmV); }
      int ne = 0, g = 0;
      for (int item = item0; item < p.n_items && ok; item += item_step) {
        const int T = tiles_of(item);
        if (T == 0) continue;
        int b, hkv, split, j0;
        geometry(item, b, hkv, split, j0, T);
        if (ne >= 1) ok = mbar_wait_warp(&qr_free[k], (uint32_t)((ne - 1) & 1), status);
        if (!ok) break;
        if (lane == 0) {
          mbar_arrive_expect_tx(&qr_full[k], (uint32_t)R * 128u * 2u);
          for (int pn = 0; pn < 2; ++pn)
            tma_load_4d(sQ + pn * HALF * 128, &tmQ, &qr_full[k], pn * 64, hkv * G, 0, b);
        }
        for (int t = 0; t < T && ok; ++t, ++g) {
          const int s = g % NK;
          const uint32_t ph = (uint32_t)((g / NK) & 1);
          const int x = (j0 - t) * p.ppt + lane;   // (a table entry past the row's end reads as "no page": zeros)
          const int pg = (lane < p.ppt && x < p.max_pages) ? __ldg(p.block_table + (size_t)b * p.max_pages + x) : -1;
          ok = mbar_wait_warp(&kr_empty[k][s], ph ^ 1u, status);
          if (!ok) break;
          if (lane < 8) t_page[k][g & 7][lane] = pg;
          __syncwarp();
          if (lane == 0) mbar_arrive_expect_tx(&kr_full[k][s], RB);
          __syncwarp();
          if (lane < p.ppt) tma_load_4d(sKr + s * RB + lane * p.prows * 128, &tmK, &kr_full[k][s], 0, 0, hkv, pg);
          if (kDense) {
            ok = mbar_wait_warp(&v_empty[k][s], ph ^ 1u, status);
            if (!ok) break;
            if (lane == 0) mbar_arrive_expect_tx(&v_full[k][s], RB);
            __syncwarp();
            if (lane < p.ppt) tma_load_4d(sVr + s * RB + lane * p.prows * 128, &tmV, &v_full[k][s], 0, 0, hkv, pg);
          }
        }
        ++ne;
      }
    } else if (job == 0) {
      // ---- TMA producer
      if (lane == 0) {
        tma_prefetch_desc(&tmQ); tma_prefetch_desc(&tmK); tma_prefetch_desc(&tmV);
        int ne = 0, g = 0;
        for (int item = item0; item < p.n_items && ok; item += item_step) {
          const int T = tiles_of(item);
          if (T == 0) continue;
          int b, hkv, split, j0;
          geometry(item, b, hkv, split, j0, T);
          // (one landing buffer: the S warp converts an item's queries at once, long before the next item starts)
          if (ne >= 1) ok = mbar_wait(&qr_free[k], (uint32_t)((ne - 1) & 1), status);
          if (!ok) break;
          mbar_arrive_expect_tx(&qr_full[k], (uint32_t)R * 128u * 2u);   // two panels of R rows x 128 bytes
          for (int pn = 0; pn < 2; ++pn)
            tma_load_4d(sQ + pn * HALF * 128, &tmQ, &qr_full[k], pn * 64, hkv * G, 0, b);
          for (int t = 0; t < T && ok; ++t, ++g) {
            const int s = g % NK;
            const uint32_t ph = (uint32_t)((g / NK) & 1);
            int row, outer, sidx;
            tile_coord(b, hkv, j0 - t, row, outer, sidx);   // (a page lookup is in flight while the slot is waited for)
            ok = mbar_wait(&kr_empty[k][s], ph ^ 1u, status);
            if (!ok) break;
            // The S warp and the vote warp take the tile's coordinates from here; they are at most seven tiles behind
            // (K ring, S^T ring, votes outstanding) and see the stores through the K tile's barrier.
            t_row[k][g & 7] = row; t_outer[k][g & 7] = outer; t_sidx[k][g & 7] = sidx;
            mbar_arrive_expect_tx(&kr_full[k][s], RB);
            tma_load_4d(sKr + s * RB, &tmK, &kr_full[k][s], 0, row, hkv, outer);
            if (kDense) {   // every tile is retained: V follows K
              ok = mbar_wait(&v_empty[k][s], ph ^ 1u, status);
              if (!ok) break;
              mbar_arrive_expect_tx(&v_full[k][s], RB);
              tma_load_4d(sVr + s * RB, &tmV, &v_full[k][s], 0, row, hkv, outer);
            }
          }
          ++ne;
        }
      }
    } else if (job == 1) {
      // ---- Q of an item -> two e4m3 rows per head; S^T = K8 Q8^T of every tile
      constexpr uint32_t idesc_qk = make_idesc_e4m3(128, 16, false, false);
      const uint64_t dQ0 = make_smem_desc(smem_u32(sQ8), 16, 1024);
      const uint64_t dK0 = make_smem_desc(smem_u32(sKr), 16, 1024);
      int ne = 0, g = 0;
      for (int item = item0; item < p.n_items && ok; item += item_step) {
        const int T = tiles_of(item);
        if (T == 0) continue;
        const int ip = ne & 1;
        int b_ = 0, hkv_ = 0, split_, j0_ = 0, nk_ = 0;
        if constexpr (kSmall) { geometry(item, b_, hkv_, split_, j0_, T); nk_ = keys_of(b_); }
        uint8_t* q8 = sQ8 + ip * Cfg::kQ8Bytes;
        // the item's queries have landed: row qh (128 bf16 in two 64-column panels, rows qh and HALF + qh of the
        // landing buffer; lane = four consecutive columns) becomes rows qh and HALF + qh of the e4m3 operand, once the
        // MMAs of the item that had the operand's slot before have read it
        ok = mbar_wait_warp(&qr_full[k], (uint32_t)(ne & 1), status);
        if (ok && ne >= 2) ok = mbar_wait_warp(&q8_free[k][ip], (uint32_t)(((ne >> 1) - 1) & 1), status);
        if (!ok) break;
        for (int qh = 0; qh < R; ++qh) {
          const int e0 = lane * 4;
          const int prow = qh + HALF * (e0 >> 6);     // row of the landing buffer: head qh of panel e0 / 64
          const uint8_t* src = sQ + prow * 128 + (((((e0 & 63) >> 3)) ^ (prow & 7)) << 4) + (e0 & 7) * 2;
          const uint2 w2 = *reinterpret_cast<const uint2*>(src);
          float a[4] = {__uint_as_float(w2.x << 16), __uint_as_float(w2.x & 0xffff0000u), __uint_as_float(w2.y << 16),
                        __uint_as_float(w2.y & 0xffff0000u)};
          float mx = fmaxf(fmaxf(fabsf(a[0]), fabsf(a[1])), fmaxf(fabsf(a[2]), fabsf(a[3])));
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
          // 2^k brings the row's largest magnitude into [128, 256)  (k = 0 for a zero row; kept inside fp32's exponents)
          const int ef = (int)((__float_as_uint(mx) >> 23) & 0xffu);
          const int kk = ef == 0 ? 0 : min(max(134 - ef, -100), 100);
          const float up = __uint_as_float((uint32_t)(kk + 127) << 23), down = __uint_as_float((uint32_t)(127 - kk) << 23);
          const uint2 s01 = split_e4m3x2(a[0] * up, a[1] * up), s23 = split_e4m3x2(a[2] * up, a[3] * up);
          const int r2 = HALF + qh;
          *reinterpret_cast<uint32_t*>(q8 + qh * 128 + (((e0 >> 4) ^ (qh & 7)) << 4) + (e0 & 15)) = s01.x | (s23.x << 16);
          *reinterpret_cast<uint32_t*>(q8 + r2 * 128 + (((e0 >> 4) ^ (r2 & 7)) << 4) + (e0 & 15)) = s01.y | (s23.y << 16);
          if (lane == 0) q_inv[k][ip][qh] = down;
        }
        fence_proxy_async_smem();
        __syncwarp();
        if (leader) mbar_arrive(&qr_free[k]);
        const uint64_t dQ = desc_advance(dQ0, ip * Cfg::kQ8Bytes);
        for (int t = 0; t < T && ok; ++t, ++g) {
          const int sb = g & 3, kc = g % NK;
          if (g >= 4) {
            ok = mbar_wait_warp(&s_free[k][sb], (uint32_t)(((g >> 2) - 1) & 1), status);
            // (the vote of the tile that had this slot has been read: its flag may be overwritten)
            if (!kDense && ok) ok = mbar_wait_warp(&vote_read[k][sb], (uint32_t)(((g >> 2) - 1) & 1), status);
          }
          if (ok) ok = mbar_wait_warp(&kr_full[k][kc], (uint32_t)((g / NK) & 1), status);
          if (!ok) break;
          if constexpr (kSmall) {   // one pair of scales per page of the tile, and the largest V scale
            const int pg = lane < 8 ? *(volatile int*)&t_page[k][g & 7][lane] : -1;
            const bool there = lane < p.ppt && pg >= 0 && pg < p.num_pages;
            const float vsc = there ? __ldg(p.vscale + (size_t)pg * p.Hkv + hkv_) : 1.f;
            if (lane < 8) {
              sc_k[k][sb][lane] = there ? __ldg(p.kscale + (size_t)pg * p.Hkv + hkv_) : 1.f;
              sc_v[k][sb][lane] = vsc;
            }
            // the reference of the 8-bit probabilities follows the largest V scale among the pages that hold a key of
            // the sequence: a page that is not there (scale 1) or lies wholly past the sequence's end (any scale) would
            // push every real key's probability toward e4m3's subnormals
            const bool counts = there && ((j0_ - t) * 128 + lane * p.prows) < nk_;
            float vmx = counts ? vsc : 0.f;
#pragma unroll
            for (int o = 4; o > 0; o >>= 1) vmx = fmaxf(vmx, __shfl_xor_sync(0xffffffffu, vmx, o));
            if (lane == 0) sc_vmax[k][sb] = vmx > 0.f ? vmx : 1.f;
            __threadfence_block();
          } else if (leader) {   // the tile's scales travel with its scores (a page without scales holds zeros: any scale does)
            const int sidx = *(volatile int*)&t_sidx[k][g & 7];
            sc_k[k][sb][0] = sidx >= 0 ? __ldg(p.kscale + sidx) : 1.f;
            sc_v[k][sb][0] = sidx >= 0 ? __ldg(p.vscale + sidx) : 1.f;
            __threadfence_block();
          }
          __syncwarp();
          tc_fence_after();
          const uint32_t dS = tS + (uint32_t)sb * 16u;
          const uint64_t dK = desc_advance(dK0, kc * RB);
#pragma unroll
          for (int kq = 0; kq < 4; ++kq)     // 32 e4m3 elements of the head size per instruction
            mma_ss_f8(dS, desc_advance(dK, kq * 32), desc_advance(dQ, kq * 32), idesc_qk, kq > 0, leader);
          if (leader) {
            tc_commit(&kr_empty[k][kc]);
            tc_commit(&s_full[k][sb]);
            if (t == T - 1) tc_commit(&q8_free[k][ip]);
          }
          __syncwarp();
        }
        ++ne;
      }
    } else if (job == 2) {
      // ---- the votes (MALA kernel): a retained tile's raw V copy is requested, the decision is passed on
      if (!kDense) {
        int g = 0, nv = 0;                       // tiles so far; raw V copies requested -- ring slot nv % NV
        for (int item = item0; item < p.n_items && ok; item += item_step) {
          const int T = tiles_of(item);
          if (T == 0) continue;
          int b, hkv, split, j0;
          geometry(item, b, hkv, split, j0, T);
          for (int t = 0; t < T && ok; ++t, ++g) {
            ok = mbar_wait_warp(&vote_bar[k][g & 3], (uint32_t)((g >> 2) & 1), status);
            if (ok && g >= 8) ok = mbar_wait_warp(&ret_free[k][g & 7], (uint32_t)(((g >> 3) - 1) & 1), status);
            if (!ok) break;
            const bool retain = __shfl_sync(0xffffffffu, *(volatile int*)&flag[k][0][g & 7] |
                                                                  (kSplit ? *(volatile int*)&flag[k][1][g & 7] : 0), 0) != 0;
            __syncwarp();
            if (leader) mbar_arrive(&vote_read[k][g & 3]);
            if (retain) {
              const int vs = nv % NV;
              if (nv >= NV) ok = mbar_wait_warp(&v_empty[k][vs], (uint32_t)(((nv / NV) - 1) & 1), status);
              if (!ok) break;
              if constexpr (kSmall) {
                if (lane == 0) mbar_arrive_expect_tx(&v_full[k][vs], RB);
                __syncwarp();
                if (lane < p.ppt)
                  tma_load_4d(sVr + vs * RB + lane * p.prows * 128, &tmV, &v_full[k][vs], 0, 0, hkv,
                              *(volatile int*)&t_page[k][g & 7][lane]);
              } else if (leader) {
                mbar_arrive_expect_tx(&v_full[k][vs], RB);
                tma_load_4d(sVr + vs * RB, &tmV, &v_full[k][vs], 0, *(volatile int*)&t_row[k][g & 7], hkv,
                            *(volatile int*)&t_outer[k][g & 7]);
              }
              ++nv;
            }
            if (leader) {
              *(volatile int*)&ret_ring[k][g & 7] = retain ? 1 : 0;
              mbar_arrive(&ret_full[k][g & 7]);
            }
            __syncwarp();
          }
        }
      }
    } else {
      // ---- O^T += V8^T P8^T of every retained tile, into the accumulator of the item
      constexpr uint32_t idesc_pv = make_idesc_e4m3(128, 16, true, true);
      const uint64_t dV0 = make_smem_desc(smem_u32(sVr), 16384, 1024);   // V tile read MN-major (M = channel)
      // P8^T read MN-major too, without swizzle: 16 bytes (the 16 columns) per key, core matrices of 8 keys 128 bytes apart
      const uint64_t dP0 = make_smem_desc(smem_u32(sP), 128, 128) & ~((uint64_t)7 << 61);
      int ne = 0, g = 0, npv = 0;                // items, tiles, PVs so far: raw V stage npv % NV, P8^T slot npv % PP
      for (int item = item0; item < p.n_items && ok; item += item_step) {
        const int T = tiles_of(item);
        if (T == 0) continue;
        const int ip = ne & 1;
        int r_item = 0;
        for (int t = 0; t < T && ok; ++t, ++g) {
          bool retain = true;
          if (!kDense) {
            ok = mbar_wait_warp(&ret_full[k][g & 7], (uint32_t)((g >> 3) & 1), status);
            if (!ok) break;
            retain = __shfl_sync(0xffffffffu, *(volatile int*)&ret_ring[k][g & 7], 0) != 0;
            __syncwarp();
            if (leader) mbar_arrive(&ret_free[k][g & 7]);
          }
          if (retain) {
            const int ps = npv % PP, vc = npv % NV;
            ok = mbar_wait_warp(&p_full[k][ps], (uint32_t)((npv / PP) & 1), status);
            if (ok) ok = mbar_wait_warp(&v_full[k][vc], (uint32_t)((npv / NV) & 1), status);
            // (the accumulator is that of the item two before, which has to have been written out)
            if (ok && r_item == 0 && ne >= 2) ok = mbar_wait_warp(&o_free[k][ip], (uint32_t)(((ne >> 1) - 1) & 1), status);
            if (!ok) break;
            tc_fence_after();
            const uint32_t dO = tO + (uint32_t)ip * 16u;
            const uint64_t dV = desc_advance(dV0, vc * RB), dP = desc_advance(dP0, ps * Cfg::kP8Bytes);
            const uint32_t acc0 = r_item > 0 ? 1u : 0u;
#pragma unroll
            for (int kq = 0; kq < 4; ++kq)     // 32 keys per instruction: 32 rows of the V tile, 32 bytes of a P8^T row
              mma_ss_f8(dO, desc_advance(dV, kq * 4096), desc_advance(dP, kq * 512), idesc_pv, kq > 0 ? 1u : acc0, leader);
            if (leader) { tc_commit(&v_empty[k][vc]); tc_commit(&p_free[k][ps]); }
            ++npv;
            ++r_item;
          }
          if (t == T - 1 && leader) tc_commit(&item_done[k][ip]);
          __syncwarp();
        }
        ++ne;
      }
      if (leader) tc_commit(&fin_bar[k]);
      __syncwarp();
      mbar_wait_warp(&fin_bar[k], 0, status);
    }
    if (!ok) { const long long t0 = clock64(); while (clock64() - t0 < 400000) {} }
  } else if (warp >= 4 * NG + 4 * NG * HS) {
    // ------------------------------------------------------------------ epilogue group: thread = output channel
    // An item is written out when its last PV has completed and its stream has left its state: the partial output,
    // normalised by the split's own normalizer, and the log-sum-exp are stored and the item's accumulator and state
    // slot handed back.  The CTA's items are taken in their order, i.e. the streams in turn.
    const int w = warp & 3;
    const uint32_t lane_base = (uint32_t)w * 32u;
    const int kt = (int)lane_base + lane;
    const bool head = (kt == 0);
    int ne_k[NG];
#pragma unroll
    for (int i = 0; i < NG; ++i) ne_k[i] = 0;
    bool ok = true;
    int k = 0;
    for (int item = (int)blockIdx.x; item < p.n_items && ok; item += (int)gridDim.x, k = (k + 1 == NG) ? 0 : k + 1) {
      const int T = tiles_of(item);
      int b, hkv, split, j0;
      geometry(item, b, hkv, split, j0, T);
      // row q of the item: token q / G, head q % G of the group; its partials lie rowoff(q) rows after the item's first
      const size_t prow0 = ((size_t)b * (kMulti ? p.Sq : 1) * p.Hq + hkv * G) * p.num_splits + split;
      auto rowoff = [&](int q) -> size_t {
        if constexpr (kMulti) { const int tok = q / G; return ((size_t)tok * p.Hq + (size_t)(q - tok * G)) * p.num_splits; }
        else return (size_t)q * p.num_splits;
      };
      const size_t stat_row = (size_t)(b * p.Hkv + hkv) * p.num_splits + split;
      if (T == 0) {   // a split without keys: (0, -inf)
#pragma unroll
        for (int q = 0; q < GH; ++q)
          if (q < R) {
            p.o_part[(prow0 + rowoff(q)) * 128 + kt] = 0.f;
            if (kt == q) p.lse_part[prow0 + rowoff(q)] = -INFINITY;
          }
        if (head && p.retained) p.retained[stat_row] = 0u;
        continue;
      }
      int ne = 0;
#pragma unroll
      for (int i = 0; i < NG; ++i) if (i == k) { ne = ne_k[i]; ++ne_k[i]; }
      const int ip = ne & 1;
      ok = mbar_wait(&item_done[k][ip], (uint32_t)((ne >> 1) & 1), status);
      ok = ok && mbar_wait(&st_full[k][ip], (uint32_t)((ne >> 1) & 1), status);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      float ms[GH], ls[GH], ys[GH];
      lds_row<GH>(st_m[k][ip], ms);
      lds_row<GH>(st_l[k][ip], ls);
      lds_row<GH>(st_y[k][ip], ys);
      const int r_all = *(volatile int*)&st_r[k][ip];
      uint32_t o[LDN];
      tmem_ld_cols<LDN>(tmem_addr(tb, lane_base, (uint32_t)k * Cfg::kColsPerStream + 64u + (uint32_t)ip * 16u), o);
      tmem_wait_ld();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&o_free[k][ip]);
#pragma unroll
      for (int q = 0; q < GH; ++q)
        if (q < R) {   // O^T is in units of 2^yref / 64, l in units of 2^m
          const float num = fmaf(__uint_as_float(o[HALF + q]), 0.0625f, __uint_as_float(o[q])) * fast_exp2(ys[q] - ms[q]);
          const bool seen = !kMulti || ls[q] > 0.f;   // (a row that saw no key of the split: (0, -inf))
          p.o_part[(prow0 + rowoff(q)) * 128 + kt] = seen ? num / (ls[q] * kPScale) : 0.f;
          if (kt == q) p.lse_part[prow0 + rowoff(q)] = seen ? (ms[q] + __log2f(ls[q])) * 0.6931471805599453f : -INFINITY;
        }
      if (head) {
        if (p.retained) p.retained[stat_row] = (uint32_t)r_all;
        if (p.totals) {
          atomicAdd(&p.totals[0], (unsigned long long)r_all);
          atomicAdd(&p.totals[1], (unsigned long long)T);
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ softmax group of stream k: thread = key of the tile
    const int k = (warp - 4 * NG) / (4 * HS);
    const int half = kSplit ? (((warp - 4 * NG) >> 2) & 1) : 0;   // which four of the (up to) eight heads
    const int hb = half * 4;
    const int item0 = (int)blockIdx.x + k * (int)gridDim.x;
    uint8_t* sP = sP_of(k);
    const uint32_t colS = (uint32_t)k * Cfg::kColsPerStream, colO0 = colS + 64u;
    const int w = warp & 3;
    const uint32_t lane_base = (uint32_t)w * 32u;
    const int kt = (int)lane_base + lane;
    const int pi = kSmall ? kt / p.prows : 0;  // small pages: the page of the tile this key lies in
    const float c2 = p.scale_log2;
    const bool head = (kt == 0);               // (of this half: casts its vote, leaves its state)
    constexpr int kLanesPerRow = 32 / GS;
    const int pub_row = lane / kLanesPerRow;
    const bool publisher = (lane % kLanesPerRow) == 0;
    int ne = 0, g = 0;                           // items and tiles of this stream so far
    int rg = 0;                                  // retained tiles so far: P8^T slot rg % PP
    uint32_t xc = 0;                             // exchanges so far (buffer and barrier phase xc & 1)
    bool ok = true;
    // The one exchange of a tile between the four warps: each warp's row maxima of this tile and its row sums of
    // the last retained tile (which the test of this tile needs in the normalizer).  Returns the maxima in tmax and
    // adds the sums to l.
    float psum_w = 0.f;                          // this warp's sum of row pub_row, last retained tile
    bool pending_sum = false;
    auto exchange = [&](float mx_w, float (&tmax)[GS], float (&l)[GS], float (&lgl)[GS]) -> bool {
      const int xb = xc & 1;
      if (publisher) { xch[k][half][xb][w][pub_row] = mx_w; xch[k][half][xb][w][8 + pub_row] = psum_w; }
      __syncwarp();
      if (lane == 0) mbar_arrive(&grp_bar[k][half]);
      bool kk = mbar_wait(&grp_bar[k][half], xc & 1, status);
      kk = __all_sync(0xffffffffu, kk);
      ++xc;
      if (!kk) return false;
      float a0[GS], a1[GS], a2[GS], a3[GS];
      lds_row<GS>(xch[k][half][xb][0], a0); lds_row<GS>(xch[k][half][xb][1], a1);
      lds_row<GS>(xch[k][half][xb][2], a2); lds_row<GS>(xch[k][half][xb][3], a3);
#pragma unroll
      for (int q = 0; q < GS; ++q) tmax[q] = fmaxf(fmaxf(a0[q], a1[q]), fmaxf(a2[q], a3[q]));
      if (pending_sum) {
        lds_row<GS>(xch[k][half][xb][0] + 8, a0); lds_row<GS>(xch[k][half][xb][1] + 8, a1);
        lds_row<GS>(xch[k][half][xb][2] + 8, a2); lds_row<GS>(xch[k][half][xb][3] + 8, a3);
#pragma unroll
        for (int q = 0; q < GS; ++q) {
          l[q] += (a0[q] + a1[q]) + (a2[q] + a3[q]);
          lgl[q] = __log2f(l[q]);
        }
        pending_sum = false;
      }
      return true;
    };
    for (int item = item0; item < p.n_items && ok; item += item_step) {
      const int T = tiles_of(item);
      if (T == 0) continue;
      int b, hkv, split, j0;
      geometry(item, b, hkv, split, j0, T);
      const int ip = ne & 1;
      const uint32_t colO = colO0 + (uint32_t)ip * 16u;
      uint32_t* bm_row = p.bitmask ? p.bitmask + ((size_t)(b * p.Hkv + hkv) * p.num_splits + split) * p.words : nullptr;
      const int nk = keys_of(b);                 // keys of the sequence: the L of Eq. 3 and the tail mask
      const float theta = kDense ? -INFINITY : (p.log2_tau - log2f((float)max(nk, 1)));
      // several tokens: row q sees the keys before position lim[q] = nk - (Sq - 1 - its token), which is its L
      int lim[kMulti ? GS : 1];
      float theta_q[kMulti ? GS : 1];
      if constexpr (kMulti) {
#pragma unroll
        for (int q = 0; q < GS; ++q) {
          const int tok = (hb + q < R) ? (hb + q) / G : 0;
          lim[q] = nk - (p.Sq - 1 - tok);
          theta_q[q] = kDense ? -INFINITY : (p.log2_tau - log2f((float)max(lim[q], 1)));
        }
      }
      auto lim_of = [&](int q) -> int { if constexpr (kMulti) return lim[q]; else return nk; };
      auto theta_of = [&](int q) -> float { if constexpr (kMulti) return theta_q[q]; else return theta; };
      int r = 0;                                 // tiles of the item retained so far
      float m_ref[GS], l[GS], yref[GS], lgl[GS], c2q[GS];
#pragma unroll
      for (int q = 0; q < GS; ++q) { m_ref[q] = -INFINITY; l[q] = 0.f; yref[q] = 0.f; lgl[q] = -INFINITY; c2q[q] = c2; }
      float lacc[kLocalSums ? GS : 1];           // this thread's share of the row sums
#pragma unroll
      for (int q = 0; q < (kLocalSums ? GS : 1); ++q) lacc[q] = 0.f;
      for (int t = 0; t < T; ++t, ++g) {
        const int sb = g & 3;
        ok = mbar_wait(&s_full[k][sb], (uint32_t)((g >> 2) & 1), status);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after();
        // the leading parts and the remainders of this thread's heads
        uint32_t sr[kSplit ? 4 : LDN], sr2[kSplit ? 4 : 1];
        if constexpr (kSplit) {
          tmem_ld_cols<4>(tmem_addr(tb, lane_base, colS + (uint32_t)sb * 16u + (uint32_t)hb), sr);
          tmem_ld_cols<4>(tmem_addr(tb, lane_base, colS + (uint32_t)sb * 16u + 8u + (uint32_t)hb), sr2);
        } else {
          tmem_ld_cols<LDN>(tmem_addr(tb, lane_base, colS + (uint32_t)sb * 16u), sr);
        }
        auto rem_of = [&](int q) -> float {
          if constexpr (kSplit) return __uint_as_float(sr2[q]);
          else return __uint_as_float(sr[HALF + q]);
        };
        // (small pages: the key's own page's scales; the reference of P' follows the tile's largest V scale)
        const float ks = *(volatile float*)&sc_k[k][sb][pi], lvk = __log2f(*(volatile float*)&sc_v[k][sb][pi]);
        const float lv = kSmall ? __log2f(*(volatile float*)&sc_vmax[k][sb]) : lvk;
        tmem_wait_ld();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&s_free[k][sb]);
        if (t == 0) {
#pragma unroll
          for (int q = 0; q < GS; ++q) c2q[q] = c2 * *(volatile float*)&q_inv[k][ip][hb + q];
        }
        const int kpos = (j0 - t) * 128 + kt;
        float x[GS], tmax[GS];
        {
          float mx[GS];
#pragma unroll
          for (int q = 0; q < GS; ++q) {   // the two e4m3 rows of the head, the row's 2^-k and the K tile's scale
            x[q] = (kpos < lim_of(q) && hb + q < R) ? fmaf(rem_of(q), 0.0625f, __uint_as_float(sr[q])) * (c2q[q] * ks) : -INFINITY;
            mx[q] = x[q];
          }
          RowReduce<GS, 16, true>::run(mx, lane);
          ok = exchange(mx[0], tmax, l, lgl);
          if (!ok) break;
        }
        // Eq. 3 against the split's partial normalizer: skip iff rowmax - (m + log l) < log(tau / Nk) for every head
        bool retain = true;
        if (!kDense && r > 0) {
          retain = false;
#pragma unroll
          for (int q = 0; q < GS; ++q)   // (several tokens: a row without a visible key in the tile does not constrain it)
            retain = retain || (hb + q < R && (!kMulti || tmax[q] > -INFINITY) &&
                                !(((tmax[q] - (m_ref[q] + lgl[q])) - theta_of(q)) < 0.f));
        }
        if (!kDense && head) {
          *(volatile int*)&flag[k][half][g & 7] = retain ? 1 : 0;
          mbar_arrive(&vote_bar[k][g & 3]);
        }
        if (!kDense && kSplit && !retain) {   // this half's heads would skip the tile: the other half's decide
          ok = mbar_wait(&vote_bar[k][g & 3], (uint32_t)((g >> 2) & 1), status);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          retain = (*(volatile int*)&flag[k][0][g & 7] | *(volatile int*)&flag[k][1][g & 7]) != 0;
          retain = __all_sync(0xffffffffu, retain);
        }
        if (!retain) continue;
        if (head && half == 0 && bm_row) atomicOr(bm_row + ((T - 1 - t) >> 5), 1u << ((T - 1 - t) & 31));
        const int ps = rg % PP;
        if (r == 0) {
#pragma unroll
          for (int q = 0; q < GS; ++q) {   // (nothing accumulated yet; finite also for a row that sees no key yet)
            m_ref[q] = kMulti ? fmaxf(tmax[q], -1e30f) : tmax[q];
            yref[q] = m_ref[q] + lv;
          }
        } else {
          // a maximum too far above a reference: the reference is raised, l follows here and O^T (whose earlier PVs
          // have to be complete) in TMEM
          float alpha[GS];
          bool touch = false;
#pragma unroll
          for (int q = 0; q < GS; ++q) {
            alpha[q] = 1.f;
            if (hb + q < R && (tmax[q] + lv > yref[q] + kPGap || tmax[q] > m_ref[q] + kMGap)) {
              const float mn = fmaxf(m_ref[q], tmax[q]), yn = fmaxf(yref[q], tmax[q] + lv);
              const float lf = fast_exp2(m_ref[q] - mn);
              l[q] *= lf;
              if constexpr (kLocalSums) lacc[q] *= lf;
              alpha[q] = fast_exp2(yref[q] - yn);
              touch = touch || yn > yref[q];
              m_ref[q] = mn;
              yref[q] = yn;
            }
          }
          if (touch) {
            ok = mbar_wait(&p_free[k][(rg - 1) % PP], (uint32_t)(((rg - 1) / PP) & 1), status);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            if constexpr (kSplit) {
              uint32_t o[4], o2[4];
              tmem_ld_cols<4>(tmem_addr(tb, lane_base, colO + (uint32_t)hb), o);
              tmem_ld_cols<4>(tmem_addr(tb, lane_base, colO + 8u + (uint32_t)hb), o2);
              tmem_wait_ld();
#pragma unroll
              for (int q = 0; q < 4; ++q) {
                o[q] = __float_as_uint(__uint_as_float(o[q]) * alpha[q]);
                o2[q] = __float_as_uint(__uint_as_float(o2[q]) * alpha[q]);
              }
              tmem_st_cols<4>(tmem_addr(tb, lane_base, colO + (uint32_t)hb), o);
              tmem_st_cols<4>(tmem_addr(tb, lane_base, colO + 8u + (uint32_t)hb), o2);
            } else {
              uint32_t o[LDN];
              tmem_ld_cols<LDN>(tmem_addr(tb, lane_base, colO), o);
              tmem_wait_ld();
#pragma unroll
              for (int q = 0; q < GS; ++q) {
                o[q] = __float_as_uint(__uint_as_float(o[q]) * alpha[q]);
                o[HALF + q] = __float_as_uint(__uint_as_float(o[HALF + q]) * alpha[q]);
              }
              tmem_st_cols<LDN>(tmem_addr(tb, lane_base, colO), o);
            }
            tmem_wait_st();
            tc_fence_before();
          }
        }
        if (rg >= PP) {
          ok = mbar_wait(&p_free[k][ps], (uint32_t)(((rg / PP) - 1) & 1), status);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
        }
        float e[GS], pp[GS];
#pragma unroll
        for (int q = 0; q < GS; ++q) {
          e[q] = (hb + q < R) ? fast_exp2(x[q] - m_ref[q]) : 0.f;
          // P' = 64 exp2(x + lv - yref) = e * 64 exp2(m + lv - yref): the tile's V scale rides on the probability
          pp[q] = (hb + q < R) ? e[q] * (kPScale * fast_exp2((m_ref[q] + lvk) - yref[q])) : 0.f;
        }
        {   // the key's 16 bytes: leading parts of the heads, their remainders (zeros behind them with up to four heads;
            // with more, each half of the group writes its four bytes of either)
          uint32_t lead = 0u, rem = 0u;
          if constexpr (GS == 1) {
            const uint2 s0 = split_e4m3x2(pp[0], 0.f);
            lead = s0.x & 0xffu; rem = s0.y & 0xffu;
          } else {
#pragma unroll
            for (int q = 0; q < GS; q += 2) {
              const uint2 s01 = split_e4m3x2(pp[q], pp[q + 1]);
              lead |= (s01.x & 0xffffu) << (8 * q);
              rem |= (s01.y & 0xffffu) << (8 * q);
            }
          }
          uint8_t* prow = sP + ps * Cfg::kP8Bytes + kt * 16;
          if constexpr (kSplit) {
            *reinterpret_cast<uint32_t*>(prow + hb) = lead;
            *reinterpret_cast<uint32_t*>(prow + 8 + hb) = rem;
          } else {
            *reinterpret_cast<uint4*>(prow) = make_uint4(lead, rem, 0u, 0u);
          }
        }
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(&p_full[k][ps]);
        if constexpr (kLocalSums) {
          // no test needs the normalizer before the item's end: every thread keeps the sums of its own key column
#pragma unroll
          for (int q = 0; q < GS; ++q) lacc[q] += e[q];
        } else {
          RowReduce<GS, 16, false>::run(e, lane);   // (the sums cross the group with the next tile's maxima)
          psum_w = e[0];
          pending_sum = true;
        }
        ++r;
        ++rg;
      }
      if (!ok) break;
      if constexpr (kLocalSums) {
        RowReduce<GS, 16, false>::run(lacc, lane);
        psum_w = lacc[0];
        pending_sum = true;
      }
      if (pending_sum) {   // the last retained tile's sums
        float unused[GS];
        ok = exchange(-INFINITY, unused, l, lgl);
        if (!ok) break;
      }
      // The item's state for its write-out; the slot is that of the stream's item two before, which has to have been
      // written out.  Only the thread that writes the state waits for that: the write-out of THIS item, which follows
      // the arrival below, completes the same barrier again, and a thread that looked at it only then would take the
      // phase it waits for to be still outstanding.
      if (head) {
        if (ne >= 2) ok = mbar_wait(&o_free[k][ip], (uint32_t)(((ne >> 1) - 1) & 1), status);
        if (ok) {
#pragma unroll
          for (int q = 0; q < GS; ++q) { st_m[k][ip][hb + q] = m_ref[q]; st_l[k][ip][hb + q] = l[q]; st_y[k][ip][hb + q] = yref[q]; }
          if (half == 0) *(volatile int*)&st_r[k][ip] = r;
          mbar_arrive(&st_full[k][ip]);
        }
      }
      ok = __all_sync(0xffffffffu, ok);
      ++ne;
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tb, Cfg::kTmemCols);
}

}  // namespace mala
