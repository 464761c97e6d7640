// Split-KV decode ("Fused decoding execution"): the persistent split kernel lives in
// mala_decode_split.cuh; this file holds the normalizer-aware merge of the split partials, the
// workspace layout and the launch code.
#pragma once
#include <cuda_runtime.h>

#include "../../include/mala.h"
#include "mala_decode_split.cuh"
#include "mala_decode_fp8.cuh"
#include "tensor_map.h"

namespace mala {

// lse = log sum_s exp(lse_s), o = sum_s exp(lse_s - lse) o_s; one block per (b, token, query head), one thread
// per output column.
template <int D>
__global__ void __launch_bounds__(D)
decode_merge_kernel(const float* __restrict__ o_part, const float* __restrict__ lse_part, __nv_bfloat16* __restrict__ o,
                    int64_t o_sb, int64_t o_sn, int64_t o_sh, float* __restrict__ lse_out, int Sq, int Hq,
                    int num_splits, int d) {   // d <= D: columns of o
  const int bh = blockIdx.x, h = bh % Hq, tok = (bh / Hq) % Sq, b = bh / (Hq * Sq), c = threadIdx.x;
  const float* lp = lse_part + (size_t)bh * num_splits;
  float mx = -INFINITY;
  for (int s = 0; s < num_splits; ++s) mx = fmaxf(mx, lp[s]);
  float Z = 0.f, acc = 0.f;
  for (int s = 0; s < num_splits; ++s) {
    const float ls = lp[s];
    if (ls == -INFINITY) continue;
    const float w = exp2f((ls - mx) * 1.4426950408889634f);
    Z += w;
    acc += w * o_part[((size_t)bh * num_splits + s) * D + c];
  }
  // (a sequence without keys has no split with mass: its output is 0 and its log-normalizer -inf)
  if (c < d) o[b * o_sb + tok * o_sn + h * o_sh + c] = __float2bfloat16(Z > 0.f ? acc / Z : 0.f);
  if (lse_out && c == 0) lse_out[bh] = Z > 0.f ? mx + logf(Z) : -INFINITY;
}

inline size_t decode_align256(size_t x) { return (x + 255) & ~(size_t)255; }

// (B: sequences x new tokens per sequence)
inline size_t decode_workspace_bytes(int B, int Hq, int d, int S) {   // d: the padded head size
  return decode_align256((size_t)B * Hq * S * d * sizeof(float)) + decode_align256((size_t)B * Hq * S * sizeof(float));
}

inline bool decode_set_attributes() {
  bool ok = true;
#define MALA_DEC_ATTR(DENSE, GP, MULTI) \
  ok = ok && cudaFuncSetAttribute(mala_decode_split_kernel<DENSE, GP, MULTI, 128>, cudaFuncAttributeMaxDynamicSharedMemorySize, DecCfg::kSmemBytes) == cudaSuccess; \
  ok = ok && cudaFuncSetAttribute(mala_decode_split_kernel<DENSE, GP, MULTI, 64>, cudaFuncAttributeMaxDynamicSharedMemorySize, DecCfg::kSmemBytes) == cudaSuccess; \
  ok = ok && cudaFuncSetAttribute(mala_decode_split_kernel<DENSE, GP, MULTI, 256>, cudaFuncAttributeMaxDynamicSharedMemorySize, DecCfgT<256>::kSmemBytes) == cudaSuccess;
#define MALA_DEC_ATTR_GP(GP) MALA_DEC_ATTR(false, GP, false) MALA_DEC_ATTR(true, GP, false) MALA_DEC_ATTR(false, GP, true) MALA_DEC_ATTR(true, GP, true)
  MALA_DEC_ATTR_GP(1) MALA_DEC_ATTR_GP(2) MALA_DEC_ATTR_GP(4) MALA_DEC_ATTR_GP(8) MALA_DEC_ATTR_GP(16)
#define MALA_F8_ATTR(DENSE, GP) \
  ok = ok && cudaFuncSetAttribute(mala_decode_fp8_kernel<DENSE, GP, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, DecF8Cfg<2, DENSE>::kSmemBytes) == cudaSuccess && cudaFuncSetAttribute(mala_decode_fp8_kernel<DENSE, GP, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, DecF8Cfg<2, DENSE>::kSmemBytes) == cudaSuccess && cudaFuncSetAttribute(mala_decode_fp8_kernel<DENSE, GP, true, 2, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, DecF8Cfg<2, DENSE>::kSmemBytes) == cudaSuccess && cudaFuncSetAttribute(mala_decode_fp8_kernel<DENSE, GP, false, 2, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, DecF8Cfg<2, DENSE>::kSmemBytes) == cudaSuccess;
  MALA_F8_ATTR(false, 1) MALA_F8_ATTR(true, 1) MALA_F8_ATTR(false, 2) MALA_F8_ATTR(true, 2) MALA_F8_ATTR(false, 4) MALA_F8_ATTR(true, 4)
  MALA_F8_ATTR(false, 8) MALA_F8_ATTR(true, 8)
#undef MALA_F8_ATTR
#undef MALA_DEC_ATTR_GP
#undef MALA_DEC_ATTR
  return ok;
}

// A cache held in pages: kc / vc are [num_pages, page_size, Hkv, d] (sb = page stride), sequence b keeps its keys
// 128*x .. in page block_table[b * bt_stride + x / (page_size / 128)], and holds seqlens[b] <= Nk keys.
struct DecPaging {
  const int* block_table;   // null: one contiguous cache per sequence
  const int* seqlens;       // null: every sequence holds Nk keys
  int bt_stride, page_size, num_pages;
};

// Launches the split kernel and the merge on `stream`.  o_part / lse_part: caller-provided scratch of
// decode_workspace_bytes() bytes in total (o_part first).  Nk: the longest cache (the splits are laid out for it).
inline int decode_launch_with_scratch(mala_tin q, mala_tin kc, mala_tin vc, mala_tout o, float* lse_opt,
                                      const mala_stats* st, int B, int Hq, int Hkv, int Nk, int d, float scale,
                                      float tau, int num_splits, float* o_part, float* lse_part, int* status,
                                      cudaStream_t stream, const DecPaging* pg = nullptr, int Sq = 1) {
  if (!head_size_ok(d, 256)) return MALA_ERR_UNSUPPORTED;
  const int D = padded_head_size(d);
  const int G = Hq / Hkv;
  if (Sq < 1 || G * Sq > 16 || Sq > Nk) return MALA_ERR_UNSUPPORTED;
  const bool paged = pg && pg->block_table;
  // pages of whole tiles, or 8, 16, 32 or 64 keys (a tile is then put together from several pages)
  if (paged && (pg->page_size < 8 || (pg->page_size % 128 != 0 && 128 % pg->page_size != 0) || pg->num_pages <= 0 ||
                pg->bt_stride <= 0))
    return MALA_ERR_UNSUPPORTED;
  const int box_rows = paged && pg->page_size < 128 ? pg->page_size : 128;
  const int per = (Nk + num_splits - 1) / num_splits;
  const int tps = (per + 127) / 128;
  if ((long long)B * Hkv * num_splits > 0x7fffffffLL) return MALA_ERR_UNSUPPORTED;

  CUtensorMap tq, tk, tv;
  // q [B,Sq,Hq,d]: one box of the group's G heads x Sq tokens
  if (!make_tensor_map_q_rows(&tq, q.p, B, Sq, Hq, d, q.sb, Sq > 1 ? q.sn : 0, q.sh, G) ||
      !make_tensor_map_bnhd(&tk, kc.p, paged ? pg->num_pages : B, paged ? pg->page_size : Nk, Hkv, d, kc.sb, kc.sn,
                            kc.sh, box_rows) ||
      !make_tensor_map_bnhd(&tv, vc.p, paged ? pg->num_pages : B, paged ? pg->page_size : Nk, Hkv, d, vc.sb, vc.sn,
                            vc.sh, box_rows))
    return MALA_ERR_TENSOR_MAP;

  DecParams p;
  p.o_part = o_part; p.lse_part = lse_part;
  p.retained = st ? st->retained_per_block : nullptr;
  p.bitmask = st ? st->tile_bitmask : nullptr;
  p.totals = st ? (unsigned long long*)st->totals : nullptr;
  p.status = status;
  p.seqlens = pg ? pg->seqlens : nullptr;
  p.block_table = paged ? pg->block_table : nullptr;
  p.bt_stride = paged ? pg->bt_stride : 0;
  p.tpp = paged && pg->page_size >= 128 ? pg->page_size / 128 : 1;
  p.ppt = 128 / box_rows;
  p.prows = box_rows;
  p.Sq = Sq;
  p.B = B; p.Hq = Hq; p.Hkv = Hkv; p.Nk = Nk; p.tps = tps; p.num_splits = num_splits; p.words = (tps + 31) / 32;
  p.n_items = B * Hkv * num_splits;
  p.scale_log2 = scale * 1.4426950408889634f;
  p.log2_tau = tau > 0.f ? log2f(tau) : -INFINITY;
  if (p.bitmask &&
      cudaMemsetAsync(p.bitmask, 0, (size_t)B * Hkv * num_splits * p.words * sizeof(uint32_t), stream) != cudaSuccess)
    return MALA_ERR_CUDA;

  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
    return MALA_ERR_CUDA;
  const int grid = p.n_items < sms ? p.n_items : sms;   // persistent: one CTA per SM
  const int R = G * Sq;   // rows of a work item
#define MALA_DEC_LAUNCH3(DENSE, GP, MULTI)                                                                           \
  {                                                                                                                  \
    if (D == 256) mala_decode_split_kernel<DENSE, GP, MULTI, 256><<<grid, DecCfg::kThreads, DecCfgT<256>::kSmemBytes, stream>>>(tq, tk, tv, p); \
    else if (D == 128) mala_decode_split_kernel<DENSE, GP, MULTI, 128><<<grid, DecCfg::kThreads, DecCfg::kSmemBytes, stream>>>(tq, tk, tv, p); \
    else mala_decode_split_kernel<DENSE, GP, MULTI, 64><<<grid, DecCfg::kThreads, DecCfg::kSmemBytes, stream>>>(tq, tk, tv, p);           \
  }
#define MALA_DEC_LAUNCH2(DENSE, GP)          \
  {                                          \
    if (Sq > 1) MALA_DEC_LAUNCH3(DENSE, GP, true) \
    else MALA_DEC_LAUNCH3(DENSE, GP, false)  \
  }
#define MALA_DEC_LAUNCH(GP)            \
  {                                    \
    if (tau == 0.f) MALA_DEC_LAUNCH2(true, GP) \
    else MALA_DEC_LAUNCH2(false, GP)   \
  }
  if (R <= 1) MALA_DEC_LAUNCH(1)
  else if (R <= 2) MALA_DEC_LAUNCH(2)
  else if (R <= 4) MALA_DEC_LAUNCH(4)
  else if (R <= 8) MALA_DEC_LAUNCH(8)
  else MALA_DEC_LAUNCH(16)
#undef MALA_DEC_LAUNCH
#undef MALA_DEC_LAUNCH2
#undef MALA_DEC_LAUNCH3
  if (cudaGetLastError() != cudaSuccess) return MALA_ERR_CUDA;
  if (D == 256)
    decode_merge_kernel<256><<<B * Sq * Hq, 256, 0, stream>>>(o_part, lse_part, (__nv_bfloat16*)o.p, o.sb,
                                                              Sq > 1 ? o.sn : 0, o.sh, lse_opt, Sq, Hq, num_splits, d);
  else if (D == 128)
    decode_merge_kernel<128><<<B * Sq * Hq, 128, 0, stream>>>(o_part, lse_part, (__nv_bfloat16*)o.p, o.sb,
                                                              Sq > 1 ? o.sn : 0, o.sh, lse_opt, Sq, Hq, num_splits, d);
  else
    decode_merge_kernel<64><<<B * Sq * Hq, 64, 0, stream>>>(o_part, lse_part, (__nv_bfloat16*)o.p, o.sb,
                                                            Sq > 1 ? o.sn : 0, o.sh, lse_opt, Sq, Hq, num_splits, d);
  return cudaGetLastError() == cudaSuccess ? MALA_OK : MALA_ERR_CUDA;
}

// Decode over an e4m3 cache with one fp32 scale per (sequence, KV head, 128-key tile): kc / vc are 8-bit [B,Nk,Hkv,d]
// views (strides in elements), kscale / vscale fp32 [B,Hkv,ceil(Nk/128)].  Up to four query heads per KV head.
// pg != null: kc / vc are [num_pages, page_size, Hkv, d] (page_size a multiple of 128, or 16, 32 or 64), the scales
// [num_pages, Hkv, max(1, page_size/128)], and Nk = bt_stride * page_size lays out the splits.
inline int decode_fp8_launch(mala_tin q, mala_tin kc, mala_tin vc, const float* kscale, const float* vscale, mala_tout o,
                             float* lse_opt, const mala_stats* st, int B, int Hq, int Hkv, int Nk, int d, float scale,
                             float tau, int num_splits, void* ws, int* status, cudaStream_t stream,
                             const DecPaging* pg = nullptr, int Sq = 1) {
  const int G = Hq / Hkv;
  const int R = G * Sq;   // rows of a work item
  if (Sq < 1 || R > 8 || Sq > Nk || d % 16 != 0 || d > 128 || d < 16) return MALA_ERR_UNSUPPORTED;
  if (Sq > 1 && pg) return MALA_ERR_UNSUPPORTED;   // (several tokens per step: contiguous caches only)
  const bool small = pg && pg->page_size < 128;
  if (pg && !(pg->page_size % 128 == 0 || pg->page_size == 16 || pg->page_size == 32 || pg->page_size == 64))
    return MALA_ERR_UNSUPPORTED;
  const int box_rows = small ? pg->page_size : 128;
  const int per = (Nk + num_splits - 1) / num_splits;
  const int tps = (per + 127) / 128;
  if ((long long)B * Hkv * num_splits > 0x7fffffffLL || (long long)B * Hkv * ((Nk + 127) / 128) > 0x7fffffffLL)
    return MALA_ERR_UNSUPPORTED;
  CUtensorMap tq, tk, tv;
  if (!make_tensor_map_q_rows(&tq, q.p, B, Sq, Hq, d, q.sb, Sq > 1 ? q.sn : 0, q.sh, G) ||
      !make_tensor_map_u8_bnhd(&tk, kc.p, pg ? pg->num_pages : B, pg ? pg->page_size : Nk, Hkv, d, kc.sb, kc.sn, kc.sh, box_rows) ||
      !make_tensor_map_u8_bnhd(&tv, vc.p, pg ? pg->num_pages : B, pg ? pg->page_size : Nk, Hkv, d, vc.sb, vc.sn, vc.sh, box_rows))
    return MALA_ERR_TENSOR_MAP;
  DecF8Params p;
  p.block_table = pg ? pg->block_table : nullptr;
  p.seqlens = pg ? pg->seqlens : nullptr;
  p.num_pages = pg ? pg->num_pages : 0;
  p.max_pages = pg ? pg->bt_stride : 0;
  p.tpp = (pg && !small) ? pg->page_size / 128 : 1;
  p.by_tpp.set((uint32_t)p.tpp);
  p.ppt = 128 / box_rows;
  p.prows = box_rows;
  p.Sq = Sq;
  p.o_part = (float*)ws;
  p.lse_part = (float*)((uint8_t*)ws + decode_align256((size_t)B * Sq * Hq * num_splits * 128 * sizeof(float)));
  p.retained = st ? st->retained_per_block : nullptr;
  p.bitmask = st ? st->tile_bitmask : nullptr;
  p.totals = st ? (unsigned long long*)st->totals : nullptr;
  p.status = status;
  p.kscale = kscale; p.vscale = vscale;
  p.B = B; p.Hq = Hq; p.Hkv = Hkv; p.Nk = Nk; p.tps = tps; p.num_splits = num_splits; p.words = (tps + 31) / 32;
  p.n_items = B * Hkv * num_splits; p.nt = (Nk + 127) / 128;
  p.by_splits.set((uint32_t)num_splits);
  p.by_hkv.set((uint32_t)Hkv);
  p.scale_log2 = scale * 1.4426950408889634f;
  p.log2_tau = tau > 0.f ? log2f(tau) : -INFINITY;
  if (p.bitmask &&
      cudaMemsetAsync(p.bitmask, 0, (size_t)B * Hkv * num_splits * p.words * sizeof(uint32_t), stream) != cudaSuccess)
    return MALA_ERR_CUDA;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
    return MALA_ERR_CUDA;
  const int grid = p.n_items < sms ? p.n_items : sms;
#define MALA_F8_LAUNCH(DENSE, GP)                                                                                      \
  do {                                                                                                                  \
    if (Sq > 1) mala_decode_fp8_kernel<DENSE, GP, false, 2, false, true><<<grid, DecF8Cfg<2, DENSE, (GP > 4)>::kThreads, DecF8Cfg<2, DENSE>::kSmemBytes, stream>>>(tq, tk, tv, p); \
    else if (small) mala_decode_fp8_kernel<DENSE, GP, true, 2, true><<<grid, DecF8Cfg<2, DENSE, (GP > 4)>::kThreads, DecF8Cfg<2, DENSE>::kSmemBytes, stream>>>(tq, tk, tv, p); \
    else if (pg) mala_decode_fp8_kernel<DENSE, GP, true><<<grid, DecF8Cfg<2, DENSE, (GP > 4)>::kThreads, DecF8Cfg<2, DENSE>::kSmemBytes, stream>>>(tq, tk, tv, p); \
    else mala_decode_fp8_kernel<DENSE, GP, false><<<grid, DecF8Cfg<2, DENSE, (GP > 4)>::kThreads, DecF8Cfg<2, DENSE>::kSmemBytes, stream>>>(tq, tk, tv, p);  \
  } while (0)
  const bool dense = (tau == 0.f);
  if (R <= 1) { if (dense) MALA_F8_LAUNCH(true, 1); else MALA_F8_LAUNCH(false, 1); }
  else if (R <= 2) { if (dense) MALA_F8_LAUNCH(true, 2); else MALA_F8_LAUNCH(false, 2); }
  else if (R <= 4) { if (dense) MALA_F8_LAUNCH(true, 4); else MALA_F8_LAUNCH(false, 4); }
  else { if (dense) MALA_F8_LAUNCH(true, 8); else MALA_F8_LAUNCH(false, 8); }
#undef MALA_F8_LAUNCH
  if (cudaGetLastError() != cudaSuccess) return MALA_ERR_CUDA;
  decode_merge_kernel<128><<<B * Sq * Hq, 128, 0, stream>>>(p.o_part, p.lse_part, (__nv_bfloat16*)o.p, o.sb,
                                                           Sq > 1 ? o.sn : 0, o.sh, lse_opt, Sq, Hq, num_splits, d);
  return cudaGetLastError() == cudaSuccess ? MALA_OK : MALA_ERR_CUDA;
}

inline int decode_launch(mala_tin q, mala_tin kc, mala_tin vc, mala_tout o, float* lse_opt, const mala_stats* st, int B,
                         int Hq, int Hkv, int Nk, int d, float scale, float tau, int num_splits, void* ws, int* status,
                         cudaStream_t stream, const DecPaging* pg = nullptr, int Sq = 1) {
  float* o_part = (float*)ws;
  float* lse_part =
      (float*)((uint8_t*)ws + decode_align256((size_t)B * Sq * Hq * num_splits * padded_head_size(d) * sizeof(float)));
  return decode_launch_with_scratch(q, kc, vc, o, lse_opt, st, B, Hq, Hkv, Nk, d, scale, tau, num_splits, o_part,
                                    lse_part, status, stream, pg, Sq);
}

}  // namespace mala
