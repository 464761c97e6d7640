// Host-side creation of TMA tensor maps for bf16 tensors viewed as [B, N, H, d] with arbitrary
// element strides (last dimension contiguous).  The driver entry point is looked up at run time so
// the library has no link-time dependency on libcuda.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace mala {

typedef CUresult (*PFN_tensorMapEncodeTiled)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                             const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                             CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                             CUtensorMapFloatOOBfill);

inline PFN_tensorMapEncodeTiled tensor_map_encoder() {
  static PFN_tensorMapEncodeTiled fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = (PFN_tensorMapEncodeTiled)p;
  }
  return fn;
}

// Tensor map over a bf16 [B, N, H, d] view: coordinates (c, n, h, b), box = 64 columns x box_rows rows,
// 128-byte swizzle, out-of-range rows read as zero.  Returns false if the driver rejects it
// (base not 16-byte aligned, a stride not a multiple of 16 bytes, ...).
// Head sizes: any multiple of 8 up to dmax (128; the forward and the decode step also take 256).  The kernels are built
// for D = 64, 128 and 256 columns; a smaller head runs on the next of them with the missing columns read as zeros (TMA
// fills what lies beyond the tensor map's inner extent d) and never stored.
inline bool head_size_ok(int d, int dmax = 128) { return d >= 8 && d <= dmax && d % 8 == 0; }
inline int padded_head_size(int d) { return d <= 64 ? 64 : (d <= 128 ? 128 : 256); }

inline bool make_tensor_map_bnhd(CUtensorMap* out, const void* base, int B, int N, int H, int d, int64_t sb,
                                 int64_t sn, int64_t sh, int box_rows) {
  PFN_tensorMapEncodeTiled enc = tensor_map_encoder();
  if (!enc) return false;
  cuuint64_t dims[4] = {(cuuint64_t)d, (cuuint64_t)N, (cuuint64_t)H, (cuuint64_t)B};
  // strides of dimensions 1..3 in bytes; a stride of a size-1 dimension only needs to be legal
  auto legal = [&](int64_t s, int n) -> cuuint64_t { return (n == 1 || s <= 0) ? (cuuint64_t)d * 2 : (cuuint64_t)s * 2; };
  cuuint64_t strides[3] = {legal(sn, N), legal(sh, H), legal(sb, B)};
  cuuint32_t box[4] = {64u, (cuuint32_t)box_rows, 1u, 1u};
  cuuint32_t estr[4] = {1u, 1u, 1u, 1u};
  CUresult r = enc(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

// Tensor map over an 8-bit [B, N, H, d] view (strides in elements = bytes): coordinates (c, n, h, b), box = 128 columns
// x box_rows rows (128: one 16 KB tile; fewer: one page smaller than a tile), 128-byte swizzle; columns beyond d and rows
// beyond N read as zero.
inline bool make_tensor_map_u8_bnhd(CUtensorMap* out, const void* base, int B, int N, int H, int d, int64_t sb,
                                    int64_t sn, int64_t sh, int box_rows = 128) {
  PFN_tensorMapEncodeTiled enc = tensor_map_encoder();
  if (!enc) return false;
  cuuint64_t dims[4] = {(cuuint64_t)d, (cuuint64_t)N, (cuuint64_t)H, (cuuint64_t)B};
  auto legal = [&](int64_t s, int n) -> cuuint64_t { return (n == 1 || s <= 0) ? (cuuint64_t)((d + 15) / 16 * 16) : (cuuint64_t)s; };
  cuuint64_t strides[3] = {legal(sn, N), legal(sh, H), legal(sb, B)};
  cuuint32_t box[4] = {128u, (cuuint32_t)box_rows, 1u, 1u};
  cuuint32_t estr[4] = {1u, 1u, 1u, 1u};
  CUresult r = enc(out, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<void*>(base), dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

// Tensor map over the bf16 queries of a decode step, [B, S, H, d]: coordinates (c, h, s, b), box = 64 columns x G
// heads x S tokens, which lands in shared memory as S * G consecutive 128-byte rows (row s * G + g), 128-byte swizzle.
inline bool make_tensor_map_q_rows(CUtensorMap* out, const void* base, int B, int S, int H, int d, int64_t sb,
                                   int64_t sn, int64_t sh, int G) {
  PFN_tensorMapEncodeTiled enc = tensor_map_encoder();
  if (!enc) return false;
  cuuint64_t dims[4] = {(cuuint64_t)d, (cuuint64_t)H, (cuuint64_t)S, (cuuint64_t)B};
  auto legal = [&](int64_t s, int n) -> cuuint64_t { return (n == 1 || s <= 0) ? (cuuint64_t)d * 2 : (cuuint64_t)s * 2; };
  cuuint64_t strides[3] = {legal(sh, H), legal(sn, S), legal(sb, B)};
  cuuint32_t box[4] = {64u, (cuuint32_t)G, (cuuint32_t)S, 1u};
  cuuint32_t estr[4] = {1u, 1u, 1u, 1u};
  CUresult r = enc(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

// Tensor map over fp32 tiles: `ntiles` row-major [128 rows x cols] blocks, `tile_stride_bytes` apart, first one at
// `base`.  Coordinates (col, row, tile), box = 32 columns x 128 rows x 1 tile (128 bytes wide), 128-byte swizzle.
// Used for TMA reduce-add of fp32 panels.
inline bool make_tensor_map_f32_tiles(CUtensorMap* out, const void* base, uint64_t ntiles, int cols,
                                      uint64_t tile_stride_bytes) {
  PFN_tensorMapEncodeTiled enc = tensor_map_encoder();
  if (!enc) return false;
  cuuint64_t dims[3] = {(cuuint64_t)cols, 128u, (cuuint64_t)ntiles};
  cuuint64_t strides[2] = {(cuuint64_t)cols * 4, (cuuint64_t)tile_stride_bytes};
  cuuint32_t box[3] = {32u, 128u, 1u};
  cuuint32_t estr[3] = {1u, 1u, 1u};
  CUresult r = enc(out, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<void*>(base), dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

}  // namespace mala
