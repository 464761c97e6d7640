#pragma once
#include "../../include/mala.h"
#include "sm100_ptx.cuh"
namespace mala {
inline bool decode_set_attributes() { return true; }
inline size_t decode_workspace_bytes(int B, int Hq, int d, int S) { return 256; }
inline int decode_launch(mala_tin, mala_tin, mala_tin, mala_tout, float*, const mala_stats*, int, int, int, int, int,
                         float, float, int, void*, int*, cudaStream_t) {
  return MALA_ERR_UNSUPPORTED;
}
}  // namespace mala
