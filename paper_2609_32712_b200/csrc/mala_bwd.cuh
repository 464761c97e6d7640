#pragma once
#include "../../include/mala.h"
#include "sm100_ptx.cuh"
namespace mala {
inline bool bwd_set_attributes() { return true; }
inline size_t bwd_workspace_bytes(int B, int Hq, int N, int d) { return 256; }
inline int bwd_launch(mala_tin, mala_tin, mala_tin, mala_tin, mala_tin, const float*, mala_tout, mala_tout, mala_tout,
                      const mala_stats*, int, int, int, int, int, int, float, float, void*, int*, cudaStream_t) {
  return MALA_ERR_UNSUPPORTED;
}
}  // namespace mala
