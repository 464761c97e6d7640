// Host side of libmala: argument validation, TMA tensor-map creation, workspace carving and kernel
// launches behind the C ABI declared in include/mala.h.  No torch types, no allocation, no sync.
#include <cuda_runtime.h>
#include <math.h>
#include <stdio.h>
#include <stdlib.h>
#include <mutex>

#include <nvtx3/nvToolsExt.h>

#include "../../include/mala.h"
#include "mala_bwd.cuh"
#include "mala_decode.cuh"
#include "mala_fwd.cuh"
#include "tensor_map.h"

namespace mala {

// Sticky per-device status word written by kernels whose bounded waits expire.
__device__ int g_mala_status;

// The kernels' bounded wait on a barrier that nobody arrives on (test support, see mala_test_expire_wait): the wait
// gives up after limit_cycles, records the time-out in the status word and the kernel leaves through its normal exit.
__global__ void expire_wait_kernel(int* status, long long limit_cycles) {
  __shared__ uint64_t bar;
  if (threadIdx.x == 0) { mbar_init(&bar, 1); mbar_fence_init(); }
  __syncthreads();
  if (threadIdx.x == 0) mbar_wait(&bar, 0, status, limit_cycles);
  __syncthreads();
}

static std::mutex g_mu;
static int* g_status_ptr[64];
static bool g_attr_done[64];

// Built-in scratch of mala_decode_static: the split partials of one decode call.  Every device that
// loads the library holds these bytes until the process exits.  In host code the array's name is only
// a stand-in for the symbol, not a device address, so its address is looked up per device below.
static __device__ __align__(256) unsigned char g_decode_scratch[MALA_STATIC_SCRATCH_BYTES];
static unsigned char* g_decode_scratch_ptr[64];

// Device address of the built-in scratch on device `dev` (which must be current); looked up once.
static int static_scratch_address(int dev, unsigned char** out) {
  std::lock_guard<std::mutex> lock(g_mu);
  if (!g_decode_scratch_ptr[dev]) {
    unsigned char* ptr = nullptr;
    if (cudaGetSymbolAddress((void**)&ptr, g_decode_scratch) != cudaSuccess || !ptr) return MALA_ERR_CUDA;
    g_decode_scratch_ptr[dev] = ptr;
  }
  *out = g_decode_scratch_ptr[dev];
  return MALA_OK;
}

static int current_device_checked(int* dev_out) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return MALA_ERR_CUDA;
  if (dev < 0 || dev >= 64) return MALA_ERR_UNSUPPORTED;
  int major = 0;
  if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return MALA_ERR_CUDA;
  if (major != 10) return MALA_ERR_WRONG_ARCH;
  *dev_out = dev;
  return MALA_OK;
}

template <typename K>
static bool set_smem(K kernel, int bytes) {
  return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) == cudaSuccess;
}

// One-time per-device set-up: status word address and dynamic shared memory limits.
static int device_setup(int dev, int** status_out) {
  std::lock_guard<std::mutex> lock(g_mu);
  if (!g_status_ptr[dev]) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_mala_status) != cudaSuccess) return MALA_ERR_CUDA;
    g_status_ptr[dev] = (int*)ptr;
  }
  if (!g_attr_done[dev]) {
    bool ok = true;
    ok = ok && set_smem(mala_fwd_kernel<128, true>, FwdCfg<128, true>::kSmemBytes);
    ok = ok && set_smem(mala_fwd_kernel<128, false>, FwdCfg<128, false>::kSmemBytes);
    ok = ok && set_smem(mala_fwd_kernel<64, false>, FwdCfg<64, false>::kSmemBytes);
    ok = ok && set_smem(mala_fwd_kernel<64, true>, FwdCfg<64, true>::kSmemBytes);
    ok = ok && set_smem(mala_fwd_kernel<128, true, true>, FwdCfg<128, true>::kSmemBytes);
    ok = ok && set_smem(mala_fwd_kernel<128, false, true>, FwdCfg<128, false>::kSmemBytes);
    ok = ok && set_smem(mala_fwd_kernel<64, false, true>, FwdCfg<64, false>::kSmemBytes);
    ok = ok && set_smem(mala_fwd_kernel<64, true, true>, FwdCfg<64, true>::kSmemBytes);
    ok = ok && set_smem(mala_fwd_kernel<256, true>, FwdCfg<256, true>::kSmemBytes);
    ok = ok && set_smem(mala_fwd_kernel<256, false>, FwdCfg<256, false>::kSmemBytes);
    ok = ok && set_smem(mala_fwd_kernel<256, true, true>, FwdCfg<256, true>::kSmemBytes);
    ok = ok && set_smem(mala_fwd_kernel<256, false, true>, FwdCfg<256, false>::kSmemBytes);
    ok = ok && bwd_set_attributes();
    ok = ok && decode_set_attributes();
    if (!ok) return MALA_ERR_CUDA;
    g_attr_done[dev] = true;
  }
  *status_out = g_status_ptr[dev];
  return MALA_OK;
}

static bool aligned16(const void* p) { return (((uintptr_t)p) & 15) == 0; }
static bool stride_ok(int64_t s) { return s >= 0 && (s % 8) == 0; }

// bf16 [B,N,H,d] view: pointer and strides legal for TMA and 16-byte vector access
static int check_view(const void* p, int64_t sb, int64_t sn, int64_t sh, int B, int N, int H) {
  if (!p) return MALA_ERR_INVALID_ARG;
  if (!aligned16(p)) return MALA_ERR_MISALIGNED;
  if ((B > 1 && !stride_ok(sb)) || (N > 1 && !stride_ok(sn)) || (H > 1 && !stride_ok(sh))) return MALA_ERR_MISALIGNED;
  if ((B > 1 && sb == 0) || (N > 1 && sn == 0) || (H > 1 && sh == 0)) return MALA_ERR_INVALID_ARG;
  return MALA_OK;
}

static int check_common(int B, int Hq, int Hkv, int N, int d, float scale, float tau, int dmax = 128) {
  if (B <= 0 || Hq <= 0 || Hkv <= 0 || N <= 0) return MALA_ERR_INVALID_ARG;
  if (!(tau >= 0.f) || !isfinite(tau)) return MALA_ERR_INVALID_ARG;
  if (!(scale > 0.f) || !isfinite(scale)) return MALA_ERR_INVALID_ARG;
  if (!head_size_ok(d, dmax)) return MALA_ERR_UNSUPPORTED;
  if (Hq % Hkv != 0) return MALA_ERR_UNSUPPORTED;
  if (B > 65535 || Hq > 65535) return MALA_ERR_UNSUPPORTED;
  return MALA_OK;
}

// Two environment variables, read once, change what a call does around its launches (both off by default):
//   MALA_NVTX=1   every call that launches kernels is an NVTX range of its own name on the calling thread
//   MALA_DEBUG=1  synchronous error reporting: the call waits for its stream, and a CUDA error or a recorded device
//                 time-out comes back as the call's own return value (MALA_ERR_CUDA / MALA_ERR_DEVICE_TIMEOUT) with a line
//                 on stderr, instead of surfacing at a later call.  (The call then synchronises, which it otherwise
//                 never does; the status word stays set until mala_device_status clears it.)
static int env_flag(const char* name) {
  const char* v = getenv(name);
  return (v && v[0] && v[0] != '0') ? 1 : 0;
}
static int nvtx_on() { static const int v = env_flag("MALA_NVTX"); return v; }
static int debug_on() { static const int v = env_flag("MALA_DEBUG"); return v; }

struct ApiScope {
  const char* name;
  cudaStream_t stream;
  bool pushed;
  ApiScope(const char* n, void* s) : name(n), stream((cudaStream_t)s), pushed(false) {
    if (nvtx_on()) { nvtxRangePushA(name); pushed = true; }
  }
  ~ApiScope() { if (pushed) nvtxRangePop(); }
  int finish(int rc) const {
    if (rc != MALA_OK || !debug_on()) return rc;
    cudaError_t e = cudaStreamSynchronize(stream);
    if (e == cudaSuccess) e = cudaGetLastError();
    if (e != cudaSuccess) {
      fprintf(stderr, "[mala debug] %s: CUDA error %d (%s)\n", name, (int)e, cudaGetErrorString(e));
      return MALA_ERR_CUDA;
    }
    int code = 0;
    if (mala_device_status(&code, 0) != MALA_OK) return MALA_ERR_CUDA;
    if (code != 0) {
      fprintf(stderr, "[mala debug] %s: device status %d (a bounded wait expired)\n", name, code);
      return MALA_ERR_DEVICE_TIMEOUT;
    }
    return MALA_OK;
  }
};

#define MALA_TRY(expr)              \
  do {                              \
    const int rc_ = (expr);         \
    if (rc_ != MALA_OK) return rc_; \
  } while (0)

static const float kLog2e = 1.4426950408889634f;

// Forward (prefill) launch: two query blocks per CTA (one with D = 256).
template <int D, bool kDense>
static int launch_fwd(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv, const FwdParams& p,
                      cudaStream_t stream) {
  dim3 grid(FwdCfg<D, kDense>::kOne ? p.Tr : (p.Tr + 1) / 2, p.Hq, p.B * (p.num_splits > 1 ? p.num_splits : 1));
  if (p.ppt > 1)
    mala_fwd_kernel<D, kDense, true><<<grid, FwdCfg<D, kDense>::kThreads, FwdCfg<D, kDense>::kSmemBytes, stream>>>(tq, tk, tv, p);
  else
    mala_fwd_kernel<D, kDense><<<grid, FwdCfg<D, kDense>::kThreads, FwdCfg<D, kDense>::kSmemBytes, stream>>>(tq, tk, tv, p);
  return cudaGetLastError() == cudaSuccess ? MALA_OK : MALA_ERR_CUDA;
}

}  // namespace mala

using namespace mala;

extern "C" {

int mala_version(void) { return 100; }

const char* mala_strerror(int code) {
  switch (code) {
    case MALA_OK: return "ok";
    case MALA_ERR_INVALID_ARG: return "invalid argument";
    case MALA_ERR_UNSUPPORTED: return "unsupported configuration";
    case MALA_ERR_MISALIGNED: return "pointer or stride not 16-byte aligned";
    case MALA_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
    case MALA_ERR_WRONG_ARCH: return "device is not sm_100";
    case MALA_ERR_CUDA: return "CUDA runtime error";
    case MALA_ERR_TENSOR_MAP: return "TMA tensor map rejected";
    case MALA_ERR_DEVICE_TIMEOUT: return "bounded device-side wait expired";
    case MALA_ERR_STATIC_SCRATCH_EXCEEDED: return "problem needs more than the library's built-in scratch";
    default: return "unknown error";
  }
}

int mala_decode_suggest_splits(int B, int Hkv, int Nk, int sm_count) {
  if (B <= 0 || Hkv <= 0 || Nk <= 0) return MALA_ERR_INVALID_ARG;
  if (sm_count <= 0) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sm_count <= 0)
      return MALA_ERR_CUDA;
  }
  const long long T = (Nk + 127) / 128, groups = (long long)B * Hkv;
  auto queue = [&](long long S) { return ((groups * S + sm_count - 1) / sm_count) * ((T + S - 1) / S); };
  long long hi = T / 2 > 1 ? T / 2 : 1;                       // at least two tiles per split
  if (hi > 65535) hi = 65535;
  long long lo = (6LL * sm_count + groups - 1) / groups;       // at least six items per SM ...
  if (lo > hi) lo = 1;                                         // ... where the cache is long enough for that
  long long best = queue(lo);
  for (long long S = lo + 1; S <= hi; ++S) best = queue(S) < best ? queue(S) : best;
  for (long long S = lo; S <= hi; ++S)
    if (queue(S) * 100 <= best * 104) return (int)S;
  return (int)lo;
}

int mala_tile_shape(int op, int d, int* Bq, int* Bk) {
  if (!Bq || !Bk) return MALA_ERR_INVALID_ARG;
  if (!head_size_ok(d, op == MALA_OP_BWD ? 128 : 256)) return MALA_ERR_UNSUPPORTED;
  if (op == MALA_OP_FWD || op == MALA_OP_BWD) { *Bq = 128; *Bk = 128; return MALA_OK; }
  if (op == MALA_OP_DECODE) { *Bq = 0; *Bk = 128; return MALA_OK; }
  return MALA_ERR_UNSUPPORTED;
}

size_t mala_workspace_bytes(int op, int B, int Hq, int Hkv, int N, int d, int num_splits) {
  if (B <= 0 || Hq <= 0 || Hkv <= 0 || N <= 0 || !head_size_ok(d, op == MALA_OP_BWD ? 128 : 256)) return 0;
  const int D = padded_head_size(d);
  if (op == MALA_OP_FWD) return num_splits > 1 ? fwd_split_workspace_bytes(B, Hq, N, D, num_splits) : 256;
  if (op == MALA_OP_BWD) return bwd_workspace_bytes(B, Hq, N, D);
  if (op == MALA_OP_DECODE) return num_splits > 0 ? decode_workspace_bytes(B, Hq, D, num_splits) : 0;
  return 0;
}

int mala_device_status(int* code_out, int clear) {
  if (!code_out) return MALA_ERR_INVALID_ARG;
  int dev = 0;
  MALA_TRY(current_device_checked(&dev));
  int* status = nullptr;
  MALA_TRY(device_setup(dev, &status));
  if (cudaDeviceSynchronize() != cudaSuccess) return MALA_ERR_CUDA;
  int v = 0;
  if (cudaMemcpy(&v, status, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return MALA_ERR_CUDA;
  *code_out = v;
  if (clear && v != 0) {
    const int zero = 0;
    if (cudaMemcpy(status, &zero, sizeof(int), cudaMemcpyHostToDevice) != cudaSuccess) return MALA_ERR_CUDA;
  }
  return MALA_OK;
}

int mala_test_expire_wait(long long limit_cycles, void* cuda_stream) {
  if (limit_cycles <= 0 || limit_cycles > 100000000LL) return MALA_ERR_INVALID_ARG;
  int dev = 0;
  MALA_TRY(current_device_checked(&dev));
  int* status = nullptr;
  MALA_TRY(device_setup(dev, &status));
  expire_wait_kernel<<<1, 32, 0, (cudaStream_t)cuda_stream>>>(status, limit_cycles);
  return cudaGetLastError() == cudaSuccess ? MALA_OK : MALA_ERR_CUDA;
}

// Lengths of a call with N queries and Nk keys: causal needs the queries to be the last N positions of the Nk.
static int check_lengths(int N, int Nk, int causal) {
  if (N <= 0 || Nk <= 0) return MALA_ERR_INVALID_ARG;
  if (causal && Nk < N) return MALA_ERR_UNSUPPORTED;
  return MALA_OK;
}

// Keys and values in pages for the forward: k, v are [num_pages, page_size, Hkv, d].
struct FwdPaging {
  const int32_t* block_table;
  const int32_t* seqlens_k;
  int num_pages, page_size, max_pages_per_seq;
};

// cu != null: B packed sequences in [1, total, H, d] tensors, N = Nk = the longest one.
static int fwd_impl(mala_tin q, mala_tin k, mala_tin v, mala_tout o, float* lse, const mala_stats* st, int B, int Hq,
                    int Hkv, int N, int Nk, int d, int causal, float scale, float tau, void* cuda_stream,
                    const int32_t* cu = nullptr, int total = 0, int num_splits = 1, void* ws = nullptr,
                    size_t ws_bytes = 0, const int32_t* cu_k = nullptr, int total_k = 0,
                    const FwdPaging* pg = nullptr) {
  if (num_splits < 1) return MALA_ERR_INVALID_ARG;
  if (num_splits > 1) {
    if (cu || num_splits > 65535 || (long long)B * num_splits > 65535) return MALA_ERR_UNSUPPORTED;
    if (!ws) return MALA_ERR_INVALID_ARG;
    if ((((uintptr_t)ws) & 255) != 0) return MALA_ERR_MISALIGNED;
    if (B > 0 && Hq > 0 && N > 0 && head_size_ok(d, 256) &&
        ws_bytes < fwd_split_workspace_bytes(B, Hq, N, padded_head_size(d), num_splits))
      return MALA_ERR_WORKSPACE_TOO_SMALL;
  }
  MALA_TRY(check_common(B, Hq, Hkv, N, d, scale, tau, 256));
  MALA_TRY(check_lengths(N, Nk, causal));
  if (!lse) return MALA_ERR_INVALID_ARG;
  const int Bt = cu ? 1 : B, Nt = cu ? total : N, Nkt = cu ? (cu_k ? total_k : total) : Nk;   // extents of the tensors
  MALA_TRY(check_view(q.p, q.sb, q.sn, q.sh, Bt, Nt, Hq));
  MALA_TRY(check_view(k.p, k.sb, k.sn, k.sh, pg ? pg->num_pages : Bt, pg ? pg->page_size : Nkt, Hkv));
  MALA_TRY(check_view(v.p, v.sb, v.sn, v.sh, pg ? pg->num_pages : Bt, pg ? pg->page_size : Nkt, Hkv));
  MALA_TRY(check_view(o.p, o.sb, o.sn, o.sh, Bt, Nt, Hq));
  int dev = 0;
  MALA_TRY(current_device_checked(&dev));
  int* status = nullptr;
  MALA_TRY(device_setup(dev, &status));
  cudaStream_t stream = (cudaStream_t)cuda_stream;

  CUtensorMap tq, tk, tv;
  const int box_rows = (pg && pg->page_size < 128) ? pg->page_size : 128;   // pages smaller than a tile: one copy per page
  if (!make_tensor_map_bnhd(&tq, q.p, Bt, Nt, Hq, d, q.sb, q.sn, q.sh, 128) ||
      !make_tensor_map_bnhd(&tk, k.p, pg ? pg->num_pages : Bt, pg ? pg->page_size : Nkt, Hkv, d, k.sb, k.sn, k.sh, box_rows) ||
      !make_tensor_map_bnhd(&tv, v.p, pg ? pg->num_pages : Bt, pg ? pg->page_size : Nkt, Hkv, d, v.sb, v.sn, v.sh, box_rows))
    return MALA_ERR_TENSOR_MAP;

  const int D = padded_head_size(d);
  FwdParams p;
  p.d = d;
  p.cu = cu; p.total = total; p.cu_k = cu_k;
  p.block_table = pg ? pg->block_table : nullptr;
  p.seqlens_k = pg ? pg->seqlens_k : nullptr;
  p.bt_stride = pg ? pg->max_pages_per_seq : 0;
  p.tpp = (pg && pg->page_size >= 128) ? pg->page_size / 128 : 1;
  p.ppt = 128 / box_rows; p.prows = box_rows;
  p.num_splits = num_splits;
  p.tps = ((Nk + 127) / 128 + num_splits - 1) / num_splits;
  p.o_part = num_splits > 1 ? (float*)ws : nullptr;
  p.lse_part = num_splits > 1
                   ? (float*)((uint8_t*)ws + (((size_t)B * Hq * num_splits * N * D * sizeof(float) + 255) & ~(size_t)255))
                   : nullptr;
  p.o = (__nv_bfloat16*)o.p; p.o_sb = o.sb; p.o_sn = o.sn; p.o_sh = o.sh;
  p.lse = lse;
  p.retained = st ? st->retained_per_block : nullptr;
  p.bitmask = st ? st->tile_bitmask : nullptr;
  p.totals = st ? (unsigned long long*)st->totals : nullptr;
  p.status = status;
  p.B = B; p.Hq = Hq; p.Hkv = Hkv; p.N = N; p.causal = causal ? 1 : 0;
  p.Nk = Nk; p.Tk = (Nk + 127) / 128; p.words = (p.Tk + 31) / 32;
  p.koff = causal ? (Nk - N) / 128 : 0;
  p.qshift = causal ? (Nk - N) % 128 : 0;        // the query blocks follow the key positions
  p.Tr = (N + p.qshift + 127) / 128;
  if (cu_k || pg) {   // per sequence on the device; the grid and the telemetry are laid out for the longest ones
    p.koff = 0; p.qshift = 0;
    p.Tr = (N + 127 + 127) / 128;
  }
  p.scale_log2 = scale * kLog2e;
  p.log2_tau = tau > 0.f ? log2f(tau) : -INFINITY;
  if (p.bitmask) {
    if (cudaMemsetAsync(p.bitmask, 0, (size_t)B * Hq * p.Tr * p.words * sizeof(uint32_t), stream) != cudaSuccess)
      return MALA_ERR_CUDA;
  }
  if (num_splits > 1 && p.retained &&   // (the ranges add to it)
      cudaMemsetAsync(p.retained, 0, (size_t)B * Hq * p.Tr * sizeof(uint32_t), stream) != cudaSuccess)
    return MALA_ERR_CUDA;
  const bool dense = (tau == 0.f);
  int rc;
  if (D == 256) rc = dense ? launch_fwd<256, true>(tq, tk, tv, p, stream) : launch_fwd<256, false>(tq, tk, tv, p, stream);
  else if (D == 128) rc = dense ? launch_fwd<128, true>(tq, tk, tv, p, stream) : launch_fwd<128, false>(tq, tk, tv, p, stream);
  else rc = dense ? launch_fwd<64, true>(tq, tk, tv, p, stream) : launch_fwd<64, false>(tq, tk, tv, p, stream);
  if (rc != MALA_OK || num_splits == 1) return rc;
  const unsigned rows = (unsigned)((long long)B * Hq * N);
  if (D == 256)
    fwd_merge_splits_kernel<256><<<rows, 256, 0, stream>>>(p.o_part, p.lse_part, p.o, p.o_sb, p.o_sn, p.o_sh, lse, Hq, N,
                                                           num_splits, p.tps, p.Tk, p.koff, p.qshift, p.causal, d);
  else if (D == 128)
    fwd_merge_splits_kernel<128><<<rows, 128, 0, stream>>>(p.o_part, p.lse_part, p.o, p.o_sb, p.o_sn, p.o_sh, lse, Hq, N,
                                                           num_splits, p.tps, p.Tk, p.koff, p.qshift, p.causal, d);
  else
    fwd_merge_splits_kernel<64><<<rows, 64, 0, stream>>>(p.o_part, p.lse_part, p.o, p.o_sb, p.o_sn, p.o_sh, lse, Hq, N,
                                                         num_splits, p.tps, p.Tk, p.koff, p.qshift, p.causal, d);
  return cudaGetLastError() == cudaSuccess ? MALA_OK : MALA_ERR_CUDA;
}

int mala_fwd(mala_tin q, mala_tin k, mala_tin v, mala_tout o, float* lse, const mala_stats* st, int B, int Hq,
             int Hkv, int N, int d, int causal, float scale, float tau, void* ws, size_t ws_bytes,
             void* cuda_stream) {
  ApiScope scope("mala_fwd", cuda_stream);
  (void)ws; (void)ws_bytes;
  return scope.finish(fwd_impl(q, k, v, o, lse, st, B, Hq, Hkv, N, N, d, causal, scale, tau, cuda_stream));
}

int mala_fwd_chunk(mala_tin q, mala_tin k, mala_tin v, mala_tout o, float* lse, const mala_stats* st, int B, int Hq,
                   int Hkv, int Nq, int Nk, int d, int causal, float scale, float tau, void* ws, size_t ws_bytes,
                   void* cuda_stream) {
  ApiScope scope("mala_fwd_chunk", cuda_stream);
  (void)ws; (void)ws_bytes;
  return scope.finish(fwd_impl(q, k, v, o, lse, st, B, Hq, Hkv, Nq, Nk, d, causal, scale, tau, cuda_stream));
}

static int bwd_impl(mala_tin q, mala_tin k, mala_tin v, mala_tin o, mala_tin dout, const float* lse, mala_tout dq,
                    mala_tout dk, mala_tout dv, const mala_stats* st, int B0, int Hq, int Hkv, int N0, int Nk0, int d,
                    int causal, float scale, float tau, void* ws, size_t ws_bytes, void* cuda_stream,
                    const int32_t* cu = nullptr, int total = 0, const int32_t* cu_k = nullptr, int total_k = 0) {
  MALA_TRY(check_common(B0, Hq, Hkv, N0, d, scale, tau));
  MALA_TRY(check_lengths(N0, Nk0, causal));
  if (!lse || !ws) return MALA_ERR_INVALID_ARG;
  // extents of the tensors and of the workspace (packed sequences: one batch entry of `total` rows)
  const int B = cu ? 1 : B0, N = cu ? total : N0, Nk = cu ? (cu_k ? total_k : total) : Nk0;
  MALA_TRY(check_view(q.p, q.sb, q.sn, q.sh, B, N, Hq));
  MALA_TRY(check_view(k.p, k.sb, k.sn, k.sh, B, Nk, Hkv));
  MALA_TRY(check_view(v.p, v.sb, v.sn, v.sh, B, Nk, Hkv));
  MALA_TRY(check_view(o.p, o.sb, o.sn, o.sh, B, N, Hq));
  MALA_TRY(check_view(dout.p, dout.sb, dout.sn, dout.sh, B, N, Hq));
  MALA_TRY(check_view(dq.p, dq.sb, dq.sn, dq.sh, B, N, Hq));
  MALA_TRY(check_view(dk.p, dk.sb, dk.sn, dk.sh, B, Nk, Hkv));
  MALA_TRY(check_view(dv.p, dv.sb, dv.sn, dv.sh, B, Nk, Hkv));
  if ((((uintptr_t)ws) & 255) != 0) return MALA_ERR_MISALIGNED;
  // (a causal chunk that starts inside a tile: the query blocks follow the positions, (Nk - N) % 128 more rows)
  const int pad_rows = (causal && !cu) ? (Nk0 - N0) % 128 : 0;
  if (ws_bytes < bwd_base_workspace_bytes(B, Hq, cu ? total + (cu_k ? 384 : 128) * B0 : N + pad_rows, padded_head_size(d)))
    return MALA_ERR_WORKSPACE_TOO_SMALL;
  int dev = 0;
  MALA_TRY(current_device_checked(&dev));
  int* status = nullptr;
  MALA_TRY(device_setup(dev, &status));
  return bwd_launch(q, k, v, o, dout, lse, dq, dk, dv, st, B0, Hq, Hkv, N0, Nk0, d, causal ? 1 : 0, scale, tau, ws,
                    ws_bytes, status, (cudaStream_t)cuda_stream, cu, total, cu_k, total_k);
}

int mala_fwd_chunk_split(mala_tin q, mala_tin k, mala_tin v, mala_tout o, float* lse, const mala_stats* st, int B,
                         int Hq, int Hkv, int Nq, int Nk, int d, int causal, float scale, float tau, int num_splits,
                         void* ws, size_t ws_bytes, void* cuda_stream) {
  ApiScope scope("mala_fwd_chunk_split", cuda_stream);
  return scope.finish(fwd_impl(q, k, v, o, lse, st, B, Hq, Hkv, Nq, Nk, d, causal, scale, tau, cuda_stream, nullptr, 0, num_splits,
                  ws, ws_bytes));
}

int mala_bwd(mala_tin q, mala_tin k, mala_tin v, mala_tin o, mala_tin dout, const float* lse, mala_tout dq,
             mala_tout dk, mala_tout dv, const mala_stats* st, int B, int Hq, int Hkv, int N, int d, int causal,
             float scale, float tau, void* ws, size_t ws_bytes, void* cuda_stream) {
  ApiScope scope("mala_bwd", cuda_stream);
  return scope.finish(bwd_impl(q, k, v, o, dout, lse, dq, dk, dv, st, B, Hq, Hkv, N, N, d, causal, scale, tau, ws, ws_bytes,
                  cuda_stream));
}

int mala_bwd_chunk(mala_tin q, mala_tin k, mala_tin v, mala_tin o, mala_tin dout, const float* lse, mala_tout dq,
                   mala_tout dk, mala_tout dv, const mala_stats* st, int B, int Hq, int Hkv, int Nq, int Nk, int d,
                   int causal, float scale, float tau, void* ws, size_t ws_bytes, void* cuda_stream) {
  ApiScope scope("mala_bwd_chunk", cuda_stream);
  return scope.finish(bwd_impl(q, k, v, o, dout, lse, dq, dk, dv, st, B, Hq, Hkv, Nq, Nk, d, causal, scale, tau, ws, ws_bytes,
                  cuda_stream));
}

static int check_packed(const int32_t* cu_seqlens, int B, int total, int max_seqlen) {
  if (!cu_seqlens || B <= 0 || total <= 0 || max_seqlen <= 0) return MALA_ERR_INVALID_ARG;
  if ((((uintptr_t)cu_seqlens) & 3) != 0) return MALA_ERR_MISALIGNED;
  if (max_seqlen > total || (long long)total + 128LL * B > 0x7fffffffLL) return MALA_ERR_UNSUPPORTED;
  return MALA_OK;
}

int mala_fwd_varlen(mala_tin q, mala_tin k, mala_tin v, const int32_t* cu_seqlens, mala_tout o, float* lse,
                    const mala_stats* st, int B, int Hq, int Hkv, int total, int max_seqlen, int d, int causal,
                    float scale, float tau, void* ws, size_t ws_bytes, void* cuda_stream) {
  ApiScope scope("mala_fwd_varlen", cuda_stream);
  (void)ws; (void)ws_bytes;
  MALA_TRY(check_packed(cu_seqlens, B, total, max_seqlen));
  return scope.finish(fwd_impl(q, k, v, o, lse, st, B, Hq, Hkv, max_seqlen, max_seqlen, d, causal, scale, tau, cuda_stream,
                  cu_seqlens, total));
}

int mala_fwd_varlen_prefix(mala_tin q, mala_tin k, mala_tin v, const int32_t* cu_seqlens_q, const int32_t* cu_seqlens_k,
                           mala_tout o, float* lse, const mala_stats* st, int B, int Hq, int Hkv, int total_q,
                           int total_k, int max_seqlen_q, int max_seqlen_k, int d, int causal, float scale, float tau,
                           void* ws, size_t ws_bytes, void* cuda_stream) {
  ApiScope scope("mala_fwd_varlen_prefix", cuda_stream);
  (void)ws; (void)ws_bytes;
  MALA_TRY(check_packed(cu_seqlens_q, B, total_q, max_seqlen_q));
  MALA_TRY(check_packed(cu_seqlens_k, B, total_k, max_seqlen_k));
  if (causal && max_seqlen_k < max_seqlen_q) return MALA_ERR_UNSUPPORTED;
  return scope.finish(fwd_impl(q, k, v, o, lse, st, B, Hq, Hkv, max_seqlen_q, max_seqlen_k, d, causal, scale, tau, cuda_stream,
                  cu_seqlens_q, total_q, 1, nullptr, 0, cu_seqlens_k, total_k));
}

int mala_fwd_paged(mala_tin q, mala_tin kpages, mala_tin vpages, const int32_t* cu_seqlens_q, const int32_t* block_table,
                   const int32_t* seqlens_k, mala_tout o, float* lse, const mala_stats* st, int B, int Hq, int Hkv,
                   int total_q, int max_seqlen_q, int num_pages, int page_size, int max_pages_per_seq, int d, int causal,
                   float scale, float tau, void* ws, size_t ws_bytes, void* cuda_stream) {
  ApiScope scope("mala_fwd_paged", cuda_stream);
  (void)ws; (void)ws_bytes;
  MALA_TRY(check_packed(cu_seqlens_q, B, total_q, max_seqlen_q));
  if (!block_table || !seqlens_k || num_pages <= 0 || page_size <= 0 || max_pages_per_seq <= 0) return MALA_ERR_INVALID_ARG;
  if ((((uintptr_t)block_table) & 3) != 0 || (((uintptr_t)seqlens_k) & 3) != 0) return MALA_ERR_MISALIGNED;
  // pages of whole tiles, or 8, 16, 32 or 64 keys (a tile is then put together from several pages)
  if (page_size < 8 || (page_size % 128 != 0 && 128 % page_size != 0) ||
      (long long)max_pages_per_seq * page_size > 0x7fffffffLL)
    return MALA_ERR_UNSUPPORTED;
  const int max_k = max_pages_per_seq * page_size;
  if (causal && max_k < max_seqlen_q) return MALA_ERR_UNSUPPORTED;
  FwdPaging pg;
  pg.block_table = block_table; pg.seqlens_k = seqlens_k; pg.num_pages = num_pages; pg.page_size = page_size;
  pg.max_pages_per_seq = max_pages_per_seq;
  return scope.finish(fwd_impl(q, kpages, vpages, o, lse, st, B, Hq, Hkv, max_seqlen_q, max_k, d, causal, scale, tau, cuda_stream,
                  cu_seqlens_q, total_q, 1, nullptr, 0, nullptr, 0, &pg));
}

int mala_bwd_varlen(mala_tin q, mala_tin k, mala_tin v, mala_tin o, mala_tin dout, const float* lse,
                    const int32_t* cu_seqlens, mala_tout dq, mala_tout dk, mala_tout dv, const mala_stats* st, int B,
                    int Hq, int Hkv, int total, int max_seqlen, int d, int causal, float scale, float tau, void* ws,
                    size_t ws_bytes, void* cuda_stream) {
  ApiScope scope("mala_bwd_varlen", cuda_stream);
  MALA_TRY(check_packed(cu_seqlens, B, total, max_seqlen));
  return scope.finish(bwd_impl(q, k, v, o, dout, lse, dq, dk, dv, st, B, Hq, Hkv, max_seqlen, max_seqlen, d, causal, scale, tau,
                  ws, ws_bytes, cuda_stream, cu_seqlens, total));
}

int mala_bwd_varlen_prefix(mala_tin q, mala_tin k, mala_tin v, mala_tin o, mala_tin dout, const float* lse,
                           const int32_t* cu_seqlens_q, const int32_t* cu_seqlens_k, mala_tout dq, mala_tout dk,
                           mala_tout dv, const mala_stats* st, int B, int Hq, int Hkv, int total_q, int total_k,
                           int max_seqlen_q, int max_seqlen_k, int d, int causal, float scale, float tau, void* ws,
                           size_t ws_bytes, void* cuda_stream) {
  ApiScope scope("mala_bwd_varlen_prefix", cuda_stream);
  MALA_TRY(check_packed(cu_seqlens_q, B, total_q, max_seqlen_q));
  MALA_TRY(check_packed(cu_seqlens_k, B, total_k, max_seqlen_k));
  if ((long long)total_q + 384LL * B > 0x7fffffffLL) return MALA_ERR_UNSUPPORTED;
  if (causal && max_seqlen_k < max_seqlen_q) return MALA_ERR_UNSUPPORTED;
  return scope.finish(bwd_impl(q, k, v, o, dout, lse, dq, dk, dv, st, B, Hq, Hkv, max_seqlen_q, max_seqlen_k, d, causal, scale, tau,
                  ws, ws_bytes, cuda_stream, cu_seqlens_q, total_q, cu_seqlens_k, total_k));
}

int mala_decode(mala_tin q, mala_tin kcache, mala_tin vcache, mala_tout o, float* lse_opt, const mala_stats* st,
                int B, int Hq, int Hkv, int Nk, int d, float scale, float tau, int num_splits, void* ws,
                size_t ws_bytes, void* cuda_stream) {
  ApiScope scope("mala_decode", cuda_stream);
  MALA_TRY(check_common(B, Hq, Hkv, Nk, d, scale, tau, 256));
  if (num_splits <= 0 || !ws) return MALA_ERR_INVALID_ARG;
  if (Hq / Hkv > 16 || num_splits > 65535) return MALA_ERR_UNSUPPORTED;
  MALA_TRY(check_view(q.p, q.sb, 8, q.sh, B, 1, Hq));
  MALA_TRY(check_view(kcache.p, kcache.sb, kcache.sn, kcache.sh, B, Nk, Hkv));
  MALA_TRY(check_view(vcache.p, vcache.sb, vcache.sn, vcache.sh, B, Nk, Hkv));
  MALA_TRY(check_view(o.p, o.sb, 8, o.sh, B, 1, Hq));
  if ((((uintptr_t)ws) & 255) != 0) return MALA_ERR_MISALIGNED;
  if (ws_bytes < decode_workspace_bytes(B, Hq, padded_head_size(d), num_splits)) return MALA_ERR_WORKSPACE_TOO_SMALL;
  int dev = 0;
  MALA_TRY(current_device_checked(&dev));
  int* status = nullptr;
  MALA_TRY(device_setup(dev, &status));
  return scope.finish(decode_launch(q, kcache, vcache, o, lse_opt, st, B, Hq, Hkv, Nk, d, scale, tau, num_splits, ws, status,
                       (cudaStream_t)cuda_stream));
}

int mala_decode_fp8(mala_tin q, mala_tin kcache8, mala_tin vcache8, const float* kscale, const float* vscale,
                    mala_tout o, float* lse_opt, const mala_stats* st, int B, int Hq, int Hkv, int Nk, int d, float scale,
                    float tau, int num_splits, void* ws, size_t ws_bytes, void* cuda_stream) {
  ApiScope scope("mala_decode_fp8", cuda_stream);
  MALA_TRY(check_common(B, Hq, Hkv, Nk, d, scale, tau));
  if (num_splits <= 0 || !ws || !kscale || !vscale) return MALA_ERR_INVALID_ARG;
  if (Hq / Hkv > 8 || d % 16 != 0 || num_splits > 65535) return MALA_ERR_UNSUPPORTED;
  MALA_TRY(check_view(q.p, q.sb, 8, q.sh, B, 1, Hq));
  // 8-bit views: strides in elements = bytes, multiples of 16
  auto check8 = [&](const mala_tin& t) -> int {
    if (!t.p) return MALA_ERR_INVALID_ARG;
    if (!aligned16(t.p)) return MALA_ERR_MISALIGNED;
    if ((B > 1 && t.sb % 16) || (Nk > 1 && t.sn % 16) || (Hkv > 1 && t.sh % 16)) return MALA_ERR_MISALIGNED;
    if ((B > 1 && t.sb <= 0) || (Nk > 1 && t.sn <= 0) || (Hkv > 1 && t.sh <= 0)) return MALA_ERR_INVALID_ARG;
    return MALA_OK;
  };
  MALA_TRY(check8(kcache8));
  MALA_TRY(check8(vcache8));
  MALA_TRY(check_view(o.p, o.sb, 8, o.sh, B, 1, Hq));
  if ((((uintptr_t)ws) & 255) != 0 || (((uintptr_t)kscale) & 3) != 0 || (((uintptr_t)vscale) & 3) != 0) return MALA_ERR_MISALIGNED;
  if (ws_bytes < decode_workspace_bytes(B, Hq, 128, num_splits)) return MALA_ERR_WORKSPACE_TOO_SMALL;
  int dev = 0;
  MALA_TRY(current_device_checked(&dev));
  int* status = nullptr;
  MALA_TRY(device_setup(dev, &status));
  return scope.finish(decode_fp8_launch(q, kcache8, vcache8, kscale, vscale, o, lse_opt, st, B, Hq, Hkv, Nk, d, scale, tau, num_splits,
                           ws, status, (cudaStream_t)cuda_stream));
}

int mala_decode_fp8_multi(mala_tin q, mala_tin kcache8, mala_tin vcache8, const float* kscale, const float* vscale,
                          mala_tout o, float* lse_opt, const mala_stats* st, int B, int Hq, int Hkv, int Nk, int Sq, int d,
                          float scale, float tau, int num_splits, void* ws, size_t ws_bytes, void* cuda_stream) {
  ApiScope scope("mala_decode_fp8_multi", cuda_stream);
  MALA_TRY(check_common(B, Hq, Hkv, Nk, d, scale, tau));
  if (num_splits <= 0 || Sq <= 0 || !ws || !kscale || !vscale) return MALA_ERR_INVALID_ARG;
  if ((Hq / Hkv) * Sq > 8 || Sq > Nk || d % 16 != 0 || num_splits > 65535) return MALA_ERR_UNSUPPORTED;
  MALA_TRY(check_view(q.p, q.sb, q.sn, q.sh, B, Sq, Hq));
  auto check8 = [&](const mala_tin& t) -> int {   // 8-bit views: strides in elements = bytes, multiples of 16
    if (!t.p) return MALA_ERR_INVALID_ARG;
    if (!aligned16(t.p)) return MALA_ERR_MISALIGNED;
    if ((B > 1 && t.sb % 16) || (Nk > 1 && t.sn % 16) || (Hkv > 1 && t.sh % 16)) return MALA_ERR_MISALIGNED;
    if ((B > 1 && t.sb <= 0) || (Nk > 1 && t.sn <= 0) || (Hkv > 1 && t.sh <= 0)) return MALA_ERR_INVALID_ARG;
    return MALA_OK;
  };
  MALA_TRY(check8(kcache8));
  MALA_TRY(check8(vcache8));
  MALA_TRY(check_view(o.p, o.sb, o.sn, o.sh, B, Sq, Hq));
  if ((((uintptr_t)ws) & 255) != 0 || (((uintptr_t)kscale) & 3) != 0 || (((uintptr_t)vscale) & 3) != 0) return MALA_ERR_MISALIGNED;
  if (ws_bytes < decode_workspace_bytes(B * Sq, Hq, 128, num_splits)) return MALA_ERR_WORKSPACE_TOO_SMALL;
  int dev = 0;
  MALA_TRY(current_device_checked(&dev));
  int* status = nullptr;
  MALA_TRY(device_setup(dev, &status));
  return scope.finish(decode_fp8_launch(q, kcache8, vcache8, kscale, vscale, o, lse_opt, st, B, Hq, Hkv, Nk, d, scale, tau,
                                        num_splits, ws, status, (cudaStream_t)cuda_stream, nullptr, Sq));
}

int mala_decode_fp8_paged(mala_tin q, mala_tin kpages8, mala_tin vpages8, const float* kscale, const float* vscale,
                          const int32_t* block_table, const int32_t* seqlens, mala_tout o, float* lse_opt,
                          const mala_stats* st, int B, int Hq, int Hkv, int num_pages, int page_size,
                          int max_pages_per_seq, int d, float scale, float tau, int num_splits, void* ws, size_t ws_bytes,
                          void* cuda_stream) {
  ApiScope scope("mala_decode_fp8_paged", cuda_stream);
  if (num_pages <= 0 || page_size <= 0 || max_pages_per_seq <= 0 || !block_table) return MALA_ERR_INVALID_ARG;
  // pages of whole tiles, or of 16, 32 or 64 keys (a tile is then put together from several pages)
  if (!(page_size % 128 == 0 || page_size == 16 || page_size == 32 || page_size == 64) ||
      (long long)max_pages_per_seq * page_size > 0x7fffffffLL ||
      (long long)num_pages * Hkv * (page_size < 128 ? 1 : page_size / 128) > 0x7fffffffLL)
    return MALA_ERR_UNSUPPORTED;
  const int Nk = max_pages_per_seq * page_size;   // the longest cache a sequence can hold
  MALA_TRY(check_common(B, Hq, Hkv, Nk, d, scale, tau));
  if (num_splits <= 0 || !ws || !kscale || !vscale) return MALA_ERR_INVALID_ARG;
  if (Hq / Hkv > 8 || d % 16 != 0 || num_splits > 65535) return MALA_ERR_UNSUPPORTED;
  if ((((uintptr_t)block_table) & 3) != 0 || (((uintptr_t)seqlens) & 3) != 0) return MALA_ERR_MISALIGNED;
  MALA_TRY(check_view(q.p, q.sb, 8, q.sh, B, 1, Hq));
  auto check8 = [&](const mala_tin& t) -> int {   // 8-bit views: strides in elements = bytes, multiples of 16
    if (!t.p) return MALA_ERR_INVALID_ARG;
    if (!aligned16(t.p)) return MALA_ERR_MISALIGNED;
    if ((num_pages > 1 && t.sb % 16) || (page_size > 1 && t.sn % 16) || (Hkv > 1 && t.sh % 16)) return MALA_ERR_MISALIGNED;
    if ((num_pages > 1 && t.sb <= 0) || (page_size > 1 && t.sn <= 0) || (Hkv > 1 && t.sh <= 0)) return MALA_ERR_INVALID_ARG;
    return MALA_OK;
  };
  MALA_TRY(check8(kpages8));
  MALA_TRY(check8(vpages8));
  MALA_TRY(check_view(o.p, o.sb, 8, o.sh, B, 1, Hq));
  if ((((uintptr_t)ws) & 255) != 0 || (((uintptr_t)kscale) & 3) != 0 || (((uintptr_t)vscale) & 3) != 0) return MALA_ERR_MISALIGNED;
  if (ws_bytes < decode_workspace_bytes(B, Hq, 128, num_splits)) return MALA_ERR_WORKSPACE_TOO_SMALL;
  int dev = 0;
  MALA_TRY(current_device_checked(&dev));
  int* status = nullptr;
  MALA_TRY(device_setup(dev, &status));
  DecPaging pg;
  pg.block_table = block_table; pg.seqlens = seqlens; pg.bt_stride = max_pages_per_seq; pg.page_size = page_size;
  pg.num_pages = num_pages;
  return scope.finish(decode_fp8_launch(q, kpages8, vpages8, kscale, vscale, o, lse_opt, st, B, Hq, Hkv, Nk, d, scale, tau,
                           num_splits, ws, status, (cudaStream_t)cuda_stream, &pg));
}

int mala_decode_multi(mala_tin q, mala_tin kcache, mala_tin vcache, mala_tout o, float* lse_opt, const mala_stats* st,
                      int B, int Hq, int Hkv, int Nk, int Sq, int d, float scale, float tau, int num_splits, void* ws,
                      size_t ws_bytes, void* cuda_stream) {
  ApiScope scope("mala_decode_multi", cuda_stream);
  MALA_TRY(check_common(B, Hq, Hkv, Nk, d, scale, tau, 256));
  if (num_splits <= 0 || Sq <= 0 || !ws) return MALA_ERR_INVALID_ARG;
  if ((Hq / Hkv) * Sq > 16 || Sq > Nk || num_splits > 65535) return MALA_ERR_UNSUPPORTED;
  MALA_TRY(check_view(q.p, q.sb, q.sn, q.sh, B, Sq, Hq));
  MALA_TRY(check_view(kcache.p, kcache.sb, kcache.sn, kcache.sh, B, Nk, Hkv));
  MALA_TRY(check_view(vcache.p, vcache.sb, vcache.sn, vcache.sh, B, Nk, Hkv));
  MALA_TRY(check_view(o.p, o.sb, o.sn, o.sh, B, Sq, Hq));
  if ((((uintptr_t)ws) & 255) != 0) return MALA_ERR_MISALIGNED;
  if (ws_bytes < decode_workspace_bytes(B * Sq, Hq, padded_head_size(d), num_splits)) return MALA_ERR_WORKSPACE_TOO_SMALL;
  int dev = 0;
  MALA_TRY(current_device_checked(&dev));
  int* status = nullptr;
  MALA_TRY(device_setup(dev, &status));
  return scope.finish(decode_launch(q, kcache, vcache, o, lse_opt, st, B, Hq, Hkv, Nk, d, scale, tau, num_splits, ws, status,
                       (cudaStream_t)cuda_stream, nullptr, Sq));
}

int mala_decode_paged(mala_tin q, mala_tin kpages, mala_tin vpages, const int32_t* block_table,
                      const int32_t* seqlens, mala_tout o, float* lse_opt, const mala_stats* st, int B, int Hq,
                      int Hkv, int num_pages, int page_size, int max_pages_per_seq, int Sq, int d, float scale,
                      float tau, int num_splits, void* ws, size_t ws_bytes, void* cuda_stream) {
  ApiScope scope("mala_decode_paged", cuda_stream);
  if (num_pages <= 0 || page_size <= 0 || max_pages_per_seq <= 0 || Sq <= 0 || !block_table) return MALA_ERR_INVALID_ARG;
  if (page_size < 8 || (page_size % 128 != 0 && 128 % page_size != 0) ||
      (long long)max_pages_per_seq * page_size > 0x7fffffffLL)
    return MALA_ERR_UNSUPPORTED;
  const int Nk = max_pages_per_seq * page_size;   // the longest cache a sequence can hold
  MALA_TRY(check_common(B, Hq, Hkv, Nk, d, scale, tau, 256));
  if (num_splits <= 0 || !ws) return MALA_ERR_INVALID_ARG;
  if ((Hq / Hkv) * Sq > 16 || num_splits > 65535) return MALA_ERR_UNSUPPORTED;
  if ((((uintptr_t)block_table) & 3) != 0 || (((uintptr_t)seqlens) & 3) != 0) return MALA_ERR_MISALIGNED;
  MALA_TRY(check_view(q.p, q.sb, Sq > 1 ? q.sn : 8, q.sh, B, Sq, Hq));
  MALA_TRY(check_view(kpages.p, kpages.sb, kpages.sn, kpages.sh, num_pages, page_size, Hkv));
  MALA_TRY(check_view(vpages.p, vpages.sb, vpages.sn, vpages.sh, num_pages, page_size, Hkv));
  MALA_TRY(check_view(o.p, o.sb, Sq > 1 ? o.sn : 8, o.sh, B, Sq, Hq));
  if ((((uintptr_t)ws) & 255) != 0) return MALA_ERR_MISALIGNED;
  if (ws_bytes < decode_workspace_bytes(B * Sq, Hq, padded_head_size(d), num_splits)) return MALA_ERR_WORKSPACE_TOO_SMALL;
  int dev = 0;
  MALA_TRY(current_device_checked(&dev));
  int* status = nullptr;
  MALA_TRY(device_setup(dev, &status));
  DecPaging pg;
  pg.block_table = block_table; pg.seqlens = seqlens; pg.bt_stride = max_pages_per_seq; pg.page_size = page_size;
  pg.num_pages = num_pages;
  return scope.finish(decode_launch(q, kpages, vpages, o, lse_opt, st, B, Hq, Hkv, Nk, d, scale, tau, num_splits, ws, status,
                       (cudaStream_t)cuda_stream, &pg, Sq));
}

int mala_decode_static(mala_tin q, mala_tin kcache, mala_tin vcache, mala_tout o, float* lse_opt, int B, int Hq,
                       int Hkv, int Nk, int d, float scale, float tau, int num_splits, void* cuda_stream) {
  ApiScope scope("mala_decode_static", cuda_stream);
  MALA_TRY(check_common(B, Hq, Hkv, Nk, d, scale, tau, 256));
  if (num_splits <= 0) return MALA_ERR_INVALID_ARG;
  if (Hq / Hkv > 16 || num_splits > 65535) return MALA_ERR_UNSUPPORTED;
  MALA_TRY(check_view(q.p, q.sb, 8, q.sh, B, 1, Hq));
  MALA_TRY(check_view(kcache.p, kcache.sb, kcache.sn, kcache.sh, B, Nk, Hkv));
  MALA_TRY(check_view(vcache.p, vcache.sb, vcache.sn, vcache.sh, B, Nk, Hkv));
  MALA_TRY(check_view(o.p, o.sb, 8, o.sh, B, 1, Hq));
  if (decode_workspace_bytes(B, Hq, padded_head_size(d), num_splits) > (size_t)MALA_STATIC_SCRATCH_BYTES)
    return MALA_ERR_STATIC_SCRATCH_EXCEEDED;
  int dev = 0;
  MALA_TRY(current_device_checked(&dev));
  int* status = nullptr;
  MALA_TRY(device_setup(dev, &status));
  unsigned char* scratch = nullptr;
  MALA_TRY(static_scratch_address(dev, &scratch));
  float* o_part = (float*)scratch;
  float* lse_part = (float*)(scratch + decode_align256((size_t)B * Hq * num_splits * padded_head_size(d) * sizeof(float)));
  // every (batch, head, split) entry of both arrays is written by the split kernel (empty splits
  // included) before the merge reads it, so nothing left over from an earlier call is ever read
  return scope.finish(decode_launch_with_scratch(q, kcache, vcache, o, lse_opt, nullptr, B, Hq, Hkv, Nk, d, scale, tau, num_splits,
                                    o_part, lse_part, status, (cudaStream_t)cuda_stream));
}

}  // extern "C"
