// A table-lookup mpGEMV entry point for callers that cannot allocate device memory.
//
// Some hosts of this library must not, or cannot, call cudaMalloc: code running inside a region
// where the allocator is frozen (a memory pool whose size was fixed at start-up, a real-time loop
// that forbids calls which may block or fail), plug-ins that are handed input and output buffers but
// no allocator, and processes whose device memory is already fully committed to model weights.
// bitnet_mpgemm needs a caller-supplied workspace whenever K is split across CTAs; this variant
// keeps that scratch in a fixed array inside the library's device image instead.
#include <mutex>

#include "common.cuh"

namespace bitnet {
namespace {

// Partial sums [T<=8][M] int32, one arrival counter per row, then the lookup tables of up to four
// token pairs (2 KB per 32-group tile), for M and K up to the stated limits.
constexpr int64_t kNoAllocMaxM = BITNET_NOALLOC_MAX_M;
constexpr int64_t kNoAllocMaxK = BITNET_NOALLOC_MAX_K;
constexpr int64_t kNoAllocMaxT = 8;
constexpr size_t kScratchBytes =
    (size_t)(kNoAllocMaxT + 1) * 4 * kNoAllocMaxM + 4 * (size_t)(kNoAllocMaxK / 64 + 2) * 2048;

static __device__ __align__(256) unsigned char g_noalloc_scratch[kScratchBytes];

// In host code `g_noalloc_scratch` is only a handle for the runtime, not an address the GPU can use;
// the device address is looked up once per device, with that device current.
int scratch_address(void** out) {
  static void* addr[64] = {nullptr};
  static std::mutex mu;
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return note_cuda_error(e);
  if (dev < 0 || dev >= 64) return BITNET_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lock(mu);
  if (!addr[dev]) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
    if (e != cudaSuccess) return note_cuda_error(e);
    addr[dev] = p;
  }
  *out = addr[dev];
  return BITNET_OK;
}

}  // namespace
}  // namespace bitnet

using namespace bitnet;

extern "C" int bitnet_mpgemv_tl_noalloc(bitnet_fmt_t fmt, const void* packed, float w_scale, int64_t M,
                                        int64_t K, int bk3, const int8_t* q, const float* act_scale,
                                        int64_t T, float* y, int32_t* acc_out, void* stream) {
  if (fmt != BITNET_FMT_TL1 && fmt != BITNET_FMT_TL2) return BITNET_ERR_INVALID_ARG;
  if (!packed || !q || !act_scale || !y || T < 1 || M < 1 || K < 1) return BITNET_ERR_INVALID_ARG;
  if (!aligned16(packed) || !aligned16(q) || !aligned16(y) || (acc_out && !aligned16(acc_out)))
    return BITNET_ERR_INVALID_ARG;
  if (M > kNoAllocMaxM || K > kNoAllocMaxK || T > kNoAllocMaxT) return BITNET_ERR_WORKSPACE;  // beyond the scratch
  TlGeom g;
  if (!tl_geom(fmt, M, K, bk3, &g)) return BITNET_ERR_UNSUPPORTED_SHAPE;
  void* scratch = nullptr;
  int rc = scratch_address(&scratch);
  if (rc != BITNET_OK) return rc;
  cudaStream_t st = (cudaStream_t)stream;
  const size_t need = gemv_tl_workspace_bytes(fmt, T, M, K);
  if (need > kScratchBytes) return BITNET_ERR_WORKSPACE;
  // The array keeps whatever the previous call left; partial sums and arrival counters must start at 0
  // (the tables behind them are rewritten in full by every call).
  cudaError_t e = cudaMemsetAsync(scratch, 0, (size_t)(T + 1) * 4 * (size_t)M, st);
  if (e != cudaSuccess) return note_cuda_error(e);
  return launch_gemv_tl(fmt, (const uint8_t*)packed, w_scale, M, K, g, q, act_scale, (int)T, y, acc_out, scratch,
                        kScratchBytes, st);
}
