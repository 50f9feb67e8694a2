// Shared host/device helpers of the bitnet_b200 library (internal).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "bitnet_b200.h"

namespace bitnet {

inline __host__ __device__ int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }

// Geometry of a TL blob (Sec. 3.1.2: block-fitting split ThreeK / TwoK; 32-row tiles).
struct TlGeom {
  int64_t three_k;      // columns coded as triples (TL2)
  int64_t two_k;        // columns coded as pairs (TL1)
  int64_t tiles3;       // 640-byte tiles per 32-row block
  int64_t tiles2;       // 512-byte tiles per 32-row block
  int64_t block_bytes;  // bytes per 32-row block
};

inline __host__ bool tl_geom(int fmt, int64_t M, int64_t K, int bk3, TlGeom* g) {
  if (M <= 0 || K <= 0 || (M % 32) != 0 || (K % 2) != 0) return false;
  if (bk3 == 0) bk3 = 96;
  if (bk3 < 0 || (bk3 % 96) != 0) return false;
  if (fmt == BITNET_FMT_TL2) {
    g->three_k = (K / bk3) * bk3;
    g->two_k = K - g->three_k;
  } else if (fmt == BITNET_FMT_TL1) {
    g->three_k = 0;
    g->two_k = K;
  } else {
    return false;
  }
  g->tiles3 = g->three_k / 96;
  g->tiles2 = ceil_div(g->two_k, 64);
  g->block_bytes = g->tiles3 * 640 + g->tiles2 * 512;
  return true;
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Records a failing CUDA call for bitnet_last_cuda_error(); returns the library status.
int note_cuda_error(cudaError_t e);
inline int check_launch() {
  cudaError_t e = cudaPeekAtLastError();
  return e == cudaSuccess ? BITNET_OK : note_cuda_error(cudaGetLastError());
}

// Device properties looked up once per device.
struct DevInfo {
  int sm_count;
  int max_smem_optin;
};
const DevInfo& dev_info();

// ---- kernel launchers (one per .cu file) ----------------------------------------------------
int launch_quant_act(const float* x, int64_t T, int64_t K, int per_tensor, int8_t* q, float* act_scale,
                     int32_t* act_sum, cudaStream_t st);
int launch_pack_i2s(const int8_t* w, int64_t M, int64_t K, uint8_t* packed, int* dev_status,
                    cudaStream_t st);
int launch_unpack_i2s(const uint8_t* packed, int64_t M, int64_t K, int8_t* w, int* dev_status,
                      cudaStream_t st);
int launch_pack_tl(int fmt, const int8_t* w, int64_t M, int64_t K, const TlGeom& g, uint8_t* packed,
                   int* dev_status, cudaStream_t st);
int launch_unpack_tl(int fmt, const uint8_t* packed, int64_t M, int64_t K, const TlGeom& g, int8_t* w,
                     int* dev_status, cudaStream_t st);

// Decode GEMV, T <= 8.
size_t gemv_i2s_workspace_bytes(int64_t T, int64_t M, int64_t K);
int launch_gemv_i2s(const uint8_t* packed, float w_scale, int64_t M, int64_t K, const int8_t* q,
                    const float* act_scale, int T, float* y, int32_t* acc_out, void* ws, size_t ws_bytes,
                    cudaStream_t st);
size_t gemv_tl_workspace_bytes(int fmt, int64_t T, int64_t M, int64_t K);
int launch_gemv_tl(int fmt, const uint8_t* packed, float w_scale, int64_t M, int64_t K, const TlGeom& g,
                   const int8_t* q, const float* act_scale, int T, float* y, int32_t* acc_out, void* ws,
                   size_t ws_bytes, cudaStream_t st);
int launch_tl_build_lut(int fmt, const int8_t* q_row, int64_t K, const TlGeom& g, int16_t* lut,
                        cudaStream_t st);

// Prefill GEMM (I2_S, int8 tensor cores).
int launch_gemm_i2s_prefill(const uint8_t* packed, float w_scale, int64_t M, int64_t K, const int8_t* q,
                            const float* act_scale, int64_t T, float* y, int32_t* acc_out,
                            cudaStream_t st);

}  // namespace bitnet
