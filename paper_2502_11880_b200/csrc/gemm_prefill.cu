// Prefill mpGEMM (many tokens), I2_S: Alg. 1 Phase 2 at large T.
//
// This file holds the plain dp4a kernel (one thread per output): a reference point for the tensor-core
// kernel of gemm_prefill_tc.cu and the path taken when BITNET_PREFILL=simt is set in the environment.
#include <cstdlib>
#include <cstring>

#include "common.cuh"

namespace bitnet {
namespace {

__device__ __forceinline__ int dp4a_us(unsigned a, int b, int c) {
  int d;
  asm("dp4a.u32.s32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
  return d;
}

// block = 32 rows (x) by 8 tokens (y); each thread walks K for one output.
__global__ void __launch_bounds__(256) gemm_i2s_simt_kernel(const uint8_t* __restrict__ packed, int64_t kp, int M, int K,
                                                            const int8_t* __restrict__ q,
                                                            const float* __restrict__ act_scale, float w_scale,
                                                            int T, float* __restrict__ y,
                                                            int32_t* __restrict__ acc_out) {
  const int m = blockIdx.x * 32 + threadIdx.x;
  const int t = blockIdx.y * 8 + threadIdx.y;
  if (m >= M || t >= T) return;
  const int* qr = reinterpret_cast<const int*>(q + (int64_t)t * K);
  int a0 = 0, a1 = 0, a2 = 0, a3 = 0, qs = 0;
  for (int c = 0; c * 256 < K; ++c) {
    const uint32_t* wr = reinterpret_cast<const uint32_t*>(packed + i2s_row_chunk_offset(m, c, kp));
    const int nwords = min(16, (K - c * 256) / 16);     // words of this chunk that lie inside K
    for (int j = 0; j < nwords; ++j) {
      const unsigned w = wr[j];
      const int* qb = qr + c * 64 + 8 * (j >> 1) + (j & 1);   // slot s multiplies activation word qb[2s]
      const int q0 = qb[0], q1 = qb[2], q2 = qb[4], q3 = qb[6];
      a0 = dp4a_us(w & 0x03030303u, q0, a0);
      a1 = dp4a_us(w & 0x0C0C0C0Cu, q1, a1);
      a2 = dp4a_us(w & 0x30303030u, q2, a2);
      a3 = dp4a_us(w & 0xC0C0C0C0u, q3, a3);
      qs = __dp4a(q0, 0x01010101, qs);
      qs = __dp4a(q1, 0x01010101, qs);
      qs = __dp4a(q2, 0x01010101, qs);
      qs = __dp4a(q3, 0x01010101, qs);
    }
  }
  const int acc = a0 + (a1 >> 2) + (a2 >> 4) + (a3 >> 6) - qs;
  y[(int64_t)t * M + m] = __fmul_rn((float)acc, __fmul_rn(act_scale[t], w_scale));
  if (acc_out) acc_out[(int64_t)t * M + m] = acc;
}

}  // namespace

int launch_gemm_i2s_simt(const uint8_t* packed, float w_scale, int64_t M, int64_t K, const int8_t* q,
                         const float* act_scale, int64_t T, float* y, int32_t* acc_out, cudaStream_t st) {
  dim3 grid((unsigned)ceil_div(M, 32), (unsigned)ceil_div(T, 8));
  gemm_i2s_simt_kernel<<<grid, dim3(32, 8), 0, st>>>(packed, i2s_kp(K), (int)M, (int)K, q, act_scale, w_scale, (int)T,
                                                    y, acc_out);
  return check_launch();
}

}  // namespace bitnet
