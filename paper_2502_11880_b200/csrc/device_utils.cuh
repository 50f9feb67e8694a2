// Device-side helpers shared by the decode kernels (internal): asynchronous copies, named barriers, the
// legacy int8 tensor-core MMA and the quantiser's rounding (Alg. 1 Phase 1).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace bitnet {

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// 16-byte asynchronous copy global -> shared with an L2 cache policy (weights: evict first).
__device__ __forceinline__ void cp16(uint32_t dst, const void* src, uint64_t pol) {
  asm volatile("cp.async.cg.shared.global.L2::cache_hint [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "l"(pol)
               : "memory");
}
// The same without a policy (data that is read again soon: quantised activations).
__device__ __forceinline__ void cp16_keep(uint32_t dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ uint64_t policy_evict_first() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
// Barrier `id` (1..15) among `nthreads` threads of the CTA (whole warps).
__device__ __forceinline__ void group_barrier(int id, int nthreads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}

// D(16x8, s32) += A(16x32, u8, row) * B(32x8, s8, col).  Lane (g = lane/4, t = lane%4):
// a0 = row g, k 4t..4t+3; a1 = row g+8, same k; a2, a3 = the same rows, k 16+4t..; b0 = k 4t..4t+3 of
// column g, b1 = k 16+4t..; c0,c1 = row g, columns 2t, 2t+1; c2,c3 = row g+8.
__device__ __forceinline__ void mma_u8s8(int (&c)[4], unsigned a0, unsigned a1, unsigned a2, unsigned a3, int b0,
                                         int b1) {
  asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// q = clamp(rint(x * s), -128, 127): one rounded binary32 product, ties to even.
__device__ __forceinline__ int quant1(float x, float s) {
  return max(-128, min(127, __float2int_rn(__fmul_rn(x, s))));
}
// Four codes in one word: the saturating pack does the clamp (same result as quant1 on every input).
__device__ __forceinline__ int quant4_packed(const float4& v, float s) {
  const int a0 = __float2int_rn(__fmul_rn(v.x, s)), a1 = __float2int_rn(__fmul_rn(v.y, s));
  const int a2 = __float2int_rn(__fmul_rn(v.z, s)), a3 = __float2int_rn(__fmul_rn(v.w, s));
  int hi, w;
  asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(hi) : "r"(a3), "r"(a2), "r"(0));
  asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(w) : "r"(a1), "r"(a0), "r"(hi));
  return w;
}
// The same word from four separate clamps (kept where the compiler schedules it better than the pack).
__device__ __forceinline__ int quant4(const float4& v, float s) {
  return (quant1(v.x, s) & 255) | ((quant1(v.y, s) & 255) << 8) | ((quant1(v.z, s) & 255) << 16) |
         ((quant1(v.w, s) & 255) << 24);
}
// Where word r (four columns) of a staged activation row lies in the I2_S decode kernels: within every 256-column
// chunk the 16-byte pieces are kept as [piece p][lane quarter t] instead of [t][p], so that the four quarters' loads
// of one piece (and, with a row stride of 64 bytes modulo 128, the rows of two tokens) cover the 32 banks exactly once.
__device__ __forceinline__ int staged_word(int r) { return (r & ~63) | ((r & 12) << 2) | ((r & 48) >> 2) | (r & 3); }
__device__ __forceinline__ float absmax4(const float4& v) {
  return fmaxf(fmaxf(fabsf(v.x), fabsf(v.y)), fmaxf(fabsf(v.z), fabsf(v.w)));
}

}  // namespace bitnet
