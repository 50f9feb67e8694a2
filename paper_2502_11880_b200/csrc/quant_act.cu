// Activation quantiser: Alg. 1 Phase 1 ("Quantization"), absmax int8 (Sec. 2.1, Sec. 3.2.2).
//
// One CTA per token.  Pass 1 reduces max|x| over the row (exact, order free); pass 2 re-reads the
// row (L1/L2 resident), multiplies by s = 127/amax with a single rounded binary32 product, rounds
// to nearest even, clamps, stores int8 and reduces the sum of the codes.  No fast-math anywhere:
// the division, the product and the conversion are the IEEE round-to-nearest forms, so the bytes
// match a scalar CPU evaluation of the same formula.
#include <stdlib.h>

#include "common.cuh"
#include "device_utils.cuh"

namespace bitnet {
namespace {

constexpr int QTHREADS = 512;

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ int warp_sum(int v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}


// amax over a [rows][K] slab starting at x; result in every thread.
__device__ float block_amax(const float* __restrict__ x, int64_t n, float* red) {
  float m = 0.0f;
  const int tid = threadIdx.x;
  if ((n & 3) == 0 && ((reinterpret_cast<uintptr_t>(x) & 15u) == 0)) {
    const float4* x4 = reinterpret_cast<const float4*>(x);
    for (int64_t i = tid; i < n / 4; i += blockDim.x) {
      float4 v = __ldcg(x4 + i);
      m = fmaxf(m, fmaxf(fmaxf(fabsf(v.x), fabsf(v.y)), fmaxf(fabsf(v.z), fabsf(v.w))));
    }
  } else {
    for (int64_t i = tid; i < n; i += blockDim.x) m = fmaxf(m, fabsf(__ldcg(x + i)));
  }
  m = warp_max(m);
  if ((tid & 31) == 0) red[tid >> 5] = m;
  __syncthreads();
  if (tid < 32) {
    float v = (tid < (blockDim.x >> 5)) ? red[tid] : 0.0f;
    v = warp_max(v);
    if (tid == 0) red[0] = v;
  }
  __syncthreads();
  float r = red[0];
  __syncthreads();
  return r;
}

// per_tensor pass A: one CTA per token folds its row maximum into *amax_bits (bit pattern of a
// non-negative float orders like the unsigned integer).
__global__ void __launch_bounds__(QTHREADS) amax_kernel(const float* __restrict__ x, int64_t K,
                                                        unsigned* amax_bits) {
  __shared__ float red[32];
  float m = block_amax(x + (int64_t)blockIdx.x * K, K, red);
  if (threadIdx.x == 0) atomicMax(amax_bits, __float_as_uint(m));
}

__global__ void __launch_bounds__(QTHREADS)
quant_act_kernel(const float* __restrict__ x, int64_t K, int8_t* __restrict__ q, float* __restrict__ act_scale,
                 int32_t* __restrict__ act_sum, const unsigned* __restrict__ tensor_amax_bits) {
  __shared__ float red[32];
  __shared__ int redi[32];
  const int64_t t = blockIdx.x;
  const float* xr = x + t * K;
  int8_t* qr = q + t * K;
  const int tid = threadIdx.x;

  // programmatic dependent launch: let the next kernel start its prologue, then wait for the kernel
  // that produced x (both are no-ops under a plain launch)
  if (tid == 0) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");

  float amax;
  if (tensor_amax_bits) {
    amax = __uint_as_float(*tensor_amax_bits);
  } else {
    amax = block_amax(xr, K, red);
  }
  const float amax_c = fmaxf(amax, 1e-5f);
  const float s = __fdiv_rn(127.0f, amax_c);

  int sum = 0;
  if ((K & 3) == 0 && ((reinterpret_cast<uintptr_t>(xr) & 15u) == 0) &&
      ((reinterpret_cast<uintptr_t>(qr) & 3u) == 0)) {
    const float4* x4 = reinterpret_cast<const float4*>(xr);
    char4* q4 = reinterpret_cast<char4*>(qr);
    for (int64_t i = tid; i < K / 4; i += blockDim.x) {
      float4 v = __ldcg(x4 + i);
      int a = quant1(v.x, s), b = quant1(v.y, s), c = quant1(v.z, s), d = quant1(v.w, s);
      sum += a + b + c + d;
      q4[i] = make_char4((signed char)a, (signed char)b, (signed char)c, (signed char)d);
    }
  } else {
    for (int64_t i = tid; i < K; i += blockDim.x) {
      int a = quant1(__ldcg(xr + i), s);
      sum += a;
      qr[i] = (int8_t)a;
    }
  }
  sum = warp_sum(sum);
  if ((tid & 31) == 0) redi[tid >> 5] = sum;
  __syncthreads();
  if (tid < 32) {
    int v = (tid < (blockDim.x >> 5)) ? redi[tid] : 0;
    v = warp_sum(v);
    if (tid == 0) {
      if (act_sum) act_sum[t] = v;
      // per-tensor mode writes the scales in a separate pass (act_scale[0] carries the maximum)
      if (!tensor_amax_bits) act_scale[t] = __fdiv_rn(amax_c, 127.0f);
    }
  }
}

// Single-pass variant for rows that fit the CTA's registers (K <= 32 * NT floats): NT threads per token, each
// keeps 8 float4 of the row between the absmax reduction and the rounding, so x is read from memory once and
// small rows use small CTAs (many tokens per SM in the prefill case).  Same operations in the same order
// as quant_act_kernel: the bytes are identical.
template <int NT>
__global__ void __launch_bounds__(NT) quant_act_reg_kernel(const float* __restrict__ x, int64_t K, int8_t* __restrict__ q,
                                                           float* __restrict__ act_scale, int32_t* __restrict__ act_sum) {
  constexpr int VPT = 8;
  __shared__ float red[32];
  __shared__ int redi[32];
  const int64_t t = blockIdx.x;
  const float4* x4 = reinterpret_cast<const float4*>(x + t * K);
  int* q4 = reinterpret_cast<int*>(q + t * K);
  const int tid = threadIdx.x, n4 = (int)(K / 4);
  if (tid == 0) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  float4 v[VPT];
#pragma unroll
  for (int r = 0; r < VPT; ++r) {
    const int i = tid + r * NT;
    v[r] = (i < n4) ? __ldcg(x4 + i) : make_float4(0.f, 0.f, 0.f, 0.f);
  }
  float m = 0.0f;
#pragma unroll
  for (int r = 0; r < VPT; ++r)
    m = fmaxf(m, fmaxf(fmaxf(fabsf(v[r].x), fabsf(v[r].y)), fmaxf(fabsf(v[r].z), fabsf(v[r].w))));
  m = warp_max(m);
  if ((tid & 31) == 0) red[tid >> 5] = m;
  __syncthreads();
  float amax = 0.0f;
#pragma unroll
  for (int w = 0; w < NT / 32; ++w) amax = fmaxf(amax, red[w]);
  const float amax_c = fmaxf(amax, 1e-5f);
  const float s = __fdiv_rn(127.0f, amax_c);
  int sum = 0;
#pragma unroll
  for (int r = 0; r < VPT; ++r) {
    const int i = tid + r * NT;
    if (i < n4) {
      const int a = quant1(v[r].x, s), b = quant1(v[r].y, s), c = quant1(v[r].z, s), d = quant1(v[r].w, s);
      sum += a + b + c + d;
      q4[i] = (a & 255) | ((b & 255) << 8) | ((c & 255) << 16) | ((d & 255) << 24);
    }
  }
  sum = warp_sum(sum);
  if ((tid & 31) == 0) redi[tid >> 5] = sum;
  __syncthreads();
  if (tid == 0) {
    int tot = 0;
#pragma unroll
    for (int w = 0; w < NT / 32; ++w) tot += redi[w];
    if (act_sum) act_sum[t] = tot;
    act_scale[t] = __fdiv_rn(amax_c, 127.0f);
  }
}

// Few tokens, long rows: a cluster of C CTAs shares one row (decode batches leave most SMs idle with one CTA
// per token, and a row of 28672 floats is a 5 us round trip for a single CTA).  Each CTA keeps its segment of
// the row in registers, the segments' maxima meet through distributed shared memory (every CTA writes its
// partial into every peer), and after the cluster barrier every CTA holds the row's amax: the same
// operations on the same values as quant_act_reg_kernel, so the bytes are identical.  The partial code sums
// meet in rank 0 the same way.
template <int NT, int C>
__global__ void __launch_bounds__(NT) quant_act_cluster_kernel(const float* __restrict__ x, int64_t K,
                                                               int8_t* __restrict__ q, float* __restrict__ act_scale,
                                                               int32_t* __restrict__ act_sum) {
  constexpr int VPT = 8;
  __shared__ float red[32];
  __shared__ int redi[32];
  __shared__ float part[C];      // partial maxima of all ranks (written by the peers)
  __shared__ int psum[C];        // partial code sums of all ranks (rank 0's copy is the one that is read)
  const int64_t t = blockIdx.y;
  const int rank = blockIdx.x;   // grid.x == cluster size: the rank in the cluster
  const float4* x4 = reinterpret_cast<const float4*>(x + t * K);
  int* q4 = reinterpret_cast<int*>(q + t * K);
  const int tid = threadIdx.x, n4 = (int)(K / 4);
  const int seg = (n4 + C - 1) / C, lo = rank * seg, hi = (lo + seg < n4) ? lo + seg : n4;
  if (tid == 0) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  // A peer's shared memory may be written only once that peer is known to be running: every CTA announces itself
  // here, and the matching wait stands right before the first remote store (it hides behind the loads of x).
  asm volatile("barrier.cluster.arrive.relaxed.aligned;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  float4 v[VPT];
#pragma unroll
  for (int r = 0; r < VPT; ++r) {
    const int i = lo + tid + r * NT;
    v[r] = (i < hi) ? __ldcg(x4 + i) : make_float4(0.f, 0.f, 0.f, 0.f);
  }
  float m = 0.0f;
#pragma unroll
  for (int r = 0; r < VPT; ++r)
    m = fmaxf(m, fmaxf(fmaxf(fabsf(v[r].x), fabsf(v[r].y)), fmaxf(fabsf(v[r].z), fabsf(v[r].w))));
  m = warp_max(m);
  if ((tid & 31) == 0) red[tid >> 5] = m;
  __syncthreads();
  asm volatile("barrier.cluster.wait.aligned;" ::: "memory");   // every CTA of the cluster has started
  if (tid < C) {
    float mc = 0.0f;
#pragma unroll
    for (int w = 0; w < NT / 32; ++w) mc = fmaxf(mc, red[w]);
    // thread p sends this CTA's maximum to rank p
    const uint32_t mine = (uint32_t)__cvta_generic_to_shared(&part[rank]);
    uint32_t remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(mine), "r"(tid));
    asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(remote), "f"(mc) : "memory");
  }
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
  float amax = 0.0f;
#pragma unroll
  for (int p = 0; p < C; ++p) amax = fmaxf(amax, part[p]);
  const float amax_c = fmaxf(amax, 1e-5f);
  const float s = __fdiv_rn(127.0f, amax_c);
  int sum = 0;
#pragma unroll
  for (int r = 0; r < VPT; ++r) {
    const int i = lo + tid + r * NT;
    if (i < hi) {
      const int a = quant1(v[r].x, s), b = quant1(v[r].y, s), c = quant1(v[r].z, s), d = quant1(v[r].w, s);
      sum += a + b + c + d;
      q4[i] = (a & 255) | ((b & 255) << 8) | ((c & 255) << 16) | ((d & 255) << 24);
    }
  }
  sum = warp_sum(sum);
  if ((tid & 31) == 0) redi[tid >> 5] = sum;
  __syncthreads();
  if (tid == 0) {
    int tot = 0;
#pragma unroll
    for (int w = 0; w < NT / 32; ++w) tot += redi[w];
    const uint32_t mine = (uint32_t)__cvta_generic_to_shared(&psum[rank]);
    uint32_t remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(mine), "r"(0));
    asm volatile("st.shared::cluster.s32 [%0], %1;" ::"r"(remote), "r"(tot) : "memory");
  }
  // nobody leaves before every peer's writes into its shared memory have landed; rank 0 then adds up
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
  if (rank == 0 && tid == 0) {
    int tot = 0;
#pragma unroll
    for (int p = 0; p < C; ++p) tot += psum[p];
    if (act_sum) act_sum[t] = tot;
    act_scale[t] = __fdiv_rn(amax_c, 127.0f);
  }
}

template <int NT, int C>
cudaError_t launch_cluster(const float* x, int64_t T, int64_t K, int8_t* q, float* act_scale, int32_t* act_sum,
                           cudaStream_t st) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(C, (unsigned)T);
  cfg.blockDim = dim3(NT);
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = C;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = early_start_enabled(st) ? 2 : 1;
  return cudaLaunchKernelEx(&cfg, quant_act_cluster_kernel<NT, C>, x, K, q, act_scale, act_sum);
}

template <int NT>
cudaError_t launch_reg(const float* x, int64_t T, int64_t K, int8_t* q, float* act_scale, int32_t* act_sum, cudaStream_t st) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)T);
  cfg.blockDim = dim3(NT);
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = early_start_enabled(st) ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, quant_act_reg_kernel<NT>, x, K, q, act_scale, act_sum);
}

// The rows of a LIST of activation matrices in one launch (Alg. 1 Phase 1 for every linear of a grouped call whose
// kernel wants the codes ready): one CTA per row, the row's matrix found by a binary search over the items' first
// rows.  Same operations in the same order as quant_act_kernel: the bytes are identical.
constexpr int QLIST_ITEMS = 800;
struct QListEntry {
  const float* x;
  int8_t* q;
  float* act_scale;
  int K, first_row;
};
struct QListArgs {
  int n, rows;
  QListEntry it[QLIST_ITEMS];
};
static_assert(sizeof(QListArgs) <= 32764, "kernel parameter limit");

__global__ void __launch_bounds__(QTHREADS) quant_act_list_kernel(const __grid_constant__ QListArgs a) {
  __shared__ float red[32];
  const int tid = threadIdx.x;
  if (tid == 0) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  int lo = 0, hi = a.n - 1;
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if (a.it[mid].first_row <= (int)blockIdx.x) lo = mid; else hi = mid - 1;
  }
  const QListEntry& d = a.it[lo];
  const int64_t t = (int)blockIdx.x - d.first_row, K = d.K;
  const float* xr = d.x + t * K;
  int8_t* qr = d.q + t * K;
  const float amax_c = fmaxf(block_amax(xr, K, red), 1e-5f);
  const float s = __fdiv_rn(127.0f, amax_c);
  if ((K & 3) == 0 && ((reinterpret_cast<uintptr_t>(xr) & 15u) == 0) && ((reinterpret_cast<uintptr_t>(qr) & 3u) == 0)) {
    const float4* x4 = reinterpret_cast<const float4*>(xr);
    int* q4 = reinterpret_cast<int*>(qr);
    for (int64_t i = tid; i < K / 4; i += blockDim.x) q4[i] = quant4_packed(__ldcg(x4 + i), s);
  } else {
    for (int64_t i = tid; i < K; i += blockDim.x) qr[i] = (int8_t)quant1(__ldcg(xr + i), s);
  }
  if (tid == 0) d.act_scale[t] = __fdiv_rn(amax_c, 127.0f);
}

__global__ void fill_scale_kernel(float* act_scale, int64_t T) {
  __shared__ float sc;
  if (threadIdx.x == 0) {
    float amax = __uint_as_float(*reinterpret_cast<unsigned*>(act_scale));
    sc = __fdiv_rn(fmaxf(amax, 1e-5f), 127.0f);
  }
  __syncthreads();
  for (int64_t i = threadIdx.x; i < T; i += blockDim.x) act_scale[i] = sc;
}

}  // namespace

int launch_quant_act_list(const QuantListItem* items, int64_t n, cudaStream_t st) {
  static thread_local QListArgs a;   // 19 KB: off the stack
  for (int64_t i0 = 0; i0 < n;) {
    int cnt = 0;
    int64_t rows = 0;
    while (i0 + cnt < n && cnt < QLIST_ITEMS && rows + items[i0 + cnt].T <= 0x3fffffff) {
      const QuantListItem& s = items[i0 + cnt];
      if (!s.x || !s.q || !s.act_scale || s.T < 1 || s.K < 1 || s.K > 0x7fffffff) return BITNET_ERR_INVALID_ARG;
      a.it[cnt] = QListEntry{s.x, s.q, s.act_scale, (int)s.K, (int)rows};
      rows += s.T;
      ++cnt;
    }
    if (cnt == 0) return BITNET_ERR_INVALID_ARG;
    a.n = cnt;
    a.rows = (int)rows;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)rows);
    cfg.blockDim = dim3(QTHREADS);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = early_start_enabled(st) ? 1 : 0;
    log_launch("quant_act_list_kernel items=%d rows=%lld", cnt, (long long)rows);
    cudaError_t e = cudaLaunchKernelEx(&cfg, quant_act_list_kernel, a);
    if (e != cudaSuccess) return note_cuda_error(e);
    i0 += cnt;
  }
  return check_launch();
}

int launch_quant_act(const float* x, int64_t T, int64_t K, int per_tensor, int8_t* q, float* act_scale,
                     int32_t* act_sum, cudaStream_t st) {
  if (per_tensor && T > 1) {
    // act_scale[0] doubles as the running maximum until the last pass overwrites every entry
    cudaError_t e = cudaMemsetAsync(act_scale, 0, sizeof(float), st);
    if (e != cudaSuccess) return note_cuda_error(e);
    amax_kernel<<<(unsigned)T, QTHREADS, 0, st>>>(x, K, reinterpret_cast<unsigned*>(act_scale));
    quant_act_kernel<<<(unsigned)T, QTHREADS, 0, st>>>(x, K, q, act_scale, act_sum,
                                                       reinterpret_cast<const unsigned*>(act_scale));
    fill_scale_kernel<<<1, 256, 0, st>>>(act_scale, T);
  } else if ((K & 3) == 0 && K <= 32 * 1024 && aligned16(x) && (reinterpret_cast<uintptr_t>(q) & 3u) == 0) {
    // rows are 16-byte aligned when x is and K % 4 == 0
    cudaError_t e;
    static const bool use_clusters = [] { const char* v = getenv("BITNET_QUANT_CLUSTERS"); return !v || atoi(v) != 0; }();
    // 4 to 8 tokens with rows of 8192 floats or more: 4 or 8 CTAs per row (100B-shaped layer at 8 tokens: 79.6
    // instead of 81.6 us, at 6 tokens 78.0 instead of 79.9; one CTA per row is as fast or faster for a single token,
    // 54.6 vs 55.6, and at 16 and 64 tokens, 100.8 vs 103.0 and 236 vs 238)
    if (log_enabled()) log_launch("quant_act T=%lld K=%lld", (long long)T, (long long)K);
    if (use_clusters && T >= 4 && T <= 8 && K >= 16384 && K <= 8 * 128 * 32) e = launch_cluster<128, 8>(x, T, K, q, act_scale, act_sum, st);
    else if (use_clusters && T >= 4 && T <= 8 && K >= 8192 && K <= 4 * 128 * 32) e = launch_cluster<128, 4>(x, T, K, q, act_scale, act_sum, st);
    else if (K <= 32 * 128) e = launch_reg<128>(x, T, K, q, act_scale, act_sum, st);
    else if (K <= 32 * 256) e = launch_reg<256>(x, T, K, q, act_scale, act_sum, st);
    else if (K <= 32 * 512) e = launch_reg<512>(x, T, K, q, act_scale, act_sum, st);
    else e = launch_reg<1024>(x, T, K, q, act_scale, act_sum, st);
    if (e != cudaSuccess) return note_cuda_error(e);
  } else {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)T);
    cfg.blockDim = dim3(QTHREADS);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = early_start_enabled(st) ? 1 : 0;
    const unsigned* no_amax = nullptr;
    cudaError_t e = cudaLaunchKernelEx(&cfg, quant_act_kernel, x, K, q, act_scale, act_sum, no_amax);
    if (e != cudaSuccess) return note_cuda_error(e);
  }
  return check_launch();
}

}  // namespace bitnet
