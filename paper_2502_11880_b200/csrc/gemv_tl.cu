// TL1 / TL2 mpGEMV for decode (1..8 tokens): element-wise LUT mpGEMM, Alg. 2, with the tables of
// Alg. 3 (pairs, 9 sums) and Alg. 4 (triples, 14 sums after mirror consolidation); Eq. 3:
//     acc = sum over groups of Lookup(LUT_group, index), the sign bit of a triple negating the value.
//
// Phase 1 ("Table-setup" / "PreCompute"): a small kernel enumerates, for every group of the token's
// int8 activations, the 16-slot table of partial sums -- slot i of a triple table is
// d0*a0 + d1*a1 + d2*a2 with (d0,d1,d2) the balanced-ternary digits of i, slot i of a pair table is
// (i/3-1)*a0 + (i%3-1)*a1 -- once, into the workspace (it is the same for every output row; building
// it in every CTA would cost as much as the lookups of ~16 rows).  Sums stay exact (|sum| <= 384), as
// in the lossless TL*_1 variants.  Two tokens share one 32-bit slot as hi*65536 + lo: integer add and
// negate act on both halves at once, so one lookup serves two tokens.
//
// Phase 2 (accumulation).  A CTA owns a K-slice (a run of 32-group tiles) and copies the slice of
// the tables into shared memory with one bulk asynchronous copy.  Lanes are rows: a warp takes one
// tile of a 32-row block, every lane reads its row's 16 index bytes (+ 4 sign bytes) with one
// coalesced request per plane (the next tile's words are requested before the current tile is
// processed) and resolves its 32 nibbles against the SAME group table -- 16 slots in 16 distinct
// banks, so lookups never conflict.  The conditional negate is v ^ m with m = 0 / -1 taken from the
// sign bit by one bit-field extract; the "+1" of two's-complement negation is added once per tile as
// popcount(sign word).  Warps of a CTA cover different tiles; their per-row sums meet in shared
// memory, and K-slices of different CTAs meet in an int32 workspace by atomicAdd, finalised by
// whichever slice arrives last (no waiting).
#include "common.cuh"
#include "device_utils.cuh"

namespace bitnet {
namespace {

constexpr int WARPS = 8;
constexpr int THREADS = WARPS * 32;
constexpr int MAX_SLICE_TILES = 48;   // 2 KB of tables per tile and token pair -> 96 KB, two CTAs per SM
constexpr uint32_t WAIT_LIMIT = 1u << 22;

static __device__ int g_tl_error = 0;

struct TlArgs {
  const uint8_t* packed;
  TlGeom g;
  int M;
  int64_t K;
  const int* table;  // [tiles][32 groups][16 slots] of this token pair
  const float* act_scale;
  float w_scale;
  int nt;            // tokens in this pass (1 or 2)
  float* y;
  int32_t* acc_out;
  int32_t* ws_acc;
  unsigned* ws_ticket;
  int nslices;
  int tiles_per_slice;
};

// Entry i of a group's table for activations (a0,a1,a2); pair tables pass a2 = 0 and is3 = false.
__device__ __forceinline__ int lut_entry(bool is3, int i, int a0, int a1, int a2) {
  if (is3) {
    if (i > 13) return 0;
    const int d0 = (i + 4) / 9;
    const int rem = i - 9 * d0;
    const int d1 = (rem + 7) / 3 - 2;
    const int d2 = rem - 3 * d1;
    return d0 * a0 + d1 * a1 + d2 * a2;
  }
  if (i > 8) return 0;
  return (i / 3 - 1) * a0 + (i % 3 - 1) * a1;
}

// Activations of tile `tile` (global tile number), group grp, token row qrow (global memory).
__device__ __forceinline__ void group_acts(const TlGeom& g, int64_t K, const int8_t* qrow, int tile, int grp,
                                           bool* is3, int* a0, int* a1, int* a2) {
  if (tile < g.tiles3) {
    const int64_t k = (int64_t)tile * 96 + 3 * grp;
    *is3 = true;
    *a0 = qrow[k];
    *a1 = qrow[k + 1];
    *a2 = qrow[k + 2];
  } else {
    const int64_t k = g.three_k + (int64_t)(tile - g.tiles3) * 64 + 2 * grp;
    *is3 = false;
    *a2 = 0;
    if (k < K) {
      *a0 = qrow[k];
      *a1 = qrow[k + 1];
    } else {
      *a0 = 0;
      *a1 = 0;
    }
  }
}

// Phase 1: one thread per table slot; blockIdx.y = token pair.  table[pair][slot] = lo + 65536 * hi.
__global__ void tl_table_kernel(const int8_t* __restrict__ q, int T, int64_t K, TlGeom g, int* __restrict__ table,
                                int64_t nslots, int* __restrict__ head, int64_t head_ints) {
  // early start: resident before the previous kernel (the quantiser) has finished, reads its codes after the wait
  if (threadIdx.x == 0) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  // The split-K sums and arrival counters of this call start at zero whatever an earlier call (of another shape,
  // whose tables may have lain here) left in the workspace.
  for (int64_t i = ((int64_t)blockIdx.y * gridDim.x + blockIdx.x) * blockDim.x + threadIdx.x; i < head_ints;
       i += (int64_t)gridDim.x * gridDim.y * blockDim.x)
    head[i] = 0;
  const int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= nslots) return;
  const int i = (int)(e & 15), grp = (int)((e >> 4) & 31);
  const int tile = (int)(e >> 9);
  const int t0 = 2 * blockIdx.y;
  bool is3;
  int a0, a1, a2;
  group_acts(g, K, q + (int64_t)t0 * K, tile, grp, &is3, &a0, &a1, &a2);
  int v = lut_entry(is3, i, a0, a1, a2);
  if (t0 + 1 < T) {
    group_acts(g, K, q + (int64_t)(t0 + 1) * K, tile, grp, &is3, &a0, &a1, &a2);
    v += lut_entry(is3, i, a0, a1, a2) * 65536;
  }
  table[(int64_t)blockIdx.y * nslots + e] = v;
}


__device__ __forceinline__ int sign_mask(unsigned sg, int bit) {   // 0 or -1 from one bit
  int m;
  asm("bfe.s32 %0, %1, %2, 1;" : "=r"(m) : "r"(sg), "r"(bit));
  return m;
}

// The four index words of row `r` of a tile (they lie 16 bytes apart: the tile interleaves four rows per piece).
__device__ __forceinline__ uint4 load_row_words(const uint8_t* tp, int r) {
  const unsigned* p = reinterpret_cast<const unsigned*>(tp + tl_word_off(r, 0));
  return make_uint4(__ldg(p), __ldg(p + 4), __ldg(p + 8), __ldg(p + 12));
}

// Waits for phase 0 of an mbarrier, at most `limit` polls.  A wait that gives up records BITNET_ERR_TIMEOUT in the
// device flag (read by bitnet_device_status) and returns false: the kernel then returns instead of hanging.
__device__ __forceinline__ bool bounded_wait(uint64_t* bar, uint32_t limit) {
  bool got = false;
  for (uint32_t it = 0; it < limit && !got; ++it) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], 0;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar))
        : "memory");
    got = ok != 0;
  }
  if (!got && threadIdx.x == 0) atomicExch(&g_tl_error, BITNET_ERR_TIMEOUT);
  return got;
}

// Test hook: a barrier that expects 16 bytes which nobody ever copies.  The bounded wait runs out, the flag is set,
// the kernel returns; nothing is in flight at any point.
__global__ void wait_timeout_probe_kernel(uint32_t limit) {
  __shared__ uint64_t bar;
  if (threadIdx.x == 0) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&bar)) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(&bar)), "r"(16u) : "memory");
  }
  __syncthreads();
  bounded_wait(&bar, limit);
}

__global__ void __launch_bounds__(THREADS, 2) gemv_tl_kernel(const TlArgs a) {
  extern __shared__ __align__(128) int smem[];
  int* tab = smem;                                   // [tiles_per_slice][32][16]
  int* red = smem + a.tiles_per_slice * 512;         // [2][WARPS][32][2]: the sums of two row blocks in flight
  uint64_t* bar = reinterpret_cast<uint64_t*>(red + 2 * WARPS * 64);
  const int lane = threadIdx.x & 31;
  const int warp = threadIdx.x >> 5;
  const int slice = blockIdx.y;
  const int tiles_total = (int)(a.g.tiles3 + a.g.tiles2);
  const int tile0 = slice * a.tiles_per_slice;
  const int ntiles = min(a.tiles_per_slice, tiles_total - tile0);

  // early start: everything this kernel reads besides the weights (tables, scales) and everything it writes
  // (y, the split-K sums and tickets) belongs to earlier kernels until the wait returns
  if (threadIdx.x == 0) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  // ---- the tables of this slice: one bulk copy global -> shared
  if (threadIdx.x == 0) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(bar)) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    const uint32_t bytes = (uint32_t)ntiles * 2048u;
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(tab)), "l"(a.table + (int64_t)tile0 * 512), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
  }
  __syncthreads();
  if (!bounded_wait(bar, WAIT_LIMIT)) return;

  const float sc0 = __fmul_rn(a.act_scale[0], a.w_scale);
  const float sc1 = (a.nt == 2) ? __fmul_rn(a.act_scale[1], a.w_scale) : 0.0f;
  const int64_t t3bytes = a.g.tiles3 * 640;

  // ---- Phase 2: lookups.  The warp's work list is (row block, tile) pairs; the next pair's index and
  // sign words are requested before the current pair is processed.
  auto tile_ptr = [&](int rb, int tl) -> const uint8_t* {
    const int tile = tile0 + tl;
    const uint8_t* blk = a.packed + (int64_t)rb * a.g.block_bytes;
    return (tile < a.g.tiles3) ? blk + (int64_t)tile * 640 : blk + t3bytes + (int64_t)(tile - a.g.tiles3) * 512;
  };
  const int nrb = a.M / 32;
  int rb = blockIdx.x, tl = warp;
  uint4 iw = make_uint4(0, 0, 0, 0);
  unsigned sg = 0;
  bool have = rb < nrb && tl < ntiles;
  if (have) {
    const uint8_t* tp = tile_ptr(rb, tl);
    iw = load_row_words(tp, lane);
    sg = (tile0 + tl < a.g.tiles3) ? __ldg(reinterpret_cast<const unsigned*>(tp + tl_sign_off(lane))) : 0u;
  }
  for (int nb = 0; rb < nrb; rb += gridDim.x, ++nb) {
    int lo = 0, hi = 0;
    int* redb = red + (nb & 1) * (WARPS * 64);
    while (tl < ntiles) {
      const uint4 ciw = iw;
      const unsigned csg = sg;
      const int ctl = tl;
      // next element of the work list: the next tile of this row block, else this warp's first tile of
      // the CTA's next row block
      int nrbi = rb, ntl = tl + WARPS;
      if (ntl >= ntiles) {
        nrbi = rb + gridDim.x;
        ntl = warp;
      }
      if (nrbi < nrb && ntl < ntiles) {
        const uint8_t* tp = tile_ptr(nrbi, ntl);
        iw = load_row_words(tp, lane);
        sg = (tile0 + ntl < a.g.tiles3) ? __ldg(reinterpret_cast<const unsigned*>(tp + tl_sign_off(lane))) : 0u;
      }
      const unsigned words[4] = {ciw.x, ciw.y, ciw.z, ciw.w};
      const char* tt = reinterpret_cast<const char*>(tab + ctl * 512);
      int s = __popc(csg);   // the +1 of every two's-complement negation below, for both halves at once
#pragma unroll
      for (int w4 = 0; w4 < 4; ++w4) {
#pragma unroll
        for (int n = 0; n < 8; ++n) {
          const int grp = w4 * 8 + n;
          // byte offset of the slot: 4 * nibble n of the word
          const unsigned off = (n == 0) ? ((words[w4] << 2) & 0x3Cu) : ((words[w4] >> (4 * n - 2)) & 0x3Cu);
          const int v = *reinterpret_cast<const int*>(tt + grp * 64 + off);
          s += v ^ sign_mask(csg, tl_sign_bit(grp));
        }
      }
      // split the packed pair: s = H * 65536 + L with |L| < 32768
      const int l16 = (int)(short)(s & 0xFFFF);
      lo += l16;
      hi += (s - l16) >> 16;
      tl += WARPS;
      if (tl >= ntiles) break;
    }
    tl = warp;
    redb[(warp * 32 + lane) * 2 + 0] = lo;
    redb[(warp * 32 + lane) * 2 + 1] = hi;
    // One barrier per row block: the warp whose turn it is adds the partial sums while the others go on; the
    // buffer is written again two row blocks later, after the next barrier, which that warp reaches only when
    // it has finished reading.
    __syncthreads();
    if (warp == (nb % WARPS)) {
      int tot[2] = {0, 0};
#pragma unroll
      for (int w = 0; w < WARPS; ++w) {
        tot[0] += redb[(w * 32 + lane) * 2 + 0];
        tot[1] += redb[(w * 32 + lane) * 2 + 1];
      }
      const int row = rb * 32 + lane;
      if (a.nslices == 1) {
        a.y[row] = __fmul_rn((float)tot[0], sc0);
        if (a.acc_out) a.acc_out[row] = tot[0];
        if (a.nt == 2) {
          a.y[a.M + row] = __fmul_rn((float)tot[1], sc1);
          if (a.acc_out) a.acc_out[a.M + row] = tot[1];
        }
      } else {
        atomicAdd(a.ws_acc + row, tot[0]);
        if (a.nt == 2) atomicAdd(a.ws_acc + a.M + row, tot[1]);
        __threadfence();
        const unsigned old = atomicAdd(a.ws_ticket + row, 1u);
        if (old == (unsigned)(a.nslices - 1)) {
          __threadfence();
          const int v0 = atomicExch(a.ws_acc + row, 0);
          a.y[row] = __fmul_rn((float)v0, sc0);
          if (a.acc_out) a.acc_out[row] = v0;
          if (a.nt == 2) {
            const int v1 = atomicExch(a.ws_acc + a.M + row, 0);
            a.y[a.M + row] = __fmul_rn((float)v1, sc1);
            if (a.acc_out) a.acc_out[a.M + row] = v1;
          }
          atomicExch(a.ws_ticket + row, 0u);
        }
      }
    }
  }
}

__global__ void tl_build_lut_kernel(const int8_t* q_row, int64_t K, TlGeom g, int16_t* lut, int64_t nslots) {
  const int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= nslots) return;
  const int i = (int)(e & 15), grp = (int)((e >> 4) & 31);
  const int tile = (int)(e >> 9);
  bool is3;
  int a0, a1, a2;
  group_acts(g, K, q_row, tile, grp, &is3, &a0, &a1, &a2);
  lut[e] = (int16_t)lut_entry(is3, i, a0, a1, a2);
}

inline void slicing(const TlGeom& g, int* nslices, int* tiles_per_slice) {
  const int tiles = (int)(g.tiles3 + g.tiles2);
  *nslices = (tiles + MAX_SLICE_TILES - 1) / MAX_SLICE_TILES;
  *tiles_per_slice = (tiles + *nslices - 1) / *nslices;
}

// bytes of the accumulator/ticket area and of the table area of the workspace (upper bounds that do
// not depend on bk3: no format has more than K/64 + 2 tiles)
inline size_t acc_area_bytes(int64_t T, int64_t M) { return (size_t)((T * M + M) * 4 + 255) & ~(size_t)255; }
inline size_t table_area_bytes(int64_t T, int64_t K) { return (size_t)((T + 1) / 2) * (size_t)(K / 64 + 2) * 2048; }

}  // namespace

size_t gemv_tl_workspace_bytes(int fmt, int64_t T, int64_t M, int64_t K) {
  TlGeom g;
  if (!tl_geom(fmt, M, K, 0, &g)) return 0;
  const int64_t Tc = T > 8 ? 8 : T;
  return acc_area_bytes(Tc, M) + table_area_bytes(Tc, K);
}

int launch_gemv_tl(int fmt, const uint8_t* packed, float w_scale, int64_t M, int64_t K, const TlGeom& g,
                   const int8_t* q, const float* act_scale, int T, float* y, int32_t* acc_out, void* ws,
                   size_t ws_bytes, cudaStream_t st) {
  (void)fmt;
  const int64_t tiles = g.tiles3 + g.tiles2;
  const size_t acc_bytes = acc_area_bytes(T, M);
  const int npairs = (T + 1) / 2;
  if (!ws || ws_bytes < acc_bytes + (size_t)npairs * (size_t)tiles * 2048) return BITNET_ERR_WORKSPACE;
  int* table = reinterpret_cast<int*>(reinterpret_cast<uint8_t*>(ws) + acc_bytes);

  // Phase 1: tables of every token pair
  const int64_t nslots = tiles * 512;
  cudaLaunchAttribute pdl[1];
  pdl[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  pdl[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t tcfg = {};
  tcfg.gridDim = dim3((unsigned)ceil_div(nslots, 256), (unsigned)npairs);
  tcfg.blockDim = dim3(256);
  tcfg.stream = st;
  tcfg.attrs = pdl;
  tcfg.numAttrs = early_start_enabled(st) ? 1 : 0;
  cudaError_t le = cudaLaunchKernelEx(&tcfg, tl_table_kernel, q, T, K, g, table, nslots, reinterpret_cast<int*>(ws),
                                      (int64_t)T * M + M);
  int rc = le == cudaSuccess ? BITNET_OK : note_cuda_error(le);
  if (rc != BITNET_OK) return rc;

  // Phase 2: lookups, one launch per token pair
  TlArgs a;
  a.packed = packed;
  a.g = g;
  a.M = (int)M;
  a.K = K;
  a.w_scale = w_scale;
  slicing(g, &a.nslices, &a.tiles_per_slice);
  a.ws_ticket = reinterpret_cast<unsigned*>(reinterpret_cast<int32_t*>(ws) + (int64_t)T * M);
  const size_t smem = (size_t)a.tiles_per_slice * 2048 + 2 * WARPS * 64 * sizeof(int) + 16;
  static bool attr_set[64] = {false};
  int dev = 0;
  cudaGetDevice(&dev);
  if (!attr_set[dev & 63]) {
    cudaError_t e = cudaFuncSetAttribute(gemv_tl_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         MAX_SLICE_TILES * 2048 + 2 * WARPS * 64 * (int)sizeof(int) + 16);
    if (e != cudaSuccess) return note_cuda_error(e);
    attr_set[dev & 63] = true;
  }
  const int sms = dev_info().sm_count;
  int gx = (2 * sms + a.nslices - 1) / a.nslices;
  if (gx > (int)(M / 32)) gx = (int)(M / 32);
  for (int p = 0; p < npairs; ++p) {
    const int t0 = 2 * p;
    a.table = table + (int64_t)p * nslots;
    a.act_scale = act_scale + t0;
    a.nt = (T - t0 >= 2) ? 2 : 1;
    a.y = y + (int64_t)t0 * M;
    a.acc_out = acc_out ? acc_out + (int64_t)t0 * M : nullptr;
    a.ws_acc = reinterpret_cast<int32_t*>(ws) + (int64_t)t0 * M;
    log_launch("gemv_tl_kernel fmt=%d tokens=%d M=%lld K=%lld grid=%lld x %d K-slices smem=%zu", fmt, a.nt, (long long)M,
               (long long)K, (long long)gx, a.nslices, (size_t)smem);
    cudaLaunchConfig_t gcfg = {};
    gcfg.gridDim = dim3((unsigned)gx, (unsigned)a.nslices);
    gcfg.blockDim = dim3(THREADS);
    gcfg.dynamicSmemBytes = smem;
    gcfg.stream = st;
    gcfg.attrs = pdl;
    gcfg.numAttrs = early_start_enabled(st) ? 1 : 0;
    le = cudaLaunchKernelEx(&gcfg, gemv_tl_kernel, a);
    rc = le == cudaSuccess ? BITNET_OK : note_cuda_error(le);
    if (rc != BITNET_OK) return rc;
  }
  return BITNET_OK;
}

int launch_tl_build_lut(int fmt, const int8_t* q_row, int64_t K, const TlGeom& g, int16_t* lut,
                        cudaStream_t st) {
  (void)fmt;
  const int64_t nslots = (g.tiles3 + g.tiles2) * 512;
  tl_build_lut_kernel<<<(unsigned)ceil_div(nslots, 256), 256, 0, st>>>(q_row, K, g, lut, nslots);
  return check_launch();
}

int gemv_tl_status(int* out) {
  cudaError_t e = cudaMemcpyFromSymbol(out, g_tl_error, sizeof(int));
  return e == cudaSuccess ? BITNET_OK : note_cuda_error(e);
}
int gemv_tl_status_clear() {
  const int zero = 0;
  cudaError_t e = cudaMemcpyToSymbol(g_tl_error, &zero, sizeof(int));
  return e == cudaSuccess ? BITNET_OK : note_cuda_error(e);
}
int launch_wait_timeout_probe(cudaStream_t st) {
  wait_timeout_probe_kernel<<<1, 64, 0, st>>>(1u << 14);
  return check_launch();
}

}  // namespace bitnet
