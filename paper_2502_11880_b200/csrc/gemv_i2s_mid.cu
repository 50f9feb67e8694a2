// I2_S mpGEMM for batches of 6 to 64 tokens (Alg. 1, Phase 2, between decode and prefill).
//
// Still a scan of the packed weights, but with T tokens per weight byte the int8 tensor cores (mma.sync
// m16n8k32, u8 x s8), not HBM, become the limit from about 24 tokens on.  Differences to the decode kernel:
//   * NT = ceil(T / 8) token tiles per weight fragment; from two tiles on the 2-bit fields are shifted down so
//     that slots share accumulators (two sets, or one from five tiles on; a decode kernel keeps one per slot);
//   * up to two token tiles, the B fragments (activations) of a tile are read from shared memory once for
//     RU = 2 adjacent 16-row units (one MMA needs 256 B of B, exactly what the shared-memory pipe delivers in the
//     MMA's two cycles); from three tiles on, one unit per step with the cheaper field extraction measured faster;
//   * the staged codes are stored transposed within each 256-column chunk, token rows 64 bytes apart mod 128:
//     the four lanes of a B load read 64 consecutive bytes and every quarter-warp covers all banks once;
//   * T x K codes do not fit in shared memory, so K is cut into NS slices.  CTAs [sl * cps, (sl + 1) * cps) own
//     slice sl, stage its codes once, and CTA j of them owns an equal share of the units; the CTA's sequence of
//     (unit group, chunk) steps is cut into sixteen equal runs, one per warp, whatever units that cuts, and each
//     warp streams its run through a private cp.async ring.  The int32 partial sums meet in a zeroed [T][M]
//     workspace through integer atomics (order-independent, hence bit-exact);
//   * closing rescale (Alg. 1's last line): up to 8 tokens the last-arriving CTA of a row range does it, beyond
//     that a second kernel over all SMs; either way the workspace is left zeroed.
// The "- sum(q)" term of the code = w + 1 representation is subtracted per slice before the atomics.
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdlib.h>

#include "common.cuh"
#include "device_utils.cuh"

namespace bitnet {
namespace {

constexpr int MW = 16;                 // warps per CTA
constexpr int MTHREADS = MW * 32;
constexpr int FINISH_IN_KERNEL_MAX_NT = 1;   // up to 8 tokens the scan kernel rescales its own sums
constexpr int HDR = 512;               // bytes of shared memory before the staged codes: csum[64]

struct MArgs {
  const uint8_t* packed;
  int64_t unit_bytes;    // bytes of one 16-row unit of the blob = 4 * Kp
  int M;
  int64_t K;
  const int8_t* q;       // [T][K] int8
  const float* act_scale;
  float w_scale;
  int T;
  float* y;
  int32_t* acc_out;
  int32_t* ws;           // [T][M] partial sums, zero on entry and left zero
  int* cnt;              // [cps] CTAs (slices) that have added their share of a row range; zero on entry, left zero
  int nchunks;           // 256-column chunks per row
  int NS;                // K-slices
  int cps;               // CTAs per slice (grid = NS * cps)
  int nunits;            // ceil(M / 16)
  int qst;               // bytes between staged token rows
};


// NT token tiles of 8; RU 16-row units per item; DEPTH ring slots (of RU KB) per warp;
// NSL accumulator sets per token tile: 4 = one per 2-bit slot (fields used in place, weights 1, 4, 16, 64),
// 2 = slots {0,1} and {2,3} (one shift per word), 1 = every field shifted down to bits 0-1.
//
// Work split.  CTAs [sl * cps, (sl + 1) * cps) own K-slice sl; CTA j of them owns an equal share of the
// slice's items (groups of RU units).  A CTA's work is the sequence of steps (item, chunk of the slice), item
// by item; warp w takes the w-th sixteenth of that sequence, whatever items it cuts: every partial sum goes
// to the workspace through an integer atomic, so an item may be shared by two warps (or two CTAs' slices).
template <int NT, int RU, int DEPTH, int NSL>
__global__ void __launch_bounds__(MTHREADS, 1) gemv_i2s_mid_kernel(const MArgs a) {
  extern __shared__ __align__(128) uint8_t smem[];
  int* csum = reinterpret_cast<int*>(smem);                // [NT * 8] sum of the staged codes per token
  int8_t* qs = reinterpret_cast<int8_t*>(smem + HDR);      // [NT * 8][qst]
  constexpr int TP = NT * 8;
  constexpr int SLOT = RU * 1024;
  uint8_t* rings = smem + HDR + (((size_t)TP * a.qst + 127) & ~(size_t)127);

  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int g = lane >> 2, t = lane & 3;
  const int sl = (int)blockIdx.x / a.cps, j = (int)blockIdx.x % a.cps;
  const int nitems = (a.nunits + RU - 1) / RU;             // items of one slice
  const int p_lo = (int)((int64_t)nitems * j / a.cps), p_hi = (int)((int64_t)nitems * (j + 1) / a.cps);
  const int c_lo = (int)((int64_t)sl * a.nchunks / a.NS), c_hi = (int)((int64_t)(sl + 1) * a.nchunks / a.NS);
  const int nw = c_hi - c_lo;
  const int64_t steps = (int64_t)(p_hi - p_lo) * nw;
  const int s_lo = (int)(steps * warp / MW), s_hi = (int)(steps * (warp + 1) / MW);

  if (threadIdx.x == 0) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  const uint32_t ring = smem_u32(rings + (size_t)warp * DEPTH * SLOT) + lane * 16;
  const uint32_t qs_u32 = smem_u32(qs);
  const uint8_t* const ring_ptr = rings + (size_t)warp * DEPTH * SLOT + lane * 16;

  // weights of item p, unit r of it, chunk c of the slice: lane's 16 bytes of rows 0-7 (+512: rows 8-15)
  const uint8_t* const base = a.packed + (int64_t)c_lo * 1024 + lane * 16;
  auto fill = [&](uint32_t slot_addr, int p, int c) {
#pragma unroll
    for (int r = 0; r < RU; ++r) {
      const int u = p * RU + r;
      if (u < a.nunits) {
        const uint8_t* src = base + (int64_t)u * a.unit_bytes + (int64_t)c * 1024;
        cp16(slot_addr + r * 1024, src, pol);
        cp16(slot_addr + r * 1024 + 512, src + 512, pol);
      }
    }
  };
  // the weights do not depend on the staged codes: request the warp's first steps now
  int pf_p = p_lo + s_lo / nw, pf_c = s_lo % nw, pf_s = s_lo;   // the step requested next
  auto request = [&](uint32_t slot_addr) {
    if (pf_s < s_hi) {
      fill(slot_addr, pf_p, pf_c);
      ++pf_s;
      if (++pf_c == nw) pf_c = 0, ++pf_p;
    }
    cp_commit();
  };
#pragma unroll
  for (int d = 0; d < DEPTH; ++d) request(ring + d * SLOT);

  // everything below reads what earlier kernels in the stream wrote (the codes, the workspace)
  asm volatile("griddepcontrol.wait;" ::: "memory");
  // ---- stage the codes of columns [256 c_lo, 256 c_hi) of every token; zero beyond K and beyond T
  {
    const int per_row = nw * 16;                         // 16-byte pieces per token
    const int64_t k0 = (int64_t)c_lo * 256;
    for (int idx = threadIdx.x; idx < TP * per_row; idx += MTHREADS) {
      const int tok = idx / per_row, jj = idx - tok * per_row;
      const int64_t k = k0 + (int64_t)jj * 16;
      // piece jj % 16 = 4t + 2h + sp of a chunk goes to place 4(2h + sp) + t: the four lanes t of one B load
      // then read 64 consecutive bytes, and with rows 64 bytes (mod 128) apart every quarter-warp of a
      // 16-byte load covers all banks once
      const uint32_t dst = qs_u32 + tok * a.qst + (jj & ~15) * 16 + (((jj & 3) << 2) | ((jj >> 2) & 3)) * 16;
      if (tok < a.T && k + 16 <= a.K) {
        cp16_keep(dst, a.q + (int64_t)tok * a.K + k);
      } else {
        asm volatile("st.shared.v4.u32 [%0], {%1,%1,%1,%1};" ::"r"(dst), "r"(0) : "memory");
      }
    }
    cp_commit();
    cp_wait<0>();
    __syncthreads();
    // per-token sum of the staged codes (the correction for code = w + 1)
    for (int tok = warp; tok < TP; tok += MW) {
      int sum = 0;
      const uint4* row = reinterpret_cast<const uint4*>(qs + (size_t)tok * a.qst);
      for (int i = lane; i < per_row; i += 32) {
        const uint4 v = row[i];
        sum = __dp4a((int)v.x, 0x01010101, sum);
        sum = __dp4a((int)v.y, 0x01010101, sum);
        sum = __dp4a((int)v.z, 0x01010101, sum);
        sum = __dp4a((int)v.w, 0x01010101, sum);
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
      if (lane == 0) csum[tok] = sum;
    }
    __syncthreads();
  }

  // token g of tile 0 under this lane's weight columns
  const int8_t* const q_lane = qs + g * a.qst + t * 16;
  const int tile_stride = 8 * a.qst;
  uint32_t slot_off = 0;
  int C[RU][NT][NSL][4];

  // One step: the oldest ring slot (chunk c of the current item) through the tensor cores, then the slot is
  // refilled with the step DEPTH places further on.
  auto step = [&](const int8_t* qp) {
    cp_wait<DEPTH - 1>();
    unsigned w[RU][4], v[RU][4];
#pragma unroll
    for (int r = 0; r < RU; ++r) {
      const uint4 lo4 = *reinterpret_cast<const uint4*>(ring_ptr + slot_off + r * 1024);
      const uint4 hi4 = *reinterpret_cast<const uint4*>(ring_ptr + slot_off + r * 1024 + 512);
      w[r][0] = lo4.x, w[r][1] = lo4.y, w[r][2] = lo4.z, w[r][3] = lo4.w;
      v[r][0] = hi4.x, v[r][1] = hi4.y, v[r][2] = hi4.z, v[r][3] = hi4.w;
    }
    // Words 2h, 2h+1 of the lane's 16 bytes and slots 2sp, 2sp+1: 16 of the lane's 64 columns.  One group =
    // those B loads for all token tiles, then 2 x NT x RU MMAs that go to NT x RU different accumulators
    // before any of them is used again.
#pragma unroll
    for (int h = 0; h < 2; ++h) {
#pragma unroll
      for (int sp = 0; sp < 2; ++sp) {
        uint4 qb[NT];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
          qb[nt] = *reinterpret_cast<const uint4*>(qp + nt * tile_stride + h * 128 + sp * 64);
#pragma unroll
        for (int s2 = 0; s2 < 2; ++s2) {
          const int sl4 = 2 * sp + s2;                 // the slot
          unsigned A[RU][4];
#pragma unroll
          for (int r = 0; r < RU; ++r) {
            const unsigned src4[4] = {w[r][2 * h], v[r][2 * h], w[r][2 * h + 1], v[r][2 * h + 1]};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              if (NSL == 4) A[r][i] = src4[i] & (0x03030303u << (2 * sl4));
              else if (NSL == 2) A[r][i] = (src4[i] >> (2 * s2)) & (0x03030303u << (4 * sp));
              else A[r][i] = (src4[i] >> (2 * sl4)) & 0x03030303u;
            }
          }
#pragma unroll
          for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int r = 0; r < RU; ++r)
              mma_u8s8(C[r][nt][NSL == 4 ? sl4 : (NSL == 2 ? sp : 0)], A[r][0], A[r][1], A[r][2], A[r][3],
                       s2 ? (int)qb[nt].z : (int)qb[nt].x, s2 ? (int)qb[nt].w : (int)qb[nt].y);
        }
      }
    }
    request(ring + slot_off);
    slot_off = (slot_off + SLOT == DEPTH * SLOT) ? 0 : slot_off + SLOT;
  };

  auto clear = [&]() {
#pragma unroll
    for (int r = 0; r < RU; ++r)
#pragma unroll
      for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int s = 0; s < NSL; ++s)
#pragma unroll
          for (int i = 0; i < 4; ++i) C[r][nt][s][i] = 0;
  };
  // Adds the accumulators (the sums over chunks [c_first, c_end) of item p and this slice) to the workspace
  // (integer sums: any order gives the same).
  // fragment: c[0] = (row g, token 2t), c[1] = (row g, token 2t+1), c[2], c[3] = the same for row g+8
  auto flush = [&](int p, int c_first) {
    // "- sum(q)" belongs to the whole slice: the warp that holds the slice's first chunk subtracts it
    const bool with_corr = c_first == 0;
#pragma unroll
    for (int r = 0; r < RU; ++r) {
      const int row0 = (p * RU + r) * 16;
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          int val;
          if (NSL == 4) val = C[r][nt][0][i] + (C[r][nt][1][i] >> 2) + (C[r][nt][2][i] >> 4) + (C[r][nt][NSL - 1][i] >> 6);
          else if (NSL == 2) val = C[r][nt][0][i] + (C[r][nt][NSL - 1][i] >> 4);
          else val = C[r][nt][0][i];
          const int tok = nt * 8 + 2 * t + (i & 1);
          const int row = row0 + g + 8 * (i >> 1);
          if (tok < a.T && row < a.M) {
            if (with_corr) val -= csum[tok];
            atomicAdd(a.ws + (int64_t)tok * a.M + row, val);
          }
        }
      }
    }
  };
  int p = p_lo + s_lo / nw, c = s_lo % nw, c_first = c;
  clear();
  for (int s = s_lo; s < s_hi; ++s) {
    step(q_lane + c * 256);
    if (++c == nw || s + 1 == s_hi) {
      flush(p, c_first);
      clear();
      c = 0, c_first = 0, ++p;
    }
  }
  cp_wait<0>();

  // ---- closing rescale (Alg. 1's last line), small batches.  The NS CTAs with the same j (one per K-slice)
  // add into the same rows; the one that arrives last finds the complete sums, writes
  // y = float(acc) * (act_scale[t] * w_scale) and puts the zeros back for the next call.  Only cps CTAs do
  // this, each at the bandwidth of one SM: measured on the 100B shapes against a second kernel over all SMs,
  // 8 tokens 81.6 vs 84.1 us per layer, 16 tokens 101.3 vs 100.6, 64 tokens 275 vs 223.
  if (NT > FINISH_IN_KERNEL_MAX_NT) return;
  int* last_flag = reinterpret_cast<int*>(smem + 256);
  __threadfence();                       // this thread's additions are visible before the CTA is counted
  __syncthreads();
  if (threadIdx.x == 0) *last_flag = (atomicAdd(a.cnt + j, 1) == a.NS - 1);
  __syncthreads();
  if (*last_flag) {
    __threadfence();
    const int row_lo = p_lo * RU * 16;
    const int row_hi = p_hi * RU * 16 < a.M ? p_hi * RU * 16 : a.M;
    const int nrows = row_hi - row_lo, total = a.T * nrows;
    constexpr int U = 4;
    for (int e0 = threadIdx.x; e0 < total; e0 += U * MTHREADS) {
      int val[U];
      int64_t off[U];
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const int e = e0 + u * MTHREADS;
        const int tok = e / nrows;
        off[u] = (int64_t)tok * a.M + row_lo + (e - tok * nrows);
        val[u] = e < total ? __ldcg(a.ws + off[u]) : 0;
      }
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const int e = e0 + u * MTHREADS;
        if (e < total) {
          a.ws[off[u]] = 0;
          a.y[off[u]] = __fmul_rn((float)val[u], __fmul_rn(__ldg(a.act_scale + e / nrows), a.w_scale));
          if (a.acc_out) a.acc_out[off[u]] = val[u];
        }
      }
    }
    if (threadIdx.x == 0) a.cnt[j] = 0;
  }
}

// The closing rescale of Alg. 1 over the finished sums: y = float(acc) * (act_scale[t] * w_scale); puts the
// zeros back into the workspace for the next call.
__global__ void __launch_bounds__(256) finish_mid_kernel(int32_t* __restrict__ ws, const float* __restrict__ act_scale,
                                                         float w_scale, int T, int M, float* __restrict__ y,
                                                         int32_t* __restrict__ acc_out) {
  if (threadIdx.x == 0) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int64_t n = (int64_t)T * M;
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  if ((M & 3) == 0) {
    for (int64_t i = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * 4; i < n; i += stride * 4) {
      const int4 v = *reinterpret_cast<const int4*>(ws + i);
      *reinterpret_cast<int4*>(ws + i) = make_int4(0, 0, 0, 0);
      const float sc = __fmul_rn(act_scale[i / M], w_scale);
      float4 o;
      o.x = __fmul_rn((float)v.x, sc), o.y = __fmul_rn((float)v.y, sc);
      o.z = __fmul_rn((float)v.z, sc), o.w = __fmul_rn((float)v.w, sc);
      *reinterpret_cast<float4*>(y + i) = o;
      if (acc_out) *reinterpret_cast<int4*>(acc_out + i) = v;
    }
  } else {
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) {
      const int v = ws[i];
      ws[i] = 0;
      y[i] = __fmul_rn((float)v, __fmul_rn(act_scale[i / M], w_scale));
      if (acc_out) acc_out[i] = v;
    }
  }
}


// bytes of the [T][M] sums at the head of the workspace; one arrival counter per CTA of a slice follows
constexpr size_t MID_WS_COUNTERS = 1024;
inline size_t mid_ws_sums(int T, int64_t M) { return (((size_t)T * (size_t)M * 4) + 15) & ~(size_t)15; }

int env_int(const char* name, int dflt) {
  const char* v = getenv(name);
  return (v && *v) ? atoi(v) : dflt;
}

struct MidCfg { int NT, RU, DEPTH; };
// Measured on the 100B shapes (us per layer, RU 2 vs 1): NT = 2: 91 vs 91 (ring of 8) or 106 (ring of 4); NT = 3:
// 117 vs 114; NT = 4: 145 vs 132 (ring of 8): from three token tiles on, one unit per step with the cheaper
// two-set field extraction wins over sharing the B loads between two units.
inline MidCfg mid_cfg(int T) {
  const int NT = (T + 7) / 8;
  if (NT <= 2) return {NT, 2, 4};
  if (NT == 3) return {NT, 1, 4};
  if (NT == 4) return {NT, 1, 8};
  return {NT, 1, 4};
}

struct MidPlan {
  MidCfg c;
  int nchunks, NS, cps, nunits, grid, qst;
  size_t smem;
};

bool make_mid_plan(int T, int64_t M, int64_t K, MidPlan* p) {
  if (T < 1 || T > 64 || K < 16 || (K % 16) != 0 || M < 1) return false;   // (K < 1 would leave no chunk to slice)
  p->c = mid_cfg(T);
  const int TP = p->c.NT * 8;
  p->nchunks = (int)(i2s_kp(K) / 256);
  p->nunits = (int)ceil_div(M, 16);
  const size_t optin = (size_t)dev_info().max_smem_optin;
  const size_t rings = (size_t)MW * p->c.DEPTH * p->c.RU * 1024;
  if (optin < rings + HDR + 4096) return false;
  const size_t qcap = optin - rings - HDR - 128;
  const int sc_max = (int)((qcap / TP - 64) / 256);         // chunks of a slice whose codes fit
  if (sc_max < 1) return false;
  const int ns_min = (int)ceil_div(p->nchunks, sc_max);
  const int sms = dev_info().sm_count;
  if (ns_min > sms || (size_t)sms * 4 > MID_WS_COUNTERS) return false;
  // the smallest number of slices that fits, unless one or two more leave fewer SMs without a CTA
  const int64_t items = ceil_div(p->nunits, p->c.RU);
  int ns = ns_min, best_idle = sms;
  for (int cand = ns_min; cand <= ns_min + 2 && cand <= p->nchunks && cand <= sms; ++cand) {
    const int64_t cps = items < sms / cand ? items : sms / cand;
    const int idle = sms - (int)(cps * cand);
    if (idle < best_idle) best_idle = idle, ns = cand;
  }
  static const int forced = env_int("BITNET_MID_NS", 0);   // read once
  if (forced >= ns_min && forced <= p->nchunks && forced <= sms) ns = forced;
  p->NS = ns;
  p->cps = (int)(items < sms / ns ? items : sms / ns);
  p->grid = p->cps * ns;
  p->qst = (int)ceil_div(p->nchunks, ns) * 256 + 64;
  p->smem = HDR + (((size_t)TP * p->qst + 127) & ~(size_t)127) + rings;
  return p->smem <= optin;
}

template <int NT, int RU, int DEPTH, int NSL>
int launch_mid(const MArgs& a, const MidPlan& p, cudaStream_t st) {
  static bool attr_set[64] = {false};
  int dev = 0;
  cudaGetDevice(&dev);
  if (!attr_set[dev & 63]) {
    cudaError_t e = cudaFuncSetAttribute(gemv_i2s_mid_kernel<NT, RU, DEPTH, NSL>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, dev_info().max_smem_optin);
    if (e != cudaSuccess) return note_cuda_error(e);
    attr_set[dev & 63] = true;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)p.grid);
  cfg.blockDim = dim3(MTHREADS);
  cfg.dynamicSmemBytes = p.smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = early_start_enabled(st) ? 1 : 0;
  cudaError_t e = cudaLaunchKernelEx(&cfg, gemv_i2s_mid_kernel<NT, RU, DEPTH, NSL>, a);
  return e == cudaSuccess ? BITNET_OK : note_cuda_error(e);
}

}  // namespace

// y = float(sums) * (act_scale[t] * w_scale) over a [T][M] int32 array, which is left zeroed.
int launch_rescale_sums(int32_t* sums, const float* act_scale, float w_scale, int64_t T, int64_t M, float* y,
                        int32_t* acc_out, cudaStream_t st) {
  const int64_t n4 = (T * M + 3) / 4;
  const int64_t want = (n4 + 255) / 256;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(want < 8 * 148 ? want : 8 * 148));
  cfg.blockDim = dim3(256);
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = early_start_enabled(st) ? 1 : 0;
  cudaError_t e = cudaLaunchKernelEx(&cfg, finish_mid_kernel, sums, act_scale, w_scale, (int)T, (int)M, y, acc_out);
  return e == cudaSuccess ? BITNET_OK : note_cuda_error(e);
}

bool gemv_i2s_mid_supported(int T, int64_t M, int64_t K) {
  MidPlan p;
  return make_mid_plan(T, M, K, &p);
}

size_t gemv_i2s_mid_workspace_bytes(int T, int64_t M, int64_t K) {
  MidPlan p;
  if (!make_mid_plan(T, M, K, &p)) return 0;
  return mid_ws_sums(T, M) + MID_WS_COUNTERS;
}

int launch_gemv_i2s_mid(const uint8_t* packed, float w_scale, int64_t M, int64_t K, const int8_t* q,
                        const float* act_scale, int T, float* y, int32_t* acc_out, void* ws, size_t ws_bytes,
                        cudaStream_t st) {
  MidPlan p;
  if (!make_mid_plan(T, M, K, &p)) return BITNET_ERR_UNSUPPORTED_SHAPE;
  const size_t need = mid_ws_sums(T, M) + MID_WS_COUNTERS;
  if (!ws || ws_bytes < need) return BITNET_ERR_WORKSPACE;
  MArgs a;
  a.packed = packed;
  a.unit_bytes = 4 * i2s_kp(K);
  a.M = (int)M;
  a.K = K;
  a.q = q;
  a.act_scale = act_scale;
  a.w_scale = w_scale;
  a.T = T;
  a.y = y;
  a.acc_out = acc_out;
  a.ws = reinterpret_cast<int32_t*>(ws);
  a.cnt = reinterpret_cast<int*>(reinterpret_cast<uint8_t*>(ws) + mid_ws_sums(T, M));
  a.nchunks = p.nchunks;
  a.NS = p.NS;
  a.cps = p.cps;
  a.nunits = p.nunits;
  a.qst = p.qst;
  log_launch("gemv_i2s_mid_kernel<NT=%d,RU=%d,DEPTH=%d> T=%d M=%lld K=%lld grid=%d K-slices=%d CTAs/slice=%d smem=%zu%s",
             p.c.NT, p.c.RU, p.c.DEPTH, T, (long long)M, (long long)K, p.grid, p.NS, p.cps, p.smem,
             p.c.NT <= FINISH_IN_KERNEL_MAX_NT ? "" : " + finish_mid_kernel");
  int rc;
  switch (p.c.NT) {
    case 1: rc = launch_mid<1, 2, 4, 4>(a, p, st); break;
    case 2: rc = launch_mid<2, 2, 4, 2>(a, p, st); break;
    case 3: rc = launch_mid<3, 1, 4, 2>(a, p, st); break;
    case 4: rc = launch_mid<4, 1, 8, 2>(a, p, st); break;
    case 5: rc = launch_mid<5, 1, 4, 1>(a, p, st); break;
    case 6: rc = launch_mid<6, 1, 4, 1>(a, p, st); break;
    case 7: rc = launch_mid<7, 1, 4, 1>(a, p, st); break;
    case 8: rc = launch_mid<8, 1, 4, 1>(a, p, st); break;
    default: return BITNET_ERR_UNSUPPORTED_SHAPE;
  }
  if (rc || p.c.NT <= FINISH_IN_KERNEL_MAX_NT) return rc;
  return launch_rescale_sums(a.ws, act_scale, w_scale, T, M, y, acc_out, st);
}

}  // namespace bitnet
