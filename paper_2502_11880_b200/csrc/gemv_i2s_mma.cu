// I2_S mpGEMV for decode (1..8 tokens), streaming kernel: Alg. 1 Phase 2 from the 2-bit blob, with
// the quantiser (Phase 1) optionally fused in.
//
// Memory side.  Persistent CTAs, one per SM, whose ring buffer takes the SM's shared memory (~220 KB
// per SM, ~32 MB over the GPU).  The matrix is cut into units of 16 rows -- the blob stores a unit
// contiguously and chunk-major (1024 bytes per 256-column chunk, 64 bytes per row), so any K-slab of
// a unit (at most 32 chunks = 32 KB) is ONE bulk asynchronous copy (cp.async.bulk global -> shared,
// completion counted on an mbarrier) into a ring slot.  Unit u belongs to CTA u mod gridDim.  Issuing
// a bulk copy costs the issuing lane a few hundred cycles whatever its size, hence large copies, and
// there is no producer thread: the warp that is last to finish reading a slot refills it.  Weights
// never depend on the previous kernel in the stream; under programmatic dependent launch the CTA
// starts as soon as an SM is free, and only the activation loads wait for that kernel
// (griddepcontrol.wait).
//
// Compute side.  16 warps in groups that work on alternate units.  A unit is the A operand of int8
// tensor-core MMAs (mma.sync m16n8k32, u8 x s8 -> s32): lane (g = lane/4, t = lane%4) reads 16 bytes =
// 64 weights of row g and of row g+8 -- the 32 lanes read 512 contiguous bytes each time, conflict
// free.  Masking a packed word with 0x03030303 << 2s leaves, without any shift, the four codes of slot
// s scaled by 4^s: exactly one A register (one row, four consecutive k).  The B operand is the
// activations: column n of B is token n, so lane (g,t) keeps token g's 64 activations for its
// k-column in registers, the same for every unit the CTA processes; the blob's word order makes the
// two activation words of an MMA adjacent.  One MMA does the work of 32 dp4a and the reduction over k
// happens inside the tensor core, so there are no shuffle reductions, and batches of 1..8 tokens cost
// the same.  Four accumulator fragments carry the slot scales 1, 4, 16, 64; each is an exact multiple
// of its scale, so arithmetic shifts undo it, and sum(code*q) - sum(q) = sum(w*q).  The warps of a
// group cover different chunks; their fragments meet in shared memory (atomicAdd + arrival counter)
// and the last warp rescales and stores y = acc * act_scale[t] * w_scale.  K longer than one slab
// is walked slab by slab for the same unit, the accumulators staying in registers and the activation
// registers being reloaded from shared memory, so nothing is exchanged between CTAs and no workspace
// is needed.
//
// Fused quantiser: with fp32 activations given, every CTA computes the absmax and the int8 codes
// itself (the row stays in registers between the two passes) while its first weight tiles are in
// flight; CTA 0 also stores the codes and scales for the caller.
//
// Every wait on an mbarrier is bounded; a wait that gives up raises a device flag that
// bitnet_device_status() reports, and the thread leaves the kernel.
#include <cstdlib>
#include <cstring>

#include "common.cuh"
#include "device_utils.cuh"

namespace bitnet {
namespace {

constexpr int CW = 16;                   // warps (all consume)
constexpr int WPT_MAX = 8;               // warps that share one unit
constexpr int THREADS = CW * 32;
constexpr int MAX_SLOTS = 12;            // ring slots, one unit-slab (16 rows x up to 32 chunks) each
constexpr int XREG = 16;                 // float4 registers per thread of the fused quantiser's fast path
constexpr int ACC_RING = 16;             // cross-warp accumulator entries (more than the units warps can drift apart)
constexpr uint32_t WAIT_LIMIT = 1u << 22;

static __device__ int g_stream_error = 0;


struct MmaArgs {
  const uint8_t* packed;
  int64_t unit_bytes;    // bytes of one 16-row block of the blob = 4 * Kp
  int M;
  int64_t K;
  const int8_t* q;       // quantised activations [T][K] (input, or output of the fused quantiser)
  const float* act_scale;
  const float* x;        // fp32 activations [T][K]: non-null selects the fused quantiser
  int8_t* q_out;         // fused mode: CTA 0 stores the codes and scales here
  float* scale_out;
  int use_qs;            // activations staged in shared memory ([T][Kp] int8)
  float w_scale;
  int T;
  float* y;
  int32_t* acc_out;
  int nchunks;           // 256-column chunks per row (Kp / 256)
  int nq;                // K-slabs per unit
  int slab_chunks;       // chunks per slab
  int stage_bytes;       // slab_chunks * 1024 = ring slot size
  int wpt;               // warps per unit (each covers KS chunks of a slab)
  int ngroups;           // warp groups; group g takes the CTA's units g, g + ngroups, ...
  int nunits;            // ceil(M / 16)
  int slots;             // ring slots
};

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// Bounded wait for the phase with the given parity; false = gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
  for (uint32_t it = 0; it < WAIT_LIMIT; ++it) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    if (ok) return true;
  }
  return false;
}
__device__ __forceinline__ void st_release_cta(int* p, int v) {
  asm volatile("st.release.cta.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(p)), "r"(v) : "memory");
}
// Bounded wait until *p == want (acquire).
__device__ __forceinline__ bool wait_issued(const int* p, int want) {
  const uint32_t addr = smem_u32(p);
  for (uint32_t it = 0; it < WAIT_LIMIT; ++it) {
    int v;
    asm volatile("ld.acquire.cta.shared::cta.b32 %0, [%1];" : "=r"(v) : "r"(addr) : "memory");
    if (v == want) return true;
  }
  return false;
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar, uint64_t pol) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
      ::"r"(dst), "l"(src), "r"(bytes), "r"(bar), "l"(pol)
      : "memory");
}

// KS = chunks (256 weights each) a warp covers per slab.
template <int KS>
__global__ void __launch_bounds__(THREADS, 1) gemv_i2s_mma_kernel(const MmaArgs a) {
  extern __shared__ __align__(128) uint8_t smem[];
  // layout: [full barriers][readers-done counters][acc counters][acc sums][quantiser scratch][codes][ring]
  uint64_t* full = reinterpret_cast<uint64_t*>(smem);
  int* rcnt = reinterpret_cast<int*>(full + MAX_SLOTS);
  int* issued = rcnt + MAX_SLOTS;                              // 1 + the tile last requested into each slot
  int* cnt = issued + MAX_SLOTS;
  int* acc = cnt + ACC_RING;                                   // [ACC_RING][T][16]
  const uint32_t head = (uint32_t)((MAX_SLOTS * 16 + ACC_RING * 4 * (1 + a.T * 16) + 127) & ~127);
  float* qscale = reinterpret_cast<float*>(smem + head);       // [8] act_scale per token
  float* qred = qscale + 8;                                    // [8][16] partial maxima / multipliers
  int8_t* qs_mem = reinterpret_cast<int8_t*>(smem + head + 1024);
  const int kp = a.nchunks * 256;
  uint8_t* ring = smem + head + 1024 + (a.use_qs ? ((a.T * kp + 127) & ~127) : 0);

  const int lane = threadIdx.x & 31;
  const int warp = threadIdx.x >> 5;
  const int n_units = (a.nunits - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;
  const int total = a.nq * n_units;            // tiles this CTA streams, in order: unit-major, then slab

  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  // Issues the copy of tile `seq` (one K-slab of one unit, contiguous in the blob) into `slot`.
  auto fill = [&](int seq, int slot) {
    const int ul = seq / a.nq;
    const int ph = seq - ul * a.nq;
    const int c0 = ph * a.slab_chunks;
    const uint32_t bytes = (uint32_t)min(a.slab_chunks, a.nchunks - c0) * 1024u;
    const uint8_t* src = a.packed + ((int64_t)blockIdx.x + (int64_t)ul * gridDim.x) * a.unit_bytes + (int64_t)c0 * 1024;
    const uint32_t bar = smem_u32(full + slot);
    mbar_expect_tx(bar, bytes);
    bulk_g2s(smem_u32(ring + (size_t)slot * a.stage_bytes), src, bytes, bar, pol);
    // Publish which tile the slot's barrier now counts for.  A parity wait tells two phases apart only;
    // a group that has not itself read the slot's previous tile must not mistake that tile's phase
    // (or the fresh barrier) for this one, so readers first wait for this number.
    st_release_cta(issued + slot, seq + 1);
  };

  if (threadIdx.x == 0) {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the next kernel may begin its prologue
    for (int s = 0; s < a.slots; ++s) mbar_init(smem_u32(full + s), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  for (int i = threadIdx.x; i < 2 * MAX_SLOTS + ACC_RING * (1 + a.T * 16); i += THREADS) rcnt[i] = 0;
  __syncthreads();

  const int group = warp / a.wpt;
  const bool idle = group >= a.ngroups;   // warps that do not fit a whole group only help in the prologue
  const int wk = warp % a.wpt;            // this warp's chunks inside a slab: wk*KS .. wk*KS+KS-1
  const int g = lane >> 2, t = lane & 3;
  // One warp per slot requests the initial contents of the ring.  The weights do not depend on the previous
  // kernel in the stream, so this happens before the wait below: a CTA that starts while that kernel's
  // last CTAs are still running already streams.
  if (lane == 0 && warp < a.slots && warp < total) fill(warp, warp);

  // ---------------- activations come from the previous kernel in the stream
  asm volatile("griddepcontrol.wait;" ::: "memory");

  if (a.use_qs) {
    if (a.x && a.T == 1 && a.K <= 4 * XREG * THREADS) {
      // ---- fused quantiser (Alg. 1 Phase 1), one token, one round trip: the row stays in registers
      // between the amax pass and the rounding pass.  Same operations and order as the stand-alone
      // kernel: s = 127 / max(amax, 1e-5), q = clamp(rint(x * s)).
      const float4* x4 = reinterpret_cast<const float4*>(a.x);
      const int n4 = (int)(a.K / 4);
      float4 xv[XREG];
#pragma unroll
      for (int r = 0; r < XREG; ++r) {
        const int i = threadIdx.x + r * THREADS;
        xv[r] = (i < n4) ? __ldcg(x4 + i) : make_float4(0.f, 0.f, 0.f, 0.f);
      }
      float m = 0.0f;
#pragma unroll
      for (int r = 0; r < XREG; ++r)
        m = fmaxf(m, fmaxf(fmaxf(fabsf(xv[r].x), fabsf(xv[r].y)), fmaxf(fabsf(xv[r].z), fabsf(xv[r].w))));
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
      if (lane == 0) qred[warp] = m;
      __syncthreads();
      float amax = 0.0f;
#pragma unroll
      for (int w2 = 0; w2 < CW; ++w2) amax = fmaxf(amax, qred[w2]);
      const float amax_c = fmaxf(amax, 1e-5f);
      const float sq = __fdiv_rn(127.0f, amax_c);
      if (threadIdx.x == 0) {
        const float inv = __fdiv_rn(amax_c, 127.0f);
        qscale[0] = inv;
        if (blockIdx.x == 0 && a.scale_out) a.scale_out[0] = inv;
      }
#pragma unroll
      for (int r = 0; r < XREG; ++r) {
        const int i = threadIdx.x + r * THREADS;
        if (i < kp / 4) {
          const int word = quant4(xv[r], sq);                 // columns K..Kp-1 came in as zeros
          reinterpret_cast<int*>(qs_mem)[i] = word;
          if (blockIdx.x == 0 && a.q_out && i < n4) reinterpret_cast<int*>(a.q_out)[i] = word;
        }
      }
    } else if (a.x) {
      // ---- fused quantiser, general form: amax per token, then a second pass over x
      for (int tok = 0; tok < a.T; ++tok) {
        const float4* x4 = reinterpret_cast<const float4*>(a.x + (int64_t)tok * a.K);
        float m = 0.0f;
        for (int i = threadIdx.x; i < (int)(a.K / 4); i += THREADS) {
          const float4 v = __ldcg(x4 + i);
          m = fmaxf(m, fmaxf(fmaxf(fabsf(v.x), fabsf(v.y)), fmaxf(fabsf(v.z), fabsf(v.w))));
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
        if (lane == 0) qred[tok * CW + warp] = m;
      }
      __syncthreads();
      if (threadIdx.x < a.T) {
        float m = 0.0f;
        for (int w2 = 0; w2 < CW; ++w2) m = fmaxf(m, qred[threadIdx.x * CW + w2]);
        const float amax_c = fmaxf(m, 1e-5f);
        qred[threadIdx.x * CW] = __fdiv_rn(127.0f, amax_c);
        const float inv = __fdiv_rn(amax_c, 127.0f);
        qscale[threadIdx.x] = inv;
        if (blockIdx.x == 0 && a.scale_out) a.scale_out[threadIdx.x] = inv;
      }
      __syncthreads();
      for (int tok = 0; tok < a.T; ++tok) {
        const float sq = qred[tok * CW];
        const float4* x4 = reinterpret_cast<const float4*>(a.x + (int64_t)tok * a.K);
        for (int i = threadIdx.x; i < kp / 4; i += THREADS) {
          int word = 0;
          if (i < (int)(a.K / 4)) {
            word = quant4(__ldcg(x4 + i), sq);
            if (blockIdx.x == 0 && a.q_out) reinterpret_cast<int*>(a.q_out + (int64_t)tok * a.K)[i] = word;
          }
          reinterpret_cast<int*>(qs_mem + tok * kp)[i] = word;
        }
      }
    } else {
      // ---- stage the given codes (zero beyond K): every warp and every slab reads them from shared memory
      for (int tok = 0; tok < a.T; ++tok) {
        const int* q4 = reinterpret_cast<const int*>(a.q + (int64_t)tok * a.K);
        for (int i = threadIdx.x; i < kp / 4; i += THREADS)
          reinterpret_cast<int*>(qs_mem + tok * kp)[i] = (i < (int)(a.K / 4)) ? __ldcg(q4 + i) : 0;
      }
      if (threadIdx.x < a.T) qscale[threadIdx.x] = __ldcg(a.act_scale + threadIdx.x);
    }
    __syncthreads();
  }
  if (idle) return;

  // rescale factors of the tokens this lane stores when its warp finishes a unit (token (lane>>4) + 2i)
  float sc[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int tok = (lane >> 4) + 2 * i;
    const float as = (tok < a.T) ? (a.use_qs ? qscale[tok] : __ldcg(a.act_scale + tok)) : 0.0f;
    sc[i] = __fmul_rn(as, a.w_scale);
  }
  const int lane_off = (wk * KS) * 1024 + g * 64 + t * 16;

  // activations of one slab: token g, the 64 values under this lane's 16-byte weight column, per chunk
  int qr[KS][16];
  bool ksok[KS];
  int qs_even = 0, qs_odd = 0;   // sums of the activations of tokens 2t and 2t+1 over this warp's chunks
  auto load_q = [&](int ph) {
    const int slab_n = min(a.slab_chunks, a.nchunks - ph * a.slab_chunks);
    int qs = 0;
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
      const int cl = wk * KS + ks;                                          // chunk inside the slab
      const int64_t k0 = (int64_t)(ph * a.slab_chunks + cl) * 256 + t * 64;  // first of the lane's 64 columns
      ksok[ks] = cl < slab_n;
      if (ksok[ks] && k0 < a.K && g < a.T) {
        const uint4* qp = a.use_qs ? reinterpret_cast<const uint4*>(qs_mem + g * kp + k0)
                                   : reinterpret_cast<const uint4*>(a.q + (int64_t)g * a.K + k0);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const uint4 v = a.use_qs ? qp[i] : __ldcg(qp + i);
          qr[ks][4 * i + 0] = (int)v.x;
          qr[ks][4 * i + 1] = (int)v.y;
          qr[ks][4 * i + 2] = (int)v.z;
          qr[ks][4 * i + 3] = (int)v.w;
        }
      } else {
#pragma unroll
        for (int i = 0; i < 16; ++i) qr[ks][i] = 0;
      }
#pragma unroll
      for (int i = 0; i < 16; ++i) qs = __dp4a(qr[ks][i], 0x01010101, qs);
    }
    qs += __shfl_xor_sync(0xffffffffu, qs, 1);
    qs += __shfl_xor_sync(0xffffffffu, qs, 2);
    qs_even = __shfl_sync(0xffffffffu, qs, (2 * t) * 4);
    qs_odd = __shfl_sync(0xffffffffu, qs, (2 * t + 1) * 4);
  };
  if (a.nq == 1) load_q(0);

  for (int ul = group; ul < n_units; ul += a.ngroups) {
    int seq = ul * a.nq;
    int slot = seq % a.slots;
    uint32_t par = (uint32_t)(seq / a.slots) & 1u;
    int C[4][4];
#pragma unroll
    for (int s = 0; s < 4; ++s)
#pragma unroll
      for (int i = 0; i < 4; ++i) C[s][i] = 0;
    int corr_even = 0, corr_odd = 0;
    for (int ph = 0; ph < a.nq; ++ph, ++seq) {
      if (a.nq > 1) load_q(ph);
      corr_even += qs_even;
      corr_odd += qs_odd;
      if (!wait_issued(issued + slot, seq + 1) || !mbar_wait(smem_u32(full + slot), par)) {
        if (lane == 0) atomicExch(&g_stream_error, BITNET_ERR_TIMEOUT);
        return;
      }
      const uint8_t* pa = ring + lane_off + slot * a.stage_bytes;
#pragma unroll
      for (int ks = 0; ks < KS; ++ks) {
        const uint4 W = ksok[ks] ? *reinterpret_cast<const uint4*>(pa + ks * 1024) : make_uint4(0, 0, 0, 0);
        const uint4 V = ksok[ks] ? *reinterpret_cast<const uint4*>(pa + ks * 1024 + 512) : make_uint4(0, 0, 0, 0);
        const unsigned w4[4] = {W.x, W.y, W.z, W.w};
        const unsigned v4[4] = {V.x, V.y, V.z, V.w};
        // words 2h, 2h+1 of the lane's 16 bytes, slot s: weights 32h + 8s + (0..7) of its 64 columns,
        // i.e. activation words 8h + 2s and 8h + 2s + 1
#pragma unroll
        for (int h = 0; h < 2; ++h) {
#pragma unroll
          for (int s = 0; s < 4; ++s) {
            const unsigned m = 0x03030303u << (2 * s);
            mma_u8s8(C[s], w4[2 * h] & m, v4[2 * h] & m, w4[2 * h + 1] & m, v4[2 * h + 1] & m,
                     qr[ks][8 * h + 2 * s], qr[ks][8 * h + 2 * s + 1]);
          }
        }
      }
      // Every weight of this warp's share has been read (the values are in registers).  The warp that is
      // last to finish with the slot refills it with the tile that comes `slots` later.
      __syncwarp();
      if (lane == 0) {
        if (atomicAdd(rcnt + slot, 1) == a.wpt - 1) {
          atomicExch(rcnt + slot, 0);
          if (seq + a.slots < total) {
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            fill(seq + a.slots, slot);
          }
        }
      }
      if (++slot == a.slots) {
        slot = 0;
        par ^= 1u;
      }
    }
    // fragment: c[0] = (row g, token 2t), c[1] = (row g, token 2t+1), c[2], c[3] = the same for row g+8
    int c[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) c[i] = C[0][i] + (C[1][i] >> 2) + (C[2][i] >> 4) + (C[3][i] >> 6);
    c[0] -= corr_even;
    c[2] -= corr_even;
    c[1] -= corr_odd;
    c[3] -= corr_odd;

    const int e = ul % ACC_RING;
    int* ea = acc + e * a.T * 16;
    if (2 * t < a.T) {
      atomicAdd(ea + (2 * t) * 16 + g, c[0]);
      atomicAdd(ea + (2 * t) * 16 + g + 8, c[2]);
    }
    if (2 * t + 1 < a.T) {
      atomicAdd(ea + (2 * t + 1) * 16 + g, c[1]);
      atomicAdd(ea + (2 * t + 1) * 16 + g + 8, c[3]);
    }
    __syncwarp();
    int last = 0;
    if (lane == 0) {
      __threadfence_block();
      last = atomicAdd(cnt + e, 1) == a.wpt - 1;
    }
    last = __shfl_sync(0xffffffffu, last, 0);
    if (last) {
      // every warp of the group has delivered: rescale and store the 16 rows of this unit
      __threadfence_block();
      const int row0 = ((int)blockIdx.x + ul * (int)gridDim.x) * 16;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int idx = lane + 32 * i;
        if (idx < a.T * 16) {
          const int tok = idx >> 4, row = row0 + (idx & 15);
          const int v = atomicExch(ea + idx, 0);
          if (row < a.M) {
            a.y[(int64_t)tok * a.M + row] = __fmul_rn((float)v, sc[i]);
            if (a.acc_out) a.acc_out[(int64_t)tok * a.M + row] = v;
          }
        }
      }
      if (lane == 0) atomicExch(cnt + e, 0);
    }
  }
}

struct Plan {
  int KS, nchunks, nq, slab_chunks, stage_bytes, wpt, ngroups, nunits, slots, grid, use_qs;
  size_t smem;
};

constexpr size_t MAX_QS_BYTES = 64 * 1024;   // activations staged in shared memory up to this size

// false if this kernel does not cover the shape: the caller falls back to the split-K kernel.
bool make_plan(int T, int64_t M, int64_t K, bool fused, Plan* p) {
  p->nchunks = (int)(i2s_kp(K) / 256);
  p->nq = (p->nchunks + 31) / 32;
  p->slab_chunks = (p->nchunks + p->nq - 1) / p->nq;
  p->KS = (p->slab_chunks + WPT_MAX - 1) / WPT_MAX;
  p->wpt = (p->slab_chunks + p->KS - 1) / p->KS;
  p->ngroups = CW / p->wpt;
  p->stage_bytes = p->slab_chunks * 1024;
  p->nunits = (int)ceil_div(M, 16);
  p->grid = dev_info().sm_count < p->nunits ? dev_info().sm_count : p->nunits;
  const size_t qs_bytes = ((size_t)T * p->nchunks * 256 + 127) & ~(size_t)127;
  // staged activations whenever they fit (required by the fused quantiser)
  p->use_qs = (qs_bytes <= MAX_QS_BYTES) ? 1 : 0;
  if (fused && !p->use_qs) return false;
  const size_t head = (((size_t)MAX_SLOTS * 16 + (size_t)ACC_RING * 4 * (1 + T * 16) + 127) & ~(size_t)127) + 1024 +
                      (p->use_qs ? qs_bytes : 0);
  const size_t budget = (size_t)dev_info().max_smem_optin - 1024;
  if (head + 2 * (size_t)p->stage_bytes > budget) return false;
  int slots = (int)((budget - head) / (size_t)p->stage_bytes);
  if (slots > MAX_SLOTS) slots = MAX_SLOTS;
  p->slots = slots;
  p->smem = head + (size_t)slots * p->stage_bytes;
  return true;
}

template <int KS>
int launch_mma(const MmaArgs& a, const Plan& p, cudaStream_t st) {
  static bool attr_set[64] = {false};
  int dev = 0;
  cudaGetDevice(&dev);
  if (!attr_set[dev & 63]) {
    cudaError_t e = cudaFuncSetAttribute(gemv_i2s_mma_kernel<KS>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         dev_info().max_smem_optin);
    if (e != cudaSuccess) return note_cuda_error(e);
    attr_set[dev & 63] = true;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)p.grid);
  cfg.blockDim = dim3(THREADS);
  cfg.dynamicSmemBytes = p.smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = early_start_enabled(st) ? 1 : 0;
  cudaError_t e = cudaLaunchKernelEx(&cfg, gemv_i2s_mma_kernel<KS>, a);
  return e == cudaSuccess ? BITNET_OK : note_cuda_error(e);
}

}  // namespace

// The warp-private-ring kernel takes every shape it supports (measured faster or equal at every batch size up
// to 8); this file's kernel, which keeps the activations in registers, takes the rest (K below 2048, or
// more staged activations than the other kernel has room for).  BITNET_I2S_STREAM=ring / =warp forces one of them.
static bool prefer_wring(int T) {
  static int v = -1;
  if (v < 0) {
    const char* e = getenv("BITNET_I2S_STREAM");
    v = (e && strcmp(e, "ring") == 0) ? 0 : (e && strcmp(e, "warp") == 0) ? 2 : 1;
  }
  return v == 2 || (v == 1 && T <= 8);
}

bool gemv_i2s_stream_supported(int T, int64_t M, int64_t K, bool fused) {
  if (prefer_wring(T) && gemv_i2s_wring_supported(T, M, K)) return true;
  Plan p;
  return T >= 1 && T <= 8 && make_plan(T, M, K, fused, &p);
}

// x != nullptr: fused quantiser (q, act_scale are then outputs); otherwise q, act_scale are inputs.
int launch_gemv_i2s_stream(const uint8_t* packed, float w_scale, int64_t M, int64_t K, const float* x, int8_t* q,
                           float* act_scale, int T, float* y, int32_t* acc_out, cudaStream_t st) {
  if (prefer_wring(T) && gemv_i2s_wring_supported(T, M, K))
    return launch_gemv_i2s_wring(packed, w_scale, M, K, x, q, act_scale, T, y, acc_out, st);
  Plan p;
  if (T < 1 || T > 8 || !make_plan(T, M, K, x != nullptr, &p)) return BITNET_ERR_UNSUPPORTED_SHAPE;
  MmaArgs a;
  a.packed = packed;
  a.unit_bytes = 4 * i2s_kp(K);
  a.M = (int)M;
  a.K = K;
  a.q = q;
  a.act_scale = act_scale;
  a.x = x;
  a.q_out = x ? q : nullptr;
  a.scale_out = x ? act_scale : nullptr;
  a.use_qs = p.use_qs;
  a.w_scale = w_scale;
  a.T = T;
  a.y = y;
  a.acc_out = acc_out;
  a.nchunks = p.nchunks;
  a.nq = p.nq;
  a.slab_chunks = p.slab_chunks;
  a.stage_bytes = p.stage_bytes;
  a.wpt = p.wpt;
  a.ngroups = p.ngroups;
  a.nunits = p.nunits;
  a.slots = p.slots;
  switch (p.KS) {
    case 1: return launch_mma<1>(a, p, st);
    case 2: return launch_mma<2>(a, p, st);
    case 3: return launch_mma<3>(a, p, st);
    case 4: return launch_mma<4>(a, p, st);
    default: return BITNET_ERR_UNSUPPORTED_SHAPE;
  }
}

int gemv_i2s_stream_status(int* out) {
  cudaError_t e = cudaMemcpyFromSymbol(out, g_stream_error, sizeof(int));
  return e == cudaSuccess ? BITNET_OK : note_cuda_error(e);
}
int gemv_i2s_stream_status_clear() {
  const int zero = 0;
  cudaError_t e = cudaMemcpyToSymbol(g_stream_error, &zero, sizeof(int));
  return e == cudaSuccess ? BITNET_OK : note_cuda_error(e);
}


}  // namespace bitnet
