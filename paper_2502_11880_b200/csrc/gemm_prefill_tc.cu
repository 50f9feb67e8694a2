// Prefill mpGEMM (many tokens), I2_S: Alg. 1 Phase 2 at large T on the int8 tensor cores.
//
//   acc[t,m] = sum_k q[t,k] * w[m,k]        (tcgen05.mma kind::i8, s8 x s8 -> s32 in tensor memory)
//   y[t,m]   = acc[t,m] * act_scale[t] * w_scale
//
// The paper does not treat the prefill stage (its Limitations section); the definition is the same
// as for decode, so the design is this build's.  One persistent CTA per SM walks output tiles of
// 128 out-features x 256 tokens.  Per 128-column K block:
//   * warp 0   : one TMA tensor copy brings the 256 x 128 int8 activation tile straight into the
//                128-byte-swizzled K-major layout the MMA wants (operand B);
//   * warps 2-9: two threads per weight row: each reads 16 of the row's 32 packed bytes from the blob
//                (L2 resident: the whole blob is ~15 MB), expands the 2-bit codes to int8 -1/0/+1 in
//                registers and writes the row of operand A into shared memory in the same swizzled
//                layout (4 conflict-free 16-byte stores), then fence.proxy.async + mbarrier arrive;
//   * warp 1   : one thread issues four tcgen05.mma (M=128, N=256, K=32) per K block, accumulating in
//                tensor memory, and tcgen05.commit releases the stage to the producers;
//   * warps 10-13: epilogue -- tcgen05.ld the finished 128 x 256 accumulator (lane = out-feature,
//                column = token), rescale with the tile's per-token factors (staged in shared memory while the
//                MMAs still run), and hand 32 x 32 boxes of y to bulk tensor stores through a 4 KB staging
//                buffer per warp (plain stores when the raw accumulators are wanted or M % 4 != 0; integer
//                atomics into the workspace when a tile's K is cut into parts).  Two accumulators (2 x 256 of
//                the 512 tensor-memory columns) let the epilogue of a tile overlap the MMAs of the next.
// Work items are whole tiles, or, when the output has fewer tiles than three quarters of the SMs, parts of a
// tile's K whose sums meet in the workspace and are rescaled by a second kernel.
// Every mbarrier wait is bounded; a wait that gives up sets a CTA-wide abort flag and the device
// status word, all roles leave their loops, and the CTA frees its tensor memory before it exits.
#include <cuda.h>

#include <cstdlib>
#include <cstring>

#include "common.cuh"
#include "device_utils.cuh"

namespace bitnet {
namespace {

#ifndef A_IN_TMEM_
#define A_IN_TMEM_ 0
#endif
// Build-time variant (-DA_IN_TMEM_=1, parity-tested, off): operand A (the unpacked weights) goes from the unpack
// warps' registers straight into tensor memory (tcgen05.st) instead of a shared-memory tile.  Shared memory
// is what binds this kernel: per K block the MMAs read 48 KB of operands and the producers write 48 KB,
// against 128 B/clk; with A's 16 KB of generic stores left out (wrong results, timing only) the kernel ran in 93
// instead of 115 us, with A's operand reads left out as well in 88.  But the A ring takes 128 of the 512
// tensor-memory columns, so the two accumulators shrink to 192 tokens, every weight tile is unpacked for a
// third more token tiles, and a K block through tcgen05.st does not fill faster than one through st.shared
// (0.46 vs 0.55 us): 129 us against 112.  With one 256-column accumulator the epilogue (8 us per tile, all
// CTAs writing at once) is exposed: 145 us.
constexpr bool A_IN_TMEM = A_IN_TMEM_ != 0;
constexpr int TILE_M = 128;     // out-features per tile (MMA M, tensor-memory lanes)
constexpr int TILE_T = A_IN_TMEM ? 192 : 256;   // tokens per tile (MMA N, tensor-memory columns)
constexpr int KBLK = 128;       // K columns per pipeline stage = one 128-byte swizzle row of int8
constexpr int STAGES = 4;
constexpr int NACC = 2;                          // accumulators of TILE_T columns: the epilogue of a tile overlaps the next tile's MMAs
constexpr int A_COL0 = NACC * TILE_T;            // first tensor-memory column of the A ring (32 columns per stage)
static_assert(!A_IN_TMEM || A_COL0 + 32 * 4 <= 512, "tensor memory: accumulators + A ring");
constexpr int A_BYTES = A_IN_TMEM ? 0 : TILE_M * KBLK;   // shared-memory bytes of a stage's A tile (16 KB)
constexpr int B_BYTES = TILE_T * KBLK;   // 32 KB
constexpr int UNPACK_WARPS = 8;           // warps that fill one stage: two threads per weight row
#ifndef UNPACK_GROUPS_
#define UNPACK_GROUPS_ 1
#endif
constexpr int UNPACK_GROUPS = UNPACK_GROUPS_;   // group g fills the K blocks kb = g (mod UNPACK_GROUPS); a second group
                                                // measured no faster (115 vs 112 us): the fill is not latency-bound
// warp 0 TMA, warp 1 MMA, then the unpack warps, then 4 epilogue warps (their index mod 4 is their lane quarter)
constexpr int THREADS = (2 + UNPACK_WARPS * UNPACK_GROUPS + 4) * 32;
static_assert(STAGES % UNPACK_GROUPS == 0, "a stage always belongs to the same group");
constexpr uint32_t WAIT_LIMIT = 1u << 22;

static __device__ int g_prefill_error = 0;

struct PrefillArgs {
  const uint8_t* packed;
  int64_t kp;            // K padded to 256 (blob geometry)
  int M;
  int K;
  int T;
  const float* act_scale;
  float w_scale;
  float* y;
  int32_t* acc_out;
  int tiles_m, tiles_t, nkb;
  int tma_store;         // y leaves through shared memory and bulk tensor stores (needs M % 4 == 0, no acc_out)
  int ksplit;            // > 1: an item is 1/ksplit of a tile's K blocks; partial sums go to ws with integer atomics
  int32_t* ws;           // [T][M] sums, zero on entry (ksplit > 1); a second kernel rescales them
};

struct __align__(8) Barriers {
  uint64_t full_a[STAGES], empty[STAGES], tmem_full[2], tmem_empty[2];
  uint32_t tmem_base;
  int abort_flag;
};

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
// Bounded wait; false = gave up (or another role already aborted).
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
  const uint32_t addr = smem_u32(bar);
  for (uint32_t it = 0; it < WAIT_LIMIT; ++it) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(addr), "r"(parity)
        : "memory");
    if (ok) return true;
    if ((it & 1023u) == 1023u && *abort_flag) return false;
  }
  return false;
}

// Shared-memory matrix descriptor for a K-major operand tile whose rows are 128 bytes, 128-byte
// swizzle: start address, stride between 8-row groups = 1024 bytes, descriptor version 1.
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);          // bits 0-13: start address / 16
  d |= (uint64_t)1 << 16;                            // bits 16-29: leading byte offset / 16 (unused here)
  d |= (uint64_t)(1024 >> 4) << 32;                  // bits 32-45: stride byte offset / 16
  d |= (uint64_t)1 << 46;                            // bits 46-47: descriptor version (tcgen05)
  d |= (uint64_t)2 << 61;                            // bits 61-63: 128-byte swizzle
  return d;
}

// Instruction descriptor: D = s32, A = s8, B = s8, both K-major, N = 256, M = 128.
constexpr uint32_t IDESC = (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(TILE_T >> 3) << 17) |
                           ((uint32_t)(TILE_M >> 4) << 24);

__device__ __forceinline__ void umma_i8(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(IDESC), "r"(accumulate)
      : "memory");
}
// the same with operand A in tensor memory (lane = row, 8 columns = 32 int8 along K)
__device__ __forceinline__ void umma_i8_ta(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::i8 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(bdesc), "r"(IDESC), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
               : "memory");
}

// signed bytes (-1, 0, +1) of slot s of a packed word: codes 0,1,2 minus one, without borrows between bytes
__device__ __forceinline__ uint32_t slot_s8(uint32_t w, int s) {
  const uint32_t c = ((w >> (2 * s)) & 0x03030303u) | 0x80808080u;
  return (c - 0x01010101u) ^ 0x80808080u;
}

__global__ void __launch_bounds__(THREADS, 1)
gemm_i2s_tc_kernel(const __grid_constant__ CUtensorMap qmap, const __grid_constant__ CUtensorMap ymap,
                   const PrefillArgs a) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* tileA = smem;                               // STAGES x 16 KB
  uint8_t* tileB = smem + STAGES * A_BYTES;            // STAGES x 32 KB
  Barriers* bars = reinterpret_cast<Barriers*>(smem + STAGES * (A_BYTES + B_BYTES));
  volatile int* abort_flag = &bars->abort_flag;

  __shared__ float ep_scale[4][TILE_T];                // epilogue: act_scale[t] * w_scale of the current tile
  __shared__ __align__(128) float ep_stage[4][32][32]; // epilogue: 32 tokens x 32 rows of y per warp, [token][row]

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int ntiles = a.tiles_m * a.tiles_t;
  // Work items: tile `item % ntiles`, K blocks [kb_lo, kb_hi) = part `item / ntiles` of ksplit (even bounds).
  const int nitems = ntiles * a.ksplit;
  auto kb_lo_of = [&](int item) { return 2 * (int)((int64_t)(item / ntiles) * (a.nkb / 2) / a.ksplit); };
  auto kb_hi_of = [&](int item) { return 2 * (int)((int64_t)(item / ntiles + 1) * (a.nkb / 2) / a.ksplit); };

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      // one barrier per stage for both operands: an arrival per unpack warp, one of the TMA producer (+ its bytes)
      mbar_init(&bars->full_a[s], UNPACK_WARPS + 1);
      mbar_init(&bars->empty[s], 1);       // tcgen05.commit
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(&bars->tmem_full[b], 1);   // tcgen05.commit
      mbar_init(&bars->tmem_empty[b], 4);  // one arrival per epilogue warp
    }
    bars->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    __syncwarp();
    // the whole tensor memory of the SM: two 128 x 256 s32 accumulators
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(smem_u32(&bars->tmem_base))
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = bars->tmem_base;

  // Early start (programmatic dependent launch): the weight unpackers and the MMA issuer touch nothing that an
  // earlier kernel in the stream writes; the TMA producer (codes) and the epilogue (scales, y, workspace) wait.
  if (threadIdx.x == 0) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer: activation tiles (operand B)
    if (lane == 0) {
      asm volatile("griddepcontrol.wait;" ::: "memory");
      uint32_t it = 0;
      for (int item = blockIdx.x; item < nitems && !*abort_flag; item += gridDim.x) {
        const int tile = item % ntiles;
        const int t0 = (tile / a.tiles_m) * TILE_T;
        for (int kb = kb_lo_of(item), kb_end = kb_hi_of(item); kb < kb_end; ++kb, ++it) {
          const int s = it % STAGES;
          if (!mbar_wait(&bars->empty[s], ((it / STAGES) & 1u) ^ 1u, abort_flag)) {
            atomicExch(&g_prefill_error, BITNET_ERR_TIMEOUT);
            bars->abort_flag = 1;
            break;
          }
          mbar_expect_tx(&bars->full_a[s], B_BYTES);
          asm volatile(
              "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
              ::"r"(smem_u32(tileB + s * B_BYTES)), "l"(&qmap), "r"(kb * KBLK), "r"(t0),
              "r"(smem_u32(&bars->full_a[s]))
              : "memory");
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      uint32_t it = 0, nt = 0;
      for (int item = blockIdx.x; item < nitems && !*abort_flag; item += gridDim.x, ++nt) {
        const int buf = nt % NACC;
        const int kb_lo = kb_lo_of(item), kb_hi = kb_hi_of(item);
        bool ok = mbar_wait(&bars->tmem_empty[buf], ((nt / NACC) & 1u) ^ 1u, abort_flag);
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t d_tmem = tmem_base + buf * TILE_T;
        for (int kb = kb_lo; ok && kb < kb_hi; ++kb, ++it) {
          const int s = it % STAGES;
          const uint32_t par = (it / STAGES) & 1u;
          ok = mbar_wait(&bars->full_a[s], par, abort_flag);   // weights unpacked and activations landed
          if (!ok) break;
          const uint64_t adesc = make_desc(smem_u32(tileA + s * A_BYTES));
          const uint64_t bdesc = make_desc(smem_u32(tileB + s * B_BYTES));
#pragma unroll
          for (int k4 = 0; k4 < KBLK / 32; ++k4) {  // 32 bytes further along K: +2 in the address field, +8 columns
            if (A_IN_TMEM)
              umma_i8_ta(d_tmem, tmem_base + A_COL0 + s * 32 + 8 * k4, bdesc + 2 * k4, (kb > kb_lo || k4 > 0) ? 1u : 0u);
            else
              umma_i8(d_tmem, adesc + 2 * k4, bdesc + 2 * k4, (kb > kb_lo || k4 > 0) ? 1u : 0u);
          }
          umma_commit(&bars->empty[s]);            // stage reusable once these MMAs have read it
        }
        if (!ok) {
          atomicExch(&g_prefill_error, BITNET_ERR_TIMEOUT);
          bars->abort_flag = 1;
          break;
        }
        umma_commit(&bars->tmem_full[buf]);        // accumulator complete
      }
    }
  } else if (warp < 2 + UNPACK_WARPS * UNPACK_GROUPS) {
    // ------------------------------------------------------------ unpackers: weight rows (operand A)
    const int grp = (threadIdx.x - 64) / (UNPACK_WARPS * 32);
    const int u = (threadIdx.x - 64) % (UNPACK_WARPS * 32);   // 0..255: row u/2 of the tile, half u%2 of its 128 columns
    // Through tensor memory a warp can only write the 32 lanes of its quarter (warp index mod 4): lane = row
    // within the quarter, and the two warps of a group that share a quarter take one half of the K block each.
    const int r = A_IN_TMEM ? (warp & 3) * 32 + lane : u >> 1;
    const int hf = A_IN_TMEM ? (u >> 7) : (u & 1);
    uint32_t it0 = 0;                              // pipeline index of the tile's K block 0 (nkb is even)
    for (int item = blockIdx.x; item < nitems && !*abort_flag; item += gridDim.x) {
      const int tile = item % ntiles;
      const int kb_lo = kb_lo_of(item), kb_hi = kb_hi_of(item);
      const int m = (tile % a.tiles_m) * TILE_M + r;
      const bool row_ok = m < a.M;
      // K block kb = half kb&1 of chunk kb/2: 32 bytes of the row, of which this thread takes 16
      const uint8_t* rowp = a.packed + i2s_row_chunk_offset(row_ok ? m : 0, 0, a.kp) + hf * 16;
      // packed words of K blocks kb .. kb+PF-1 are kept in flight: an L2 round trip is longer than one block
      constexpr int PF = 4;
      constexpr int G = UNPACK_GROUPS;
      const uint4 zero_w = make_uint4(0x55555555u, 0x55555555u, 0x55555555u, 0x55555555u);   // code 1 = weight 0
      auto fetch = [&](int kb) {
        return (row_ok && kb < kb_hi)
                   ? __ldg(reinterpret_cast<const uint4*>(rowp + (int64_t)(kb >> 1) * 1024 + (kb & 1) * 32))
                   : zero_w;
      };
      uint4 nx[PF];
#pragma unroll
      for (int p = 0; p < PF; ++p) nx[p] = fetch(kb_lo + grp + p * G);
      bool ok = true;
      for (int kb = kb_lo + grp; kb < kb_hi; kb += G) {
        const uint32_t it = it0 + (uint32_t)(kb - kb_lo);
        const uint4 cw = nx[0];
#pragma unroll
        for (int p = 0; p + 1 < PF; ++p) nx[p] = nx[p + 1];
        nx[PF - 1] = fetch(kb + PF * G);
        const int s = it % STAGES;
        if (!mbar_wait(&bars->empty[s], ((it / STAGES) & 1u) ^ 1u, abort_flag)) {
          ok = false;
          break;
        }
        const uint32_t w[4] = {cw.x, cw.y, cw.z, cw.w};
        if (A_IN_TMEM) {
          // 64 int8 of the row in K order = 16 tensor-memory columns: chunk c4 of 16 columns takes words
          // 2*(c4/2), 2*(c4/2)+1 of the 16 packed bytes, slots 2h, 2h+1 (h = c4 % 2)
          uint32_t o[16];
#pragma unroll
          for (int c4 = 0; c4 < 4; ++c4) {
            const uint32_t w0 = w[2 * (c4 >> 1)], w1 = w[2 * (c4 >> 1) + 1];
            const int h = c4 & 1;
            o[4 * c4 + 0] = slot_s8(w0, 2 * h);
            o[4 * c4 + 1] = slot_s8(w1, 2 * h);
            o[4 * c4 + 2] = slot_s8(w0, 2 * h + 1);
            o[4 * c4 + 3] = slot_s8(w1, 2 * h + 1);
          }
          const uint32_t taddr = tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + A_COL0 + s * 32 + hf * 16;
          asm volatile(
              "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, "
              "%14, %15, %16};"
              ::"r"(taddr), "r"(o[0]), "r"(o[1]), "r"(o[2]), "r"(o[3]), "r"(o[4]), "r"(o[5]), "r"(o[6]), "r"(o[7]),
                "r"(o[8]), "r"(o[9]), "r"(o[10]), "r"(o[11]), "r"(o[12]), "r"(o[13]), "r"(o[14]), "r"(o[15])
              : "memory");
          asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
          asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
          __syncwarp();
          if (lane == 0) mbar_arrive(&bars->full_a[s]);
          continue;
        }
        uint8_t* rowA = tileA + s * A_BYTES + (r >> 3) * 1024 + (r & 7) * 128;
#pragma unroll
        for (int c4 = 0; c4 < 4; ++c4) {
          // 16 consecutive columns of the block, chunk c = 4*hf + c4: words 2P, 2P+1 (P = c/2) of the 32
          // bytes, i.e. words 2*(c4/2), 2*(c4/2)+1 of this thread's 16, slots 2h, 2h+1 (h = c%2)
          const uint32_t w0 = w[2 * (c4 >> 1)], w1 = w[2 * (c4 >> 1) + 1];
          const int h = c4 & 1;
          const uint4 o = make_uint4(slot_s8(w0, 2 * h), slot_s8(w1, 2 * h), slot_s8(w0, 2 * h + 1), slot_s8(w1, 2 * h + 1));
          const int c = 4 * hf + c4;
          *reinterpret_cast<uint4*>(rowA + ((c ^ (r & 7)) << 4)) = o;
        }
        // make the generic-proxy stores visible to the tensor core (async proxy), then signal
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if (lane == 0) mbar_arrive(&bars->full_a[s]);
      }
      if (!ok) {
        atomicExch(&g_prefill_error, BITNET_ERR_TIMEOUT);
        bars->abort_flag = 1;
        break;
      }
      it0 += (uint32_t)(kb_hi - kb_lo);
    }
  } else {
    // ------------------------------------------------------------ epilogue
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int quarter = warp & 3;                  // tensor-memory lanes 32*quarter .. 32*quarter+31
    uint32_t nt = 0;
    for (int item = blockIdx.x; item < nitems && !*abort_flag; item += gridDim.x, ++nt) {
      const int tile = item % ntiles;
      const int buf = nt % NACC;
      const int m = (tile % a.tiles_m) * TILE_M + quarter * 32 + lane;
      const int t0 = (tile / a.tiles_m) * TILE_T;
      // this tile's per-token factors act_scale[t] * w_scale, one copy per epilogue warp, fetched while the
      // tile's MMAs still run (a global load per stored element, even one that hits L1, made the epilogue the
      // slowest stage of the pipeline: 130 instead of 88 us for the whole GEMM with every other stage idle)
      float* const my_scale = ep_scale[quarter];
      __syncwarp();
      for (int i = lane; i < TILE_T; i += 32)
        my_scale[i] = (t0 + i < a.T) ? __fmul_rn(__ldg(a.act_scale + t0 + i), a.w_scale) : 0.0f;
      __syncwarp();
      if (!mbar_wait(&bars->tmem_full[buf], (nt / NACC) & 1u, abort_flag)) {
        atomicExch(&g_prefill_error, BITNET_ERR_TIMEOUT);
        bars->abort_flag = 1;
        break;
      }
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + buf * TILE_T;
#pragma unroll 1
      for (int c0 = 0; c0 < TILE_T; c0 += 32) {
        uint32_t v[32];
        asm volatile(
            "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
            "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
            "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
            : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
              "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
              "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
              "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
            : "r"(taddr + c0)
            : "memory");
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
        if (a.tma_store) {
          // 32 tokens x 32 rows through shared memory, then one bulk tensor store (rows and tokens beyond M
          // and T are clipped by the tensor map): one instruction instead of 32 strided 128-byte stores
          if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");   // previous box read out
          __syncwarp();
#pragma unroll
          for (int j = 0; j < 32; ++j) ep_stage[quarter][j][lane] = __fmul_rn((float)(int)v[j], my_scale[c0 + j]);
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
          __syncwarp();
          if (lane == 0) {
            asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];"
                         ::"l"(&ymap), "r"((tile % a.tiles_m) * TILE_M + quarter * 32), "r"(t0 + c0),
                           "r"(smem_u32(&ep_stage[quarter][0][0]))
                         : "memory");
            asm volatile("cp.async.bulk.commit_group;" ::: "memory");
          }
        } else if (a.ksplit > 1) {
          // part of a tile's K: add the raw sums (integers: any order gives the same); rescaled afterwards
          if (m < a.M) {
#pragma unroll
            for (int j = 0; j < 32; ++j) {
              const int t = t0 + c0 + j;
              if (t < a.T) atomicAdd(a.ws + (int64_t)t * a.M + m, (int)v[j]);
            }
          }
        } else if (m < a.M) {
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            const int t = t0 + c0 + j;
            if (t < a.T) {
              const int acc = (int)v[j];
              a.y[(int64_t)t * a.M + m] = __fmul_rn((float)acc, my_scale[c0 + j]);
              if (a.acc_out) a.acc_out[(int64_t)t * a.M + m] = acc;
            }
          }
        }
      }
      // the accumulator has been read: hand the buffer back to the MMA issuer
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      __syncwarp();
      if (lane == 0) mbar_arrive(&bars->tmem_empty[buf]);
    }
    if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");   // the last boxes have left
  }

  // ---- teardown: every role has left its loop (all waits are bounded); free the tensor memory
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem_base) : "memory");
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess)
      p = nullptr;
    return reinterpret_cast<EncodeTiledFn>(p);
  }();
  return fn;
}

}  // namespace

int encode_q_tile_map(void* out, const int8_t* q, int64_t K, int64_t T, int box_t) {
  EncodeTiledFn enc = encode_fn();
  if (!enc) return note_cuda_error(cudaErrorNotSupported);
  const cuuint64_t gdim[2] = {(cuuint64_t)K, (cuuint64_t)T};
  const cuuint64_t gstride[1] = {(cuuint64_t)K};            // bytes between token rows
  const cuuint32_t box[2] = {KBLK, (cuuint32_t)box_t};
  const cuuint32_t estr[2] = {1, 1};
  CUresult r = enc(static_cast<CUtensorMap*>(out), CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<int8_t*>(q), gdim, gstride, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? BITNET_OK : note_cuda_error(cudaErrorInvalidValue);
}

int launch_gemm_i2s_simt(const uint8_t* packed, float w_scale, int64_t M, int64_t K, const int8_t* q,
                         const float* act_scale, int64_t T, float* y, int32_t* acc_out, cudaStream_t st);

static bool no_tma_store() {
  static const bool off = [] { const char* e = getenv("BITNET_PREFILL_TMA_STORE"); return e && atoi(e) == 0; }();
  return off;
}

// Parts per tile's K: with fewer tiles than SMs (short prompts, small layers) whole tiles leave SMs idle and
// the time is that of one tile's K blocks; parts of at least 8 K blocks fill the machine instead.
static int prefill_ksplit(int64_t T, int64_t M, int64_t K) {
  static const int forced = [] { const char* e = getenv("BITNET_PREFILL_KSPLIT"); return e ? atoi(e) : 0; }();
  const int64_t ntiles = ceil_div(M, TILE_M) * ceil_div(T, TILE_T);
  const int64_t nkb = i2s_kp(K) / KBLK;
  const int sms = dev_info().sm_count;
  int64_t ks = 1;
  if (forced > 0) ks = forced;
  else if (ntiles * 4 <= sms * 3) ks = sms / ntiles;          // at most three quarters of the SMs would work
  // (with more tiles than that the atomics and the rescale pass over T x M cost more than the idle SMs)
  if (ks > nkb / 8) ks = nkb / 8;
  return ks < 1 ? 1 : (int)ks;
}

size_t gemm_i2s_prefill_workspace_bytes(int64_t T, int64_t M, int64_t K) {
  return prefill_ksplit(T, M, K) > 1 ? (size_t)T * (size_t)M * 4 : 0;
}

int launch_gemm_i2s_prefill(const uint8_t* packed, float w_scale, int64_t M, int64_t K, const int8_t* q,
                            const float* act_scale, int64_t T, float* y, int32_t* acc_out, void* ws, size_t ws_bytes,
                            cudaStream_t st) {
  static const bool force_simt = [] {
    const char* e = getenv("BITNET_PREFILL");
    return e && strcmp(e, "simt") == 0;
  }();
  if (force_simt) return launch_gemm_i2s_simt(packed, w_scale, M, K, q, act_scale, T, y, acc_out, st);
  int ksplit = prefill_ksplit(T, M, K);
  if (ksplit > 1 && (!ws || ws_bytes < (size_t)T * (size_t)M * 4)) ksplit = 1;
  EncodeTiledFn enc = encode_fn();
  if (!enc) return note_cuda_error(cudaErrorNotSupported);
  CUtensorMap qmap;
  const cuuint64_t gdim[2] = {(cuuint64_t)K, (cuuint64_t)T};
  const cuuint64_t gstride[1] = {(cuuint64_t)K};            // bytes between token rows
  const cuuint32_t box[2] = {KBLK, TILE_T};
  const cuuint32_t estr[2] = {1, 1};
  CUresult r = enc(&qmap, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<int8_t*>(q), gdim, gstride, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return note_cuda_error(cudaErrorInvalidValue);

  // y[T][M] fp32 as a tensor of 32 x 32 boxes for the epilogue's bulk stores
  const bool tma_store = ksplit == 1 && acc_out == nullptr && (M % 4) == 0 && !no_tma_store();
  CUtensorMap ymap = qmap;
  if (tma_store) {
    const cuuint64_t ydim[2] = {(cuuint64_t)M, (cuuint64_t)T};
    const cuuint64_t ystride[1] = {(cuuint64_t)M * 4};
    const cuuint32_t ybox[2] = {32, 32};
    r = enc(&ymap, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, y, ydim, ystride, ybox, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return note_cuda_error(cudaErrorInvalidValue);
  }

  PrefillArgs a;
  a.tma_store = tma_store ? 1 : 0;
  a.ksplit = ksplit;
  a.ws = reinterpret_cast<int32_t*>(ws);
  a.packed = packed;
  a.kp = i2s_kp(K);
  a.M = (int)M;
  a.K = (int)K;
  a.T = (int)T;
  a.act_scale = act_scale;
  a.w_scale = w_scale;
  a.y = y;
  a.acc_out = acc_out;
  a.tiles_m = (int)ceil_div(M, TILE_M);
  a.tiles_t = (int)ceil_div(T, TILE_T);
  a.nkb = (int)(a.kp / KBLK);
  const size_t smem = (size_t)STAGES * (A_BYTES + B_BYTES) + sizeof(Barriers) + 1024;
  static bool attr_set[64] = {false};
  int dev = 0;
  cudaGetDevice(&dev);
  if (!attr_set[dev & 63]) {
    cudaError_t e = cudaFuncSetAttribute(gemm_i2s_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return note_cuda_error(e);
    attr_set[dev & 63] = true;
  }
  int grid = dev_info().sm_count;
  const int nitems = a.tiles_m * a.tiles_t * ksplit;
  if (grid > nitems) grid = nitems;
  log_launch("gemm_i2s_tc_kernel T=%lld M=%lld K=%lld grid=%d tiles=%d K-parts=%d output=%s%s", (long long)T, (long long)M,
             (long long)K, grid, a.tiles_m * a.tiles_t, ksplit, tma_store ? "bulk tensor stores" : "plain stores",
             ksplit > 1 ? " + finish_mid_kernel" : "");
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)grid);
  cfg.blockDim = dim3(THREADS);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = early_start_enabled(st) ? 1 : 0;
  cudaError_t le = cudaLaunchKernelEx(&cfg, gemm_i2s_tc_kernel, qmap, ymap, a);
  int rc = le == cudaSuccess ? BITNET_OK : note_cuda_error(le);
  if (rc || ksplit == 1) return rc;
  return launch_rescale_sums(a.ws, act_scale, w_scale, T, M, y, acc_out, st);
}


int gemm_prefill_status(int* out) {
  cudaError_t e = cudaMemcpyFromSymbol(out, g_prefill_error, sizeof(int));
  return e == cudaSuccess ? BITNET_OK : note_cuda_error(e);
}
int gemm_prefill_status_clear() {
  const int zero = 0;
  cudaError_t e = cudaMemcpyToSymbol(g_prefill_error, &zero, sizeof(int));
  return e == cudaSuccess ? BITNET_OK : note_cuda_error(e);
}

}  // namespace bitnet
