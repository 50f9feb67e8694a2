// I2_S mpGEMM for 17 to 128 tokens over a list of linears: Alg. 1 Phase 2 with the weights streamed from HBM once
// and multiplied on the fifth-generation tensor cores (tcgen05.mma kind::i8, accumulators in tensor memory).
//
//   acc[t,m] = sum_k q[t,k] * w[m,k],   y[t,m] = acc[t,m] * act_scale[t] * w_scale
//
// Between decode (1..8 tokens: the weight stream is everything, mma.sync keeps up) and prefill (hundreds of tokens:
// the tensor cores are everything) the work per weight byte is small enough that the blob should cross HBM once,
// yet too large for mma.sync: m16n8k32 needs 2 T MMAs per 1-KB chunk.  The paper treats neither stage; the design
// is this build's.  One persistent CTA per SM walks tiles of 128 out-features x all of K, tile j of the list's
// tile sequence going to CTA j mod grid:
//   * warps 0-15 (writers): thread = (row of the tile, half of a 128-column K block).  It keeps the row's packed
//     words of the next eight steps in flight (16-byte cp.async copies into a private ring slot: 64 KB per SM),
//     turns the 2-bit codes into bytes 0/1/2 (a shift and a mask per word: the codes go to the tensor core as
//     UNSIGNED 8-bit values, the "- sum(q)" of code = w + 1 is applied in the epilogue) and writes them straight
//     into tensor memory (tcgen05.st): operand A never touches shared memory as bytes.  The same threads copy the
//     activation tile (64 tokens x 128 codes) of each K block, two steps ahead, into shared memory in the
//     128-byte-swizzled K-major layout (operand B; cp.async with zero fill beyond T and K) and add up the codes of
//     their own pieces once landed, which gives sum(q) per token;
//   * warps 16-19: issuers, taking the steps in turn.  Per step (two K blocks) one elected lane issues eight
//     tcgen05.mma (M = 128, N = 64, K = 32; A from tensor memory, B from shared memory) and releases the stage pair
//     with one tcgen05.commit.  An issuer's wait-fence-issue-commit round costs about 500 cycles whatever the MMAs
//     do (at 64 tokens they occupy the tensor pipe for 32 cycles each: measured 22 cycles of issue per MMA, over
//     200 for the wait, fence and commit around them), so several warps share the steps; every MMA accumulates (the
//     epilogue leaves the accumulators zeroed), so their order does not matter;
//   * warps 20-23: epilogue -- tcgen05.ld the finished 128 x 64 accumulator, zero it, subtract sum(q), rescale,
//     store y.
// Two accumulators (2 x 64 columns) overlap a tile's epilogue with the next tile's MMAs; the A ring takes 12 x 32
// columns.  Items with 65 to 128 tokens run the same kernel with 128-token tiles (template TN = 128: two activation
// pieces per writer thread and K block, accumulators of 128 columns, 8 stages): 11 ms per 100B sweep against 22 ms
// for the prefill kernel, which such lists fell to before.  What binds is the writers' instruction stream (about 100 per warp and step: 7.6 ms per 100B sweep at any
// token count from 17 to 64, against 9.6 to 19.4 ms for the mma.sync kernel of gemv_i2s_mid.cu).  Every mbarrier wait is bounded; a wait that gives up sets a CTA-wide abort flag and the device status
// word, all roles leave their loops, and the CTA frees its tensor memory before it exits.
#include <cstdlib>
#include <cstring>

#include "common.cuh"
#include "device_utils.cuh"

namespace bitnet {
namespace {

constexpr int TILE_M = 128;     // out-features per tile (MMA M, tensor-memory lanes)
// tokens per tile (MMA N, tensor-memory columns of an accumulator): the kernel template's TN, 64 or 128
constexpr int KBLK = 128;       // K columns per pipeline stage = one 128-byte swizzle row of int8
constexpr int MAX_STAGES = 12;               // stages: 12 at 64 tokens, 8 at 128 (tensor memory: 2 TN + 32 stages = 512 columns)
constexpr int NACC = 2;
constexpr int TMEM_COLS = 512;
constexpr int MAX_N = 128;
constexpr int WRITER_WARPS = 16;
constexpr int MMA_WARPS = 4;                 // issuers: warp i takes the steps i, i + 4, ... of a tile
constexpr int THREADS = (WRITER_WARPS + MMA_WARPS + 4) * 32;   // + 4 epilogue warps
constexpr int DA = 8;                        // steps (pairs of K blocks) of packed words in flight per thread
constexpr int DB = 2;                        // steps by which the activation copies run ahead
constexpr int SLOTS_A = DA + 1;              // ring slots: the copy for step s + DA never lands in the slot step s reads
constexpr int RING_A_BYTES = SLOTS_A * WRITER_WARPS * 32 * 16;   // 72 KB: one 16-byte slot per writer thread and step
constexpr int NITEMS = 400;                  // items per launch (argument block of 32 KB)
constexpr uint32_t WAIT_LIMIT = 1u << 22;

static __device__ int g_stream_tc_error = 0;

struct TItem {
  const uint8_t* packed;
  const int8_t* q;        // [T][K] codes
  const float* act_scale; // [T]
  float* y;               // [T][ldy]
  int32_t* acc_out;       // nullable
  float w_scale;
  int M, K, T;
  int first_tile;         // tiles of the items before this one
  int ldy;
};
static_assert(sizeof(TItem) == 64, "argument block layout");

struct TArgs {
  int n, total_tiles;
  TItem it[NITEMS];
};
static_assert(sizeof(TArgs) <= 32764, "kernel parameter limit");

struct __align__(8) Bars {
  uint64_t full[MAX_STAGES], empty[MAX_STAGES], tmem_full[NACC], tmem_empty[NACC], qsum_ready[NACC];
  uint32_t tmem_base;
  int abort_flag;
};

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// Bounded wait; false = gave up (or another role already aborted).  `hint_ns`: how long one probe may keep the thread
// suspended before it reports "not yet" (roles that wait for a whole tile probe rarely: their polling would take
// issue slots from the writers).
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag, uint32_t hint_ns = 0) {
  const uint32_t addr = smem_u32(bar);
  for (uint32_t it = 0; it < WAIT_LIMIT; ++it) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(addr), "r"(parity), "r"(hint_ns)
        : "memory");
    if (ok) return true;
    if ((it & 255u) == 255u && *abort_flag) return false;
  }
  return false;
}

// Shared-memory matrix descriptor for a K-major operand tile whose rows are 128 bytes, 128-byte swizzle: start
// address, stride between 8-row groups = 1024 bytes, descriptor version 1.
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);
  d |= (uint64_t)1 << 16;
  d |= (uint64_t)(1024 >> 4) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}

// Instruction descriptor: D = s32, A = u8 (the codes 0, 1, 2), B = s8, both K-major, N tokens, M = 128.
__host__ __device__ constexpr uint32_t idesc_of(int n) {
  return (2u << 4) | (0u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(TILE_M >> 4) << 24);
}

// operand A in tensor memory (lane = row, 8 columns = 32 codes along K), operand B through a descriptor.  The
// whole warp runs the issuing loop and one elected lane issues (`leader` != 0): with warp-uniform operands the
// compiler keeps addresses and descriptors in uniform registers instead of moving them there per instruction.
__device__ __forceinline__ void umma_u8s8_ta(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc,
                                             uint32_t accumulate, uint32_t leader) {
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "setp.ne.b32 q, %5, 0;\n\t"
      "@q tcgen05.mma.cta_group::1.kind::i8 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(leader)
      : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t* bar, uint32_t leader) {
  asm volatile(
      "{\n\t.reg .pred q;\n\t"
      "setp.ne.b32 q, %1, 0;\n\t"
      "@q tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n\t}"
      ::"r"(smem_u32(bar)), "r"(leader)
      : "memory");
}
__device__ __forceinline__ uint32_t elect_one() {
  uint32_t pred;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "elect.sync _|p, 0xffffffff;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(pred));
  return pred;
}

// item that holds tile `job` of the list's tile sequence
__device__ __forceinline__ int locate(const TArgs& a, int job) {
  int lo = 0, hi = a.n - 1;
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if (a.it[mid].first_tile <= job) lo = mid; else hi = mid - 1;
  }
  return lo;
}

template <int TN>
__global__ void __launch_bounds__(THREADS, 1) gemm_i2s_stream_tc_kernel(const __grid_constant__ TArgs a) {
  constexpr int TILE_N = TN;
  constexpr int STAGES = TN == 64 ? 12 : 8;
  constexpr int A_COL0 = NACC * TILE_N;        // first tensor-memory column of the A ring (32 columns per stage)
  constexpr int B_BYTES = TILE_N * KBLK;       // 8 or 16 KB per stage
  constexpr int NP = TN / 64;                  // activation pieces per writer thread and K block (tokens tb, tb + 64)
  constexpr uint32_t IDESC = idesc_of(TN);
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* tileB = smem;                                   // STAGES x 8 KB
  uint8_t* ringA = smem + STAGES * B_BYTES;                // SLOTS_A x 512 x 16 bytes
  Bars* bars = reinterpret_cast<Bars*>(smem + STAGES * B_BYTES + RING_A_BYTES);
  volatile int* abort_flag = &bars->abort_flag;
  __shared__ int qsum_s[NACC][MAX_N];                      // sum of a token's codes over K, per accumulator in flight
  __shared__ float ep_scale[4][MAX_N];                     // epilogue: act_scale[t] * w_scale of the current tile

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(&bars->full[s], WRITER_WARPS);   // every writer warp: its pieces of B, and of A where it has some
      mbar_init(&bars->empty[s], 1);             // tcgen05.commit (used on the odd stages: one per stage pair)
    }
    for (int b = 0; b < NACC; ++b) {
      mbar_init(&bars->tmem_full[b], MMA_WARPS); // one tcgen05.commit per issuer
      mbar_init(&bars->tmem_empty[b], 4);        // one arrival per epilogue warp
      mbar_init(&bars->qsum_ready[b], WRITER_WARPS);
    }
    bars->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == WRITER_WARPS) {
    __syncwarp();
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(&bars->tmem_base)), "n"(TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = bars->tmem_base;
  // 32 lanes x 32 columns of zeros: the accumulators start (and are handed back) cleared
  auto zero32 = [](uint32_t taddr) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, "
        "%1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1};"
        ::"r"(taddr), "r"(0u)
        : "memory");
  };
  if (warp >= WRITER_WARPS + MMA_WARPS) {
    for (int c0 = 0; c0 < NACC * TILE_N; c0 += 32) zero32(tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + c0);
    asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");

  if (warp < WRITER_WARPS) {
    // ------------------------------------------------------------ writers: operands A (tensor memory) and B (shared)
    const int quarter = warp & 3;                  // tensor-memory lanes 32*quarter .. +31 = rows of the tile
    const int grp2 = (warp >> 3) & 1;              // which K block of a step this warp unpacks
    const int hf = (warp >> 2) & 1;                // which half (64 columns) of that K block
    const int r = quarter * 32 + lane;
    const int tb = threadIdx.x >> 3, cb = threadIdx.x & 7;   // activation piece: token, 16-byte piece of the 128-byte row
    const uint32_t b_off = (uint32_t)((tb >> 3) * 1024 + (tb & 7) * 128 + ((cb ^ (tb & 7)) << 4));
    const uint32_t ring_a = smem_u32(ringA) + threadIdx.x * 16;
    const uint32_t tile_b = smem_u32(tileB) + b_off;
    // Running positions instead of divisions: st0 = stage of the current step's first K block (even; its second K
    // block sits in st0 + 1), ph = how often the stage ring has been passed (mod 2), slot = the step's ring slot.
    int st0 = 0, slot = 0;
    uint32_t ph = 0;
    constexpr uint32_t SLOT_BYTES = WRITER_WARPS * 32 * 16;
    uint32_t nt = 0;
    bool ok = true;
    for (int job = blockIdx.x; ok && job < a.total_tiles && !*abort_flag; job += gridDim.x, ++nt) {
      const int ii = locate(a, job);
      const TItem& d = a.it[ii];
      const int64_t kp = i2s_kp(d.K);
      const int nsteps = (int)(kp / 256);          // a step = the two K blocks of a 256-column chunk
      const int m = (job - d.first_tile) * TILE_M + r;
      // chunk s of the row: 64 bytes; K block 2s + grp2 = its half grp2 (32 bytes), of which this thread takes 16
      // (rows beyond M read the last row: their sums are never stored)
      const uint8_t* rowp = d.packed + i2s_row_chunk_offset(m < d.M ? m : d.M - 1, 0, kp) + grp2 * 32 + hf * 16;
      const int K = d.K;
      const int8_t* qrow = d.q + (int64_t)(tb < d.T ? tb : 0) * K + cb * 16;
      const int8_t* qrow2 = d.q + (int64_t)(tb + 64 < d.T ? tb + 64 : 0) * K + cb * 16;   // (TN = 128: the thread's second token)
      const bool tok_ok = tb < d.T, tok2_ok = NP == 2 && tb + 64 < d.T;
      // the thread's two activation pieces of step s into stage pair stb (zeros beyond T, K), once that pair is free:
      // the stages are released in order, so the later one being free means both are
      auto issue_b = [&](int s, int stb, uint32_t phb) -> bool {
        if (!mbar_wait(&bars->empty[stb + 1], phb ^ 1u, abort_flag, 20)) return false;
        const int col = 2 * s * KBLK + cb * 16;
        const uint32_t by0 = (tok_ok && col + 16 <= K) ? 16u : 0u, by1 = (tok_ok && col + KBLK + 16 <= K) ? 16u : 0u;
        const int8_t* src = qrow + 2 * s * KBLK;
        const uint32_t dst = tile_b + stb * B_BYTES;
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(by0 ? src : qrow), "r"(by0) : "memory");
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst + B_BYTES), "l"(by1 ? src + KBLK : qrow), "r"(by1)
                     : "memory");
        if (NP == 2) {                             // tokens 64..127 lie 8 row groups (8 KB) further down the tile
          const uint32_t cy0 = (tok2_ok && col + 16 <= K) ? 16u : 0u, cy1 = (tok2_ok && col + KBLK + 16 <= K) ? 16u : 0u;
          const int8_t* src2 = qrow2 + 2 * s * KBLK;
          asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst + 8192), "l"(cy0 ? src2 : qrow), "r"(cy0) : "memory");
          asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst + B_BYTES + 8192), "l"(cy1 ? src2 + KBLK : qrow), "r"(cy1)
                       : "memory");
        }
        return true;
      };
      // prologue: packed words of the first DA steps (slots slot .. slot + DA - 1); activation pieces of the first DB
#pragma unroll
      for (int p = 0; p < DA; ++p) {
        const int sl = slot + p >= SLOTS_A ? slot + p - SLOTS_A : slot + p;
        if (p < nsteps) cp16_keep(ring_a + sl * SLOT_BYTES, rowp + (int64_t)p * 1024);
      }
      cp_commit();
#pragma unroll
      for (int p = 0; p < DB; ++p) {
        int stb = st0 + 2 * p;
        uint32_t phb = ph;
        if (stb >= STAGES) stb -= STAGES, phb ^= 1u;
        if (ok && p < nsteps) ok = issue_b(p, stb, phb);
        cp_commit();
      }
      int qs = 0, qs2 = 0;
      const uint8_t* pa = rowp + (int64_t)DA * 1024;   // packed words of step s + DA
      for (int s = 0; s < nsteps && ok; ++s, pa += 1024) {
        if (s + DB < nsteps) {
          int stb = st0 + 2 * DB;
          uint32_t phb = ph;
          if (stb >= STAGES) stb -= STAGES, phb ^= 1u;
          ok = issue_b(s + DB, stb, phb);
          if (!ok) break;
        }
        // step s + DA goes to the slot before this step's (DA = SLOTS_A - 1 places on)
        if (s + DA < nsteps) cp16_keep(ring_a + (slot ? slot - 1 : SLOTS_A - 1) * SLOT_BYTES, pa);
        cp_commit();
        cp_wait<DB>();                             // everything but the last DB groups has landed: step s is complete
        // the landed activation bytes go to the tensor core through the async proxy
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        {
          uint4 b0, b1;                            // this thread's own pieces, for the row sums
          asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(b0.x), "=r"(b0.y), "=r"(b0.z), "=r"(b0.w) : "r"(tile_b + st0 * B_BYTES));
          asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(b1.x), "=r"(b1.y), "=r"(b1.z), "=r"(b1.w) : "r"(tile_b + (st0 + 1) * B_BYTES));
          qs = __dp4a((int)b0.x, 0x01010101, qs);
          qs = __dp4a((int)b0.y, 0x01010101, qs);
          qs = __dp4a((int)b0.z, 0x01010101, qs);
          qs = __dp4a((int)b0.w, 0x01010101, qs);
          qs = __dp4a((int)b1.x, 0x01010101, qs);
          qs = __dp4a((int)b1.y, 0x01010101, qs);
          qs = __dp4a((int)b1.z, 0x01010101, qs);
          qs = __dp4a((int)b1.w, 0x01010101, qs);
        }
        if (NP == 2) {
          uint4 b0, b1;
          asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(b0.x), "=r"(b0.y), "=r"(b0.z), "=r"(b0.w) : "r"(tile_b + st0 * B_BYTES + 8192));
          asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(b1.x), "=r"(b1.y), "=r"(b1.z), "=r"(b1.w) : "r"(tile_b + (st0 + 1) * B_BYTES + 8192));
          qs2 = __dp4a((int)b0.x, 0x01010101, qs2);
          qs2 = __dp4a((int)b0.y, 0x01010101, qs2);
          qs2 = __dp4a((int)b0.z, 0x01010101, qs2);
          qs2 = __dp4a((int)b0.w, 0x01010101, qs2);
          qs2 = __dp4a((int)b1.x, 0x01010101, qs2);
          qs2 = __dp4a((int)b1.y, 0x01010101, qs2);
          qs2 = __dp4a((int)b1.z, 0x01010101, qs2);
          qs2 = __dp4a((int)b1.w, 0x01010101, qs2);
        }
        {
          // 64 codes of the row in K order = 16 tensor-memory columns: columns 4 c4 .. 4 c4 + 3 take the words
          // 2 (c4 / 2), 2 (c4 / 2) + 1 of the 16 packed bytes under the slots 2h, 2h + 1 (h = c4 % 2)
          uint32_t w[4];
          asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];"
                       : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3])
                       : "r"(ring_a + slot * SLOT_BYTES));
          uint32_t o[16];
#pragma unroll
          for (int c4 = 0; c4 < 4; ++c4) {
            const uint32_t w0 = w[2 * (c4 >> 1)], w1 = w[2 * (c4 >> 1) + 1];
            const int h = c4 & 1;
            o[4 * c4 + 0] = (w0 >> (4 * h)) & 0x03030303u;
            o[4 * c4 + 1] = (w1 >> (4 * h)) & 0x03030303u;
            o[4 * c4 + 2] = (w0 >> (4 * h + 2)) & 0x03030303u;
            o[4 * c4 + 3] = (w1 >> (4 * h + 2)) & 0x03030303u;
          }
          const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + A_COL0 + (st0 + grp2) * 32 + hf * 16;
          asm volatile(
              "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, "
              "%14, %15, %16};"
              ::"r"(taddr), "r"(o[0]), "r"(o[1]), "r"(o[2]), "r"(o[3]), "r"(o[4]), "r"(o[5]), "r"(o[6]), "r"(o[7]),
                "r"(o[8]), "r"(o[9]), "r"(o[10]), "r"(o[11]), "r"(o[12]), "r"(o[13]), "r"(o[14]), "r"(o[15])
              : "memory");
          asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
          asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&bars->full[st0 + 1]);   // one barrier per stage pair (the odd stage's)
        st0 += 2;
        if (st0 == STAGES) st0 = 0, ph ^= 1u;
        slot = slot + 1 == SLOTS_A ? 0 : slot + 1;
      }
      if (!ok) break;
      // sum of the codes of token tb over all of K: the 8 threads that carry the token's pieces
      qs += __shfl_xor_sync(0xffffffffu, qs, 1);
      qs += __shfl_xor_sync(0xffffffffu, qs, 2);
      qs += __shfl_xor_sync(0xffffffffu, qs, 4);
      if (cb == 0) qsum_s[nt % NACC][tb] = qs;
      if (NP == 2) {
        qs2 += __shfl_xor_sync(0xffffffffu, qs2, 1);
        qs2 += __shfl_xor_sync(0xffffffffu, qs2, 2);
        qs2 += __shfl_xor_sync(0xffffffffu, qs2, 4);
        if (cb == 0) qsum_s[nt % NACC][tb + 64] = qs2;
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&bars->qsum_ready[nt % NACC]);
    }
    if (!ok) {
      atomicExch(&g_stream_tc_error, BITNET_ERR_TIMEOUT);
      bars->abort_flag = 1;
    }
  } else if (warp < WRITER_WARPS + MMA_WARPS) {
    // ------------------------------------------------------------ MMA issuers (whole warps; one lane issues)
    {
      const int me = warp - WRITER_WARPS;
      const uint32_t leader = elect_one();
      uint32_t it0 = 0, nt = 0;                   // pipeline index of the tile's K block 0; tiles done
      bool ok = true;
      for (int job = blockIdx.x; ok && job < a.total_tiles && !*abort_flag; job += gridDim.x, ++nt) {
        const TItem& d = a.it[locate(a, job)];
        const int nsteps = (int)(i2s_kp(d.K) / 256);
        const int buf = (int)(nt % NACC);
        ok = mbar_wait(&bars->tmem_empty[buf], ((nt / NACC) & 1u) ^ 1u, abort_flag, 1000);
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t d_tmem = tmem_base + buf * TILE_N;
        // a step = two K blocks = a stage pair: one wait, one fence and one commit per step (the writers signal and
        // wait on the pair's later stage only)
        for (int sidx = me; ok && sidx < nsteps; sidx += MMA_WARPS) {
          const uint32_t it = it0 + 2u * (uint32_t)sidx;
          const int st = (int)(it % STAGES);
          ok = mbar_wait(&bars->full[st + 1], (it / STAGES) & 1u, abort_flag, 20);   // codes in tensor memory, activations landed
          if (!ok) break;
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint64_t bdesc = make_desc(smem_u32(tileB + st * B_BYTES));
#pragma unroll
          for (int k4 = 0; k4 < 2 * (KBLK / 32); ++k4)   // 32 bytes further along K: +2 in the address field, +8 columns
            umma_u8s8_ta(d_tmem, tmem_base + A_COL0 + st * 32 + 8 * k4, bdesc + (uint64_t)((k4 >> 2) * (B_BYTES >> 4) + 2 * (k4 & 3)),
                         IDESC, 1u, leader);
          umma_commit(&bars->empty[st + 1], leader);   // the pair is reusable once these MMAs have read it
        }
        if (!ok) break;
        it0 += 2u * (uint32_t)nsteps;
        umma_commit(&bars->tmem_full[buf], leader);   // this issuer's share of the accumulator is complete
      }
      if (!ok && leader) {
        atomicExch(&g_stream_tc_error, BITNET_ERR_TIMEOUT);
        bars->abort_flag = 1;
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue
    const int quarter = warp & 3;                  // tensor-memory lanes 32*quarter .. 32*quarter+31
    uint32_t nt = 0;
    for (int job = blockIdx.x; job < a.total_tiles && !*abort_flag; job += gridDim.x, ++nt) {
      const TItem& d = a.it[locate(a, job)];
      const int buf = (int)(nt % NACC);
      const int m = (job - d.first_tile) * TILE_M + quarter * 32 + lane;
      float* const my_scale = ep_scale[quarter];
      __syncwarp();
      for (int i = lane; i < TILE_N; i += 32) my_scale[i] = (i < d.T) ? __fmul_rn(__ldg(d.act_scale + i), d.w_scale) : 0.0f;
      __syncwarp();
      if (!mbar_wait(&bars->tmem_full[buf], (nt / NACC) & 1u, abort_flag, 4000) ||
          !mbar_wait(&bars->qsum_ready[buf], (nt / NACC) & 1u, abort_flag, 1000)) {
        atomicExch(&g_stream_tc_error, BITNET_ERR_TIMEOUT);
        bars->abort_flag = 1;
        break;
      }
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + buf * TILE_N;
#pragma unroll 1
      for (int c0 = 0; c0 < TILE_N; c0 += 32) {
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
        if (m < d.M) {
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            const int t = c0 + j;
            if (t < d.T) {
              const int acc = (int)v[j] - qsum_s[buf][t];          // sum(code * q) - sum(q) = sum(w * q)
              d.y[(int64_t)t * d.ldy + m] = __fmul_rn((float)acc, my_scale[t]);
              if (d.acc_out) d.acc_out[(int64_t)t * d.ldy + m] = acc;
            }
          }
        }
      }
      // the accumulator and the sums have been read: clear it and hand the buffer back
#pragma unroll
      for (int c0 = 0; c0 < TILE_N; c0 += 32) zero32(taddr + c0);
      asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      __syncwarp();
      if (lane == 0) mbar_arrive(&bars->tmem_empty[buf]);
    }
  }

  // ---- teardown: every role has left its loop (all waits are bounded); free the tensor memory
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  if (warp == WRITER_WARPS)   // (the warp that allocated)
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "n"(TMEM_COLS) : "memory");
}

}  // namespace

// Shapes the kernel takes: 9 to 64 tokens; rows long enough that a tile's K blocks outnumber the ring by far (the
// hand-over of the per-token sums between tiles relies on it).
bool gemm_i2s_stream_tc_item_supported(int64_t T, int64_t M, int64_t K) {
  return T >= 9 && T <= MAX_N && M >= 1 && M <= 0x7fffffff && K >= 2048 && (K % 64) == 0 && K <= 0x3fffffff;
}

namespace {
template <int TN>
int launch_tn(const TArgs& a, int grid, cudaStream_t st) {
  constexpr int STAGES = TN == 64 ? 12 : 8;
  const size_t smem = (size_t)STAGES * TN * KBLK + RING_A_BYTES + sizeof(Bars) + 1024;
  static bool attr_set[64] = {false};
  int dev = 0;
  cudaGetDevice(&dev);
  if (!attr_set[dev & 63]) {
    cudaError_t e = cudaFuncSetAttribute(gemm_i2s_stream_tc_kernel<TN>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return note_cuda_error(e);
    attr_set[dev & 63] = true;
  }
  gemm_i2s_stream_tc_kernel<TN><<<grid, THREADS, smem, st>>>(a);
  return check_launch();
}
}  // namespace

// One launch per run of up to NITEMS items whose token counts fall into the same class (up to 64: 64-token tiles;
// 65 to 128: 128-token tiles).
int launch_gemm_i2s_stream_tc(const StreamTcLinear* items, int64_t n, cudaStream_t st) {
  static thread_local TArgs a;      // 26 KB: off the stack
  for (int64_t i0 = 0; i0 < n;) {
    const bool wide = items[i0].T > 64;
    int cnt = 0;
    int64_t tiles = 0;
    while (i0 + cnt < n && cnt < NITEMS && (items[i0 + cnt].T > 64) == wide) {
      const StreamTcLinear& s = items[i0 + cnt];
      if (!gemm_i2s_stream_tc_item_supported(s.T, s.M, s.K)) return BITNET_ERR_UNSUPPORTED_SHAPE;
      if (tiles + ceil_div(s.M, TILE_M) > 0x3fffffff) break;
      TItem& d = a.it[cnt];
      d.packed = s.packed;
      d.q = s.q;
      d.act_scale = s.act_scale;
      d.y = s.y;
      d.acc_out = s.acc_out;
      d.w_scale = s.w_scale;
      d.M = (int)s.M;
      d.K = (int)s.K;
      d.T = s.T;
      d.first_tile = (int)tiles;
      d.ldy = (int)(s.ldy ? s.ldy : s.M);
      tiles += ceil_div(s.M, TILE_M);
      ++cnt;
    }
    if (cnt == 0) return BITNET_ERR_UNSUPPORTED_SHAPE;
    a.n = cnt;
    a.total_tiles = (int)tiles;
    int grid = dev_info().sm_count;
    if (grid > tiles) grid = (int)tiles;
    log_launch("gemm_i2s_stream_tc_kernel<%d> items=%d tiles=%lld grid=%d", wide ? 128 : 64, cnt, (long long)tiles, grid);
    const int rc = wide ? launch_tn<128>(a, grid, st) : launch_tn<64>(a, grid, st);
    if (rc) return rc;
    i0 += cnt;
  }
  return BITNET_OK;
}

int gemm_i2s_stream_tc_status(int* out) {
  cudaError_t e = cudaMemcpyFromSymbol(out, g_stream_tc_error, sizeof(int));
  return e == cudaSuccess ? BITNET_OK : note_cuda_error(e);
}
int gemm_i2s_stream_tc_status_clear() {
  const int zero = 0;
  cudaError_t e = cudaMemcpyToSymbol(g_stream_tc_error, &zero, sizeof(int));
  return e == cudaSuccess ? BITNET_OK : note_cuda_error(e);
}

}  // namespace bitnet
