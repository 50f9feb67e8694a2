// I2_S mpGEMM for 17 to 128 tokens over a list of linears: Alg. 1 Phase 2 with the weights streamed from HBM once
// and multiplied on the fifth-generation tensor cores (tcgen05.mma kind::i8, accumulators in tensor memory).
//
//   acc[t,m] = sum_k q[t,k] * w[m,k],   y[t,m] = acc[t,m] * act_scale[t] * w_scale
//
// Between decode (1..8 tokens: the weight stream is everything, mma.sync keeps up) and prefill (hundreds of tokens:
// the tensor cores are everything) the work per weight byte is small enough that the blob should cross HBM once,
// yet too large for mma.sync: m16n8k32 needs 2 T MMAs per 1-KB chunk.  The paper treats neither stage; the design
// is this build's.  One persistent CTA per SM walks tiles of 128 out-features x all of K; the list's tiles form one
// sequence, of which a CTA takes the contiguous range that holds its equal share of the work (steps).  A step is two
// 256-column chunks of the tile's rows (four K blocks of 128) at 64-token tiles, one chunk at 128-token tiles.
//   * warp 24 (producer of packed words): per step one bulk copy per 16-row unit of the tile (a unit's chunks are
//     contiguous in the blob) into a ring of shared memory, 8 chunks ahead of the writers;
//   * warp 25 (producer of activation tiles): per K block one tensor copy of 128 codes x 64 (128) tokens of q into the
//     128-byte-swizzled K-major layout of operand B, zeros beyond T and K (the tensor maps, one per item, travel in
//     the argument block), as far ahead as the ring of 3 (4) steps allows;
//   * warps 0-15 (writers): thread = (row of the tile, 16 bytes of a chunk's 64).  It turns the 2-bit codes into bytes
//     whose top two bits are the code (a left shift and a mask per word: 64 x code as UNSIGNED 8-bit values; the
//     factor 64 and the "- sum(q)" of code = w + 1 are taken out in the epilogue) and writes them straight into
//     tensor memory (tcgen05.st): operand A never touches shared memory as bytes.  In the first tile of an item the
//     writers also add up the codes of the landed activation tiles: sum(q) per token, kept for the item's other tiles;
//   * warps 16-19: issuers.  Issuer i takes the steps i, i + R, ... of the CTA's whole step sequence (R = steps in
//     the ring = issuers at work), so it always meets the same barriers, phase after phase.  Per step one elected
//     lane issues 16 (8) tcgen05.mma (M = 128, N = 64 or 128, K = 32; A from tensor memory, B from shared memory) and
//     releases the step's stages with one tcgen05.commit; every MMA accumulates (the epilogue leaves the accumulators
//     zeroed), so their order does not matter;
//   * warps 20-23: epilogue -- tcgen05.ld the finished 128 x 64 accumulator, zero it, divide by 64, subtract sum(q),
//     rescale, store y.
// Two accumulators (2 x 64 or 2 x 128 columns) overlap a tile's epilogue with the next tile's MMAs; the A ring takes
// the other 12 (8) x 32 columns.  Measured on the 100B-shaped sweep (17.1 GB of packed weights, inputs fp32, the
// list quantiser included): 4.7 ms at 32 tokens, 5.2 at 64, 8.0 at 128, against 9.6 to 19.4 ms for the mma.sync
// kernel of gemv_i2s_mid.cu and 22 ms for the prefill kernel at 128.  What binds: the writers -- about 500 cycles
// of integer work and 400 of barrier probes per step against the 712 the HBM stream allows -- then, at 128 tokens,
// the tensor pipe.  Two rules learnt by measurement: a wait for phase k of a barrier means nothing unless phase
// k - 1 is known to be over (hence issuers bound to their own stages), and a ring slot may be handed back only
// after the values loaded from it have been used, not right behind the loads.  Every mbarrier wait is bounded; a wait
// that gives up sets a CTA-wide abort flag and the device status word, all roles leave their loops, and the CTA frees
// its tensor memory before it exits.
#include <cuda.h>

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
constexpr int MMA_WARPS = 4;                 // issuer warps (NISS of them at work: see the kernel)
constexpr int PRODUCER_WARP = WRITER_WARPS + MMA_WARPS + 4;    // packed words (operand A's source); after the 4 epilogue warps
constexpr int PRODUCER_B_WARP = PRODUCER_WARP + 1;             // activation tiles (operand B)
constexpr int THREADS = (PRODUCER_B_WARP + 1) * 32;
// A step = CPS 256-column chunks of a tile's rows (2 CPS K blocks = 2 CPS stages): two chunks per step at 64-token
// tiles (12 stages = 3 steps in the ring), one at 128-token tiles (8 stages = 4 steps).  Per step a writer thread
// unpacks 16 bytes of packed words per chunk; the waits, fences and barrier arrivals are paid once per step.
__host__ __device__ constexpr int cps_of(int tn) { return tn == 64 ? 2 : 1; }
// slots of the packed-word ring = steps the producer runs ahead (8 chunks of the tile's 128 rows either way: 64 KB)
__host__ __device__ constexpr int da_of(int tn) { return 8 / cps_of(tn); }
__host__ __device__ constexpr int ring_a_bytes(int tn) { return da_of(tn) * cps_of(tn) * 8192; }
constexpr int MAX_SLOTS_A = 8;
// Steps in the ring of the activation tiles (operand B, shared memory), of operand A (tensor memory) and of the step
// barriers: 3 at 64-token tiles (12 stages of 32 columns beside two accumulators), 4 at 128-token tiles.  A longer B
// ring with its own barriers (4 steps at 64-token tiles) measured no faster and costs the writers a wait per step.
__host__ __device__ constexpr int rb_of(int tn) { return tn == 64 ? 3 : 4; }
__host__ __device__ constexpr int b_stages(int tn) { return rb_of(tn) * 2 * cps_of(tn); }
constexpr int NITEMS = 160;                  // items per launch (argument block of 32 KB: a tensor map and 72 bytes each)
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
  int64_t first_w;        // steps of the tiles of the items before this one (the measure of work the CTAs share)
};
static_assert(sizeof(TItem) == 72, "argument block layout");

struct TArgs {
  CUtensorMap qmap[NITEMS];   // the item's codes q[T][K] as tiles of 128 columns x TN tokens, 128-byte swizzle, zero fill
  int n, total_tiles;
  int64_t total_w;
  TItem it[NITEMS];
};
static_assert(sizeof(TArgs) <= 32764, "kernel parameter limit");

struct __align__(8) Bars {
  uint64_t full[MAX_STAGES], empty[MAX_STAGES];         // per step of the ring: codes written / operands read by the MMAs
  uint64_t tmem_full[NACC], tmem_empty[NACC], qsum_ready[NACC];
  uint64_t b_full[4];                                   // a step's activation tiles have landed
  uint64_t a_full[MAX_SLOTS_A], a_empty[MAX_SLOTS_A];   // packed-word ring: bytes landed / slot read by every writer warp
  uint32_t tmem_base;
  int abort_flag;
};

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
// bulk asynchronous copy global -> shared (16-byte aligned, a multiple of 16 bytes), bytes counted on `bar`
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint64_t* bar, uint64_t pol) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
      ::"r"(dst), "l"(src), "r"(bytes), "r"(smem_u32(bar)), "l"(pol)
      : "memory");
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

// Instruction descriptor: D = s32, A = u8 (64 x the codes 0, 1, 2), B = s8, both K-major, N tokens, M = 128.
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

// steps of one tile of an item with K columns
__host__ __device__ __forceinline__ int steps_of(int K, int cps) { return (int)((i2s_kp(K) / 256 + cps - 1) / cps); }

// first tile (of the list's tile sequence) whose first step lies at or after position w of the list's step sequence
__device__ __forceinline__ int tile_at(const TArgs& a, int64_t w, int cps) {
  if (w >= a.total_w) return a.total_tiles;
  int lo = 0, hi = a.n - 1;
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if (a.it[mid].first_w <= w) lo = mid; else hi = mid - 1;
  }
  const int ns = steps_of(a.it[lo].K, cps);
  return a.it[lo].first_tile + (int)((w - a.it[lo].first_w + ns - 1) / ns);
}

template <int TN>
__global__ void __launch_bounds__(THREADS, 1) gemm_i2s_stream_tc_kernel(const __grid_constant__ TArgs a) {
  constexpr int TILE_N = TN;
  constexpr int STAGES = TN == 64 ? 12 : 8;
  constexpr int CPS = cps_of(TN), GST = 2 * CPS;   // chunks and stages per step
  constexpr int DA = da_of(TN), SLOTS_A = DA, RB = rb_of(TN);
  constexpr int RA = STAGES / GST;                 // steps in the tensor-memory ring of operand A
  constexpr int STAGES_B = RB * GST;               // activation tiles (one per K block) in shared memory
  constexpr uint32_t SLOT_BYTES = CPS * 8192;      // a step's packed words of the tile: 8 units x CPS KB
  constexpr int RING_A_BYTES = ring_a_bytes(TN);
  // Issuers at work: as many as the ring holds steps, issuer i taking the steps i, i + NISS, ... of the CTA's whole
  // step sequence (counted across tiles), i.e. always the same stages.  A wait for a barrier's phase k is only
  // meaningful once phase k - 1 is known to be complete (a barrier still in phase k - 1 answers "done" to a probe
  // for the parity of k); an issuer that meets every phase of its own barriers in order knows that.
  constexpr int NISS = RB;
  static_assert(NISS <= MMA_WARPS && RA <= RB, "an issuer warp per step of the barrier ring");
  constexpr int A_COL0 = NACC * TILE_N;        // first tensor-memory column of the A ring (32 columns per stage)
  constexpr int B_BYTES = TILE_N * KBLK;       // 8 or 16 KB per stage
  constexpr int NP = TN / 64;                  // activation pieces per writer thread and K block (tokens tb, tb + 64)
  constexpr uint32_t IDESC = idesc_of(TN);
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* tileB = smem;                                   // STAGES_B x 8 or 16 KB
  uint8_t* ringA = smem + STAGES_B * B_BYTES;              // SLOTS_A steps of packed words
  Bars* bars = reinterpret_cast<Bars*>(smem + STAGES_B * B_BYTES + RING_A_BYTES);
  volatile int* abort_flag = &bars->abort_flag;
  __shared__ int qsum_s[NACC][MAX_N];                      // sum of a token's codes over K, per accumulator in flight
  __shared__ float ep_scale[4][MAX_N];                     // epilogue: act_scale[t] * w_scale of the current tile

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // this CTA's tiles: a contiguous range of the list's tile sequence holding an equal share of its steps (a CTA
  // then meets few items, and the per-token sums of an item are taken once per CTA, not once per tile)
  const int jb = tile_at(a, a.total_w * blockIdx.x / gridDim.x, CPS);
  const int je = tile_at(a, a.total_w * (blockIdx.x + 1) / gridDim.x, CPS);

  if (threadIdx.x == 0) {
    for (int s = 0; s < RB; ++s) {            // (per step of the barrier ring)
      // every writer warp: its codes are in tensor memory
      mbar_init(&bars->full[s], WRITER_WARPS);
      mbar_init(&bars->b_full[s], 1);            // the producer's arrival with the byte count
      mbar_init(&bars->empty[s], 1);             // tcgen05.commit: the step's MMAs have read their operands
    }
    for (int sl = 0; sl < SLOTS_A; ++sl) {
      mbar_init(&bars->a_full[sl], 1);           // the producer's arrival with the byte count
      mbar_init(&bars->a_empty[sl], WRITER_WARPS);
    }
    for (int b = 0; b < NACC; ++b) {
      mbar_init(&bars->tmem_full[b], NISS);      // one tcgen05.commit per issuer at work
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
  if (warp >= WRITER_WARPS + MMA_WARPS && warp < PRODUCER_WARP) {
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
    // this thread's 16 bytes of a chunk in a ring slot: the slot holds the tile's 8 units, CPS KB each, as the blob does
    const uint32_t ring_a = smem_u32(ringA) + (r >> 4) * (CPS * 1024) + (r & 15) * 64 + grp2 * 32 + hf * 16;
    const uint32_t tile_b = smem_u32(tileB) + b_off;
    // Running positions instead of divisions: st0 = first stage of the current step (a multiple of GST), ph = how
    // often the stage ring has been passed (mod 2), slot = the step's ring slot.
    int bs = 0, tg = 0, slot = 0;                  // (bs: position in the B and barrier ring; tg: in the tensor-memory ring)
    uint32_t ph = 0, pha = 0;                      // (pha: passes of the packed-word ring, mod 2)
    uint32_t g = 0;                                // steps done by this CTA
    uint32_t nt = 0;
    bool ok = true;
    int ii = jb < je ? locate(a, jb) : 0, prev_item = -1;
    int qtot = 0, qtot2 = 0;                       // sums of the codes of this thread's tokens over K, current item
    for (int job = jb; ok && job < je && !*abort_flag; ++job, ++nt) {
      while (ii + 1 < a.n && a.it[ii + 1].first_tile <= job) ++ii;
      const TItem& d = a.it[ii];
      const bool need_q = ii != prev_item;         // first tile of the item in this CTA: take the sums of the codes
      prev_item = ii;
      const int64_t kp = i2s_kp(d.K);
      const int nch = (int)(kp / 256), nsteps = (nch + CPS - 1) / CPS;
      // chunk c of a row: 64 bytes; K block 2c + grp2 = its half grp2 (32 bytes), of which this thread takes 16
      int qs = 0, qs2 = 0;
      for (int s2 = 0; s2 < nsteps && ok; ++s2) {
        // the step's packed words have landed (bulk copies of the producer warp).  (A chunk beyond the row's last, or a
        // row beyond M, is not copied: what the slot holds then meets activation codes that are all zero, or sums that
        // are never stored.)
        ok = mbar_wait(&bars->a_full[slot], pha, abort_flag, 20);
        if (!ok) break;
        // the tensor-memory columns of this step were last read by the MMAs of step g - RA
        static_assert(RA == RB, "one barrier ring for both operands");
        ok = mbar_wait(&bars->empty[bs], ph ^ 1u, abort_flag, 20);
        if (!ok) break;
        // A tile that takes the sums of the codes reads this thread's pieces of the landed activation tiles.  (After
        // the wait above: the MMAs of step g - RB being over means the barrier of the activation tiles has left the
        // phase of that step, so a probe for this step's phase cannot be answered by the one before.)
        if (need_q) {
          ok = mbar_wait(&bars->b_full[bs], ph, abort_flag, 20);
          if (!ok) break;
        }
        if (need_q) {
#pragma unroll
          for (int j = 0; j < GST; ++j) {
            uint4 b0;                              // this thread's own pieces, for the row sums
            asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(b0.x), "=r"(b0.y), "=r"(b0.z), "=r"(b0.w) : "r"(tile_b + (bs * GST + j) * B_BYTES));
            qs = __dp4a((int)b0.x, 0x01010101, qs);
            qs = __dp4a((int)b0.y, 0x01010101, qs);
            qs = __dp4a((int)b0.z, 0x01010101, qs);
            qs = __dp4a((int)b0.w, 0x01010101, qs);
            if (NP == 2) {
              uint4 b1;
              asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(b1.x), "=r"(b1.y), "=r"(b1.z), "=r"(b1.w) : "r"(tile_b + (bs * GST + j) * B_BYTES + 8192));
              qs2 = __dp4a((int)b1.x, 0x01010101, qs2);
              qs2 = __dp4a((int)b1.y, 0x01010101, qs2);
              qs2 = __dp4a((int)b1.z, 0x01010101, qs2);
              qs2 = __dp4a((int)b1.w, 0x01010101, qs2);
            }
          }
        }
        uint32_t wa[CPS][4];
#pragma unroll
        for (int c = 0; c < CPS; ++c)
          asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];"
                       : "=r"(wa[c][0]), "=r"(wa[c][1]), "=r"(wa[c][2]), "=r"(wa[c][3])
                       : "r"(ring_a + slot * SLOT_BYTES + c * 1024));
#pragma unroll
        for (int c = 0; c < CPS; ++c) {
          // 64 codes of the row in K order = 16 tensor-memory columns: columns 4 c4 .. 4 c4 + 3 take the words
          // 2 (c4 / 2), 2 (c4 / 2) + 1 of the 16 packed bytes under the slots 2h, 2h + 1 (h = c4 % 2)
          const uint32_t* w = wa[c];
          uint32_t o[16];
#pragma unroll
          for (int c4 = 0; c4 < 4; ++c4) {
            const uint32_t w0 = w[2 * (c4 >> 1)], w1 = w[2 * (c4 >> 1) + 1];
            const int h = c4 & 1;
            // the code moves to the top two bits of its byte (64 x code: one scale for all four fields, taken out in
            // the epilogue): left shifts, which the multiply-add pipe can do beside the integer pipe's masks
            o[4 * c4 + 0] = (w0 << (6 - 4 * h)) & 0xC0C0C0C0u;
            o[4 * c4 + 1] = (w1 << (6 - 4 * h)) & 0xC0C0C0C0u;
            o[4 * c4 + 2] = (w0 << (4 - 4 * h)) & 0xC0C0C0C0u;
            o[4 * c4 + 3] = (w1 << (4 - 4 * h)) & 0xC0C0C0C0u;
          }
          const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + A_COL0 + (tg * GST + 2 * c + grp2) * 32 + hf * 16;
          asm volatile(
              "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, "
              "%14, %15, %16};"
              ::"r"(taddr), "r"(o[0]), "r"(o[1]), "r"(o[2]), "r"(o[3]), "r"(o[4]), "r"(o[5]), "r"(o[6]), "r"(o[7]),
                "r"(o[8]), "r"(o[9]), "r"(o[10]), "r"(o[11]), "r"(o[12]), "r"(o[13]), "r"(o[14]), "r"(o[15])
              : "memory");
        }
        asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncwarp();
        // The ring slot goes back to the producer only here, after the codes made from its words have been stored: an
        // arrival right behind the shared-memory loads is not held back until they have read (measured: a refill
        // overtook them), the loads' results having been used is.
        if (lane == 0) {
          mbar_arrive(&bars->a_empty[slot]);
          mbar_arrive(&bars->full[bs]);
        }
        ++g;
        if (++bs == RB) bs = 0, ph ^= 1u;
        if (++tg == RA) tg = 0;
        if (++slot == SLOTS_A) slot = 0, pha ^= 1u;
      }
      if (!ok) break;
      if (need_q) {
        // sum of the codes of token tb over all of K: the 8 threads that carry the token's pieces
        qs += __shfl_xor_sync(0xffffffffu, qs, 1);
        qs += __shfl_xor_sync(0xffffffffu, qs, 2);
        qs += __shfl_xor_sync(0xffffffffu, qs, 4);
        qtot = qs;
        if (NP == 2) {
          qs2 += __shfl_xor_sync(0xffffffffu, qs2, 1);
          qs2 += __shfl_xor_sync(0xffffffffu, qs2, 2);
          qs2 += __shfl_xor_sync(0xffffffffu, qs2, 4);
          qtot2 = qs2;
        }
      }
      if (cb == 0) {
        qsum_s[nt % NACC][tb] = qtot;
        if (NP == 2) qsum_s[nt % NACC][tb + 64] = qtot2;
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
      uint32_t g0 = 0, nt = 0;                    // steps before this tile; tiles done
      bool ok = true;
      int ii = jb < je ? locate(a, jb) : 0;
      for (int job = jb; me < NISS && ok && job < je && !*abort_flag; ++job, ++nt) {
        while (ii + 1 < a.n && a.it[ii + 1].first_tile <= job) ++ii;
        const int nsteps = steps_of(a.it[ii].K, CPS);
        const int buf = (int)(nt % NACC);
        ok = mbar_wait(&bars->tmem_empty[buf], ((nt / NACC) & 1u) ^ 1u, abort_flag, 200);
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t d_tmem = tmem_base + buf * TILE_N;
        // a step = GST K blocks = GST stages: one wait, one fence and one commit per step (the writers signal and
        // wait on the step's last stage only)
        for (int sidx = (int)((me + NISS - g0 % NISS) % NISS); ok && sidx < nsteps; sidx += NISS) {
          const uint32_t g = g0 + (uint32_t)sidx;        // the step's number in the CTA's step sequence
          const int pos = (int)(g % RB), st = pos * GST, sta = (int)(g % RA) * GST;
          ok = mbar_wait(&bars->full[pos], (g / RB) & 1u, abort_flag, 200);   // codes in tensor memory, activations landed
          if (!ok) break;
          ok = mbar_wait(&bars->b_full[pos], (g / RB) & 1u, abort_flag, 20);      // the step's activation tiles have landed
          if (!ok) break;
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint64_t bdesc = make_desc(smem_u32(tileB + st * B_BYTES));
#pragma unroll
          for (int k4 = 0; k4 < GST * (KBLK / 32); ++k4)   // 32 bytes further along K: +2 in the address field, +8 columns
            umma_u8s8_ta(d_tmem, tmem_base + A_COL0 + sta * 32 + 8 * k4, bdesc + (uint64_t)((k4 >> 2) * (B_BYTES >> 4) + 2 * (k4 & 3)),
                         IDESC, 1u, leader);
          umma_commit(&bars->empty[pos], leader);   // the step's tiles and columns are reusable once these MMAs have read them
        }
        if (!ok) break;
        g0 += (uint32_t)nsteps;
        umma_commit(&bars->tmem_full[buf], leader);   // this issuer's share of the accumulator is complete
      }
      if (!ok && leader) {
        atomicExch(&g_stream_tc_error, BITNET_ERR_TIMEOUT);
        bars->abort_flag = 1;
      }
    }
  } else if (warp == PRODUCER_B_WARP) {
    // ------------------------------------------------------------ producer of the activation tiles (operand B)
    // Per step GST tiles of 128 columns x TN tokens (tensor copies: 128-byte swizzle, zeros beyond T and K), as far
    // ahead as the ring allows: a step's tiles are free once the MMAs of the step RB before have read them.
    int bs = 0;
    uint32_t ph = 0;
    bool ok = true;
    int ii = jb < je ? locate(a, jb) : 0;
    for (int job = jb; ok && job < je && !*abort_flag; ++job) {
      while (ii + 1 < a.n && a.it[ii + 1].first_tile <= job) ++ii;
      const int nsteps = steps_of(a.it[ii].K, CPS);
      const CUtensorMap* map = &a.qmap[ii];
      for (int s2 = 0; s2 < nsteps && ok; ++s2) {
        ok = mbar_wait(&bars->empty[bs], ph ^ 1u, abort_flag, 200);
        if (!ok) break;
        if (lane == 0) {
          mbar_expect_tx(&bars->b_full[bs], (uint32_t)(GST * B_BYTES));
#pragma unroll
          for (int j = 0; j < GST; ++j)
            asm volatile(
                "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                ::"r"(smem_u32(tileB + (bs * GST + j) * B_BYTES)), "l"(map), "r"((s2 * GST + j) * KBLK), "r"(0),
                  "r"(smem_u32(&bars->b_full[bs]))
                : "memory");
        }
        __syncwarp();
        if (++bs == RB) bs = 0, ph ^= 1u;
      }
    }
    if (!ok && lane == 0) {
      atomicExch(&g_stream_tc_error, BITNET_ERR_TIMEOUT);
      bars->abort_flag = 1;
    }
  } else if (warp == PRODUCER_WARP) {
    // ------------------------------------------------------------ producer of the packed-word ring
    // Per step one bulk copy per 16-row unit of the tile (a unit's chunks are contiguous in the blob: CPS KB), issued
    // by one lane each, SLOTS_A steps ahead of the writers: whole 32-byte sectors, no copy instructions in the
    // writers' instruction stream.
    const uint64_t pol = policy_evict_first();
    int slot = 0;
    uint32_t php = 0;
    bool ok = true;
    int ii = jb < je ? locate(a, jb) : 0;
    for (int job = jb; ok && job < je && !*abort_flag; ++job) {
      while (ii + 1 < a.n && a.it[ii + 1].first_tile <= job) ++ii;
      const TItem& d = a.it[ii];
      const int64_t kp = i2s_kp(d.K);
      const int nch = (int)(kp / 256), nsteps = (nch + CPS - 1) / CPS;
      const int row0 = (job - d.first_tile) * TILE_M;
      const int left = (d.M - row0 + 15) >> 4, nunits = left < 8 ? left : 8;
      const uint8_t* src = d.packed + ((int64_t)(row0 >> 4) + lane) * (4 * kp);
      const uint32_t dst = smem_u32(ringA) + lane * (CPS * 1024);
      for (int s2 = 0; s2 < nsteps && ok; ++s2) {
        ok = mbar_wait(&bars->a_empty[slot], php ^ 1u, abort_flag, 200);   // every writer warp has read the slot
        if (!ok) break;
        const int nc = nch - s2 * CPS < CPS ? nch - s2 * CPS : CPS;
        if (lane == 0) mbar_expect_tx(&bars->a_full[slot], (uint32_t)(nunits * nc) * 1024u);
        __syncwarp();
        if (lane < nunits) bulk_g2s(dst + slot * SLOT_BYTES, src + (int64_t)s2 * (CPS * 1024), (uint32_t)nc * 1024u, &bars->a_full[slot], pol);
        if (++slot == SLOTS_A) slot = 0, php ^= 1u;
      }
    }
    if (!ok && lane == 0) {
      atomicExch(&g_stream_tc_error, BITNET_ERR_TIMEOUT);
      bars->abort_flag = 1;
    }
  } else {
    // ------------------------------------------------------------ epilogue
    const int quarter = warp & 3;                  // tensor-memory lanes 32*quarter .. 32*quarter+31
    uint32_t nt = 0;
    int ii = jb < je ? locate(a, jb) : 0;
    for (int job = jb; job < je && !*abort_flag; ++job, ++nt) {
      while (ii + 1 < a.n && a.it[ii + 1].first_tile <= job) ++ii;
      const TItem& d = a.it[ii];
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
              const int acc = ((int)v[j] >> 6) - qsum_s[buf][t];   // sum(64 code * q) / 64 - sum(q) = sum(w * q)
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
  // (K: the accumulators hold 64 x sum(code * q), at most 64 * 2 * 127 * K in magnitude)
  return T >= 9 && T <= MAX_N && M >= 1 && M <= 0x7fffffff && K >= 2048 && (K % 64) == 0 && K <= 131072;
}

namespace {
template <int TN>
int launch_tn(const TArgs& a, int grid, cudaStream_t st) {
  const size_t smem = (size_t)b_stages(TN) * TN * KBLK + ring_a_bytes(TN) + sizeof(Bars) + 1024;
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
    int64_t tiles = 0, work = 0;
    const int cps = cps_of(wide ? 128 : 64);
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
      d.first_w = work;
      if (int rc = encode_q_tile_map(&a.qmap[cnt], s.q, s.K, s.T, wide ? 128 : 64)) return rc;
      work += ceil_div(s.M, TILE_M) * steps_of((int)s.K, cps);
      tiles += ceil_div(s.M, TILE_M);
      ++cnt;
    }
    if (cnt == 0) return BITNET_ERR_UNSUPPORTED_SHAPE;
    a.n = cnt;
    a.total_tiles = (int)tiles;
    a.total_w = work;
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
