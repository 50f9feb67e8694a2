// TL2 decode (1..8 tokens) at the rate of the memory stream: the 1.67-bit blob of Table 5 / Alg. 4 (4-bit index
// + 1-bit sign per weight triple, the two planes of Sec. 3.1.2) scanned once, every packed index resolved by ONE
// shared-memory table lookup into the weights it stands for, which then go through the int8 tensor cores against
// the quantised activations.  Same persistent, grouped form as the I2_S kernel (gemv_i2s_group.cu): a list of
// linears is one stream of 32-row blocks cut into equal shares per SM.
//
// Why not the activation tables of Alg. 2 here: a table of partial sums needs one lookup, one conditional negate
// and one add per triple on the integer pipe -- 5-6 instructions per 3 weights, which caps the scan at a quarter of
// the memory rate (gemv_tl.cu is that form).  The table below is indexed the other way round: by the packed bits.
//
// Decode table.  One index byte (two triples) plus its two sign bits is a 10-bit number; the table maps it to the
// six weights as 2-bit codes w+1 laid out as an "I2_S word": byte b, bit pair s of the 32-bit entry holds
// (triple 0: w0,w1,w2 -> s=0, b=0,1,2; triple 1: w0 -> s=0, b=3; w1,w2 -> s=1, b=0,1).  Two entries E, E' of
// neighbouring index bytes join as X = E + 16 E' (E' moves to s = 2, 3), and X & (0x03030303 << 2s) is an A
// register of mma.sync.m16n8k32 (u8 x s8) exactly as in the I2_S kernel: four accumulators carry the scales
// 1, 4, 16, 64, and sum(code*q) - sum(q) = sum(w*q).  Every lane keeps a private copy of the table (entry e of
// lane l at word 32e + l: bank l whatever e is), so the 32 lookups of a warp never conflict: 128 KB.
//
// Tile = 32 rows x 32 triples (640 B).  Lane (g, t) owns index word t of the rows g, g+8, g+16, g+24: one 16-byte
// piece of the index plane (the tile layout interleaves exactly these four rows), which is also the piece the lane
// copied with cp.async; the four rows' sign words are the 16-byte piece 512 + 16g.  (signs >> 2t) & 0x03030303
// puts the sign pair of index byte j into byte j, and one byte permute joins index byte and sign pair into the
// table index.  Rows g, g+8 are the A rows of the MMAs of the block's upper half, g+16, g+24 of its lower half.
//
// Activations are staged in the order the decoded words want them: per tile and lane-quarter t, 32 bytes = the
// B registers of the four scales for the two X words (24 codes + 8 zero bytes).  The pair-coded tail columns of a
// row (TL1 tiles, Table 4 / Alg. 3; at most two tiles) go through a 256-entry table (index byte -> four codes) and
// half-filled MMAs.
#include <cstdlib>
#include <cstring>

#include "common.cuh"
#include "device_utils.cuh"

namespace bitnet {
namespace {

constexpr int CW = 16;  // warps
constexpr int THREADS = CW * 32;
constexpr int XREG = 16;
constexpr int NSMALL = 44, NLARGE = 363;   // items per launch: argument blocks of 4 KB / 32 KB
constexpr int SLOT = 640;                  // ring slot = one tile
constexpr int TBL2_BYTES = 1024 * 32 * 4;

struct SItem {
  const uint8_t* packed;
  const float* x;      // fp32 activations [T][K]; null: q and act_scale are inputs
  int8_t* q;
  float* act_scale;
  float* y;
  int32_t* acc_out;
  float w_scale;
  int M, K, T;
  int tiles3, tiles2;  // triple / pair tiles per 32-row block
  int block_bytes;
  int first_unit;      // 32-row blocks of the items before this one
  int first_w;         // tiles of the items before this one
  int ldy;             // elements between the token rows of y and acc_out
};
static_assert(sizeof(SItem) == 88, "argument block layout");

template <int NMAX>
struct SArgs {
  int n, S, tmax, code_bytes;
  int total_units, total_w, r0, r1;
  SItem it[NMAX];
};
static_assert(sizeof(SArgs<NSMALL>) <= 4096 && sizeof(SArgs<NLARGE>) <= 32764, "kernel parameter limits");

__device__ __forceinline__ bool same_input(const SItem& p, const SItem& d) {
  return p.K == d.K && p.T == d.T && p.tiles3 == d.tiles3 &&
         (d.x ? p.x == d.x : (p.x == nullptr && p.q == d.q && p.act_scale == d.act_scale));
}

__device__ __forceinline__ unsigned lds32(uint32_t addr) {
  unsigned v;
  asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
  return v;
}
// Generic byte permute: selector nibbles 0..7 pick a byte of {a, b}; with bit 3 set the picked byte's sign bit is
// replicated instead (a byte below 128 gives 0).
__device__ __forceinline__ unsigned prmt(unsigned a, unsigned b, unsigned sel) {
  unsigned d;
  asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
  return d;
}
__device__ __forceinline__ void lds128(uint32_t addr, unsigned (&v)[4]) {
  asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]) : "r"(addr));
}

// The three 2-bit codes (w+1) of a triple from its index (0..13; 14, 15 do not occur) and sign: the balanced-ternary
// digits of v = +-index (Table 5: v = 9 w0 + 3 w1 + w2).
__device__ __forceinline__ void triple_codes(int idx, int neg, int* c0, int* c1, int* c2) {
  if (idx > 13) idx = 0;
  const int d0 = (idx + 4) / 9;
  const int rem = idx - 9 * d0;
  const int d1 = (rem + 7) / 3 - 2;
  const int d2 = rem - 3 * d1;
  const int sg = neg ? -1 : 1;
  *c0 = sg * d0 + 1;
  *c1 = sg * d1 + 1;
  *c2 = sg * d2 + 1;
}

// Stores the four codes of columns 4i..4i+3 of a token row into the staged (permuted) order.
//   triple-coded columns: tile = k / 96, quarter t = (k % 96) / 24; the quarter's 32 bytes are the words
//   (scale s, X word h) at 4(2s + h): h = first or second 12 columns, which hold their 12 codes as
//   s=0: 4 codes, s=1: 2 codes + 2 zero bytes, s=2: 4 codes, s=3: 2 codes + 2 zero bytes;
//   pair-coded columns follow in natural order, 64 bytes per tile.
__device__ __forceinline__ void store_codes(int8_t* row, int i, int word, int three_k4, int tiles3) {
  if (i < three_k4) {
    const int k = 4 * i;
    const int tile = k / 96, c = k - 96 * tile;
    const int t = c / 24, o = c - 24 * t;
    const int h = o >= 12 ? 1 : 0, o2 = o - 12 * h;          // o2 in {0, 4, 8}
    int8_t* blk = row + tile * 128 + t * 32 + 4 * h;
    if (o2 == 0) {
      *reinterpret_cast<int*>(blk) = word;                                       // s = 0
    } else if (o2 == 4) {
      *reinterpret_cast<int*>(blk + 8) = word & 0xFFFF;                          // s = 1 (two codes, two zeros)
      *reinterpret_cast<short*>(blk + 16) = (short)((unsigned)word >> 16);       // s = 2, bytes 0, 1
    } else {
      *reinterpret_cast<short*>(blk + 18) = (short)(word & 0xFFFF);              // s = 2, bytes 2, 3
      *reinterpret_cast<int*>(blk + 24) = (int)((unsigned)word >> 16);           // s = 3 (two codes, two zeros)
    }
  } else {
    *reinterpret_cast<int*>(row + tiles3 * 128 + 4 * (i - three_k4)) = word;
  }
}

// Stages the item's activation codes (T rows, qst bytes apart) and, per token, the scale and the sum of the codes.
// Called by all threads; contains barriers.
__device__ __forceinline__ void stage_item(const SItem& d, bool owner, int qst, int8_t* qs_mem, float* qscale, int* qsum,
                                           float* qred) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int n4 = d.K / 4;
  const int kw = (d.tiles3 * 96 + d.tiles2 * 64) / 4;     // staged columns / 4 (pair tiles padded to 64 columns)
  const int three_k4 = d.tiles3 * 24;
  if (threadIdx.x < 8) qsum[threadIdx.x] = 0;
  if (d.x && kw <= XREG * THREADS) {
    // Alg. 1 Phase 1 / Alg. 2 "Tbl-quantization", one round trip per token: s = 127 / max(amax, 1e-5),
    // q = clamp(rint(x * s))
    const int nrow = (kw + THREADS - 1) / THREADS;
    for (int tok = 0; tok < d.T; ++tok) {
      const float4* x4 = reinterpret_cast<const float4*>(d.x + (int64_t)tok * d.K);
      float4 xv[XREG];
#pragma unroll
      for (int r = 0; r < XREG; ++r) {
        const int i = threadIdx.x + r * THREADS;
        xv[r] = (r < nrow && i < n4) ? __ldcg(x4 + i) : make_float4(0.f, 0.f, 0.f, 0.f);
      }
      float m = 0.0f;
#pragma unroll
      for (int r = 0; r < XREG; ++r)
        if (r < nrow) m = fmaxf(m, absmax4(xv[r]));
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
      if (tok > 0) __syncthreads();
      if (lane == 0) qred[warp] = m;
      __syncthreads();
      float amax = 0.0f;
#pragma unroll
      for (int w2 = 0; w2 < CW; ++w2) amax = fmaxf(amax, qred[w2]);
      const float amax_c = fmaxf(amax, 1e-5f);
      const float sq = __fdiv_rn(127.0f, amax_c);
      if (threadIdx.x == 0) {
        const float inv = __fdiv_rn(amax_c, 127.0f);
        qscale[tok] = inv;
        if (owner) d.act_scale[tok] = inv;
      }
      int s = 0;
#pragma unroll
      for (int r = 0; r < XREG; ++r) {
        const int i = threadIdx.x + r * THREADS;
        if (r < nrow && i < kw) {
          const int word = quant4_packed(xv[r], sq);  // columns beyond K came in as zeros
          store_codes(qs_mem + tok * qst, i, word, three_k4, d.tiles3);
          s = __dp4a(word, 0x01010101, s);
          if (owner && i < n4) reinterpret_cast<int*>(d.q + (int64_t)tok * d.K)[i] = word;
        }
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
      if (lane == 0) atomicAdd(qsum + tok, s);
    }
  } else if (d.x) {
    for (int tok = 0; tok < d.T; ++tok) {
      const float4* x4 = reinterpret_cast<const float4*>(d.x + (int64_t)tok * d.K);
      float m = 0.0f;
      for (int i = threadIdx.x; i < n4; i += THREADS) m = fmaxf(m, absmax4(__ldcg(x4 + i)));
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
      if (lane == 0) qred[tok * CW + warp] = m;
    }
    __syncthreads();
    if (threadIdx.x < d.T) {
      float m = 0.0f;
      for (int w2 = 0; w2 < CW; ++w2) m = fmaxf(m, qred[threadIdx.x * CW + w2]);
      const float inv = __fdiv_rn(fmaxf(m, 1e-5f), 127.0f);
      qscale[threadIdx.x] = inv;
      if (owner) d.act_scale[threadIdx.x] = inv;
    }
    __syncthreads();
    for (int tok = 0; tok < d.T; ++tok) {
      float m = 0.0f;
      for (int w2 = 0; w2 < CW; ++w2) m = fmaxf(m, qred[tok * CW + w2]);
      const float sq = __fdiv_rn(127.0f, fmaxf(m, 1e-5f));
      const float4* x4 = reinterpret_cast<const float4*>(d.x + (int64_t)tok * d.K);
      int s = 0;
      for (int i = threadIdx.x; i < kw; i += THREADS) {
        int word = 0;
        if (i < n4) {
          word = quant4_packed(__ldcg(x4 + i), sq);
          if (owner) reinterpret_cast<int*>(d.q + (int64_t)tok * d.K)[i] = word;
        }
        store_codes(qs_mem + tok * qst, i, word, three_k4, d.tiles3);
        s = __dp4a(word, 0x01010101, s);
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
      if (lane == 0) atomicAdd(qsum + tok, s);
    }
  } else {
    __syncthreads();  // qsum is zero before the first atomicAdd
    for (int tok = 0; tok < d.T; ++tok) {
      const int* qrow = reinterpret_cast<const int*>(d.q + (int64_t)tok * d.K);
      int s = 0;
      for (int i = threadIdx.x; i < kw; i += THREADS) {
        const int word = (i < n4) ? __ldcg(qrow + i) : 0;
        store_codes(qs_mem + tok * qst, i, word, three_k4, d.tiles3);
        s = __dp4a(word, 0x01010101, s);
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
      if (lane == 0) atomicAdd(qsum + tok, s);
    }
    if (threadIdx.x < d.T) qscale[threadIdx.x] = __ldcg(d.act_scale + threadIdx.x);
  }
}

template <int DEPTH, int NMAX>
__global__ void __launch_bounds__(THREADS, 1) gemv_tl2_scan_kernel(const __grid_constant__ SArgs<NMAX> a) {
  extern __shared__ __align__(128) uint8_t smem[];
  int* hdr = reinterpret_cast<int*>(smem);
  float* qscale = reinterpret_cast<float*>(smem + 64);
  int* qsum = reinterpret_cast<int*>(smem + 96);
  float* qred = reinterpret_cast<float*>(smem + 128);
  unsigned* tbl1 = reinterpret_cast<unsigned*>(smem + 1024);     // [256] index byte of two pairs -> four codes
  int* red = reinterpret_cast<int*>(smem + 2048);                // [CW][2][tmax][32] partial sums
  unsigned* tbl2 = reinterpret_cast<unsigned*>(smem + 2048 + CW * 2 * a.tmax * 32 * 4);   // [1024][32 lanes]
  int8_t* qs_mem = reinterpret_cast<int8_t*>(tbl2) + TBL2_BYTES;
  uint8_t* rings = reinterpret_cast<uint8_t*>(qs_mem) + a.code_bytes;

  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int S = a.S, G = CW / S, gi = warp / S, wk = warp % S;
  const int g = lane >> 2, t = lane & 3;

  if (threadIdx.x == 0) {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    auto locate = [&](int64_t w, int* item) -> int {
      int lo = 0, hi = a.n - 1;
      while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if ((int64_t)a.it[mid].first_w <= w) lo = mid; else hi = mid - 1;
      }
      *item = lo;
      const int per = a.it[lo].tiles3 + a.it[lo].tiles2;
      return a.it[lo].first_unit + (int)((w - a.it[lo].first_w) / per);
    };
    int ib, ie;
    const int jb = locate((int64_t)blockIdx.x * a.total_w / gridDim.x, &ib);
    const int je = locate((int64_t)(blockIdx.x + 1) * a.total_w / gridDim.x, &ie);
    hdr[0] = jb;
    hdr[1] = je;
    hdr[2] = ib;
    hdr[3] = (je > a.it[ie].first_unit) ? ie : ie - 1;
  }
  __syncthreads();
  const int jb = hdr[0], je = hdr[1], item0 = hdr[2], item1 = hdr[3];
  if (jb >= je) return;

  const uint64_t pol = policy_evict_first();
  const uint32_t ring = smem_u32(rings + (size_t)warp * DEPTH * SLOT);

  // ---------------- where the group's next block lies: a cursor over the items that runs one block ahead
  int n_item = item0, n_first = 0, n_end = 0, n_bb = 0, n_t3 = 0;
  const uint8_t* n_base = nullptr;
  auto n_load = [&](int i) {
    const SItem& d = a.it[i];
    n_bb = d.block_bytes;
    n_t3 = d.tiles3;
    n_first = d.first_unit;
    n_end = (i + 1 < a.n) ? a.it[i + 1].first_unit : a.total_units;
    n_base = d.packed + (int64_t)(wk * d.tiles3 / S) * SLOT + lane * 16;
  };
  // this warp's first triple tile of block `job` (job < je, asked for in ascending order)
  auto job_ptr = [&](int job) -> const uint8_t* {
    while (job >= n_end) n_load(++n_item);
    return n_base + (int64_t)(job - n_first) * n_bb;
  };
  auto prefetch = [&](uint32_t slot, const uint8_t* src, bool triple_tile) {
    cp16(slot + lane * 16, src, pol);
    if (triple_tile && lane < 8) cp16(slot + 512 + lane * 16, src + 512, pol);
  };
  n_load(item0);
  int cj = jb + gi, nloc = 0;
  const uint8_t* cur = (cj < je) ? job_ptr(cj) : nullptr;
  // Weights depend on nothing an earlier kernel writes: fill the ring before waiting for that kernel.  Every
  // warp's run of triple tiles is at least DEPTH tiles long (the host chooses S and DEPTH that way).
#pragma unroll
  for (int d = 0; d < DEPTH; ++d) {
    if (cur) prefetch(ring + d * SLOT, cur + d * SLOT, true);
    cp_commit();
  }

  // ---------------- the decode tables (they depend on nothing either)
  for (int e = warp; e < 1024; e += CW) {
    const int byte = e & 255;
    int c00, c01, c02, c10, c11, c12;
    triple_codes(byte & 15, (e >> 8) & 1, &c00, &c01, &c02);
    triple_codes(byte >> 4, (e >> 9) & 1, &c10, &c11, &c12);
    tbl2[e * 32 + lane] = (unsigned)(c00 | (c01 << 8) | (c02 << 16) | (c10 << 24) | (c11 << 2) | (c12 << 10));
  }
  if (threadIdx.x < 256) {
    const int lo = threadIdx.x & 15, hi = threadIdx.x >> 4;
    // pair code i -> (i/3 - 1, i%3 - 1); codes above 8 do not occur and decode to (0, 0)
    const int a0 = lo <= 8 ? lo / 3 : 1, a1 = lo <= 8 ? lo % 3 : 1, b0 = hi <= 8 ? hi / 3 : 1, b1 = hi <= 8 ? hi % 3 : 1;
    tbl1[threadIdx.x] = (unsigned)(a0 | (a1 << 8) | (b0 << 16) | (b1 << 24));
  }

  asm volatile("griddepcontrol.wait;" ::: "memory");

  // ---------------- consume
  const uint32_t tbl2_lane = smem_u32(tbl2) + lane * 4;
  const uint32_t tbl1_s = smem_u32(tbl1);
  int slot = 0;                      // ring slot consumed next
  const int tmax = a.tmax;
  for (int ci = item0; ci <= item1; ++ci) {
    const SItem& d = a.it[ci];
    const int T = d.T, tiles3 = d.tiles3, tiles2 = d.tiles2;
    const int qst = tiles3 * 128 + tiles2 * 64 + 16;
    const bool owner = jb <= d.first_unit;
    if (ci == item0 || !same_input(a.it[ci - 1], d)) {
      if (ci > item0) __syncthreads();  // everyone is done with the previous item's codes
      stage_item(d, owner, qst, qs_mem, qscale, qsum, qred);
      __syncthreads();                  // (also: the decode tables are complete)
    } else if (owner && d.x && d.q != a.it[ci - 1].q) {
      // same input as the previous item, but its own output buffers for the codes: quantise once more
      __syncthreads();
      stage_item(d, owner, qst, qs_mem, qscale, qsum, qred);
      __syncthreads();
    }
    const int lo3 = wk * tiles3 / S, hi3 = (wk + 1) * tiles3 / S, n3 = hi3 - lo3;
    const int n2 = (wk == S - 1) ? tiles2 : 0;
    const int iend = (ci + 1 < a.n) ? a.it[ci + 1].first_unit : a.total_units;
    const int cend = je < iend ? je : iend;
    const int first = d.first_unit, M = d.M, ldy = d.ldy;
    const unsigned has_tok = g < T ? 1u : 0u;
    const uint32_t q_row = smem_u32(qs_mem + min(g, T - 1) * qst);
    const uint32_t q3 = q_row + lo3 * 128 + t * 32;         // B registers of the warp's first triple tile
    const uint32_t q1 = q_row + tiles3 * 128 + t * 16;      // ... of the first pair tile
    const float w_scale = d.w_scale;
    float* const y = d.y;
    int32_t* const acc_out = d.acc_out;
    const int tail_off = (tiles3 - lo3) * SLOT;             // from the warp's first triple tile to the first pair tile

    for (; cj < cend; cj += G, ++nloc) {
      int C0[4][4], C1[4][4];
#pragma unroll
      for (int s = 0; s < 4; ++s)
#pragma unroll
        for (int i = 0; i < 4; ++i) C0[s][i] = C1[s][i] = 0;
      uint32_t qp = q3;
      int qr[8] = {0, 0, 0, 0, 0, 0, 0, 0};  // B registers; lanes beyond the batch keep these zeros

      // One triple tile: wait for the oldest slot, decode, MMA, refill the slot from `pf`.
      auto step3 = [&](const uint8_t* pf, bool do_pf, bool pf_triple) {
        cp_wait<DEPTH - 1>();
        __syncwarp();                          // the sign plane was copied by lanes 0..7
        const uint32_t sl = ring + slot * SLOT;
        unsigned iw[4], sg[4];
        lds128(sl + lane * 16, iw);            // index word t of rows g, g+8, g+16, g+24
        lds128(sl + 512 + g * 16, sg);         // their sign words
        asm volatile(
            "{\n\t.reg .pred p;\n\tsetp.ne.u32 p, %9, 0;\n\t"
            "@p ld.shared.v4.u32 {%0,%1,%2,%3}, [%8];\n\t"
            "@p ld.shared.v4.u32 {%4,%5,%6,%7}, [%8+16];\n\t}"
            : "+r"(qr[0]), "+r"(qr[1]), "+r"(qr[2]), "+r"(qr[3]), "+r"(qr[4]), "+r"(qr[5]), "+r"(qr[6]), "+r"(qr[7])
            : "r"(qp), "r"(has_tok));
        unsigned xa[4], xb[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const unsigned tw = (sg[u] >> (2 * t)) & 0x03030303u;     // sign pair of index byte j in byte j
          const unsigned e0 = lds32(tbl2_lane + prmt(iw[u], tw, 0xCC40u) * 128);
          const unsigned e1 = lds32(tbl2_lane + prmt(iw[u], tw, 0xDD51u) * 128);
          const unsigned e2 = lds32(tbl2_lane + prmt(iw[u], tw, 0xEE62u) * 128);
          const unsigned e3 = lds32(tbl2_lane + prmt(iw[u], tw, 0xFF73u) * 128);
          xa[u] = e0 + 16u * e1;
          xb[u] = e2 + 16u * e3;
        }
#pragma unroll
        for (int s = 0; s < 4; ++s) {
          const unsigned m = 0x03030303u << (2 * s);
          mma_u8s8(C0[s], xa[0] & m, xa[1] & m, xb[0] & m, xb[1] & m, qr[2 * s], qr[2 * s + 1]);
          mma_u8s8(C1[s], xa[2] & m, xa[3] & m, xb[2] & m, xb[3] & m, qr[2 * s], qr[2 * s + 1]);
        }
        qp += 128;
        __syncwarp();                          // every lane has read the slot's sign plane
        if (do_pf) prefetch(sl, pf, pf_triple);
        cp_commit();
        slot = (slot + 1 == DEPTH) ? 0 : slot + 1;
      };
      // One pair tile (the K tail): index byte -> four codes; X = E0 | E1<<2 | E2<<4 | E3<<6 is a full I2_S word,
      // used as the first half of the MMA's K only.
      auto step1 = [&](uint32_t qaddr, const uint8_t* pf, bool do_pf) {
        cp_wait<DEPTH - 1>();
        __syncwarp();
        const uint32_t sl = ring + slot * SLOT;
        unsigned iw[4];
        lds128(sl + lane * 16, iw);
        int q1r[4] = {0, 0, 0, 0};
        asm volatile(
            "{\n\t.reg .pred p;\n\tsetp.ne.u32 p, %5, 0;\n\t"
            "@p ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];\n\t}"
            : "+r"(q1r[0]), "+r"(q1r[1]), "+r"(q1r[2]), "+r"(q1r[3])
            : "r"(qaddr), "r"(has_tok));
        unsigned x[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const unsigned e0 = lds32(tbl1_s + ((iw[u] << 2) & 0x3FCu));
          const unsigned e1 = lds32(tbl1_s + ((iw[u] >> 6) & 0x3FCu));
          const unsigned e2 = lds32(tbl1_s + ((iw[u] >> 14) & 0x3FCu));
          const unsigned e3 = lds32(tbl1_s + ((iw[u] >> 22) & 0x3FCu));
          x[u] = e0 | (e1 << 2) | (e2 << 4) | (e3 << 6);
        }
#pragma unroll
        for (int s = 0; s < 4; ++s) {
          const unsigned m = 0x03030303u << (2 * s);
          mma_u8s8(C0[s], x[0] & m, x[1] & m, 0u, 0u, q1r[s], 0);
          mma_u8s8(C1[s], x[2] & m, x[3] & m, 0u, 0u, q1r[s], 0);
        }
        __syncwarp();
        if (do_pf) prefetch(sl, pf, true);     // what follows a pair tile DEPTH places on is a triple tile
        cp_commit();
        slot = (slot + 1 == DEPTH) ? 0 : slot + 1;
      };

      // The warp's stream: n3 triple tiles of this block, n2 pair tiles (last warp of the group), then the next
      // block's triple tiles.  Tile i is followed, DEPTH places on, by tile i + DEPTH of that stream.
      const int nj = cj + G;
      const bool more = nj < je;
      const uint8_t* const nxt = more ? job_ptr(nj) : cur;
      const uint8_t* pf = cur + DEPTH * SLOT;
#pragma unroll 1
      for (int left = n3 - DEPTH; left > 0; --left, pf += SLOT) step3(pf, true, true);
      // d-th tile after this block's triple tiles: one of its pair tiles, or a triple tile of the next block
      const uint8_t* const tail = cur + tail_off;
#pragma unroll 1
      for (int dd = 0; dd < DEPTH; ++dd) {
        const bool in_tail = dd < n2;
        step3(in_tail ? tail + dd * 512 : nxt + (dd - n2) * SLOT, in_tail || more, !in_tail);
      }
#pragma unroll 1
      for (int j2 = 0; j2 < n2; ++j2) step1(q1 + j2 * 64, nxt + (DEPTH - n2 + j2) * SLOT, more);
      cur = nxt;

      // fragments: c[0] = (row g, token 2t), c[1] = (row g, token 2t+1), c[2], c[3] = the same for row g+8
      int* mine = red + ((warp * 2 + (nloc & 1)) * tmax) * 32;
#pragma unroll
      for (int u = 0; u < 2; ++u) {
        int c[4];
#pragma unroll
        for (int i = 0; i < 4; ++i)
          c[i] = u == 0 ? C0[0][i] + (C0[1][i] >> 2) + (C0[2][i] >> 4) + (C0[3][i] >> 6)
                        : C1[0][i] + (C1[1][i] >> 2) + (C1[2][i] >> 4) + (C1[3][i] >> 6);
        if (2 * t < T) {
          mine[(2 * t) * 32 + 16 * u + g] = c[0];
          mine[(2 * t) * 32 + 16 * u + g + 8] = c[2];
        }
        if (2 * t + 1 < T) {
          mine[(2 * t + 1) * 32 + 16 * u + g] = c[1];
          mine[(2 * t + 1) * 32 + 16 * u + g + 8] = c[3];
        }
      }
      if (S > 1) group_barrier(1 + gi, S * 32);
      else __syncwarp();
      if (wk == (nloc & (S - 1))) {
        // this block's turn to be finished by this warp: add the group's partials, rescale, store 32 rows
        const int row0 = (cj - first) * 32;
        const int* grp = red + (((gi * S) * 2 + (nloc & 1)) * tmax) * 32;
        for (int idx = lane; idx < T * 32; idx += 32) {
          int v = 0;
          for (int w2 = 0; w2 < S; ++w2) v += grp[w2 * 2 * tmax * 32 + idx];
          const int tok = idx >> 5, row = row0 + (idx & 31);
          v -= qsum[tok];
          if (row < M) {
            y[(int64_t)tok * ldy + row] = __fmul_rn((float)v, __fmul_rn(qscale[tok], w_scale));
            if (acc_out) acc_out[(int64_t)tok * ldy + row] = v;
          }
        }
      }
    }
  }
  cp_wait<0>();
  __syncthreads();   // no warp leaves the CTA before the others are done
}

int env_int_once(const char* name, int dflt) {
  const char* v = getenv(name);
  return (v && *v) ? atoi(v) : dflt;
}
int depth_cap() {
  static const int d = [] {
    const int v = env_int_once("BITNET_TL2_DEPTH", 8);
    return (v >= 3 && v <= 8 && v != 7) ? v : 8;
  }();
  return d;
}
int forced_s() {
  static const int s = [] {
    const int v = env_int_once("BITNET_TL2_S", 0);
    return (v == 1 || v == 2 || v == 4 || v == 8) ? v : 0;
  }();
  return s;
}

size_t code_bytes_of(int T, int tiles3, int tiles2) {
  return ((size_t)T * (size_t)(tiles3 * 128 + tiles2 * 64 + 16) + 127) & ~(size_t)127;
}
size_t smem_of(int tmax, size_t code_bytes, int depth) {
  return 2048 + (size_t)CW * 2 * tmax * 32 * 4 + TBL2_BYTES + code_bytes + (size_t)CW * depth * SLOT;
}

struct Shape {
  int S, depth;
};
// S and ring depth for a launch whose shortest rows have `t3` triple tiles: every warp's run of triple tiles is at
// least as long as its ring; the ring is made shallower until everything fits one SM's shared memory.
bool launch_shape(int t3, int tmax, size_t code, int64_t units, Shape* out) {
  // Warps per 32-row block: one when the launch has enough blocks to keep the 16 warps of every SM busy with
  // blocks of their own (no partial sums to join: 3.4 TB/s against 3.1 with four on the 100B sweep), more when
  // it has few.
  int S = forced_s();
  if (!S) {
    S = 1;
    while (S < 4 && units * S < (int64_t)CW * dev_info().sm_count * 4) S <<= 1;
  }
  while (S > 1 && t3 / S < 8) S >>= 1;
  const int nw = t3 / S;
  if (nw < 3) return false;
  const size_t cap = (size_t)dev_info().max_smem_optin;
  int depth = depth_cap();
  auto lower = [](int d) { return d == 8 ? 6 : d - 1; };
  while (depth > 3 && (depth > nw || smem_of(tmax, code, depth) > cap)) depth = lower(depth);
  if (depth > nw || smem_of(tmax, code, depth) > cap) return false;
  *out = Shape{S, depth};
  return true;
}

template <int DEPTH, int NMAX>
int launch_scan(const SArgs<NMAX>& a, int grid, size_t smem, cudaStream_t st) {
  static bool attr_set[64] = {false};
  int dev = 0;
  cudaGetDevice(&dev);
  if (!attr_set[dev & 63]) {
    cudaError_t e = cudaFuncSetAttribute(gemv_tl2_scan_kernel<DEPTH, NMAX>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         dev_info().max_smem_optin);
    if (e != cudaSuccess) return note_cuda_error(e);
    attr_set[dev & 63] = true;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)grid);
  cfg.blockDim = dim3(THREADS);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = early_start_enabled() ? 1 : 0;
  cudaError_t e = cudaLaunchKernelEx(&cfg, gemv_tl2_scan_kernel<DEPTH, NMAX>, a);
  return e == cudaSuccess ? BITNET_OK : note_cuda_error(e);
}

template <int NMAX>
int launch_depth(const SArgs<NMAX>& a, int depth, int grid, size_t smem, cudaStream_t st) {
  switch (depth) {
    case 3: return launch_scan<3, NMAX>(a, grid, smem, st);
    case 4: return launch_scan<4, NMAX>(a, grid, smem, st);
    case 5: return launch_scan<5, NMAX>(a, grid, smem, st);
    case 6: return launch_scan<6, NMAX>(a, grid, smem, st);
    case 8: return launch_scan<8, NMAX>(a, grid, smem, st);
    default: return BITNET_ERR_UNSUPPORTED_SHAPE;
  }
}

template <int NMAX>
int launch_run(const Tl2Linear* items, int n, Shape shape, cudaStream_t st) {
  static thread_local SArgs<NMAX> a;
  a.n = n;
  a.S = shape.S;
  a.tmax = 1;
  size_t code = 0;
  int64_t units = 0, w = 0;
  for (int i = 0; i < n; ++i) {
    const Tl2Linear& s = items[i];
    SItem& d = a.it[i];
    d.packed = s.packed;
    d.x = s.x;
    d.q = s.q;
    d.act_scale = s.act_scale;
    d.y = s.y;
    d.acc_out = s.acc_out;
    d.w_scale = s.w_scale;
    d.M = (int)s.M;
    d.K = (int)s.K;
    d.T = s.T;
    d.tiles3 = (int)s.g.tiles3;
    d.tiles2 = (int)s.g.tiles2;
    d.block_bytes = (int)s.g.block_bytes;
    d.first_unit = (int)units;
    d.first_w = (int)w;
    d.ldy = (int)(s.ldy ? s.ldy : s.M);
    units += s.M / 32;
    w += (s.M / 32) * (s.g.tiles3 + s.g.tiles2);
    if (s.T > a.tmax) a.tmax = s.T;
    const size_t cb = code_bytes_of(s.T, d.tiles3, d.tiles2);
    if (cb > code) code = cb;
  }
  a.total_units = (int)units;
  a.total_w = (int)w;
  a.code_bytes = (int)code;
  a.r0 = a.r1 = 0;
  const size_t smem = smem_of(a.tmax, code, shape.depth);
  if (smem > (size_t)dev_info().max_smem_optin) return BITNET_ERR_UNSUPPORTED_SHAPE;
  const int G = CW / a.S;
  int grid = dev_info().sm_count;
  if ((int64_t)grid * G > units) grid = (int)ceil_div(units, G);
  log_launch("gemv_tl2_scan_kernel items=%d blocks=%lld tiles=%lld grid=%d warps/block=%d ring=%d tmax=%d smem=%zu", n,
             (long long)units, (long long)w, grid, a.S, shape.depth, a.tmax, smem);
  return launch_depth<NMAX>(a, shape.depth, grid, smem, st);
}

}  // namespace

bool gemv_tl2_scan_item_supported(int T, int64_t M, int64_t K, const TlGeom& g) {
  if (T < 1 || T > 8 || M < 32 || (M % 32) != 0 || K < 4 || (K % 4) != 0 || M > 0x7fffffff || g.block_bytes > 0x7fffffff)
    return false;
  if (g.tiles2 > 2 || g.three_k > 0x3fffffff) return false;    // more pair tiles than a ring refill pattern assumes
  Shape sh;
  return launch_shape((int)g.tiles3, T, code_bytes_of(T, (int)g.tiles3, (int)g.tiles2), M / 32, &sh);
}

// Launches the scan kernel over `n` supported TL2 items: as few launches as the argument block (NLARGE items,
// 2^30 tiles) and shared memory allow.
int launch_gemv_tl2_scan(const Tl2Linear* items, int64_t n, cudaStream_t st) {
  int64_t i = 0;
  while (i < n) {
    int64_t j = i, w = 0;
    int t3_min = 1 << 30, tmax = 1;
    size_t code = 0;
    Shape sh{1, 3};
    int64_t units = 0;
    for (int64_t k = i; k < n && k - i < NLARGE; ++k) units += items[k].M / 32;   // (an estimate when the run is cut short)
    while (j < n && j - i < NLARGE) {
      const TlGeom& g = items[j].g;
      const int64_t add = (items[j].M / 32) * (g.tiles3 + g.tiles2);
      const size_t cb = code_bytes_of(items[j].T, (int)g.tiles3, (int)g.tiles2);
      const int tm = items[j].T > tmax ? items[j].T : tmax;
      const size_t cm = cb > code ? cb : code;
      const int t3 = (int)g.tiles3 < t3_min ? (int)g.tiles3 : t3_min;
      Shape sj;
      const bool fits = launch_shape(t3, tm, cm, units, &sj);
      if (!fits && j == i) return BITNET_ERR_UNSUPPORTED_SHAPE;
      if (!fits || (j > i && w + add > (1ll << 30))) break;
      w += add;
      tmax = tm;
      code = cm;
      t3_min = t3;
      sh = sj;
      ++j;
    }
    const int cnt = (int)(j - i);
    const int rc = cnt <= NSMALL ? launch_run<NSMALL>(items + i, cnt, sh, st) : launch_run<NLARGE>(items + i, cnt, sh, st);
    if (rc != BITNET_OK) return rc;
    i = j;
  }
  return BITNET_OK;
}

}  // namespace bitnet
