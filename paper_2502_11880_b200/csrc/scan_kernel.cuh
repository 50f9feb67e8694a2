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
// six weights as 2-bit codes w+1: byte b, bit pair s of the 32-bit entry holds (triple 0: w0,w1,w2 -> s=0, b=0,1,2;
// triple 1: w0 -> s=0, b=3; w1,w2 -> s=1, b=0,1).  entry & 0x03030303 is an A register of mma.sync.m16n8k32
// (u8 x s8) with four codes; the s=1 pairs of two entries are joined by one byte permute into an A register with
// four codes scaled by 4.  Two accumulators carry the scales 1 and 4, and sum(code*q) - sum(q) = sum(w*q).
// Every lane keeps a private copy of the table (entry e of lane l at word 32e + l: bank l whatever e is), so the
// 32 lookups of a warp never conflict: 128 KB.
//
// Tile = 32 rows x 32 triples (640 B).  Lane (g, t) owns index word t of the rows g, g+8, g+16, g+24: one 16-byte
// piece of the index plane (the tile layout interleaves exactly these four rows), which is also the piece the lane
// copied with cp.async; the four rows' sign words are the 16-byte piece 512 + 16g.  (signs >> 2t) & 0x03030303
// puts the sign pair of index byte j into byte j, and one byte permute joins index byte and sign pair into the
// table index.  Rows g, g+8 are the A rows of the MMAs of the block's upper half, g+16, g+24 of its lower half:
// three MMAs per half and tile (index bytes 0,1 at scale 1; bytes 2,3 at scale 1; the s=1 pairs of all four at 4).
//
// Activations are staged in the order the decoded words want them: per tile and lane-quarter t, 24 bytes = the
// B registers of those three MMAs, no padding.  The pair-coded tail columns of a row (TL1 tiles, Table 4 / Alg. 3;
// at most two tiles) go through a 256-entry table (index byte -> four codes): two MMAs per half.
//
// The same kernel serves the element-wise tables beyond ternary of App. A in their g = 2 form (F = 1): weights of
// cardinality C stored as pair indices 0 .. C^2-1 of four bits (C <= 4) or five (C = 5: the fifth bit in the plane
// where TL2 keeps its signs), tiles of 32 rows x 32 pairs.  There an index byte plus its two fifth bits selects a
// table entry that IS the A register -- four weights as bytes w + C/2 -- so a tile is 16 lookups and four MMAs per
// lane with no masking, against activations staged in their natural order; sum(code*q) - (C/2) sum(q) = sum(w*q).
//
// For C = 4 the pair index is the two 2-bit codes side by side (at a power of two, bit-wise and element-wise storage
// coincide: Table 3), so no table is needed (F = 2): one shift and four masks per index word give the A registers of
// two MMAs at the scales 1 and 16, against activations staged in the matching byte order.
// For C = 3 (TL1: Table 4's code of a pair is 3 a + b with a, b the weights + 1) the index is taken apart by byte-wise
// arithmetic (F = 3): the index nibbles of a word spread over two words of bytes x; bits 5, 6 of 11 x are a = x / 3
// (x <= 8, and 11 x stays inside its byte), so 32 a = (11 x) & 0x60 and 32 b = 32 x - 3 (32 a): four A registers of
// byte codes per index word at the scale 32, more than half of the instructions on the multiply-add pipe.
//
// This header is the whole kernel and its launcher as templates over F; gemv_tl2_scan.cu and gemv_elut_scan.cu
// instantiate them.
#pragma once
#include <cstdlib>
#include <cstring>

#include "common.cuh"
#include "device_utils.cuh"

namespace bitnet {
namespace scan {

constexpr int CW = 16;  // warps
constexpr int THREADS = CW * 32;
constexpr int XREG = 16;
constexpr int NSMALL = 42, NLARGE = 340;   // items per launch: argument blocks of 4 KB / 32 KB
constexpr int SLOT = 640;                  // ring slot = one tile
constexpr int TBL2_BYTES = 1024 * 32 * 4;

// Bytes between the staged rows of two tokens: the columns of the largest part (+ a pair-coded tail) rounded up to
// 96 (triple tiles) or 64 (pair tiles) modulo 128, so that the activation loads of a quarter- or half-warp -- the
// lane quarters of one token 24 or 16 bytes apart, the tokens one row apart -- cover the 32 banks exactly once.
__host__ __device__ inline int staged_stride(int cols, int big, int tiles2) {
  const int raw = big * cols + tiles2 * 64 + 16, want = cols == 96 ? 96 : 64;
  return ((raw - want + 127) / 128) * 128 + want;
}

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
  int nparts;          // the triple tiles of a row are walked in this many parts (the pair tiles belong to the last)
  int pad;
};
static_assert(sizeof(SItem) == 96, "argument block layout");

template <int NMAX>
struct SArgs {
  int n, S, tmax, code_bytes;
  int total_units, total_w;
  int card;        // F = 1: the weights' cardinality C
  int tile_bytes;  // bytes of a tile in the blob: 640, or 512 when the pair indices have no fifth-bit plane
  SItem it[NMAX];
};
static_assert(sizeof(SArgs<NSMALL>) <= 4096 && sizeof(SArgs<NLARGE>) <= 32764, "kernel parameter limits");

__device__ __forceinline__ bool same_input(const SItem& p, const SItem& d) {
  return p.nparts == 1 && d.nparts == 1 && p.K == d.K && p.T == d.T && p.tiles3 == d.tiles3 &&
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
__device__ __forceinline__ unsigned mad_u32(unsigned a, unsigned b, unsigned c) {
  unsigned d;
  asm("mad.lo.u32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
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

// The staged columns of one part of an item: the triple tiles [t0, t1) and, if `tail`, the pair tiles.
struct Part {
  int t0, t1;      // triple tiles
  int tiles3;      // of the whole row (where the pair-coded columns begin: column 96 * tiles3)
  int tiles2;      // pair tiles staged with this part (0 unless it is the last part)
};

// Stores the four codes of columns 4i..4i+3 of a token row into the staged (permuted) order, if the part holds them.
//   triple-coded columns: tile = k / 96, quarter t = (k % 96) / 24; the quarter's 24 bytes are six words, the B
//   registers of its three MMAs: columns o = 0..23 of the quarter go to
//     word 0 (o 0..3), word 1 (o 6..9), word 2 (o 12..15), word 3 (o 18..21)      -- the scale-1 codes,
//     word 4 (o 4, 5, 16, 17), word 5 (o 10, 11, 22, 23)                          -- the scale-4 pairs;
//   pair-coded columns follow the part's triple tiles in natural order, 64 bytes per tile.
// Returns true if the word was staged.
template <int F>
__device__ __forceinline__ bool store_codes(int8_t* row, int i, int word, const Part& pt) {
  const int k = 4 * i;
  if (F == 1) {      // pair tiles: natural order, 64 bytes per tile
    const int tile = k >> 6;
    if (tile < pt.t0 || tile >= pt.t1) return false;
    *reinterpret_cast<int*>(row + (k - 64 * pt.t0)) = word;
    return true;
  }
  if (F == 2) {
    // pair tiles decoded by masks: the 16 columns of lane quarter t are four words, word s holding the columns
    // 16t + 4j + p(s), j = 0..3, p = (1, 0, 3, 2): bit pair s of index byte j is the code of exactly that column
    const int tile = k >> 6;
    if (tile < pt.t0 || tile >= pt.t1) return false;
    const int c = k & 63, j = (c >> 2) & 3;
    int8_t* blk = row + (tile - pt.t0) * 64 + (c & 48);
    blk[4 + j] = (int8_t)word;
    blk[j] = (int8_t)(word >> 8);
    blk[12 + j] = (int8_t)(word >> 16);
    blk[8 + j] = (int8_t)(word >> 24);
    return true;
  }
  if (F == 3) {
    // pair tiles decoded by arithmetic: word d of a lane quarter's 16 bytes holds the columns 16t + 4j + d, j = 0..3
    const int tile = k >> 6;
    if (tile < pt.t0 || tile >= pt.t1) return false;
    const int c = k & 63, j = (c >> 2) & 3;
    int8_t* blk = row + (tile - pt.t0) * 64 + (c & 48);
    blk[j] = (int8_t)word;
    blk[4 + j] = (int8_t)(word >> 8);
    blk[8 + j] = (int8_t)(word >> 16);
    blk[12 + j] = (int8_t)(word >> 24);
    return true;
  }
  if (k < 96 * pt.tiles3) {
    const int tile = k / 96, c = k - 96 * tile;
    if (tile < pt.t0 || tile >= pt.t1) return false;
    const int t = c / 24, o = c - 24 * t;                     // o in {0, 4, 8, 12, 16, 20}
    int8_t* blk = row + (tile - pt.t0) * 96 + t * 24;
    const short lo = (short)(word & 0xFFFF), hi = (short)((unsigned)word >> 16);
    switch (o) {
      case 0: *reinterpret_cast<int*>(blk) = word; break;
      case 4: *reinterpret_cast<short*>(blk + 16) = lo; *reinterpret_cast<short*>(blk + 4) = hi; break;
      case 8: *reinterpret_cast<short*>(blk + 6) = lo; *reinterpret_cast<short*>(blk + 20) = hi; break;
      case 12: *reinterpret_cast<int*>(blk + 8) = word; break;
      case 16: *reinterpret_cast<short*>(blk + 18) = lo; *reinterpret_cast<short*>(blk + 12) = hi; break;
      default: *reinterpret_cast<short*>(blk + 14) = lo; *reinterpret_cast<short*>(blk + 22) = hi; break;
    }
    return true;
  }
  const int j = i - 24 * pt.tiles3;
  if (j >= 16 * pt.tiles2) return false;
  *reinterpret_cast<int*>(row + (pt.t1 - pt.t0) * 96 + 4 * j) = word;
  return true;
}

// Stages the activation codes of one part of the item (T rows, qst bytes apart) and, per token, the scale and the
// sum of the staged codes.  `first` = the item's first part: the row maximum is taken (Alg. 2 "Tbl-quantization" =
// Alg. 1 Phase 1) and, in the CTA that owns the item, codes and scales of the WHOLE row go to the caller; later parts
// reuse the multiplier kept in qmul.  Called by all threads; contains barriers.
template <int F>
__device__ __forceinline__ void stage_item(const SItem& d, bool owner, bool first, const Part& pt, int qst, int8_t* qs_mem,
                                           float* qscale, float* qmul, int* qsum, float* qred) {
  constexpr int W4 = F ? 16 : 24;                           // 4-column words per tile
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int n4 = d.K / 4;
  const int kw = d.tiles3 * W4 + d.tiles2 * 16;             // columns of the row / 4, the last tile padded
  if (threadIdx.x < 8) qsum[threadIdx.x] = 0;
  if (d.x && first && kw <= XREG * THREADS) {
    // one round trip per token: s = 127 / max(amax, 1e-5), q = clamp(rint(x * s)); the row stays in registers
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
        qmul[tok] = sq;
        if (owner) d.act_scale[tok] = inv;
      }
      int s = 0;
#pragma unroll
      for (int r = 0; r < XREG; ++r) {
        const int i = threadIdx.x + r * THREADS;
        if (r < nrow && i < kw) {
          const int word = quant4_packed(xv[r], sq);  // columns beyond K came in as zeros
          if (store_codes<F>(qs_mem + tok * qst, i, word, pt)) s = __dp4a(word, 0x01010101, s);
          if (owner && i < n4) reinterpret_cast<int*>(d.q + (int64_t)tok * d.K)[i] = word;
        }
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
      if (lane == 0) atomicAdd(qsum + tok, s);
    }
  } else if (d.x) {
    if (first) {
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
        const float amax_c = fmaxf(m, 1e-5f);
        const float inv = __fdiv_rn(amax_c, 127.0f);
        qscale[threadIdx.x] = inv;
        qmul[threadIdx.x] = __fdiv_rn(127.0f, amax_c);
        if (owner) d.act_scale[threadIdx.x] = inv;
      }
    }
    __syncthreads();
    // the part's columns (in the owning CTA's first part: every column, for the caller's copy of the codes)
    const bool all = owner && first;
    const int lo = all ? 0 : W4 * pt.t0;
    const int hi = all ? kw : (pt.tiles2 ? kw : W4 * pt.t1);
    for (int tok = 0; tok < d.T; ++tok) {
      const float sq = qmul[tok];
      const float4* x4 = reinterpret_cast<const float4*>(d.x + (int64_t)tok * d.K);
      int s = 0;
      for (int i = lo + threadIdx.x; i < hi; i += THREADS) {
        int word = 0;
        if (i < n4) {
          word = quant4_packed(__ldcg(x4 + i), sq);
          if (all) reinterpret_cast<int*>(d.q + (int64_t)tok * d.K)[i] = word;
        }
        if (store_codes<F>(qs_mem + tok * qst, i, word, pt)) s = __dp4a(word, 0x01010101, s);
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
      if (lane == 0) atomicAdd(qsum + tok, s);
    }
  } else {
    __syncthreads();  // qsum is zero before the first atomicAdd
    const int lo = W4 * pt.t0, hi = pt.tiles2 ? kw : W4 * pt.t1;
    for (int tok = 0; tok < d.T; ++tok) {
      const int* qrow = reinterpret_cast<const int*>(d.q + (int64_t)tok * d.K);
      int s = 0;
      for (int i = lo + threadIdx.x; i < hi; i += THREADS) {
        const int word = (i < n4) ? __ldcg(qrow + i) : 0;
        if (store_codes<F>(qs_mem + tok * qst, i, word, pt)) s = __dp4a(word, 0x01010101, s);
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
      if (lane == 0) atomicAdd(qsum + tok, s);
    }
    if (threadIdx.x < d.T) qscale[threadIdx.x] = __ldcg(d.act_scale + threadIdx.x);
  }
}

template <int DEPTH, int NMAX, int F>
__global__ void __launch_bounds__(THREADS, 1) gemv_tl2_scan_kernel(const __grid_constant__ SArgs<NMAX> a) {
  constexpr int COLS = F ? 64 : 96;             // columns of a tile
  const int TB = F ? a.tile_bytes : SLOT;       // bytes from a tile to the next in the blob
  const bool hb = !F || a.tile_bytes == SLOT;   // the tile has a second plane (signs / fifth index bits)
  extern __shared__ __align__(128) uint8_t smem[];
  int* hdr = reinterpret_cast<int*>(smem);
  float* qscale = reinterpret_cast<float*>(smem + 64);
  int* qsum = reinterpret_cast<int*>(smem + 96);
  float* qred = reinterpret_cast<float*>(smem + 128);
  float* qmul = reinterpret_cast<float*>(smem + 640);            // [8] 127 / amax per token
  unsigned* tbl1 = reinterpret_cast<unsigned*>(smem + 1024);     // [256] index byte of two pairs -> four codes
  // partial sums [CW][RD][tmax][32]: two buffers per warp, so that a warp may start its next block while its group
  // still adds up the last one; one (bit 8 of a.S) when every warp finishes its own blocks
  const int RD = (a.S & 0x100) ? 1 : 2;
  int* red = reinterpret_cast<int*>(smem + 2048);
  unsigned* tbl2 = reinterpret_cast<unsigned*>(smem + 2048 + CW * RD * a.tmax * 32 * 4);   // [1024][32 lanes]
  int8_t* qs_mem = reinterpret_cast<int8_t*>(tbl2) + (F >= 2 ? 0 : TBL2_BYTES);   // (the mask and arithmetic modes have no table)
  uint8_t* rings = reinterpret_cast<uint8_t*>(qs_mem) + a.code_bytes;

  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int S = a.S & 0xff, G = CW / S, gi = warp / S, wk = warp % S;
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

  // ---------------- the group's sequence of jobs: (item, part, 32-row block).  Within the CTA's range, item i
  // contributes the blocks [max(jb, first_i), min(je, end_i)); the group takes every G-th of them starting at its
  // own index, once per part of the item's triple tiles.
  auto item_end = [&](int i) { return (i + 1 < a.n) ? a.it[i + 1].first_unit : a.total_units; };
  auto range_lo = [&](int i) { const int f = a.it[i].first_unit; return (f > jb ? f : jb) + gi; };
  auto range_hi = [&](int i) { const int e = item_end(i); return e < je ? e : je; };
  // this warp's first triple tile of (item i, part p, block job)
  auto job_ptr = [&](int i, int p, int job) -> const uint8_t* {
    const SItem& d = a.it[i];
    const int t0 = p * d.tiles3 / d.nparts, npt = (p + 1) * d.tiles3 / d.nparts - t0;
    return d.packed + (int64_t)(job - d.first_unit) * d.block_bytes + (int64_t)(t0 + wk * npt / S) * TB + lane * 16;
  };
  auto next_job = [&](int& i, int& p, int& job) -> bool {
    if (job + G < range_hi(i)) {
      job += G;
      return true;
    }
    if (p + 1 < a.it[i].nparts) {
      ++p;
      job = range_lo(i);
      return true;
    }
    for (++i; i <= item1; ++i)
      if (range_lo(i) < range_hi(i)) {
        p = 0;
        job = range_lo(i);
        return true;
      }
    return false;
  };
  auto prefetch = [&](uint32_t slot, const uint8_t* src, bool triple_tile) {
    cp16(slot + lane * 16, src, pol);
    if (triple_tile && hb && lane < 8) cp16(slot + 512 + lane * 16, src + 512, pol);
  };
  int ni = item0 - 1, np = 0, nj = 0;
  bool more = false;
  for (int i = item0; i <= item1 && !more; ++i)
    if (range_lo(i) < range_hi(i)) {
      ni = i;
      np = 0;
      nj = range_lo(i);
      more = true;
    }
  const uint8_t* cur = more ? job_ptr(ni, np, nj) : nullptr;
  // Weights depend on nothing an earlier kernel writes: fill the ring before waiting for that kernel.  Every
  // warp's run of triple tiles in every part is at least DEPTH tiles long (the host chooses S and DEPTH that way).
#pragma unroll
  for (int d = 0; d < DEPTH; ++d) {
    if (cur) prefetch(ring + d * SLOT, cur + d * TB, true);
    cp_commit();
  }

  // ---------------- the decode tables (they depend on nothing either)
  for (int e = warp; e < (F >= 2 ? 0 : 1024); e += CW) {
    const int byte = e & 255;
    if (F == 1) {
      // pair index i < C^2 -> the weights (i / C, i % C) + lo as codes i / C, i % C; an index that does not occur
      // decodes to two zero weights (code C/2)
      const int C = a.card, z = C / 2;
      const int ia = (byte & 15) | (((e >> 8) & 1) << 4), ib = (byte >> 4) | (((e >> 9) & 1) << 4);
      const int a0 = ia < C * C ? ia / C : z, a1 = ia < C * C ? ia % C : z;
      const int b0 = ib < C * C ? ib / C : z, b1 = ib < C * C ? ib % C : z;
      tbl2[e * 32 + lane] = (unsigned)(a0 | (a1 << 8) | (b0 << 16) | (b1 << 24));
    } else {
      int c00, c01, c02, c10, c11, c12;
      triple_codes(byte & 15, (e >> 8) & 1, &c00, &c01, &c02);
      triple_codes(byte >> 4, (e >> 9) & 1, &c10, &c11, &c12);
      tbl2[e * 32 + lane] = (unsigned)(c00 | (c01 << 8) | (c02 << 16) | (c10 << 24) | (c11 << 2) | (c12 << 10));
    }
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
  int nloc = 0;
  const int tmax = a.tmax;
  bool staged_any = false;
  for (int ci = item0; ci <= item1; ++ci) {
    const SItem& d = a.it[ci];
    const int T = d.T, tiles3 = d.tiles3, tiles2 = d.tiles2, nparts = d.nparts;
    const int qst = staged_stride(COLS, (tiles3 + nparts - 1) / nparts, tiles2);
    const bool owner = jb <= d.first_unit;
    const int jlo = range_lo(ci), jhi = range_hi(ci);
    const int first = d.first_unit, M = d.M, ldy = d.ldy;
    const unsigned has_tok = g < T ? 1u : 0u;
    const float w_scale = d.w_scale;
    float* const y = d.y;
    int32_t* const acc_out = d.acc_out;
    const uint32_t q_row = smem_u32(qs_mem + min(g, T - 1) * qst);
    for (int part = 0; part < nparts; ++part) {
      const bool last_part = part + 1 == nparts;
      Part pt;
      pt.t0 = part * tiles3 / nparts;
      pt.t1 = (part + 1) * tiles3 / nparts;
      pt.tiles3 = tiles3;
      pt.tiles2 = last_part ? tiles2 : 0;
      const int npt = pt.t1 - pt.t0;
      if (!staged_any || part > 0 || !same_input(a.it[ci - 1], d) || (owner && d.x && d.q != a.it[ci - 1].q)) {
        if (staged_any) __syncthreads();  // everyone is done with the codes staged before (and with y as scratch)
        stage_item<F>(d, owner, part == 0, pt, qst, qs_mem, qscale, qmul, qsum, qred);
        __syncthreads();                  // (also: the decode tables are complete)
        staged_any = true;
      }
      const int s_lo = wk * npt / S, n3 = (wk + 1) * npt / S - s_lo;
      const int n2 = (wk == S - 1) ? pt.tiles2 : 0;
      const uint32_t q3 = q_row + s_lo * COLS + t * (COLS / 4);   // B registers of the warp's first tile
      const uint32_t q1 = q_row + npt * 96 + t * 16;         // ... of the first pair tile that follows triple tiles
      const int tail_off = (tiles3 - pt.t0 - s_lo) * SLOT;   // from the warp's first triple tile to the first pair tile

      for (int cj = jlo; cj < jhi; cj += G, ++nloc) {
        int C0[2][4], C1[2][4];                // [scale 1, scale 4] x fragment, upper and lower half of the block
#pragma unroll
        for (int s = 0; s < 2; ++s)
#pragma unroll
          for (int i = 0; i < 4; ++i) C0[s][i] = C1[s][i] = 0;
        uint32_t qp = q3;
        int qr[6] = {0, 0, 0, 0, 0, 0};        // B registers; lanes beyond the batch keep these zeros

        // One triple tile: wait for the oldest slot, decode, MMA, refill the slot from `pf`.
        auto step3 = [&](const uint8_t* pf, bool do_pf, bool pf_triple) {
          cp_wait<DEPTH - 1>();
          __syncwarp();                          // the sign plane was copied by lanes 0..7
          const uint32_t sl = ring + slot * SLOT;
          unsigned iw[4], sg[4] = {0u, 0u, 0u, 0u};
          lds128(sl + lane * 16, iw);            // index word t of rows g, g+8, g+16, g+24
          if (F < 2 && hb) lds128(sl + 512 + g * 16, sg); // their sign words (fifth index bits)
          if (F != 0)
            asm volatile(
                "{\n\t.reg .pred p;\n\tsetp.ne.u32 p, %5, 0;\n\t"
                "@p ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];\n\t}"
                : "+r"(qr[0]), "+r"(qr[1]), "+r"(qr[2]), "+r"(qr[3])
                : "r"(qp), "r"(has_tok));
          else
            asm volatile(
                "{\n\t.reg .pred p;\n\tsetp.ne.u32 p, %7, 0;\n\t"
                "@p ld.shared.v2.u32 {%0,%1}, [%6];\n\t"
                "@p ld.shared.v2.u32 {%2,%3}, [%6+8];\n\t"
                "@p ld.shared.v2.u32 {%4,%5}, [%6+16];\n\t}"
                : "+r"(qr[0]), "+r"(qr[1]), "+r"(qr[2]), "+r"(qr[3]), "+r"(qr[4]), "+r"(qr[5])
                : "r"(qp), "r"(has_tok));
          unsigned e[4][4];                      // [row u][index byte j]
#pragma unroll
          for (int u = 0; u < (F >= 2 ? 0 : 4); ++u) {
            const unsigned tw = (sg[u] >> (2 * t)) & 0x03030303u;     // sign pair of index byte j in byte j
            // (the entry's address by a multiply-add: the FMA pipe has room, the integer pipe is the busy one)
            e[u][0] = lds32(mad_u32(prmt(iw[u], tw, 0xCC40u), 128u, tbl2_lane));
            e[u][1] = lds32(mad_u32(prmt(iw[u], tw, 0xDD51u), 128u, tbl2_lane));
            e[u][2] = lds32(mad_u32(prmt(iw[u], tw, 0xEE62u), 128u, tbl2_lane));
            e[u][3] = lds32(mad_u32(prmt(iw[u], tw, 0xFF73u), 128u, tbl2_lane));
          }
          if (F == 3) {
            // x = index nibbles as bytes (0..8); a = x / 3 = (11 x) >> 5, b = x - 3 a: the codes of the pair's weights
            // Both kept at the scale 32 where bits 5, 6 of 11 x hold a: 32 a = (11 x) & 0x60, 32 b = 32 x - 3 (32 a)
            // (multiply-adds; every byte of the result is at most 64, so the word arithmetic is exact).
            constexpr unsigned MB = 0x0F0F0F0Fu, MA = 0x60606060u;
            unsigned alo[4], blo[4], ahi[4], bhi[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
              const unsigned xl = iw[u] & MB, xh = (iw[u] >> 4) & MB;
              alo[u] = mad_u32(xl, 11u, 0u) & MA;
              ahi[u] = mad_u32(xh, 11u, 0u) & MA;
              blo[u] = mad_u32(xl, 32u, mad_u32(alo[u], 0xFFFFFFFDu, 0u));
              bhi[u] = mad_u32(xh, 32u, mad_u32(ahi[u], 0xFFFFFFFDu, 0u));
            }
            mma_u8s8(C0[0], alo[0], alo[1], blo[0], blo[1], qr[0], qr[1]);
            mma_u8s8(C1[0], alo[2], alo[3], blo[2], blo[3], qr[0], qr[1]);
            mma_u8s8(C0[0], ahi[0], ahi[1], bhi[0], bhi[1], qr[2], qr[3]);
            mma_u8s8(C1[0], ahi[2], ahi[3], bhi[2], bhi[3], qr[2], qr[3]);
          } else if (F == 2) {
            // bit pairs 0, 1 of the index bytes at scale 1 (in place, shifted down by two), pairs 2, 3 at scale 16
            constexpr unsigned M0 = 0x03030303u, M2 = 0x30303030u;
            unsigned hi[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) hi[u] = iw[u] >> 2;
            mma_u8s8(C0[0], iw[0] & M0, iw[1] & M0, hi[0] & M0, hi[1] & M0, qr[0], qr[1]);
            mma_u8s8(C1[0], iw[2] & M0, iw[3] & M0, hi[2] & M0, hi[3] & M0, qr[0], qr[1]);
            mma_u8s8(C0[1], iw[0] & M2, iw[1] & M2, hi[0] & M2, hi[1] & M2, qr[2], qr[3]);
            mma_u8s8(C1[1], iw[2] & M2, iw[3] & M2, hi[2] & M2, hi[3] & M2, qr[2], qr[3]);
          } else if (F == 1) {
            // entry of index byte j = the codes of columns 16t + 4j .. + 3, the activation word j of the lane's quarter
            mma_u8s8(C0[0], e[0][0], e[1][0], e[0][1], e[1][1], qr[0], qr[1]);
            mma_u8s8(C1[0], e[2][0], e[3][0], e[2][1], e[3][1], qr[0], qr[1]);
            mma_u8s8(C0[0], e[0][2], e[1][2], e[0][3], e[1][3], qr[2], qr[3]);
            mma_u8s8(C1[0], e[2][2], e[3][2], e[2][3], e[3][3], qr[2], qr[3]);
          } else {
            constexpr unsigned M0 = 0x03030303u, M1 = 0x0C0C0C0Cu;
            // scale 1: index bytes 0, 1 then 2, 3; scale 4: the s=1 pairs of bytes (0, 2) and (1, 3)
            mma_u8s8(C0[0], e[0][0] & M0, e[1][0] & M0, e[0][1] & M0, e[1][1] & M0, qr[0], qr[1]);
            mma_u8s8(C1[0], e[2][0] & M0, e[3][0] & M0, e[2][1] & M0, e[3][1] & M0, qr[0], qr[1]);
            mma_u8s8(C0[0], e[0][2] & M0, e[1][2] & M0, e[0][3] & M0, e[1][3] & M0, qr[2], qr[3]);
            mma_u8s8(C1[0], e[2][2] & M0, e[3][2] & M0, e[2][3] & M0, e[3][3] & M0, qr[2], qr[3]);
            // (bytes 2, 3 of an entry carry nothing under M1, so the second entry shifted up by a multiply-add and
            // one three-input logic operation join the pairs: one integer-pipe instruction per register)
            auto join = [](unsigned ea, unsigned eb) { return (ea | mad_u32(eb, 65536u, 0u)) & M1; };
            mma_u8s8(C0[1], join(e[0][0], e[0][2]), join(e[1][0], e[1][2]), join(e[0][1], e[0][3]), join(e[1][1], e[1][3]),
                     qr[4], qr[5]);
            mma_u8s8(C1[1], join(e[2][0], e[2][2]), join(e[3][0], e[3][2]), join(e[2][1], e[2][3]), join(e[3][1], e[3][3]),
                     qr[4], qr[5]);
          }
          qp += COLS;
          __syncwarp();                          // every lane has read the slot's sign plane
          if (do_pf) prefetch(sl, pf, pf_triple);
          cp_commit();
          slot = (slot + 1 == DEPTH) ? 0 : slot + 1;
        };
        // One pair tile (the K tail): index byte -> four codes at s=0; X = E | E'<<2 holds two index bytes.
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
          unsigned xl[4], xh[4];
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            const unsigned e0 = lds32(tbl1_s + ((iw[u] << 2) & 0x3FCu));
            const unsigned e1 = lds32(tbl1_s + ((iw[u] >> 6) & 0x3FCu));
            const unsigned e2 = lds32(tbl1_s + ((iw[u] >> 14) & 0x3FCu));
            const unsigned e3 = lds32(tbl1_s + ((iw[u] >> 22) & 0x3FCu));
            xl[u] = e0 | (e1 << 2);              // columns 16t + 0..3 at s=0, 16t + 4..7 at s=1
            xh[u] = e2 | (e3 << 2);              // columns 16t + 8..11 at s=0, 16t + 12..15 at s=1
          }
          constexpr unsigned M0 = 0x03030303u, M1 = 0x0C0C0C0Cu;
          mma_u8s8(C0[0], xl[0] & M0, xl[1] & M0, xh[0] & M0, xh[1] & M0, q1r[0], q1r[2]);
          mma_u8s8(C1[0], xl[2] & M0, xl[3] & M0, xh[2] & M0, xh[3] & M0, q1r[0], q1r[2]);
          mma_u8s8(C0[1], xl[0] & M1, xl[1] & M1, xh[0] & M1, xh[1] & M1, q1r[1], q1r[3]);
          mma_u8s8(C1[1], xl[2] & M1, xl[3] & M1, xh[2] & M1, xh[3] & M1, q1r[1], q1r[3]);
          __syncwarp();
          if (do_pf) prefetch(sl, pf, true);     // what follows a pair tile DEPTH places on is a triple tile
          cp_commit();
          slot = (slot + 1 == DEPTH) ? 0 : slot + 1;
        };

        // The warp's stream: n3 triple tiles of this job, n2 pair tiles (last warp of the group, last part), then the
        // next job's triple tiles.  Tile i is followed, DEPTH places on, by tile i + DEPTH of that stream.
        more = next_job(ni, np, nj);
        const uint8_t* const nxt = more ? job_ptr(ni, np, nj) : cur;
        const uint8_t* pf = cur + DEPTH * TB;
#pragma unroll 1
        for (int left = n3 - DEPTH; left > 0; --left, pf += TB) step3(pf, true, true);
        // d-th tile after this job's triple tiles: one of its pair tiles, or a triple tile of the next job
        const uint8_t* const tail = cur + tail_off;
#pragma unroll 1
        for (int dd = 0; dd < DEPTH; ++dd) {
          const bool in_tail = dd < n2;
          step3(in_tail ? tail + dd * 512 : nxt + (dd - n2) * TB, in_tail || more, !in_tail);
        }
#pragma unroll 1
        for (int j2 = 0; j2 < n2; ++j2) step1(q1 + j2 * 64, nxt + (DEPTH - n2 + j2) * SLOT, more);
        cur = nxt;

        // fragments: c[0] = (row g, token 2t), c[1] = (row g, token 2t+1), c[2], c[3] = the same for row g+8
        const int rbuf = RD == 2 ? (nloc & 1) : 0;
        int* mine = red + ((warp * RD + rbuf) * tmax) * 32;
#pragma unroll
        for (int u = 0; u < 2; ++u) {
          int c[4];
#pragma unroll
          for (int i = 0; i < 4; ++i)
            c[i] = u == 0 ? (C0[0][i] >> (F == 3 ? 5 : 0)) + (C0[1][i] >> (F == 2 ? 4 : 2))
                          : (C1[0][i] >> (F == 3 ? 5 : 0)) + (C1[1][i] >> (F == 2 ? 4 : 2));
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
          // this block's turn to be finished by this warp: add the group's partials; the sums of an item walked in
          // parts rest in y (as integers) between the parts; the last part rescales and stores 32 rows
          const int row0 = (cj - first) * 32;
          const int* grp = red + (((gi * S) * RD + rbuf) * tmax) * 32;
          for (int idx = lane; idx < T * 32; idx += 32) {
            int v = 0;
            for (int w2 = 0; w2 < S; ++w2) v += grp[w2 * RD * tmax * 32 + idx];
            const int tok = idx >> 5, row = row0 + (idx & 31);
            v -= (F ? a.card >> 1 : 1) * qsum[tok];     // codes are weights + 1 (+ C/2)
            if (row < M) {
              float* const yp = y + (int64_t)tok * ldy + row;
              if (part > 0) v += __ldcg(reinterpret_cast<const int*>(yp));
              if (last_part) {
                *yp = __fmul_rn((float)v, __fmul_rn(qscale[tok], w_scale));
                if (acc_out) acc_out[(int64_t)tok * ldy + row] = v;
              } else {
                *reinterpret_cast<int*>(yp) = v;
              }
            }
          }
        }
      }
    }
  }
  cp_wait<0>();
  __syncthreads();   // no warp leaves the CTA before the others are done
}

inline int env_int_once(const char* name, int dflt) {
  const char* v = getenv(name);
  return (v && *v) ? atoi(v) : dflt;
}
inline int depth_cap() {
  static const int d = [] {
    const int v = env_int_once("BITNET_TL2_DEPTH", 8);
    return (v >= 3 && v <= 8 && v != 7) ? v : 8;
  }();
  return d;
}
inline int forced_s() {
  static const int s = [] {
    const int v = env_int_once("BITNET_TL2_S", 0);
    return (v == 1 || v == 2 || v == 4 || v == 8) ? v : 0;
  }();
  return s;
}

// (`rd`: buffers of partial sums per warp: 1 when the launch runs with one warp per block, else 2)
inline size_t smem_of(int tmax, size_t code_bytes, int depth, int F, int rd) {
  return 2048 + (size_t)CW * rd * tmax * 32 * 4 + (F >= 2 ? 0 : TBL2_BYTES) + code_bytes + (size_t)CW * depth * SLOT;
}
// true if a launch over `units` blocks runs with one warp per block
inline bool one_warp_per_block(int64_t units) {
  const int f = forced_s();
  return f ? f == 1 : units >= (int64_t)CW * dev_info().sm_count * 4;
}

// How one item is walked: its triple tiles in `nparts` parts (as few as let the staged codes of a part fit beside
// the decode table and a ring of at least 4 tiles per warp -- 3 if nothing else fits); `code` = bytes of the staged
// codes of its largest part, `t3` = triple tiles of its smallest part.
struct ItemPlan {
  int nparts;
  size_t code;
  int t3;
};
inline bool plan_item(int T, const TlGeom& g, int cols, int F, ItemPlan* out, int rd = 2) {
  const size_t cap = (size_t)dev_info().max_smem_optin;
  const int tiles3 = (int)g.tiles3, tiles2 = (int)g.tiles2;
  auto fits = [&](int n, int depth) {
    const int big = (tiles3 + n - 1) / n, small = tiles3 / n;
    if (small < 3) return false;
    const size_t code = ((size_t)T * (size_t)staged_stride(cols, big, tiles2) + 127) & ~(size_t)127;
    if (smem_of(T, code, depth, F, rd) > cap) return false;
    *out = ItemPlan{n, code, small};
    return true;
  };
  if (F < 2 && T > 4) {
    // table modes with many tokens: fewer parts before deeper rings (the decode binds, not the weight stream, and a
    // part costs a staging pass and a round trip of the sums through y)
    for (int n = 1; n <= 16; ++n)
      for (int want_depth = 4; want_depth >= 3; --want_depth)
        if (fits(n, want_depth)) return true;
    return false;
  }
  for (int want_depth = 4; want_depth >= 3; --want_depth)
    for (int n = 1; n <= 16; ++n) {
      if (tiles3 / n < 3) break;
      if (fits(n, want_depth)) return true;
    }
  return false;
}

struct Shape {
  int S, depth;
  int rd = 2;
};
// S and ring depth for a launch whose shortest rows have `t3` triple tiles: every warp's run of triple tiles is at
// least as long as its ring; the ring is made shallower until everything fits one SM's shared memory.
inline bool launch_shape(int t3, int tmax, size_t code, int64_t units, int F, Shape* out, int rd = 2) {
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
  if (rd == 1 && S != 1) return false;          // (one buffer of partial sums per warp needs one warp per block)
  while (depth > 3 && (depth > nw || smem_of(tmax, code, depth, F, rd) > cap)) depth = lower(depth);
  if (depth > nw || smem_of(tmax, code, depth, F, rd) > cap) return false;
  Shape sh;
  sh.S = S;
  sh.depth = depth;
  sh.rd = rd;
  *out = sh;
  return true;
}

template <int DEPTH, int NMAX, int F>
int launch_scan(const SArgs<NMAX>& a, int grid, size_t smem, cudaStream_t st) {
  static bool attr_set[64] = {false};
  int dev = 0;
  cudaGetDevice(&dev);
  if (!attr_set[dev & 63]) {
    cudaError_t e = cudaFuncSetAttribute(gemv_tl2_scan_kernel<DEPTH, NMAX, F>, cudaFuncAttributeMaxDynamicSharedMemorySize,
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
  cfg.numAttrs = early_start_enabled(st) ? 1 : 0;
  cudaError_t e = cudaLaunchKernelEx(&cfg, gemv_tl2_scan_kernel<DEPTH, NMAX, F>, a);
  return e == cudaSuccess ? BITNET_OK : note_cuda_error(e);
}

template <int NMAX, int F>
int launch_depth(const SArgs<NMAX>& a, int depth, int grid, size_t smem, cudaStream_t st) {
  switch (depth) {
    case 3: return launch_scan<3, NMAX, F>(a, grid, smem, st);
    case 4: return launch_scan<4, NMAX, F>(a, grid, smem, st);
    case 5: return launch_scan<5, NMAX, F>(a, grid, smem, st);
    case 6: return launch_scan<6, NMAX, F>(a, grid, smem, st);
    case 8: return launch_scan<8, NMAX, F>(a, grid, smem, st);
    default: return BITNET_ERR_UNSUPPORTED_SHAPE;
  }
}

template <int NMAX, int F>
int launch_run(const Tl2Linear* items, int n, int card, Shape shape, cudaStream_t st) {
  constexpr int COLS = F ? 64 : 96;
  static thread_local SArgs<NMAX> a;
  a.n = n;
  a.S = shape.S | (shape.rd == 1 ? 0x100 : 0);
  a.tmax = 1;
  size_t code = 0;
  int64_t units = 0, w = 0;
  for (int i = 0; i < n; ++i) {
    const Tl2Linear& s = items[i];
    SItem& d = a.it[i];
    ItemPlan pl;
    if (!plan_item(s.T, s.g, COLS, F, &pl, shape.rd)) return BITNET_ERR_UNSUPPORTED_SHAPE;
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
    d.nparts = pl.nparts;
    d.pad = 0;
    units += s.M / 32;
    w += (s.M / 32) * (s.g.tiles3 + s.g.tiles2);
    if (s.T > a.tmax) a.tmax = s.T;
    if (pl.code > code) code = pl.code;
  }
  a.total_units = (int)units;
  a.total_w = (int)w;
  a.code_bytes = (int)code;
  a.card = card;
  a.tile_bytes = (F && n > 0) ? (int)(items[0].g.block_bytes / items[0].g.tiles3) : SLOT;
  const size_t smem = smem_of(a.tmax, code, shape.depth, F, shape.rd);
  if (smem > (size_t)dev_info().max_smem_optin) return BITNET_ERR_UNSUPPORTED_SHAPE;
  const int G = CW / shape.S;
  int grid = dev_info().sm_count;
  if ((int64_t)grid * G > units) grid = (int)ceil_div(units, G);
  log_launch(F ? "gemv_tl2_scan_kernel<pairs> items=%d blocks=%lld tiles=%lld grid=%d warps/block=%d ring=%d tmax=%d smem=%zu"
               : "gemv_tl2_scan_kernel items=%d blocks=%lld tiles=%lld grid=%d warps/block=%d ring=%d tmax=%d smem=%zu", n,
             (long long)units, (long long)w, grid, shape.S, shape.depth, a.tmax, smem);
  return launch_depth<NMAX, F>(a, shape.depth, grid, smem, st);
}

template <int F>
bool item_supported(int T, int64_t M, int64_t K, const TlGeom& g) {
  if (T < 1 || T > 8 || M < 32 || (M % 32) != 0 || K < 4 || (K % 4) != 0 || M > 0x7fffffff || g.block_bytes > 0x7fffffff)
    return false;
  if (g.tiles2 > 2 || g.three_k > 0x3fffffff) return false;    // more pair tiles than a ring refill pattern assumes
  ItemPlan pl;
  Shape sh;
  return plan_item(T, g, F ? 64 : 96, F, &pl) && launch_shape(pl.t3, T, pl.code, M / 32, F, &sh);
}

// Launches the scan kernel over `n` supported items of one format (and, F = 1, one cardinality and tile size): as
// few launches as the argument block (NLARGE items, 2^30 tiles) and shared memory allow.
template <int F>
int launch_items(const Tl2Linear* items, int64_t n, int card, cudaStream_t st) {
  constexpr int COLS = F ? 64 : 96;
  int64_t i = 0;
  while (i < n) {
    int64_t j = i, w = 0;
    int t3_min = 1 << 30, tmax = 1;
    size_t code = 0;
    Shape sh{1, 3};
    int64_t units = 0;
    for (int64_t k = i; k < n && k - i < NLARGE; ++k) units += items[k].M / 32;   // (an estimate when the run is cut short)
    const int rd = one_warp_per_block(units) ? 1 : 2;   // buffers of partial sums per warp
    while (j < n && j - i < NLARGE) {
      const TlGeom& g = items[j].g;
      ItemPlan pl;
      if (!plan_item(items[j].T, g, COLS, F, &pl, rd)) return BITNET_ERR_UNSUPPORTED_SHAPE;
      const int64_t add = (items[j].M / 32) * (g.tiles3 + g.tiles2);
      const int tm = items[j].T > tmax ? items[j].T : tmax;
      const size_t cm = pl.code > code ? pl.code : code;
      const int t3 = pl.t3 < t3_min ? pl.t3 : t3_min;
      Shape sj;
      const bool fits = launch_shape(t3, tm, cm, units, F, &sj, rd);
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
    const int rc = cnt <= NSMALL ? launch_run<NSMALL, F>(items + i, cnt, card, sh, st)
                                 : launch_run<NLARGE, F>(items + i, cnt, card, sh, st);
    if (rc != BITNET_OK) return rc;
    i = j;
  }
  return BITNET_OK;
}

}  // namespace scan
}  // namespace bitnet
