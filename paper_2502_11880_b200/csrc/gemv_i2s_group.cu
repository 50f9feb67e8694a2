// Grouped I2_S decode (1..8 tokens): Alg. 1, Phases 1 and 2 plus the rescale, for a LIST of linear layers
// whose inputs are all there at launch, in ONE persistent kernel.
//
// Why.  A decode GEMV of a few tens of megabytes lasts 5-20 us, of which about 3 us per launch are fixed
// (launch release, the quantiser's round trip, the first tile, the tail).  Over a list of linears that fixed
// part is paid once here: the packed weights of the whole list are one stream of work that is cut into 148
// equal pieces, one per SM, and a CTA walks its piece from the first byte to the last without ever letting
// its asynchronous copies run dry, across the borders between linears.
//
// Work split.  The unit of work is a 16-row block of one linear (contiguous in the blob: 4*Kp bytes).  The
// units of all items, in item order, form one sequence; CTA c owns the contiguous range whose packed bytes
// are the c-th 1/gridDim of the total (found on the device by a binary search over the items' prefix sums,
// which the host puts into the argument block).  A CTA's range touches two or three items of a long list, so
// the activation row changes only a few times per CTA.  Inside the CTA the 16 warps form G = 16/S groups;
// group gi takes the units jb+gi, jb+gi+G, ... of the range, and the S warps of a group split a unit's K
// into slices (as in the single-linear kernel).  Every warp owns a ring of DEPTH 1-KB chunks in shared
// memory, filled by per-thread cp.async copies that the same thread reads back: the only synchronisation of
// the weight stream is cp.async.wait_group.  The prefetch position of a warp is a cursor of its own that runs
// DEPTH chunks ahead of the consume position through the same sequence of units -- over unit borders, item
// borders and the CTA-wide barriers of an item change alike.
//
// Item change.  When the CTA's range enters a new item, the CTA meets at a barrier, quantises the item's
// activation rows (fp32 -> int8 by absmax, the row held in registers between the two passes; same operations
// in the same order as the stand-alone quantiser, so bit-identical) or copies the given codes, into shared
// memory, and goes on.  An item whose input (x, K, T) equals the previous item's keeps the staged codes: linears
// that share an input (Q/K/V, gate/up) quantise it once per CTA.  The CTA whose range holds an item's first
// unit also stores the codes and scales for the caller.
//
// Compute side: as in the single-linear kernel -- a packed word under the mask 0x03030303 << 2s is an A
// register of mma.sync.m16n8k32 (u8 x s8), four accumulators carry the scales 1, 4, 16, 64, and
// sum(code*q) - sum(q) = sum(w*q); the row sum of the codes is taken once while staging.
#include <cstdlib>
#include <cstring>

#include "common.cuh"
#include "device_utils.cuh"

namespace bitnet {
namespace {

constexpr int CW = 16;  // warps
constexpr int THREADS = CW * 32;
constexpr int XREG = 16;                       // float4 registers per thread of the quantiser's one-pass form
constexpr int NSMALL = 50, NLARGE = 409;       // items per launch: argument blocks of 4 KB / 32 KB
constexpr size_t MAX_CODE_BYTES = 144 * 1024;  // staged activation codes of one item

struct GItem {
  const uint8_t* packed;
  const float* x;      // fp32 activations [T][K]; null: q and act_scale are inputs
  int8_t* q;
  float* act_scale;
  float* y;
  int32_t* acc_out;
  float w_scale;
  int M, K, T;
  int first_unit;      // units of the items before this one
  int first_w;         // 1-KB chunks of the items before this one
  int nparts;          // K is walked in this many parts (1 unless the staged codes of a whole row do not fit)
  int ldy;             // elements between the token rows of y and acc_out (M, or more for a slice of a wider output)
};
static_assert(sizeof(GItem) == 80, "argument block layout");

template <int NMAX>
struct GArgs {
  int n, S, tmax, code_bytes;
  int total_units, total_w, r0, r1;
  GItem it[NMAX];
};
static_assert(sizeof(GArgs<NSMALL>) <= 4096 && sizeof(GArgs<NLARGE>) <= 32764, "kernel parameter limits");

// bytes of the kernel's shared-memory header (range, per-token scales, sums and partial maxima) for batches of up to
// `tmax` tokens
__host__ __device__ constexpr int header_bytes(int tmax) { return tmax > 8 ? 2048 : 1024; }

__device__ __forceinline__ bool same_input(const GItem& p, const GItem& d) {
  return p.nparts == 1 && d.nparts == 1 && p.K == d.K && p.T == d.T &&
         (d.x ? p.x == d.x : (p.x == nullptr && p.q == d.q && p.act_scale == d.act_scale));
}

// Stages the activation codes of the item's columns [256 c0, 256 c1) (T rows, qst bytes apart, zero beyond K) and,
// per token, the scale and the sum of the staged codes.  `first` = the item's first part: the row maximum is taken
// (Alg. 1 Phase 1) and, in the CTA that owns the item, codes and scales of the WHOLE row go to the caller; later
// parts reuse the multiplier kept in qmul.  Called by all threads; contains barriers.
template <int NT>
__device__ __forceinline__ void stage_item(const GItem& d, bool owner, bool first, int c0, int c1, int qst, int8_t* qs_mem,
                                           float* qscale, float* qmul, int* qsum, float* qred) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int n4 = d.K / 4, w0 = c0 * 64, w1 = c1 * 64;       // staged words [w0, w1) of a row
  if (threadIdx.x < 8 * NT) qsum[threadIdx.x] = 0;
  if (d.x && first && d.K <= 4 * XREG * THREADS) {
    // one round trip per token: s = 127 / max(amax, 1e-5), q = clamp(rint(x * s)); the row stays in registers
    const int kw = (int)(i2s_kp(d.K) / 4);
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
      if (tok > 0) __syncthreads();  // everyone has read the previous token's partial maxima
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
          const int word = quant4_packed(xv[r], sq);  // columns K..Kp-1 came in as zeros
          if (i >= w0 && i < w1) {
            reinterpret_cast<int*>(qs_mem + tok * qst)[staged_word(i - w0)] = word;
            s = __dp4a(word, 0x01010101, s);
          }
          if (owner && i < n4) reinterpret_cast<int*>(d.q + (int64_t)tok * d.K)[i] = word;
        }
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
      if (lane == 0) atomicAdd(qsum + tok, s);
    }
  } else if (d.x) {
    if (first) {
      // rows too long for the registers: amax per token first
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
    // quantise: the staged columns into shared memory; in the owning CTA's first part every column for the caller
    const int lo = (owner && first) ? 0 : w0, hi = (owner && first) ? max(w1, n4) : w1;
    for (int tok = 0; tok < d.T; ++tok) {
      const float sq = qmul[tok];
      const float4* x4 = reinterpret_cast<const float4*>(d.x + (int64_t)tok * d.K);
      int s = 0;
      for (int i = lo + threadIdx.x; i < hi; i += THREADS) {
        int word = 0;
        if (i < n4) {
          word = quant4_packed(__ldcg(x4 + i), sq);
          if (owner && first) reinterpret_cast<int*>(d.q + (int64_t)tok * d.K)[i] = word;
        }
        if (i >= w0 && i < w1) {
          reinterpret_cast<int*>(qs_mem + tok * qst)[staged_word(i - w0)] = word;
          s = __dp4a(word, 0x01010101, s);
        }
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
      if (lane == 0) atomicAdd(qsum + tok, s);
    }
  } else {
    // given codes: 16 at a time (K % 64 == 0 and the parts begin on chunks: a row's words come in whole fours, and
    // staged_word keeps four consecutive words together)
    __syncthreads();  // qsum is zero before the first atomicAdd
    for (int tok = 0; tok < d.T; ++tok) {
      const int4* qrow = reinterpret_cast<const int4*>(d.q + (int64_t)tok * d.K);
      int s = 0;
      for (int i = w0 / 4 + threadIdx.x; i < w1 / 4; i += THREADS) {
        const int4 v = (4 * i < n4) ? __ldcg(qrow + i) : make_int4(0, 0, 0, 0);
        *reinterpret_cast<int4*>(reinterpret_cast<int*>(qs_mem + tok * qst) + staged_word(4 * i - w0)) = v;
        s = __dp4a(v.x, 0x01010101, s);
        s = __dp4a(v.y, 0x01010101, s);
        s = __dp4a(v.z, 0x01010101, s);
        s = __dp4a(v.w, 0x01010101, s);
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
      if (lane == 0) atomicAdd(qsum + tok, s);
    }
    if (threadIdx.x < d.T) qscale[threadIdx.x] = __ldcg(d.act_scale + threadIdx.x);
  }
}

// NT = groups of eight tokens an item may have (1: up to 8 tokens; 2: up to 16 -- every A register then feeds two
// MMAs, one per group, and the weights of a 9-to-16-token batch still cross HBM once).
template <int DEPTH, int NMAX, int NT>
__global__ void __launch_bounds__(THREADS, 1) gemv_i2s_group_kernel(const __grid_constant__ GArgs<NMAX> a) {
  extern __shared__ __align__(128) uint8_t smem[];
  constexpr int HB = header_bytes(8 * NT);
  int* hdr = reinterpret_cast<int*>(smem);             // [0] first unit, [1] end unit, [2] first item, [3] last item
  float* qscale = reinterpret_cast<float*>(smem + 64);            // [8 NT] act_scale per token
  int* qsum = reinterpret_cast<int*>(smem + 64 + 32 * NT);        // [8 NT] sum of the staged codes per token
  float* qred = reinterpret_cast<float*>(smem + 64 + 64 * NT);    // [8 NT][16] partial maxima
  float* qmul = reinterpret_cast<float*>(smem + 64 + 576 * NT);   // [8 NT] 127 / amax per token
  // partial sums [CW][RD][tmax][16]: two buffers per warp, so that a warp may start its next unit while its group
  // still adds up the last one; one when every warp finishes its own units (two-group form, one warp per unit)
  const int RD = a.r0;                                 // (set by the host: 1 or 2)
  int* red = reinterpret_cast<int*>(smem + HB);
  int8_t* qs_mem = reinterpret_cast<int8_t*>(smem + HB + CW * RD * a.tmax * 16 * 4);
  uint8_t* rings = reinterpret_cast<uint8_t*>(qs_mem) + a.code_bytes;

  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int S = a.S, G = CW / S, gi = warp / S, wk = warp % S;
  const int g = lane >> 2, t = lane & 3;

  if (threadIdx.x == 0) {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    // this CTA's range of the unit sequence: equal shares of the packed bytes, cut at unit borders
    auto locate = [&](int64_t w, int* item) -> int {
      int lo = 0, hi = a.n - 1;
      while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if ((int64_t)a.it[mid].first_w <= w) lo = mid; else hi = mid - 1;
      }
      *item = lo;
      const int nch = (int)(i2s_kp(a.it[lo].K) / 256);
      return a.it[lo].first_unit + (int)((w - a.it[lo].first_w) / nch);
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
  const uint32_t ring = smem_u32(rings + (size_t)warp * DEPTH * 1024) + lane * 16;

  // ---------------- the group's sequence of jobs.  Within the CTA's range, item i contributes the units
  // [max(jb, first_i), min(je, end_i)); the group takes every G-th of them starting at its own index, once per
  // part of the item's K.  A job is (item, part, unit).
  auto item_end = [&](int i) { return (i + 1 < a.n) ? a.it[i + 1].first_unit : a.total_units; };
  auto range_lo = [&](int i) { const int f = a.it[i].first_unit; return (f > jb ? f : jb) + gi; };
  auto range_hi = [&](int i) { const int e = item_end(i); return e < je ? e : je; };
  // first chunk of this warp's slice of (item i, part p, unit job)
  auto job_ptr = [&](int i, int p, int job) -> const uint8_t* {
    const GItem& d = a.it[i];
    const int kp = (int)i2s_kp(d.K), nch = kp / 256;
    const int c0 = p * nch / d.nparts, npc = (p + 1) * nch / d.nparts - c0;
    return d.packed + (int64_t)(job - d.first_unit) * (4 * kp) + (int64_t)(c0 + wk * npc / S) * 1024 + lane * 16;
  };
  // the job after (i, p, job) in this group's sequence; false if there is none
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
  int ni = item0 - 1, np = 0, nj = 0;     // (item, part, unit) of the job whose first chunks enter the ring next
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
  // slice of every part of every item is at least DEPTH chunks long (the host chooses S and DEPTH that way).
#pragma unroll
  for (int d = 0; d < DEPTH; ++d) {
    if (cur) {
      cp16(ring + d * 1024, cur + d * 1024, pol);
      cp16(ring + d * 1024 + 512, cur + d * 1024 + 512, pol);
    }
    cp_commit();
  }

  asm volatile("griddepcontrol.wait;" ::: "memory");

  // ---------------- consume
  uint32_t slot_off = 0;
  int nloc = 0;
  const int tmax = a.tmax;
  bool staged_any = false;
  for (int ci = item0; ci <= item1; ++ci) {
    const GItem& d = a.it[ci];
    const int T = d.T, kp = (int)i2s_kp(d.K), nch = kp / 256, nparts = d.nparts;
    const int qst = ((nch + nparts - 1) / nparts) * 256 + 64;
    const bool owner = jb <= d.first_unit;
    const int jlo = range_lo(ci), jhi = range_hi(ci);
    const int first = d.first_unit, M = d.M, ldy = d.ldy;
    const unsigned has_tok = g < T ? 1u : 0u, has_tok2 = g + 8 < T ? 1u : 0u;
    const float w_scale = d.w_scale;
    float* const y = d.y;
    int32_t* const acc_out = d.acc_out;
    for (int part = 0; part < nparts; ++part) {
      const int c0 = part * nch / nparts, c1 = (part + 1) * nch / nparts, npc = c1 - c0;
      if (!staged_any || part > 0 || !same_input(a.it[ci - 1], d)) {
        if (staged_any) __syncthreads();  // everyone is done with the codes staged before (and with y as scratch)
        stage_item<NT>(d, owner, part == 0, c0, c1, qst, qs_mem, qscale, qmul, qsum, qred);
        __syncthreads();
        staged_any = true;
      } else if (owner && d.x && d.q != a.it[ci - 1].q) {
        // same input as the previous item but its own output buffers for the codes
        for (int tok = 0; tok < T; ++tok)
          for (int i = threadIdx.x; i < d.K / 4; i += THREADS)
            reinterpret_cast<int*>(d.q + (int64_t)tok * d.K)[i] = reinterpret_cast<const int*>(qs_mem + tok * qst)[staged_word(i)];
        if (threadIdx.x < T) d.act_scale[threadIdx.x] = qscale[threadIdx.x];
      }
      const int s_lo = wk * npc / S, nw = (wk + 1) * npc / S - s_lo;
      const uint32_t q_lane = smem_u32(qs_mem + min(g, T - 1) * qst + s_lo * 256 + t * 16);
      const uint32_t q_grp2 = (uint32_t)((min(g + 8, T - 1) - min(g, T - 1)) * qst);   // (NT = 2) on to token g + 8
      const bool last_part = part + 1 == nparts;

      for (int cj = jlo; cj < jhi; cj += G, ++nloc) {
        int C[NT][4][4];
        int qr[NT][8];                         // B registers; lanes beyond the batch keep their zeros
#pragma unroll
        for (int n = 0; n < NT; ++n) {
#pragma unroll
          for (int s = 0; s < 4; ++s)
#pragma unroll
            for (int i = 0; i < 4; ++i) C[n][s][i] = 0;
#pragma unroll
          for (int i = 0; i < 8; ++i) qr[n][i] = 0;
        }
        uint32_t qp = q_lane;
        // One step: wait for the oldest chunk of the ring, put it through the tensor cores, then refill its slot
        // from `pf` (the chunk DEPTH places further down the warp's stream), if there is one.
        auto step = [&](const uint8_t* pf, bool do_pf) {
          cp_wait<DEPTH - 1>();
          unsigned w4[4], v4[4];
          asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];"
                       : "=r"(w4[0]), "=r"(w4[1]), "=r"(w4[2]), "=r"(w4[3])
                       : "r"(ring + slot_off));
          asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];"
                       : "=r"(v4[0]), "=r"(v4[1]), "=r"(v4[2]), "=r"(v4[3])
                       : "r"(ring + slot_off + 512));
#pragma unroll
          for (int h = 0; h < 2; ++h) {
            // only the lanes whose B column is a real token load activations
            asm volatile(
                "{\n\t.reg .pred p;\n\tsetp.ne.u32 p, %9, 0;\n\t"
                "@p ld.shared.v4.u32 {%0,%1,%2,%3}, [%8];\n\t"
                "@p ld.shared.v4.u32 {%4,%5,%6,%7}, [%8+64];\n\t}"
                : "+r"(qr[0][0]), "+r"(qr[0][1]), "+r"(qr[0][2]), "+r"(qr[0][3]), "+r"(qr[0][4]), "+r"(qr[0][5]), "+r"(qr[0][6]),
                  "+r"(qr[0][7])
                : "r"(qp + h * 128), "r"(has_tok));
            if (NT == 2)
              asm volatile(
                  "{\n\t.reg .pred p;\n\tsetp.ne.u32 p, %9, 0;\n\t"
                  "@p ld.shared.v4.u32 {%0,%1,%2,%3}, [%8];\n\t"
                  "@p ld.shared.v4.u32 {%4,%5,%6,%7}, [%8+64];\n\t}"
                  : "+r"(qr[NT - 1][0]), "+r"(qr[NT - 1][1]), "+r"(qr[NT - 1][2]), "+r"(qr[NT - 1][3]), "+r"(qr[NT - 1][4]),
                    "+r"(qr[NT - 1][5]), "+r"(qr[NT - 1][6]), "+r"(qr[NT - 1][7])
                  : "r"(qp + q_grp2 + h * 128), "r"(has_tok2));
#pragma unroll
            for (int s = 0; s < 4; ++s) {
              const unsigned m = 0x03030303u << (2 * s);
              const unsigned a0 = w4[2 * h] & m, a1 = v4[2 * h] & m, a2 = w4[2 * h + 1] & m, a3 = v4[2 * h + 1] & m;
#pragma unroll
              for (int n = 0; n < NT; ++n) mma_u8s8(C[n][s], a0, a1, a2, a3, qr[n][2 * s], qr[n][2 * s + 1]);
            }
          }
          qp += 256;
          // the chunk's bytes were in registers before the MMAs were issued: its slot can be refilled
          if (do_pf) {
            cp16(ring + slot_off, pf, pol);
            cp16(ring + slot_off + 512, pf + 512, pol);
          }
          cp_commit();
          slot_off = (slot_off + 1024 == DEPTH * 1024) ? 0 : slot_off + 1024;
        };

        // chunks 0 .. nw-DEPTH-1 are followed, DEPTH places on, by chunks of the same slice; the last DEPTH chunks by
        // the first DEPTH chunks of the group's next job (this item's next unit or part, or a later item), if any
        more = next_job(ni, np, nj);
        const uint8_t* const nxt = more ? job_ptr(ni, np, nj) : cur;
        const uint8_t* pf = cur + DEPTH * 1024;
#pragma unroll 2
        for (int left = nw - DEPTH; left > 0; --left, pf += 1024) step(pf, true);
#pragma unroll
        for (int dd = 0; dd < DEPTH; ++dd) step(nxt + dd * 1024, more);
        cur = nxt;

        // fragment: c[0] = (row g, token 2t), c[1] = (row g, token 2t+1), c[2], c[3] = the same for row g+8
        // (token group n: the tokens 8 n + 2t, 8 n + 2t + 1)
        const int rbuf = RD == 2 ? (nloc & 1) : 0;
        int* mine = red + ((warp * RD + rbuf) * tmax) * 16;
#pragma unroll
        for (int n = 0; n < NT; ++n) {
          int c[4];
#pragma unroll
          for (int i = 0; i < 4; ++i) c[i] = C[n][0][i] + (C[n][1][i] >> 2) + (C[n][2][i] >> 4) + (C[n][3][i] >> 6);
          const int tk = 8 * n + 2 * t;
          if (tk < T) {
            mine[tk * 16 + g] = c[0];
            mine[tk * 16 + g + 8] = c[2];
          }
          if (tk + 1 < T) {
            mine[(tk + 1) * 16 + g] = c[1];
            mine[(tk + 1) * 16 + g + 8] = c[3];
          }
        }
        if (S > 1) group_barrier(1 + gi, S * 32);
        else __syncwarp();
        if (wk == (nloc & (S - 1))) {
          // this unit's turn to be finished by this warp: add the group's partials; the sums of an item walked in
          // parts rest in y (as integers) between the parts; the last part rescales and stores 16 rows
          const int row0 = (cj - first) * 16;
          const int* grp = red + (((gi * S) * RD + rbuf) * tmax) * 16;
#pragma unroll
          for (int i = 0; i < 4 * NT; ++i) {
            const int idx = lane + 32 * i;
            if (idx < T * 16) {
              int v = 0;
              for (int w2 = 0; w2 < S; ++w2) v += grp[w2 * RD * tmax * 16 + idx];
              const int tok = idx >> 4, row = row0 + (idx & 15);
              v -= qsum[tok];
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
  }
  cp_wait<0>();
  __syncthreads();   // no warp leaves the CTA before the others are done
}

int env_int_once(const char* name, int dflt) {
  const char* v = getenv(name);
  return (v && *v) ? atoi(v) : dflt;
}
// Tuning overrides, read once: warps per unit (1, 2 or 4) and ring depth (4, 6, 8 or 12); 0 = the defaults below.
int forced_s() {
  static const int s = [] {
    const int v = env_int_once("BITNET_GROUP_S", 0);
    return (v == 1 || v == 2 || v == 4 || v == 8) ? v : 0;
  }();
  return s;
}
int depth_cap() {
  static const int d = [] {
    // Four chunks per warp in flight (64 KB per SM) measured fastest on the 100B sweep with one warp per unit: 2.42 ms
    // per step against 2.47 with three, 2.46 with five, 2.56 with six and 2.63 with eight (with four warps per unit,
    // before units went to single warps, six had been best: 2.45 against 2.59 with eight).
    const int v = env_int_once("BITNET_GROUP_DEPTH", 4);
    return (v == 4 || v == 6 || v == 8 || v == 12) ? v : 4;
  }();
  return d;
}

// Warps per unit and ring depth for a launch whose shortest rows have `nch` chunks: every warp's K-slice must be
// at least as long as its ring (the prefetch never reaches beyond the next unit), so short rows get fewer warps per
// unit, then shallower rings.
struct Shape {
  int S, depth;
  int rd = 2;      // buffers of partial sums per warp (1: two-group form with one warp per unit)
};
// `units` = 16-row units of the whole launch: with at least four units per warp of the GPU every warp takes whole
// units (no partial sums to join, no group barriers: 2.52 ms per 100B sweep against 2.72 with four warps per unit,
// 2.60 against 2.92 after seconds of sustained load); with fewer, up to four warps share a unit's K.
Shape shape_for(int64_t nch, int64_t units) {
  int S = forced_s();
  if (!S) {
    S = 1;
    while (S < 4 && units * S < (int64_t)CW * dev_info().sm_count * 4) S <<= 1;
  }
  while (S > 1 && nch / S < 8) S >>= 1;
  const int64_t nw = nch / S;      // the shortest slice
  int depth = depth_cap();
  while (depth > 4 && depth > nw) depth = depth == 12 ? 8 : depth - 2;
  Shape sh;
  sh.S = S;
  sh.depth = depth;
  return sh;
}

// true if a launch over `units` units runs with one warp per unit
bool one_warp_per_unit(int64_t units) {
  const int f = forced_s();
  return f ? f == 1 : units >= (int64_t)CW * dev_info().sm_count * 4;
}

size_t smem_of(int tmax, size_t code_bytes, int depth, int rd) {
  return (size_t)header_bytes(tmax) + (size_t)CW * rd * tmax * 16 * 4 + code_bytes + (size_t)CW * depth * 1024;
}

// How one item is walked: in `nparts` parts of its K (as few as let the staged codes of a part, T rows of at most
// ceil(nch / nparts) chunks, fit beside the warps' rings, 4 chunks each unless BITNET_GROUP_DEPTH asks for more); `code` =
// bytes of the staged codes of its largest part, `npc` = chunks of its smallest part.
struct ItemPlan {
  int nparts;
  size_t code;
  int64_t npc;
};
// (`rd`: buffers of partial sums per warp the launch will have.  With 9 to 16 tokens fewer parts come before a deeper
// ring: a part costs a staging pass over 16 rows of codes and a round trip of the sums through y.)
bool plan_item(int T, int64_t M, int64_t K, ItemPlan* out, int rd = 2) {
  if (T < 1 || T > 16 || M < 1 || K < 1 || (K % 64) != 0 || M > 0x7fffffff) return false;
  const int64_t nch = i2s_kp(K) / 256;
  const size_t cap = (size_t)dev_info().max_smem_optin;
  auto fits = [&](int n, int depth, ItemPlan* pl) {
    const int64_t big = ceil_div(nch, n), small = nch / n;
    if (small < 4) return false;
    const size_t code = ((size_t)T * (size_t)(big * 256 + 64) + 127) & ~(size_t)127;
    if (code > MAX_CODE_BYTES || smem_of(T, code, depth, rd) > cap) return false;
    *pl = ItemPlan{n, code, small};
    return true;
  };
  const int top = depth_cap() >= 6 ? 6 : 4;      // (rings deeper than the launch will use need no room)
  if (T > 8) {
    for (int n = 1; n <= 16; ++n)
      for (int want_depth = top; want_depth >= 4; want_depth -= 2)
        if (fits(n, want_depth, out)) return true;
    return false;
  }
  for (int want_depth = top; want_depth >= 4; want_depth -= 2)
    for (int n = 1; n <= 16; ++n) {
      if (nch / n < 4) break;
      if (fits(n, want_depth, out)) return true;
    }
  return false;
}

template <int DEPTH, int NMAX, int NT>
int launch_group(const GArgs<NMAX>& a, int grid, size_t smem, cudaStream_t st) {
  static bool attr_set[64] = {false};
  int dev = 0;
  cudaGetDevice(&dev);
  if (!attr_set[dev & 63]) {
    cudaError_t e = cudaFuncSetAttribute(gemv_i2s_group_kernel<DEPTH, NMAX, NT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
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
  cudaError_t e = cudaLaunchKernelEx(&cfg, gemv_i2s_group_kernel<DEPTH, NMAX, NT>, a);
  return e == cudaSuccess ? BITNET_OK : note_cuda_error(e);
}

template <int NMAX, int NT>
int launch_depth(const GArgs<NMAX>& a, int depth, int grid, size_t smem, cudaStream_t st) {
  switch (depth) {
    case 4: return launch_group<4, NMAX, NT>(a, grid, smem, st);
    case 6: return launch_group<6, NMAX, NT>(a, grid, smem, st);
    case 8: return launch_group<8, NMAX, NT>(a, grid, smem, st);
    case 12: return launch_group<12, NMAX, NT>(a, grid, smem, st);
    default: return BITNET_ERR_UNSUPPORTED_SHAPE;
  }
}

// S and ring depth for a launch whose shortest part has `npc` chunks, whose largest batch is `tmax` tokens and
// whose largest staged codes take `code` bytes; false if they do not fit one SM's shared memory.
bool launch_shape(int64_t npc, int tmax, size_t code, int64_t units, int rd, Shape* out) {
  if (npc < 4 || code > MAX_CODE_BYTES) return false;
  Shape sh = shape_for(npc, units);
  if (rd == 1 && sh.S != 1) return false;     // (one buffer of partial sums per warp needs one warp per unit)
  sh.rd = rd;
  const size_t cap = (size_t)dev_info().max_smem_optin;
  while (sh.depth > 4 && smem_of(tmax, code, sh.depth, sh.rd) > cap) sh.depth = sh.depth == 12 ? 8 : sh.depth - 2;
  if (smem_of(tmax, code, sh.depth, sh.rd) > cap) return false;
  *out = sh;
  return true;
}

// One launch over `n` items with the given shape.
template <int NMAX>
int launch_run(const GroupLinear* items, int n, Shape shape, cudaStream_t st) {
  static thread_local GArgs<NMAX> a;   // 32 KB: off the stack
  a.n = n;
  a.S = shape.S;
  a.tmax = 1;
  size_t code = 0;
  int64_t units = 0, w = 0;
  for (int i = 0; i < n; ++i) {
    const GroupLinear& s = items[i];
    GItem& d = a.it[i];
    ItemPlan pl;
    if (!plan_item(s.T, s.M, s.K, &pl, shape.rd)) return BITNET_ERR_UNSUPPORTED_SHAPE;
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
    d.first_unit = (int)units;
    d.first_w = (int)w;
    d.nparts = pl.nparts;
    d.ldy = (int)(s.ldy ? s.ldy : s.M);
    const int64_t nu = ceil_div(s.M, 16), nch = i2s_kp(s.K) / 256;
    units += nu;
    w += nu * nch;
    if (s.T > a.tmax) a.tmax = s.T;
    if (pl.code > code) code = pl.code;
  }
  a.total_units = (int)units;
  a.total_w = (int)w;
  a.code_bytes = (int)code;
  a.r0 = shape.rd;
  a.r1 = 0;
  const int depth = shape.depth;
  const size_t smem = smem_of(a.tmax, code, depth, shape.rd);
  if (smem > (size_t)dev_info().max_smem_optin) return BITNET_ERR_UNSUPPORTED_SHAPE;
  const int G = CW / a.S;
  int grid = dev_info().sm_count;
  if ((int64_t)grid * G > units) grid = (int)ceil_div(units, G);
  log_launch("gemv_i2s_group_kernel items=%d units=%lld chunks=%lld grid=%d warps/unit=%d ring=%d tmax=%d smem=%zu", n,
             (long long)units, (long long)w, grid, a.S, depth, a.tmax, smem);
  if (a.tmax > 8) {                        // 9 to 16 tokens: the two-group kernel, built for the large block only
    if (NMAX != NLARGE) return BITNET_ERR_UNSUPPORTED_SHAPE;
    return launch_depth<NMAX, NMAX == NLARGE ? 2 : 1>(a, depth, grid, smem, st);
  }
  return launch_depth<NMAX, 1>(a, depth, grid, smem, st);
}

}  // namespace

bool gemv_i2s_group_item_supported(int T, int64_t M, int64_t K) {
  ItemPlan pl;
  Shape sh;
  return plan_item(T, M, K, &pl) && launch_shape(pl.npc, T, pl.code, ceil_div(M, 16), 2, &sh);
}

// Launches the grouped kernel over `n` supported items: as few launches as the argument block (NLARGE items,
// 2^30 chunks) and shared memory (the largest batch and the longest part of a launch set its code area) allow.
// A launch runs with the warps per unit and ring depth that suit its shortest part.
int launch_gemv_i2s_group(const GroupLinear* items, int64_t n, cudaStream_t st) {
  int64_t i = 0;
  while (i < n) {
    int64_t j = i, w = 0, npc_min = 1 << 30;
    int tmax = 1;
    size_t code = 0;
    Shape sh{1, 4};
    int64_t units = 0;
    const bool wide = items[i].T > 8;      // a launch holds items of one class: up to 8 tokens, or 9 to 16
    for (int64_t k = i; k < n && k - i < NLARGE && (items[k].T > 8) == wide; ++k)
      units += ceil_div(items[k].M, 16);   // (an estimate when the run is cut short)
    const int rd = (wide && one_warp_per_unit(units)) ? 1 : 2;   // buffers of partial sums per warp
    while (j < n && j - i < NLARGE && (items[j].T > 8) == wide) {
      ItemPlan pl;
      if (!plan_item(items[j].T, items[j].M, items[j].K, &pl, rd)) return BITNET_ERR_UNSUPPORTED_SHAPE;
      const int64_t add = ceil_div(items[j].M, 16) * (i2s_kp(items[j].K) / 256);
      const int tm = items[j].T > tmax ? items[j].T : tmax;
      const size_t cm = pl.code > code ? pl.code : code;
      const int64_t nm = pl.npc < npc_min ? pl.npc : npc_min;
      Shape sj;
      const bool fits = launch_shape(nm, tm, cm, units, rd, &sj);
      if (!fits && j == i) return BITNET_ERR_UNSUPPORTED_SHAPE;
      if (!fits || (j > i && w + add > (1ll << 30))) break;
      w += add;
      tmax = tm;
      code = cm;
      npc_min = nm;
      sh = sj;
      ++j;
    }
    const int cnt = (int)(j - i);
    const int rc = (cnt <= NSMALL && !wide) ? launch_run<NSMALL>(items + i, cnt, sh, st) : launch_run<NLARGE>(items + i, cnt, sh, st);
    if (rc != BITNET_OK) return rc;
    i = j;
  }
  return BITNET_OK;
}

}  // namespace bitnet
