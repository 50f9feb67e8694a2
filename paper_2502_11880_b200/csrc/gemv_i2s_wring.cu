// I2_S mpGEMV for decode (1..8 tokens; used for batches of up to 4), warp-private rings: Alg. 1 Phase 2
// from the 2-bit blob with the quantiser (Phase 1) optionally fused in.
//
// Memory side.  The blob stores 16-row units contiguously and chunk-major (1024 bytes per 256-column
// chunk, 64 bytes per row).  A unit is shared by S warps (S a power of two), each owning a K-slice of the
// unit.  Every warp streams the chunks of its slices through a private ring in shared memory with
// per-thread asynchronous 16-byte copies (cp.async, L2 evict-first): lane l copies bytes [16l, 16l+16)
// and [512+16l, ...) of a chunk and later reads back exactly those bytes, so the only synchronisation
// of the stream is the thread's own cp.async.wait_group -- no barrier, no producer, no handshake.  The
// ring runs DEPTH chunks ahead and crosses unit boundaries.  One CTA of 16 warps per SM; the rings (128 KB)
// keep a second CTA off the SM on purpose: when the CTAs of consecutive kernels shared SMs, the hardware
// placed them unevenly and the slowest SM set the pace.
//
// Work distribution.  Unit u belongs to CTA u mod gridDim; inside the CTA the warp groups take the
// CTA's units from a shared counter, one unit ahead of use (a warp's slice is at least as long as its
// ring, so its requests never reach beyond the next unit), so a group that falls behind takes fewer units.
//
// Compute side.  A chunk of a unit is the A operand of 8 int8 tensor-core MMAs (mma.sync m16n8k32,
// u8 x s8 -> s32): lane (g = lane/4, t = lane%4) holds 64 weights of row g and of row g+8.  Masking a
// packed word with 0x03030303 << 2s leaves, without a shift, the four codes of slot s scaled by 4^s:
// one A register.  The B operand is the activations (column n = token n), read from shared memory by
// the lanes of real tokens only (columns of D beyond the batch are never stored, and a load by a few
// lanes costs the shared-memory pipe a fraction of a full-warp load).  Four accumulator fragments carry
// the scales 1, 4, 16, 64; each is an exact multiple of its scale, so arithmetic shifts undo it, and
// sum(code*q) - sum(q) = sum(w*q).  The S partial fragments of a unit meet in shared memory at a named
// barrier of the group; one warp (rotating) adds them, rescales and stores y = acc * act_scale[t] * w_scale.
//
// Kernel chain.  Under programmatic dependent launch the CTA starts as soon as its SM is free, requests
// its first weights -- which depend on nothing -- and only then waits for the previous kernel
// (griddepcontrol.wait) before it touches activations.
//
// Fused quantiser: with fp32 activations given, every CTA computes absmax and the int8 codes itself,
// while its first weight copies are in flight; CTA 0 also stores the codes and scales for the caller.
#include <cstdlib>
#include <cstring>

#include "common.cuh"
#include "device_utils.cuh"

namespace bitnet {
namespace {

constexpr int CW = 16;                   // warps
constexpr int THREADS = CW * 32;
constexpr int JQ = 4;                    // entries of a group's queue of upcoming units
constexpr int XREG_MAX = 16;                 // float4 registers per thread of the fused quantiser's fast path
constexpr size_t MAX_QS_BYTES = 144 * 1024;   // activations staged in shared memory up to this size


struct WArgs {
  const uint8_t* packed;
  int64_t unit_bytes;    // bytes of one 16-row unit of the blob = 4 * Kp
  int M;
  int64_t K;
  const int8_t* q;       // quantised activations [T][K] (input, or output of the fused quantiser)
  const float* act_scale;
  const float* x;        // fp32 activations [T][K]: non-null selects the fused quantiser
  int8_t* q_out;         // fused mode: CTA 0 stores the codes and scales here
  float* scale_out;
  float w_scale;
  int T;
  float* y;
  int32_t* acc_out;
  int nchunks;           // 256-column chunks per row (Kp / 256)
  int S;                 // warps per unit
  int KC;                // chunks per warp and unit (the last warp of a unit may have fewer, or none)
  int nunits;            // ceil(M / 16)
  int pre;               // ring slots requested before waiting for the previous kernel
};

// shared memory: [unit counter, unit queues, quantiser scratch: 2 KB][partials][codes][rings]
__host__ __device__ inline size_t red_bytes(int T) { return (size_t)CW * 2 * T * 16 * 4; }

// XREG: float4 registers per thread of the fused quantiser's fast path (rows of THREADS float4 of x)
template <int DEPTH, int XREG>
__global__ void __launch_bounds__(THREADS, 1) gemv_i2s_wring_kernel(const WArgs a) {
  extern __shared__ __align__(128) uint8_t smem[];
  int* counter = reinterpret_cast<int*>(smem);                 // next unit (index into the CTA's list) to hand out
  int* jq = reinterpret_cast<int*>(smem + 64);                 // [groups][JQ] upcoming units of each group
  float* qscale = reinterpret_cast<float*>(smem + 1152);       // [8] act_scale per token
  float* qred = qscale + 8;                                    // [8][16] partial maxima / multipliers
  int* red = reinterpret_cast<int*>(smem + 2048);              // [CW][2][T][16] partial sums
  const int kp = a.nchunks * 256;
  int8_t* qs_mem = reinterpret_cast<int8_t*>(smem + 2048 + red_bytes(a.T));
  // Token rows are kp + 64 bytes apart and the 16-byte pieces of a chunk are kept [piece][lane quarter]
  // (staged_word): the B loads of one MMA pair -- the four lane quarters of every token at the same piece -- then
  // cover the 32 shared-memory banks exactly once per eight lanes.
  const int qst = kp + 64;
  uint8_t* rings = reinterpret_cast<uint8_t*>(qs_mem) + (((size_t)a.T * qst + 127) & ~(size_t)127);

  const int lane = threadIdx.x & 31;
  const int warp = threadIdx.x >> 5;
  const int G = CW / a.S;                      // groups
  const int gi = warp / a.S;                   // this warp's group
  const int wk = warp % a.S;                   // its place in the group = its K-slice
  const int g = lane >> 2, t = lane & 3;
  const int n_units = (a.nunits - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;
  const int c_lo = wk * a.nchunks / a.S, c_hi = (wk + 1) * a.nchunks / a.S;   // this warp's K-slice, >= DEPTH chunks

  if (threadIdx.x == 0) {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the next kernel may become resident
    *counter = 2 * G;
  }
  // the first two units of each group are fixed: unit i of group gi is gi + i * G
  if (threadIdx.x < G * JQ) {
    const int i = threadIdx.x % JQ;
    jq[threadIdx.x] = (i <= 1) ? (threadIdx.x / JQ) + i * G : 0x7fffffff;
  }
  __syncthreads();

  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));

  // ---------------- the warp's stream of chunks: its slice of the group's unit 0, of unit 1, ...
  // The ring holds DEPTH consecutive chunks of that stream; slot_off is the slot of the chunk consumed next.
  const uint32_t ring = smem_u32(rings + (size_t)warp * DEPTH * 1024) + lane * 16;
  const uint8_t* const base = a.packed + (int64_t)blockIdx.x * a.unit_bytes + (int64_t)c_lo * 1024 + lane * 16;
  const int64_t unit_stride = (int64_t)gridDim.x * a.unit_bytes;
  const volatile int* my_jq = jq + gi * JQ;
  const int nw = c_hi - c_lo;
  uint32_t slot_off = 0;
  // Weights do not depend on the previous kernel in the stream: request the first chunks now.  Only a.pre
  // of the DEPTH chunks: the activation loads that follow the wait below queue behind whatever is in flight,
  // and everything after them waits for the activations.  The rest of the ring is requested right after them.
  const int j0 = my_jq[0];
  const uint8_t* const src0 = base + (int64_t)j0 * unit_stride;
  auto first_fill = [&](bool before_wait) {
#pragma unroll
    for (int d = 0; d < DEPTH; ++d) {
      if ((d < a.pre) == before_wait) {
        if (j0 < n_units) {
          cp16(ring + d * 1024, src0 + d * 1024, pol);
          cp16(ring + d * 1024 + 512, src0 + d * 1024 + 512, pol);
        }
        cp_commit();
      }
    }
  };
  first_fill(true);

  // ---------------- activations come from the previous kernel in the stream
  asm volatile("griddepcontrol.wait;" ::: "memory");

  if (a.x && a.K <= 4 * XREG * THREADS) {
    // ---- fused quantiser (Alg. 1 Phase 1), one round trip per token: the row stays in registers
    // between the amax pass and the rounding pass.  Same operations and order as the stand-alone
    // kernel: s = 127 / max(amax, 1e-5), q = clamp(rint(x * s)).
    const int n4 = (int)(a.K / 4);
    const int nrow = (max(n4, kp / 4) + THREADS - 1) / THREADS;     // rows of THREADS words that hold anything
    // With few registers per row (the short-row instance) the next token's row is requested before this
    // token's is reduced, so the tokens' round trips overlap.
    constexpr bool AHEAD = XREG <= 8;
    float4 xv[XREG], xn[AHEAD ? XREG : 1];
    auto load_row = [&](float4* dst, int tok) {
      const float4* x4 = reinterpret_cast<const float4*>(a.x + (int64_t)tok * a.K);
#pragma unroll
      for (int r = 0; r < XREG; ++r) {
        const int i = threadIdx.x + r * THREADS;
        dst[r] = (r < nrow && i < n4) ? __ldcg(x4 + i) : make_float4(0.f, 0.f, 0.f, 0.f);
      }
    };
    if (AHEAD) load_row(xv, 0);
    for (int tok = 0; tok < a.T; ++tok) {
      if (AHEAD) {
        if (tok + 1 < a.T) load_row(xn, tok + 1);
      } else {
        load_row(xv, tok);
      }
      if (tok == 0) first_fill(false);
      float m = 0.0f;
#pragma unroll
      for (int r = 0; r < XREG; ++r)
        if (r < nrow) m = fmaxf(m, fmaxf(fmaxf(fabsf(xv[r].x), fabsf(xv[r].y)), fmaxf(fabsf(xv[r].z), fabsf(xv[r].w))));
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
      if (tok > 0) __syncthreads();          // everyone has read the previous token's partial maxima
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
        if (blockIdx.x == 0 && a.scale_out) a.scale_out[tok] = inv;
      }
#pragma unroll
      for (int r = 0; r < XREG; ++r) {
        const int i = threadIdx.x + r * THREADS;
        if (r < nrow && i < kp / 4) {
          const int word = quant4_packed(xv[r], sq);          // columns K..Kp-1 came in as zeros
          reinterpret_cast<int*>(qs_mem + tok * qst)[staged_word(i)] = word;
          if (blockIdx.x == 0 && a.q_out && i < n4) reinterpret_cast<int*>(a.q_out + (int64_t)tok * a.K)[i] = word;
        }
      }
      if (AHEAD) {
#pragma unroll
        for (int r = 0; r < XREG; ++r) xv[r] = xn[r];
      }
    }
  } else if (a.x) {
    // ---- fused quantiser, general form: amax per token, then a second pass over x
    first_fill(false);
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
        reinterpret_cast<int*>(qs_mem + tok * qst)[staged_word(i)] = word;
      }
    }
  } else {
    // ---- stage the given codes (zero beyond K); the first QREG words per thread are loaded before the
    // rest of the ring is requested
    constexpr int QREG = 8;
    const int nq4 = (int)(a.K / 4), total4 = a.T * (kp / 4);     // words per token, words to stage
    int qv[QREG];
#pragma unroll
    for (int r = 0; r < QREG; ++r) {
      const int i = threadIdx.x + r * THREADS, tok = i / (kp / 4), col = i - tok * (kp / 4);
      qv[r] = (i < total4 && col < nq4) ? __ldcg(reinterpret_cast<const int*>(a.q + (int64_t)tok * a.K) + col) : 0;
    }
    const float my_scale = (threadIdx.x < a.T) ? __ldcg(a.act_scale + threadIdx.x) : 0.0f;
    first_fill(false);
#pragma unroll
    for (int r = 0; r < QREG; ++r) {
      const int i = threadIdx.x + r * THREADS;
      if (i < total4) reinterpret_cast<int*>(qs_mem + (i / (kp / 4)) * qst)[staged_word(i % (kp / 4))] = qv[r];
    }
    for (int i = threadIdx.x + QREG * THREADS; i < total4; i += THREADS) {
      const int tok = i / (kp / 4), col = i - tok * (kp / 4);
      reinterpret_cast<int*>(qs_mem + tok * qst)[staged_word(col)] = (col < nq4) ? __ldcg(reinterpret_cast<const int*>(a.q + (int64_t)tok * a.K) + col) : 0;
    }
    if (threadIdx.x < a.T) qscale[threadIdx.x] = my_scale;
  }
  __syncthreads();

  // sum of the activations of tokens 2t and 2t+1 over this warp's K-slice (the "- sum(q)" term)
  int corr_even = 0, corr_odd = 0;
  for (int tok = 0; tok < a.T; ++tok) {
    int s = 0, s2 = 0;
    const uint4* qw = reinterpret_cast<const uint4*>(qs_mem + tok * qst + c_lo * 256);
#pragma unroll 4
    for (int i = lane; i < (c_hi - c_lo) * 16; i += 32) {
      const uint4 v = qw[i];
      s = __dp4a((int)v.x, 0x01010101, s);
      s2 = __dp4a((int)v.y, 0x01010101, s2);
      s = __dp4a((int)v.z, 0x01010101, s);
      s2 = __dp4a((int)v.w, 0x01010101, s2);
    }
    s += s2;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (tok == 2 * t) corr_even = s;
    if (tok == 2 * t + 1) corr_odd = s;
  }
  // token g's codes under this lane's 16-byte weight column: 64 bytes per chunk
  const unsigned has_tok = g < a.T ? 1u : 0u;
  const uint32_t q_lane = smem_u32(qs_mem + min(g, a.T - 1) * qst + c_lo * 256 + t * 16);
  const int bar_id = 1 + gi, bar_threads = a.S * 32;

  // One step: wait for the oldest chunk of the ring, put it through the tensor cores, then refill its slot
  // from `pf` (the chunk DEPTH places further down the stream), if there is one.
  int C[4][4];
  uint32_t qp = 0;                 // shared-memory address of the lane's 64 codes of the current chunk
  int qr[8] = {0, 0, 0, 0, 0, 0, 0, 0};   // B registers; lanes beyond the batch keep these zeros
  auto step = [&](const uint8_t* pf, bool do_pf) {
    cp_wait<DEPTH - 1>();
    unsigned w4[4], v4[4];
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(w4[0]), "=r"(w4[1]), "=r"(w4[2]), "=r"(w4[3])
                 : "r"(ring + slot_off));
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v4[0]), "=r"(v4[1]), "=r"(v4[2]), "=r"(v4[3])
                 : "r"(ring + slot_off + 512));
    // words 2h, 2h+1 of the lane's 16 bytes, slot s: weights 32h + 8s + (0..7) of its 64 columns,
    // i.e. activation words 8h + 2s and 8h + 2s + 1
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      // only the lanes whose B column is a real token load (a load by a few lanes costs the shared-memory
      // pipe a fraction of a full-warp load); the other columns of D are never stored
      asm volatile(
          "{\n\t.reg .pred p;\n\tsetp.ne.u32 p, %9, 0;\n\t"
          "@p ld.shared.v4.u32 {%0,%1,%2,%3}, [%8];\n\t"
          "@p ld.shared.v4.u32 {%4,%5,%6,%7}, [%8+64];\n\t}"
          : "+r"(qr[0]), "+r"(qr[1]), "+r"(qr[2]), "+r"(qr[3]), "+r"(qr[4]), "+r"(qr[5]), "+r"(qr[6]), "+r"(qr[7])
          : "r"(qp + h * 128), "r"(has_tok));
#pragma unroll
      for (int s = 0; s < 4; ++s) {
        const unsigned m = 0x03030303u << (2 * s);
        mma_u8s8(C[s], w4[2 * h] & m, v4[2 * h] & m, w4[2 * h + 1] & m, v4[2 * h + 1] & m, qr[2 * s], qr[2 * s + 1]);
      }
    }
    qp += 256;
    // the chunk's bytes were in registers before the MMAs above were issued: its slot can be refilled
    if (do_pf) {
      cp16(ring + slot_off, pf, pol);
      cp16(ring + slot_off + 512, pf + 512, pol);
    }
    cp_commit();
    slot_off = (slot_off + 1024 == DEPTH * 1024) ? 0 : slot_off + 1024;
  };

  for (int n = 0;; ++n) {
    const int j = my_jq[n & (JQ - 1)];
    if (j >= n_units) break;
    const int jn = my_jq[(n + 1) & (JQ - 1)];
    // The group's first warp draws the unit after the next; the barrier at the end of this unit publishes
    // it before anyone looks for it.  (A warp's slice is at least as long as its ring, so its requests
    // never reach beyond the next unit.)
    if (wk == 0 && lane == 0) jq[gi * JQ + ((n + 2) & (JQ - 1))] = atomicAdd(counter, 1);

#pragma unroll
    for (int s = 0; s < 4; ++s)
#pragma unroll
      for (int i = 0; i < 4; ++i) C[s][i] = 0;
    qp = q_lane;

    // chunks 0 .. nw-DEPTH-1 are followed, DEPTH places on, by chunks of the same unit
    const uint8_t* pf = base + (int64_t)j * unit_stride + DEPTH * 1024;
#pragma unroll 2
    for (int left = nw - DEPTH; left > 0; --left, pf += 1024) { step(pf, true); }
    // the last DEPTH chunks by the first DEPTH chunks of the group's next unit, if there is one
    pf = base + (int64_t)jn * unit_stride;
    const bool more = jn < n_units;
#pragma unroll
    for (int d = 0; d < DEPTH; ++d) { step(pf + d * 1024, more); }

    // fragment: c[0] = (row g, token 2t), c[1] = (row g, token 2t+1), c[2], c[3] = the same for row g+8
    int c[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) c[i] = C[0][i] + (C[1][i] >> 2) + (C[2][i] >> 4) + (C[3][i] >> 6);
    int* mine = red + ((warp * 2 + (n & 1)) * a.T) * 16;
    if (2 * t < a.T) {
      mine[(2 * t) * 16 + g] = c[0] - corr_even;
      mine[(2 * t) * 16 + g + 8] = c[2] - corr_even;
    }
    if (2 * t + 1 < a.T) {
      mine[(2 * t + 1) * 16 + g] = c[1] - corr_odd;
      mine[(2 * t + 1) * 16 + g + 8] = c[3] - corr_odd;
    }
    if (a.S > 1) group_barrier(bar_id, bar_threads);
    else __syncwarp();
    if (wk == (n & (a.S - 1))) {
      // this unit's turn to be finished by this warp: add the group's partials, rescale, store 16 rows
      const int row0 = ((int)blockIdx.x + j * (int)gridDim.x) * 16;
      const int* grp = red + (((gi * a.S) * 2 + (n & 1)) * a.T) * 16;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int idx = lane + 32 * i;
        if (idx < a.T * 16) {
          int v = 0;
          for (int w2 = 0; w2 < a.S; ++w2) v += grp[w2 * 2 * a.T * 16 + idx];
          const int tok = idx >> 4, row = row0 + (idx & 15);
          if (row < a.M) {
            a.y[(int64_t)tok * a.M + row] = __fmul_rn((float)v, __fmul_rn(qscale[tok], a.w_scale));
            if (a.acc_out) a.acc_out[(int64_t)tok * a.M + row] = v;
          }
        }
      }
    }
  }
  cp_wait<0>();
}

struct Plan {
  int nchunks, S, KC, nunits, grid, depth;
  size_t smem;
};

// Tuning overrides from the environment, read once per process (never on the launch path again).
struct Tuning {
  int depth, kc, ctas, pre;
};
const Tuning& tuning() {
  static const Tuning t = [] {
    auto env_int = [](const char* name, int dflt) {
      const char* v = getenv(name);
      return (v && *v) ? atoi(v) : dflt;
    };
    return Tuning{env_int("BITNET_I2S_DEPTH", 0), env_int("BITNET_I2S_KC", 8), env_int("BITNET_I2S_CTAS", 1),
                  env_int("BITNET_I2S_PRE", 4)};
  }();
  return t;
}

bool make_plan(int T, int64_t M, int64_t K, Plan* p) {
  p->nchunks = (int)(i2s_kp(K) / 256);
  const int forced = tuning().depth;
  int depth = (forced == 12 || forced == 8 || forced == 6 || forced == 4) ? forced : 8;
  while (depth > 4 && 2048 + red_bytes(T) + (((size_t)T * (p->nchunks * 256 + 64) + 127) & ~(size_t)127) +
                              (size_t)CW * depth * 1024 > (size_t)dev_info().max_smem_optin)
    depth -= 2;
  if (depth == 10) depth = 8;
  if (p->nchunks < depth) return false;     // a warp's slice is at least as long as the ring
  // warps per unit: as many as leave every warp about kc_target chunks of a unit (never fewer than the ring)
  int kc_target = tuning().kc;
  if (kc_target < depth) kc_target = depth;
  int S = 1;
  while (S < CW && p->nchunks / (2 * S) >= kc_target) S *= 2;
  p->S = S;
  p->KC = (p->nchunks + S - 1) / S;
  p->nunits = (int)ceil_div(M, 16);
  const int ctas = dev_info().sm_count * tuning().ctas;
  p->grid = ctas < p->nunits ? ctas : p->nunits;
  const size_t qs_bytes = ((size_t)T * (p->nchunks * 256 + 64) + 127) & ~(size_t)127;
  if (qs_bytes > MAX_QS_BYTES) return false;
  p->depth = depth;
  p->smem = 2048 + red_bytes(T) + qs_bytes + (size_t)CW * depth * 1024;
  return p->smem <= (size_t)dev_info().max_smem_optin;
}

template <int DEPTH, int XREG>
int launch_wring(const WArgs& a, const Plan& p, cudaStream_t st) {
  static bool attr_set[64] = {false};
  int dev = 0;
  cudaGetDevice(&dev);
  if (!attr_set[dev & 63]) {
    cudaError_t e = cudaFuncSetAttribute(gemv_i2s_wring_kernel<DEPTH, XREG>, cudaFuncAttributeMaxDynamicSharedMemorySize,
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
  cudaError_t e = cudaLaunchKernelEx(&cfg, gemv_i2s_wring_kernel<DEPTH, XREG>, a);
  return e == cudaSuccess ? BITNET_OK : note_cuda_error(e);
}

}  // namespace

bool gemv_i2s_wring_supported(int T, int64_t M, int64_t K) {
  Plan p;
  return T >= 1 && T <= 8 && make_plan(T, M, K, &p);
}

// x != nullptr: fused quantiser (q, act_scale are then outputs); otherwise q, act_scale are inputs.
int launch_gemv_i2s_wring(const uint8_t* packed, float w_scale, int64_t M, int64_t K, const float* x, int8_t* q,
                          float* act_scale, int T, float* y, int32_t* acc_out, cudaStream_t st) {
  Plan p;
  if (T < 1 || T > 8 || !make_plan(T, M, K, &p)) return BITNET_ERR_UNSUPPORTED_SHAPE;
  WArgs a;
  a.packed = packed;
  a.unit_bytes = 4 * i2s_kp(K);
  a.M = (int)M;
  a.K = K;
  a.q = q;
  a.act_scale = act_scale;
  a.x = x;
  a.q_out = x ? q : nullptr;
  a.scale_out = x ? act_scale : nullptr;
  a.w_scale = w_scale;
  a.T = T;
  a.y = y;
  a.acc_out = acc_out;
  a.nchunks = p.nchunks;
  a.S = p.S;
  a.KC = p.KC;
  a.nunits = p.nunits;
  a.pre = tuning().pre;
  // short rows get the instance whose (fully unrolled) quantiser prologue is a quarter of the code
  log_launch("gemv_i2s_wring_kernel%s T=%d M=%lld K=%lld grid=%d warps/unit=%d ring=%d smem=%zu", x ? " (fused quantiser)" : "",
             T, (long long)M, (long long)K, p.grid, p.S, p.depth, p.smem);
  const bool small_x = x != nullptr && K <= 4 * 4 * THREADS;
  switch (p.depth) {
    case 4: return launch_wring<4, XREG_MAX>(a, p, st);
    case 6: return launch_wring<6, XREG_MAX>(a, p, st);
    case 12: return launch_wring<12, XREG_MAX>(a, p, st);
    case 8: return small_x ? launch_wring<8, 4>(a, p, st) : launch_wring<8, XREG_MAX>(a, p, st);
    default: return BITNET_ERR_UNSUPPORTED_SHAPE;
  }
}


}  // namespace bitnet
