// I2_S mpGEMV for decode (1..8 tokens): Alg. 1 Phase 2 evaluated from the 2-bit blob.
//
//   acc[t,m] = sum_k q[t,k] * w[m,k],   w = code - 1,  code in {0,1,2} two bits each
//            = sum_k q[t,k] * code[m,k]  -  sum_k q[t,k]
//
// Split-K fallback for shapes the streaming kernel does not cover (see gemv_i2s_mma.cu).
// Mapping.  A warp owns a row (for a K-slice of J*2048 weights): lane l loads J 16-byte vectors of
// the row (vector index slice*J*32 + j*32 + l, 64 weights each).
// The lane's activations for those weights never change from row to row, so they live in registers
// (TT tokens x J x 16 words).  A packed 32-bit word holds 16 codes; the four masks 0x03030303 << 2s
// pick, WITHOUT shifting, the four codes of slot s scaled by 4^s, and one dp4a.u32.s32 multiplies
// them with the matching activation word.  Four accumulators carry the scales
// 1, 4, 16, 64; each is an exact multiple of its scale, so arithmetic shifts undo it.  That is one
// logic op and one dp4a per four weights.  Lane partials are summed by warp shuffles.
//
// K longer than one slice is split over blockIdx.y; partial sums meet in an int32 workspace by
// atomicAdd (exact and order independent), and the slice that arrives last at a row's ticket
// converts, stores and re-zeroes that row -- no waiting anywhere.
#include <cstdlib>
#include <cstring>

#include "common.cuh"

namespace bitnet {
namespace {

constexpr int WARPS = 8;
constexpr int THREADS = WARPS * 32;

__device__ __forceinline__ int dp4a_us(unsigned a, int b, int c) {
  int d;
  asm("dp4a.u32.s32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
  return d;
}
__device__ __forceinline__ int dp4a_ss(int a, int b, int c) {
  int d;
  asm("dp4a.s32.s32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
  return d;
}
__device__ __forceinline__ uint4 ldg_stream(const uint4* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}

struct GemvArgs {
  const uint8_t* packed; // blob
  int64_t kp;            // K padded to 256 (blob geometry)
  int data_vecs;         // K / 64: vectors per row that carry weights
  int M;
  int64_t K;
  const int8_t* q;       // first token of this pass
  const float* act_scale;
  float w_scale;
  int nt;                // tokens in this pass (<= TT)
  float* y;              // first token of this pass
  int32_t* acc_out;      // nullable
  int32_t* ws_acc;       // [T][M] partial sums (split-K only), first token of this pass
  unsigned* ws_ticket;   // [M]
  int nslices;
};

// 16-byte vector v of a row = its weights [64v, 64v+64): piece v%4 of chunk v/4.
__device__ __forceinline__ const uint4* vec_ptr(const GemvArgs& a, int row, int v) {
  return reinterpret_cast<const uint4*>(a.packed + i2s_row_chunk_offset(row, v >> 2, a.kp) + (v & 3) * 16);
}

template <int TT, int J>
__global__ void __launch_bounds__(THREADS, 2) gemv_i2s_kernel(const GemvArgs a) {
  const int lane = threadIdx.x & 31;
  const int warp = threadIdx.x >> 5;
  const int slice = blockIdx.y;
  const int gw = blockIdx.x * WARPS + warp;
  const int gws = gridDim.x * WARPS;

  // this lane's vectors and activations
  int vec[J];
  bool ok[J];
  int qr[TT][J][16];
  int qsum[TT];
#pragma unroll
  for (int t = 0; t < TT; ++t) qsum[t] = 0;
#pragma unroll
  for (int j = 0; j < J; ++j) {
    vec[j] = (slice * J + j) * 32 + lane;
    ok[j] = vec[j] < a.data_vecs;
#pragma unroll
    for (int t = 0; t < TT; ++t) {
      if (ok[j] && t < a.nt) {
        const uint4* qp = reinterpret_cast<const uint4*>(a.q + (int64_t)t * a.K + (int64_t)vec[j] * 64);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const uint4 v = __ldg(qp + i);
          qr[t][j][4 * i + 0] = (int)v.x;
          qr[t][j][4 * i + 1] = (int)v.y;
          qr[t][j][4 * i + 2] = (int)v.z;
          qr[t][j][4 * i + 3] = (int)v.w;
        }
      } else {
#pragma unroll
        for (int i = 0; i < 16; ++i) qr[t][j][i] = 0;
      }
#pragma unroll
      for (int i = 0; i < 16; ++i) qsum[t] = dp4a_ss(qr[t][j][i], 0x01010101, qsum[t]);
    }
  }

  float sc[TT];
#pragma unroll
  for (int t = 0; t < TT; ++t) sc[t] = (t < a.nt) ? __fmul_rn(a.act_scale[t], a.w_scale) : 0.0f;

  int row = gw;
  uint4 cur[J], nxt[J];
#pragma unroll
  for (int j = 0; j < J; ++j) {
    cur[j] = make_uint4(0, 0, 0, 0);
    if (row < a.M && ok[j]) cur[j] = ldg_stream(vec_ptr(a, row, vec[j]));
  }
  for (; row < a.M; row += gws) {
    const int nrow = row + gws;
#pragma unroll
    for (int j = 0; j < J; ++j) {
      nxt[j] = make_uint4(0, 0, 0, 0);
      if (nrow < a.M && ok[j]) nxt[j] = ldg_stream(vec_ptr(a, nrow, vec[j]));
    }
    int acc[TT][4];
#pragma unroll
    for (int t = 0; t < TT; ++t) {
      acc[t][0] = -qsum[t];
      acc[t][1] = acc[t][2] = acc[t][3] = 0;
    }
#pragma unroll
    for (int j = 0; j < J; ++j) {
      const unsigned wv[4] = {cur[j].x, cur[j].y, cur[j].z, cur[j].w};
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const unsigned m0 = wv[c] & 0x03030303u, m1 = wv[c] & 0x0C0C0C0Cu;
        const unsigned m2 = wv[c] & 0x30303030u, m3 = wv[c] & 0xC0C0C0C0u;
#pragma unroll
        for (int t = 0; t < TT; ++t) {
          // word c of the piece, slot s multiplies activation word 8*(c/2) + 2*s + (c%2)
          acc[t][0] = dp4a_us(m0, qr[t][j][8 * (c / 2) + 0 + (c % 2)], acc[t][0]);
          acc[t][1] = dp4a_us(m1, qr[t][j][8 * (c / 2) + 2 + (c % 2)], acc[t][1]);
          acc[t][2] = dp4a_us(m2, qr[t][j][8 * (c / 2) + 4 + (c % 2)], acc[t][2]);
          acc[t][3] = dp4a_us(m3, qr[t][j][8 * (c / 2) + 6 + (c % 2)], acc[t][3]);
        }
      }
    }
    int tot[TT];
#pragma unroll
    for (int t = 0; t < TT; ++t) {
      int v = acc[t][0] + (acc[t][1] >> 2) + (acc[t][2] >> 4) + (acc[t][3] >> 6);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
      tot[t] = v;
    }
    if (lane == 0) {
      if (a.nslices == 1) {
#pragma unroll
        for (int t = 0; t < TT; ++t) {
          if (t < a.nt) {
            a.y[(int64_t)t * a.M + row] = __fmul_rn((float)tot[t], sc[t]);
            if (a.acc_out) a.acc_out[(int64_t)t * a.M + row] = tot[t];
          }
        }
      } else {
#pragma unroll
        for (int t = 0; t < TT; ++t)
          if (t < a.nt) atomicAdd(a.ws_acc + (int64_t)t * a.M + row, tot[t]);
        __threadfence();
        const unsigned old = atomicAdd(a.ws_ticket + row, 1u);
        if (old == (unsigned)(a.nslices - 1)) {
          __threadfence();
#pragma unroll
          for (int t = 0; t < TT; ++t) {
            if (t < a.nt) {
              const int v = atomicExch(a.ws_acc + (int64_t)t * a.M + row, 0);
              a.y[(int64_t)t * a.M + row] = __fmul_rn((float)v, sc[t]);
              if (a.acc_out) a.acc_out[(int64_t)t * a.M + row] = v;
            }
          }
          atomicExch(a.ws_ticket + row, 0u);
        }
      }
    }
#pragma unroll
    for (int j = 0; j < J; ++j) cur[j] = nxt[j];
  }
}

inline int slices_for(int64_t K, int J) { return (int)ceil_div(K / 64, (int64_t)J * 32); }

// tokens per pass and vectors per lane for a given batch
inline void pick(int T, int* TT, int* J) {
  if (T == 1) { *TT = 1; *J = 4; }
  else if (T == 2) { *TT = 2; *J = 2; }
  else { *TT = 4; *J = 1; }
}

template <int TT, int J>
int launch_one(GemvArgs a, cudaStream_t st) {
  const int sms = dev_info().sm_count;
  int gx = (2 * sms + a.nslices - 1) / a.nslices;
  const int need = (a.M + WARPS - 1) / WARPS;
  if (gx > need) gx = need;
  if (gx < 1) gx = 1;
  dim3 grid((unsigned)gx, (unsigned)a.nslices);
  gemv_i2s_kernel<TT, J><<<grid, THREADS, 0, st>>>(a);
  return check_launch();
}

}  // namespace

static bool use_stream_kernel(int64_t T, int64_t M, int64_t K) {
  static const bool forced_splitk = [] {
    const char* e = getenv("BITNET_I2S_KERNEL");
    return e && strcmp(e, "splitk") == 0;
  }();
  return !forced_splitk && gemv_i2s_stream_supported((int)T, M, K, false);
}

size_t gemv_i2s_workspace_bytes(int64_t T, int64_t M, int64_t K) {
  if (use_stream_kernel(T > 8 ? 8 : T, M, K)) return 0;
  int TT, J;
  pick((int)(T > 8 ? 8 : T), &TT, &J);
  if (slices_for(K, J) == 1) return 0;
  const int64_t Tc = T > 8 ? 8 : T;
  return (size_t)(Tc * M * 4 + M * 4);
}

int launch_gemv_i2s(const uint8_t* packed, float w_scale, int64_t M, int64_t K, const int8_t* q,
                    const float* act_scale, int T, float* y, int32_t* acc_out, void* ws, size_t ws_bytes,
                    cudaStream_t st) {
  if (use_stream_kernel(T, M, K))
    return launch_gemv_i2s_stream(packed, w_scale, M, K, nullptr, const_cast<int8_t*>(q), const_cast<float*>(act_scale), T, y,
                                  acc_out, st);
  int TT, J;
  pick(T, &TT, &J);
  GemvArgs a;
  a.packed = packed;
  a.kp = i2s_kp(K);
  a.data_vecs = (int)(K / 64);
  a.M = (int)M;
  a.K = K;
  a.w_scale = w_scale;
  a.nslices = slices_for(K, J);
  if (a.nslices > 1) {
    if (!ws || ws_bytes < gemv_i2s_workspace_bytes(T, M, K)) return BITNET_ERR_WORKSPACE;
  }
  a.ws_ticket = (a.nslices > 1) ? reinterpret_cast<unsigned*>(reinterpret_cast<int32_t*>(ws) + (int64_t)T * M) : nullptr;
  for (int t0 = 0; t0 < T; t0 += TT) {
    a.q = q + (int64_t)t0 * K;
    a.act_scale = act_scale + t0;
    a.nt = (T - t0 < TT) ? (T - t0) : TT;
    a.y = y + (int64_t)t0 * M;
    a.acc_out = acc_out ? acc_out + (int64_t)t0 * M : nullptr;
    a.ws_acc = (a.nslices > 1) ? reinterpret_cast<int32_t*>(ws) + (int64_t)t0 * M : nullptr;
    int rc;
    if (TT == 1) rc = launch_one<1, 4>(a, st);
    else if (TT == 2) rc = launch_one<2, 2>(a, st);
    else rc = launch_one<4, 1>(a, st);
    if (rc != BITNET_OK) return rc;
  }
  return BITNET_OK;
}

}  // namespace bitnet
