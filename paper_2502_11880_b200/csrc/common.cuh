// Shared host/device helpers of the bitnet_b200 library (internal).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "bitnet_b200.h"

namespace bitnet {

inline __host__ __device__ int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }

// Geometry of a TL blob (Sec. 3.1.2: block-fitting split ThreeK / TwoK; 32-row tiles).
struct TlGeom {
  int64_t three_k;      // columns coded as triples (TL2)
  int64_t two_k;        // columns coded as pairs (TL1)
  int64_t tiles3;       // 640-byte tiles per 32-row block
  int64_t tiles2;       // 512-byte tiles per 32-row block
  int64_t block_bytes;  // bytes per 32-row block
};

inline __host__ bool tl_geom(int fmt, int64_t M, int64_t K, int bk3, TlGeom* g) {
  if (M <= 0 || K <= 0 || (M % 32) != 0 || (K % 2) != 0) return false;
  if (bk3 == 0) bk3 = 96;
  if (bk3 < 0 || (bk3 % 96) != 0) return false;
  if (fmt == BITNET_FMT_TL2) {
    g->three_k = (K / bk3) * bk3;
    g->two_k = K - g->three_k;
  } else if (fmt == BITNET_FMT_TL1) {
    g->three_k = 0;
    g->two_k = K;
  } else {
    return false;
  }
  g->tiles3 = g->three_k / 96;
  g->tiles2 = ceil_div(g->two_k, 64);
  g->block_bytes = g->tiles3 * 640 + g->tiles2 * 512;
  return true;
}

// Positions inside a TL tile.  Row r = g + 8u of the 32-row block (g = r % 8, u = r / 8) has 16 index bytes (byte i:
// group 2i in the low nibble, 2i+1 in the high nibble), i.e. four 32-bit words.  Word t of row r lies at
// 64g + 16t + 4u: every 16-byte piece of the index plane holds word t of the rows g, g+8, g+16, g+24 -- the four
// rows a lane of an m16n8k32 MMA owns in the two 16-row halves of the block.  A triple tile's sign plane keeps row
// r's uint32 at 512 + 16g + 4u; the sign of group grp (index byte i = grp/2) is bit 8(i%4) + 2(i/4) + grp%2, so
// that (signs >> 2t) & 0x03030303 lines the sign pairs of word t's four bytes up with those bytes.
inline __host__ __device__ int tl_word_off(int r, int t) { return 64 * (r & 7) + 16 * t + 4 * (r >> 3); }
inline __host__ __device__ int tl_sign_off(int r) { return 512 + 16 * (r & 7) + 4 * (r >> 3); }
inline __host__ __device__ int tl_sign_bit(int grp) { return 8 * ((grp >> 1) & 3) + 2 * (grp >> 3) + (grp & 1); }

// Geometry of an I2_S blob: rows in blocks of 16, K padded to 256; a block is contiguous and holds
// one 1024-byte piece per 256-column chunk, row r of the block owning bytes [64r, 64r+64) of it.
// Word j (0..15) of those 64 bytes, slot s (bits [8b+2s, 8b+2s+1] of byte b) holds the weights
// kk = 32*(j/2) + 8*s + 4*(j%2) + b of the chunk, i.e. the activation word 8*(j/2) + 2*s + (j%2).
inline __host__ __device__ int64_t i2s_kp(int64_t K) { return ceil_div(K, 256) * 256; }
inline __host__ __device__ int64_t i2s_mp(int64_t M) { return ceil_div(M, 16) * 16; }
inline __host__ __device__ int64_t i2s_row_chunk_offset(int64_t m, int64_t chunk, int64_t kp) {
  return (m >> 4) * (4 * kp) + chunk * 1024 + (m & 15) * 64;
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Records a failing CUDA call for bitnet_last_cuda_error(); returns the library status.
int note_cuda_error(cudaError_t e);
inline int check_launch() {
  cudaError_t e = cudaPeekAtLastError();
  return e == cudaSuccess ? BITNET_OK : note_cuda_error(cudaGetLastError());
}

// BITNET_LOG=1: one line on stderr per kernel launch (which kernel, shape, grid, plan).  Read once.
bool log_enabled();
void log_launch(const char* fmt, ...);

// Device properties looked up once per device.
struct DevInfo {
  int sm_count;
  int max_smem_optin;
  int max_smem_per_sm;
};
const DevInfo& dev_info();

// ---- kernel launchers (one per .cu file) ----------------------------------------------------
int launch_quant_act(const float* x, int64_t T, int64_t K, int per_tensor, int8_t* q, float* act_scale,
                     int32_t* act_sum, cudaStream_t st);
// per-token quantiser over a list of matrices x[T][K] -> q[T][K], act_scale[T], in one launch per 800 matrices
struct QuantListItem {
  const float* x;
  int8_t* q;
  float* act_scale;
  int64_t K;
  int T;
};
int launch_quant_act_list(const QuantListItem* items, int64_t n, cudaStream_t st);
int launch_pack_i2s(const int8_t* w, int64_t M, int64_t K, uint8_t* packed, int* dev_status,
                    cudaStream_t st);
int launch_unpack_i2s(const uint8_t* packed, int64_t M, int64_t K, int8_t* w, int* dev_status,
                      cudaStream_t st);
int launch_pack_tl(int fmt, const int8_t* w, int64_t M, int64_t K, const TlGeom& g, uint8_t* packed,
                   int* dev_status, cudaStream_t st);
int launch_unpack_tl(int fmt, const uint8_t* packed, int64_t M, int64_t K, const TlGeom& g, int8_t* w,
                     int* dev_status, cudaStream_t st);
// TL blob -> I2_S blob of the same matrix (bitnet_i2s_packed_bytes(M, K) bytes), entirely on the device.
int launch_tl_to_i2s(const uint8_t* tl, int64_t M, int64_t K, const TlGeom& g, uint8_t* i2s, cudaStream_t st);

// Decode GEMV, T <= 8.
size_t gemv_i2s_workspace_bytes(int64_t T, int64_t M, int64_t K);
int launch_gemv_i2s(const uint8_t* packed, float w_scale, int64_t M, int64_t K, const int8_t* q,
                    const float* act_scale, int T, float* y, int32_t* acc_out, void* ws, size_t ws_bytes,
                    cudaStream_t st);
// Streaming (bulk-copy ring + tensor-core MMA) kernel.
bool gemv_i2s_stream_supported(int T, int64_t M, int64_t K, bool fused);
// x != nullptr runs the quantiser inside the kernel (q and act_scale are then outputs).
int launch_gemv_i2s_stream(const uint8_t* packed, float w_scale, int64_t M, int64_t K, const float* x, int8_t* q,
                           float* act_scale, int T, float* y, int32_t* acc_out, cudaStream_t st);
int gemv_i2s_stream_status(int* out);
// Warp-private cp.async rings + tensor-core MMA; two consecutive kernels' CTAs share an SM.
bool gemv_i2s_wring_supported(int T, int64_t M, int64_t K);
int launch_gemv_i2s_wring(const uint8_t* packed, float w_scale, int64_t M, int64_t K, const float* x, int8_t* q,
                          float* act_scale, int T, float* y, int32_t* acc_out, cudaStream_t st);
// One persistent kernel over a list of I2_S linears (1..8 tokens each) whose inputs exist at launch.
struct GroupLinear {
  const uint8_t* packed;
  const float* x;      // fp32 activations [T][K] (q, act_scale are then outputs); null: q, act_scale are inputs
  int8_t* q;
  float* act_scale;
  float* y;
  int32_t* acc_out;    // nullable
  float w_scale;
  int T;
  int64_t M, K;
  int64_t ldy;         // elements between the token rows of y / acc_out; 0 = M
};
bool gemv_i2s_group_item_supported(int T, int64_t M, int64_t K);
int launch_gemv_i2s_group(const GroupLinear* items, int64_t n, cudaStream_t st);
// One persistent kernel over a list of TL2 linears (1..8 tokens each): packed indices decoded through a shared-memory
// table into tensor-core operands.
struct Tl2Linear {
  const uint8_t* packed;
  const float* x;      // fp32 activations [T][K] (q, act_scale are then outputs); null: q, act_scale are inputs
  int8_t* q;
  float* act_scale;
  float* y;
  int32_t* acc_out;    // nullable
  float w_scale;
  int T;
  int64_t M, K;
  int64_t ldy;         // elements between the token rows of y / acc_out; 0 = M
  TlGeom g;
};
bool gemv_tl2_scan_item_supported(int T, int64_t M, int64_t K, const TlGeom& g);
int launch_gemv_tl2_scan(const Tl2Linear* items, int64_t n, cudaStream_t st);
// App. A beyond ternary, g = 2: weights of cardinality C = 3, 4, 5 as pair indices in 32-row x 32-pair tiles (512
// bytes of index nibbles; for C = 5 another 128 bytes of fifth bits).  The geometry comes back in a TlGeom whose
// tiles3 counts those tiles (tiles2 = 0); the same persistent kernel walks them.
bool elut2_geom(int C, int64_t M, int64_t K, TlGeom* g);
bool gemv_elut_scan_item_supported(int T, int64_t M, int64_t K, const TlGeom& g);
int launch_gemv_elut_scan(const Tl2Linear* items, int64_t n, int C, cudaStream_t st);
int launch_pack_elut2(int C, const int8_t* w, int64_t M, int64_t K, const TlGeom& g, uint8_t* packed, int* dev_status,
                      cudaStream_t st);
int launch_unpack_elut2(int C, const uint8_t* packed, int64_t M, int64_t K, const TlGeom& g, int8_t* w, int* dev_status,
                        cudaStream_t st);
// Batches of 9 to 64 tokens: mma.sync over K-slices, partial sums through a [T][M] int32 workspace when K is
// cut into more than one slice (gemv_i2s_mid_workspace_bytes says how much; 0 = none needed).
bool gemv_i2s_mid_supported(int T, int64_t M, int64_t K);
size_t gemv_i2s_mid_workspace_bytes(int T, int64_t M, int64_t K);
int launch_gemv_i2s_mid(const uint8_t* packed, float w_scale, int64_t M, int64_t K, const int8_t* q,
                        const float* act_scale, int T, float* y, int32_t* acc_out, void* ws, size_t ws_bytes,
                        cudaStream_t st);
// 9 to 128 tokens over a list of I2_S linears whose codes exist (q, act_scale): the weights streamed once, unpacked
// into tensor memory, tcgen05 MMAs (gemm_i2s_stream_tc.cu).
struct StreamTcLinear {
  const uint8_t* packed;
  const int8_t* q;
  const float* act_scale;
  float* y;
  int32_t* acc_out;    // nullable
  float w_scale;
  int T;
  int64_t M, K;
  int64_t ldy;         // elements between the token rows of y / acc_out; 0 = M
};
bool gemm_i2s_stream_tc_item_supported(int64_t T, int64_t M, int64_t K);
// Tensor map of the codes q[T][K] (int8) for tensor copies of 128 columns x `box_t` tokens into the 128-byte-swizzled
// K-major layout of an MMA operand; columns and tokens beyond the matrix read as zeros (gemm_prefill_tc.cu).
int encode_q_tile_map(void* out /* CUtensorMap */, const int8_t* q, int64_t K, int64_t T, int box_t);
int launch_gemm_i2s_stream_tc(const StreamTcLinear* items, int64_t n, cudaStream_t st);
int gemm_i2s_stream_tc_status(int* out);
int gemm_i2s_stream_tc_status_clear();
// Programmatic dependent launch (kernels may start their prologue, and prefetch weights, before the
// previous kernel in the stream has finished); process-wide switch, on by default.  early_start_enabled(st) is asked
// once per launch on `st`: it answers no for the first launch after a kernel of this library wrote a packed blob
// on that stream (note_blob_written), so that this launch begins only when the blob is complete and everything
// queued behind it is ordered after it.
bool early_start_enabled(cudaStream_t st);
void note_blob_written(cudaStream_t st);
size_t gemv_tl_workspace_bytes(int fmt, int64_t T, int64_t M, int64_t K);
int launch_gemv_tl(int fmt, const uint8_t* packed, float w_scale, int64_t M, int64_t K, const TlGeom& g,
                   const int8_t* q, const float* act_scale, int T, float* y, int32_t* acc_out, void* ws,
                   size_t ws_bytes, cudaStream_t st);
int launch_tl_build_lut(int fmt, const int8_t* q_row, int64_t K, const TlGeom& g, int16_t* lut,
                        cudaStream_t st);

// y = float(sums) * (act_scale[t] * w_scale) over a [T][M] int32 array of finished sums, which is left zeroed.
// y[t][m] *= scale of the segment row m lies in (n_seg <= 16 segments, ends ascending, the last = M).
int launch_scale_segments(float* y, int64_t T, int64_t M, int n_seg, const int64_t* seg_end, const float* seg_scale,
                          cudaStream_t st);
int launch_rescale_sums(int32_t* sums, const float* act_scale, float w_scale, int64_t T, int64_t M, float* y,
                        int32_t* acc_out, cudaStream_t st);

// Prefill GEMM (I2_S, int8 tensor cores).  With few output tiles for the SMs it cuts every tile's K into parts
// that meet in `ws` (zeroed [T][M] int32, gemm_i2s_prefill_workspace_bytes; without it: whole tiles only).
size_t gemm_i2s_prefill_workspace_bytes(int64_t T, int64_t M, int64_t K);
int launch_gemm_i2s_prefill(const uint8_t* packed, float w_scale, int64_t M, int64_t K, const int8_t* q,
                            const float* act_scale, int64_t T, float* y, int32_t* acc_out, void* ws, size_t ws_bytes,
                            cudaStream_t st);

int gemm_prefill_status(int* out);
int gemv_tl_status(int* out);
int gemm_prefill_status_clear();
int gemv_tl_status_clear();
int gemv_i2s_stream_status_clear();
int launch_wait_timeout_probe(cudaStream_t st);

}  // namespace bitnet
