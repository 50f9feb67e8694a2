// C ABI of libbitnet_b200.so: argument validation and dispatch.  Every step of the path runs in the
// kernels of the sibling files; nothing here computes.
#include <cstdlib>
#include <cstring>
#include <cstdarg>
#include <cstdio>
#include <atomic>
#include <mutex>

#include <vector>

#include "common.cuh"

namespace bitnet {

static thread_local int g_last_cuda_error = 0;

int note_cuda_error(cudaError_t e) {
  g_last_cuda_error = (int)e;
  return BITNET_ERR_CUDA;
}

static int g_early_start = 1;
static int g_tl2_lookup = [] { const char* e = getenv("BITNET_TL2"); return (e && strcmp(e, "lut") == 0) ? 1 : 0; }();
// Streams on which a packer (or the TL -> I2_S transcode) has been queued and no kernel of this library since.
static std::mutex g_written_mu;
static std::vector<cudaStream_t> g_written;
static std::atomic<int> g_written_n{0};
void note_blob_written(cudaStream_t st) {
  std::lock_guard<std::mutex> lock(g_written_mu);
  for (cudaStream_t s : g_written)
    if (s == st) return;
  g_written.push_back(st);
  g_written_n.store((int)g_written.size(), std::memory_order_release);
}
bool early_start_enabled(cudaStream_t st) {
  if (!g_early_start) return false;
  if (g_written_n.load(std::memory_order_acquire) == 0) return true;
  std::lock_guard<std::mutex> lock(g_written_mu);
  for (size_t i = 0; i < g_written.size(); ++i)
    if (g_written[i] == st) {
      g_written.erase(g_written.begin() + (long)i);
      g_written_n.store((int)g_written.size(), std::memory_order_release);
      return false;
    }
  return true;
}

bool log_enabled() {
  static const bool on = [] { const char* e = getenv("BITNET_LOG"); return e && atoi(e) != 0; }();
  return on;
}
void log_launch(const char* fmt, ...) {
  if (!log_enabled()) return;
  va_list ap;
  va_start(ap, fmt);
  fputs("[bitnet_b200] ", stderr);
  vfprintf(stderr, fmt, ap);
  fputc('\n', stderr);
  va_end(ap);
}

const DevInfo& dev_info() {
  static DevInfo info[64];
  static bool have[64] = {false};
  static std::mutex mu;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) {
    cudaGetLastError();
    dev = 0;
  }
  dev &= 63;
  std::lock_guard<std::mutex> lock(mu);
  if (!have[dev]) {
    // B200 figures stand in when no device can be queried (size queries on a machine without a GPU)
    info[dev].sm_count = 148;
    info[dev].max_smem_optin = 232448;
    info[dev].max_smem_per_sm = 233472;
    int v = 0;
    if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && v > 0) info[dev].sm_count = v;
    if (cudaDeviceGetAttribute(&v, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) == cudaSuccess && v > 0)
      info[dev].max_smem_optin = v;
    if (cudaDeviceGetAttribute(&v, cudaDevAttrMaxSharedMemoryPerMultiprocessor, dev) == cudaSuccess && v > 0)
      info[dev].max_smem_per_sm = v;
    cudaGetLastError();
    have[dev] = true;
  }
  return info[dev];
}

}  // namespace bitnet

using namespace bitnet;

extern "C" {

const char* bitnet_status_string(int status) {
  switch (status) {
    case BITNET_OK: return "ok";
    case BITNET_ERR_INVALID_ARG: return "invalid argument (null or misaligned pointer, bad enum or size)";
    case BITNET_ERR_UNSUPPORTED_SHAPE: return "unsupported shape for this weight format";
    case BITNET_ERR_WORKSPACE: return "workspace missing or too small";
    case BITNET_ERR_BAD_WEIGHT: return "weight outside the format's alphabet or invalid packed code";
    case BITNET_ERR_CUDA: return "CUDA call failed (see bitnet_last_cuda_error)";
    case BITNET_ERR_TIMEOUT: return "bounded device-side wait gave up";
    default: return "unknown status";
  }
}

int bitnet_last_cuda_error(void) { return g_last_cuda_error; }

int bitnet_device_status(int* status_out) {
  if (!status_out) return BITNET_ERR_INVALID_ARG;
  int a = 0, b = 0;
  int rc = gemv_i2s_stream_status(&a);
  if (rc) return rc;
  rc = gemm_prefill_status(&b);
  if (rc) return rc;
  int c = 0;
  rc = gemv_tl_status(&c);
  if (rc) return rc;
  int d = 0;
  rc = gemm_i2s_stream_tc_status(&d);
  if (rc) return rc;
  *status_out = a ? a : (b ? b : (c ? c : d));
  return BITNET_OK;
}

int bitnet_device_status_clear(void) {
  cudaError_t e = cudaDeviceSynchronize();
  if (e != cudaSuccess) return note_cuda_error(e);
  int rc = gemv_i2s_stream_status_clear();
  if (rc) return rc;
  rc = gemm_prefill_status_clear();
  if (rc) return rc;
  rc = gemm_i2s_stream_tc_status_clear();
  if (rc) return rc;
  return gemv_tl_status_clear();
}

int bitnet_debug_wait_timeout_probe(void* stream) { return launch_wait_timeout_probe((cudaStream_t)stream); }

void bitnet_set_early_start(int enable) { g_early_start = enable ? 1 : 0; }
void bitnet_set_tl2_lookup(int enable) { bitnet::g_tl2_lookup = enable ? 1 : 0; }

int bitnet_quant_act(const float* x, int64_t T, int64_t K, int per_tensor, int8_t* q, float* act_scale,
                     int32_t* act_sum, void* stream) {
  if (!x || !q || !act_scale || T < 1 || K < 1 || T > 0x7fffffff) return BITNET_ERR_INVALID_ARG;
  if (!aligned16(x) || !aligned16(q) || (reinterpret_cast<uintptr_t>(act_scale) & 3u)) return BITNET_ERR_INVALID_ARG;
  return launch_quant_act(x, T, K, per_tensor, q, act_scale, act_sum, (cudaStream_t)stream);
}

size_t bitnet_i2s_packed_bytes(int64_t M, int64_t K) {
  if (M < 1 || K < 1 || (K % 64) != 0) return 0;
  return (size_t)i2s_mp(M) * (size_t)i2s_kp(K) / 4;
}

static int i2s_shape(int64_t M, int64_t K) {
  if (M < 1 || K < 1 || M > 0x7fffffff) return BITNET_ERR_INVALID_ARG;
  if ((K % 64) != 0) return BITNET_ERR_UNSUPPORTED_SHAPE;
  return BITNET_OK;
}

int bitnet_pack_i2s(const int8_t* w, int64_t M, int64_t K, void* packed, size_t packed_bytes, int* dev_status,
                    void* stream) {
  if (!w || !packed || !aligned16(packed)) return BITNET_ERR_INVALID_ARG;
  int rc = i2s_shape(M, K);
  if (rc) return rc;
  if (packed_bytes < bitnet_i2s_packed_bytes(M, K)) return BITNET_ERR_INVALID_ARG;
  return launch_pack_i2s(w, M, K, (uint8_t*)packed, dev_status, (cudaStream_t)stream);
}

int bitnet_unpack_i2s(const void* packed, int64_t M, int64_t K, int8_t* w, int* dev_status, void* stream) {
  if (!w || !packed || !aligned16(packed)) return BITNET_ERR_INVALID_ARG;
  int rc = i2s_shape(M, K);
  if (rc) return rc;
  return launch_unpack_i2s((const uint8_t*)packed, M, K, w, dev_status, (cudaStream_t)stream);
}

static int tl_shape(int fmt, int64_t M, int64_t K, int bk3, TlGeom* g) {
  if (fmt != BITNET_FMT_TL1 && fmt != BITNET_FMT_TL2) return BITNET_ERR_INVALID_ARG;
  if (M < 1 || K < 1 || M > 0x7fffffff) return BITNET_ERR_INVALID_ARG;
  if (!tl_geom(fmt, M, K, bk3, g)) return BITNET_ERR_UNSUPPORTED_SHAPE;
  return BITNET_OK;
}

size_t bitnet_tl_packed_bytes(bitnet_fmt_t fmt, int64_t M, int64_t K, int bk3) {
  TlGeom g;
  if (tl_shape(fmt, M, K, bk3, &g)) return 0;
  return (size_t)(M / 32) * (size_t)g.block_bytes;
}

int bitnet_pack_tl(bitnet_fmt_t fmt, const int8_t* w, int64_t M, int64_t K, int bk3, void* packed,
                   size_t packed_bytes, int* dev_status, void* stream) {
  if (!w || !packed || !aligned16(packed)) return BITNET_ERR_INVALID_ARG;
  TlGeom g;
  int rc = tl_shape(fmt, M, K, bk3, &g);
  if (rc) return rc;
  if (packed_bytes < (size_t)(M / 32) * (size_t)g.block_bytes) return BITNET_ERR_INVALID_ARG;
  return launch_pack_tl(fmt, w, M, K, g, (uint8_t*)packed, dev_status, (cudaStream_t)stream);
}

int bitnet_unpack_tl(bitnet_fmt_t fmt, const void* packed, int64_t M, int64_t K, int bk3, int8_t* w,
                     int* dev_status, void* stream) {
  if (!w || !packed || !aligned16(packed)) return BITNET_ERR_INVALID_ARG;
  TlGeom g;
  int rc = tl_shape(fmt, M, K, bk3, &g);
  if (rc) return rc;
  return launch_unpack_tl(fmt, (const uint8_t*)packed, M, K, g, w, dev_status, (cudaStream_t)stream);
}

int64_t bitnet_tl_num_groups(bitnet_fmt_t fmt, int64_t K, int bk3) {
  TlGeom g;
  if (tl_shape(fmt, 32, K, bk3, &g)) return -1;
  return (g.tiles3 + g.tiles2) * 32;
}

int bitnet_tl_build_lut_debug(bitnet_fmt_t fmt, const int8_t* q_row, int64_t K, int bk3, int16_t* lut,
                              void* stream) {
  if (!q_row || !lut) return BITNET_ERR_INVALID_ARG;
  TlGeom g;
  int rc = tl_shape(fmt, 32, K, bk3, &g);
  if (rc) return rc;
  return launch_tl_build_lut(fmt, q_row, K, g, lut, (cudaStream_t)stream);
}

// Batch sizes served by the mid-batch kernel: 9 to 64 tokens, and decode batches whose codes crowd the decode
// kernel's shared memory (6 tokens or more, or more than 96 KiB of codes: measured crossover on the 100B
// shapes).  BITNET_I2S_MID_MAX_T = 0 switches the kernel off, BITNET_I2S_MID_MIN_T raises the lower limit.
static bool use_mid(int64_t T, int64_t M, int64_t K) {
  static const int lo = [] { const char* e = getenv("BITNET_I2S_MID_MIN_T"); return e ? atoi(e) : 1; }();
  static const int hi = [] { const char* e = getenv("BITNET_I2S_MID_MAX_T"); return e ? atoi(e) : 64; }();
  if (T < lo || T > hi || T > 64) return false;
  if (T <= 8 && T < 6 && T * i2s_kp(K) <= 96 * 1024) return false;
  return gemv_i2s_mid_supported((int)T, M, K);
}
static bool mid_takes(int64_t T, int64_t M, int64_t K, const void* workspace, size_t workspace_bytes) {
  return use_mid(T, M, K) && workspace && gemv_i2s_mid_workspace_bytes((int)T, M, K) <= workspace_bytes;
}

// TL2 decode batches go to the scan kernel (decode table + tensor cores) unless BITNET_TL2=lut asks for the
// activation-table form of Alg. 2 / Alg. 4, or the shape does not fit it.
static bool tl2_scan_takes(int fmt, int64_t T, int64_t M, int64_t K, const TlGeom& g) {
  return !bitnet::g_tl2_lookup && fmt == BITNET_FMT_TL2 && T >= 1 && T <= 8 && gemv_tl2_scan_item_supported((int)T, M, K, g);
}
// A TL1 blob is the pair-index blob of cardinality 3 (Table 4's code of a pair = 3 (w0+1) + (w1+1)): decode batches
// go to the scan kernel's pair mode under the same switch.  `pg` receives the geometry that kernel wants.
static bool tl1_scan_takes(int fmt, int64_t T, int64_t M, int64_t K, TlGeom* pg) {
  return !bitnet::g_tl2_lookup && fmt == BITNET_FMT_TL1 && T >= 1 && T <= 8 && elut2_geom(3, M, K, pg) &&
         gemv_elut_scan_item_supported((int)T, M, K, *pg);
}
// One decode item for either scan mode.
static Tl2Linear scan_item(const void* packed, const float* x, int8_t* q, float* act_scale, float* y, int32_t* acc_out,
                           float w_scale, int64_t T, int64_t M, int64_t K, int64_t ldy, const TlGeom& g) {
  Tl2Linear it;
  it.packed = (const uint8_t*)packed;
  it.x = x;
  it.q = q;
  it.act_scale = act_scale;
  it.y = y;
  it.acc_out = acc_out;
  it.w_scale = w_scale;
  it.T = (int)T;
  it.M = M;
  it.K = K;
  it.ldy = ldy;
  it.g = g;
  return it;
}

// From this many tokens on a TL call is cheaper as: transcode the blob to I2_S in the workspace (about 20 us for a
// 4096 x 14336 tensor), then the tcgen05 prefill kernel -- than as ceil(T / 8) scans of the blob.
static constexpr int64_t TL_PREFILL_MIN_T = 128;

size_t bitnet_mpgemm_workspace_bytes(bitnet_fmt_t fmt, int64_t T, int64_t M, int64_t K) {
  if (T < 1 || M < 1 || K < 1) return 0;
  if (fmt == BITNET_FMT_I2S) {
    size_t n = T > 8 ? gemm_i2s_prefill_workspace_bytes(T, M, K) : gemv_i2s_workspace_bytes(T, M, K);
    if (use_mid(T, M, K)) {
      const size_t m = gemv_i2s_mid_workspace_bytes((int)T, M, K);
      if (m > n) n = m;
    }
    return n;
  }
  size_t n = gemv_tl_workspace_bytes(fmt, T, M, K);
  // batches of TL_PREFILL_MIN_T tokens or more are served by the tensor-core prefill kernel from an I2_S copy of the
  // tensor made on the fly in the workspace
  if (T >= TL_PREFILL_MIN_T && (K % 64) == 0) {
    const size_t m = bitnet_i2s_packed_bytes(M, K);
    if (m > n) n = m;
  }
  return n;
}

int bitnet_workspace_init(void* workspace, size_t workspace_bytes, void* stream) {
  if (workspace_bytes == 0) return BITNET_OK;
  if (!workspace) return BITNET_ERR_INVALID_ARG;
  cudaError_t e = cudaMemsetAsync(workspace, 0, workspace_bytes, (cudaStream_t)stream);
  return e == cudaSuccess ? BITNET_OK : note_cuda_error(e);
}

int bitnet_mpgemm(bitnet_fmt_t fmt, const void* packed, float w_scale, int64_t M, int64_t K, int bk3,
                  const int8_t* q, const float* act_scale, int64_t T, float* y, int32_t* acc_out,
                  void* workspace, size_t workspace_bytes, void* stream) {
  if (!packed || !q || !act_scale || !y || T < 1) return BITNET_ERR_INVALID_ARG;
  if (!aligned16(packed) || !aligned16(q) || !aligned16(y) || (acc_out && !aligned16(acc_out)) ||
      (workspace && !aligned16(workspace)))
    return BITNET_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  if (fmt == BITNET_FMT_I2S) {
    int rc = i2s_shape(M, K);
    if (rc) return rc;
    // A single tensor with enough 128-row tiles for the SMs: the streaming tcgen05 kernel (weights read once, codes
    // unpacked into tensor memory).  Measured crossovers against the mma.sync and prefill kernels, quantiser
    // included (us): 57344 x 8192 at 24 / 32 / 64 / 128 tokens 57 / 56 / 59 / 85 against 54 / 66 / 114 / 125;
    // 28672 x 8192: 36 / 36 / 38 / 53 against 35 / 40 / 65 / 70; with fewer tiles than two thirds of the SMs
    // (8192 x 28672: 56 / 56 / 58 / 75 against 34 / 40 / 62 / 72) the kernels that split K stay ahead up to 64 tokens.
    static const bool stream_tc = [] { const char* e = getenv("BITNET_I2S_STREAM_TC"); return !(e && atoi(e) == 0); }();
    const int64_t tiles128 = ceil_div(M, 128), sms = dev_info().sm_count;
    if (stream_tc && gemm_i2s_stream_tc_item_supported(T, M, K) &&
        ((T >= 25 && T <= 64 && tiles128 * 3 >= sms * 2) || (T >= 65 && T <= 128 && tiles128 >= sms))) {
      StreamTcLinear t;
      t.packed = (const uint8_t*)packed;
      t.q = q;
      t.act_scale = act_scale;
      t.y = y;
      t.acc_out = acc_out;
      t.w_scale = w_scale;
      t.T = (int)T;
      t.M = M;
      t.K = K;
      t.ldy = 0;
      return launch_gemm_i2s_stream_tc(&t, 1, st);
    }
    // 9 to 64 tokens (and crowded decode batches): the weight scan on mma.sync; the prefill (or decode) kernel
    // takes the call when the caller's workspace is smaller than bitnet_mpgemm_workspace_bytes asked for
    if (mid_takes(T, M, K, workspace, workspace_bytes))
      return launch_gemv_i2s_mid((const uint8_t*)packed, w_scale, M, K, q, act_scale, (int)T, y, acc_out, workspace,
                                 workspace_bytes, st);
    if (T > 8)
      return launch_gemm_i2s_prefill((const uint8_t*)packed, w_scale, M, K, q, act_scale, T, y, acc_out, workspace,
                                     workspace_bytes, st);
    return launch_gemv_i2s((const uint8_t*)packed, w_scale, M, K, q, act_scale, (int)T, y, acc_out, workspace,
                           workspace_bytes, st);
  }
  TlGeom g;
  int rc = tl_shape(fmt, M, K, bk3, &g);
  if (rc) return rc;
  if (T >= TL_PREFILL_MIN_T && (K % 64) == 0 && workspace && workspace_bytes >= bitnet_i2s_packed_bytes(M, K)) {
    // many tokens: the packed tensor is turned into its I2_S form in the workspace and the tensor-core prefill
    // kernel (whole tiles per CTA: it is given no workspace of its own) does the rest; same integers
    rc = launch_tl_to_i2s((const uint8_t*)packed, M, K, g, (uint8_t*)workspace, st);
    if (rc) return rc;
    return launch_gemm_i2s_prefill((const uint8_t*)workspace, w_scale, M, K, q, act_scale, T, y, acc_out, nullptr, 0, st);
  }
  for (int64_t t0 = 0; t0 < T; t0 += 8) {
    const int nt = (int)((T - t0 < 8) ? (T - t0) : 8);
    TlGeom pg;
    if (tl2_scan_takes(fmt, nt, M, K, g)) {
      const Tl2Linear it = scan_item(packed, nullptr, const_cast<int8_t*>(q + t0 * K), const_cast<float*>(act_scale + t0),
                                     y + t0 * M, acc_out ? acc_out + t0 * M : nullptr, w_scale, nt, M, K, 0, g);
      rc = launch_gemv_tl2_scan(&it, 1, st);
    } else if (tl1_scan_takes(fmt, nt, M, K, &pg)) {
      const Tl2Linear it = scan_item(packed, nullptr, const_cast<int8_t*>(q + t0 * K), const_cast<float*>(act_scale + t0),
                                     y + t0 * M, acc_out ? acc_out + t0 * M : nullptr, w_scale, nt, M, K, 0, pg);
      rc = launch_gemv_elut_scan(&it, 1, 3, st);
    } else {
      rc = launch_gemv_tl(fmt, (const uint8_t*)packed, w_scale, M, K, g, q + t0 * K, act_scale + t0, nt,
                          y + t0 * M, acc_out ? acc_out + t0 * M : nullptr, workspace, workspace_bytes, st);
    }
    if (rc) return rc;
  }
  return BITNET_OK;
}

int bitnet_linear(bitnet_fmt_t fmt, const void* packed, float w_scale, int64_t M, int64_t K, int bk3, const float* x,
                  int64_t T, int8_t* q, float* act_scale, float* y, int32_t* acc_out, void* workspace,
                  size_t workspace_bytes, void* stream) {
  if (!packed || !x || !q || !act_scale || !y || T < 1) return BITNET_ERR_INVALID_ARG;
  if (!aligned16(packed) || !aligned16(x) || !aligned16(q) || !aligned16(y) || (acc_out && !aligned16(acc_out)) ||
      (reinterpret_cast<uintptr_t>(act_scale) & 3u))
    return BITNET_ERR_INVALID_ARG;
  if (fmt == BITNET_FMT_I2S) {
    int rc = i2s_shape(M, K);      // before any plan is made from M and K
    if (rc) return rc;
  }
  if (fmt == BITNET_FMT_I2S && T <= 8 && !mid_takes(T, M, K, workspace, workspace_bytes)) {
    static const bool no_fuse = [] {
      const char* e = getenv("BITNET_I2S_KERNEL");
      return e && strcmp(e, "splitk") == 0;
    }();
    // Decode batches (up to 8 tokens): every CTA of the GEMV quantises the rows itself (one pass per row, the row
    // held in registers), which measured faster than a separate quantiser launch at every batch size where the
    // streaming kernel applies.  BITNET_FUSE_MAX_T lowers the threshold.
    static const int fuse_max = [] { const char* e = getenv("BITNET_FUSE_MAX_T"); return e ? atoi(e) : 8; }();
    if (!no_fuse && T <= fuse_max && gemv_i2s_stream_supported((int)T, M, K, true))
      return launch_gemv_i2s_stream((const uint8_t*)packed, w_scale, M, K, x, q, act_scale, (int)T, y, acc_out,
                                    (cudaStream_t)stream);
  }
  if (fmt == BITNET_FMT_TL2 && T <= 8) {
    TlGeom g;
    int rc = tl_shape(fmt, M, K, bk3, &g);
    if (rc) return rc;
    if (tl2_scan_takes(fmt, T, M, K, g)) {       // one kernel: quantiser fused
      const Tl2Linear it = scan_item(packed, x, q, act_scale, y, acc_out, w_scale, T, M, K, 0, g);
      return launch_gemv_tl2_scan(&it, 1, (cudaStream_t)stream);
    }
  }
  if (fmt == BITNET_FMT_TL1 && T <= 8) {
    TlGeom g, pg;
    int rc = tl_shape(fmt, M, K, bk3, &g);
    if (rc) return rc;
    if (tl1_scan_takes(fmt, T, M, K, &pg)) {
      const Tl2Linear it = scan_item(packed, x, q, act_scale, y, acc_out, w_scale, T, M, K, 0, pg);
      return launch_gemv_elut_scan(&it, 1, 3, (cudaStream_t)stream);
    }
  }
  int rc = bitnet_quant_act(x, T, K, 0, q, act_scale, nullptr, stream);
  if (rc) return rc;
  return bitnet_mpgemm(fmt, packed, w_scale, M, K, bk3, q, act_scale, T, y, acc_out, workspace, workspace_bytes,
                       stream);
}

int bitnet_linear_host(bitnet_fmt_t fmt, const void* packed, float w_scale, int64_t M, int64_t K, int bk3,
                       const float* x_host, int64_t T, float* y_host, float* x_dev, int8_t* q_dev,
                       float* scale_dev, float* y_dev, void* workspace, size_t workspace_bytes, void* stream) {
  if (!x_host || !y_host || !x_dev || !q_dev || !scale_dev || !y_dev || T < 1 || M < 1 || K < 1)
    return BITNET_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  cudaError_t e = cudaMemcpyAsync(x_dev, x_host, (size_t)T * K * sizeof(float), cudaMemcpyHostToDevice, st);
  if (e != cudaSuccess) return note_cuda_error(e);
  int rc = bitnet_linear(fmt, packed, w_scale, M, K, bk3, x_dev, T, q_dev, scale_dev, y_dev, nullptr, workspace,
                         workspace_bytes, stream);
  if (rc) return rc;
  e = cudaMemcpyAsync(y_host, y_dev, (size_t)T * M * sizeof(float), cudaMemcpyDeviceToHost, st);
  return e == cudaSuccess ? BITNET_OK : note_cuda_error(e);
}

int bitnet_linear_group(const bitnet_group_item_t* items, int64_t n, void* stream) {
  if (n < 0 || (n > 0 && !items)) return BITNET_ERR_INVALID_ARG;
  for (int64_t i = 0; i < n; ++i) {
    const bitnet_group_item_t& d = items[i];
    if (!d.packed || !d.x || !d.q || !d.act_scale || !d.y || d.T < 1 || d.M < 1 || d.K < 1) return BITNET_ERR_INVALID_ARG;
    if (!aligned16(d.packed) || !aligned16(d.x) || !aligned16(d.q) || !aligned16(d.y) ||
        (d.acc_out && !aligned16(d.acc_out)) || (reinterpret_cast<uintptr_t>(d.act_scale) & 3u))
      return BITNET_ERR_INVALID_ARG;
    if (d.fmt == BITNET_FMT_I2S) {
      int rc = i2s_shape(d.M, d.K);
      if (rc) return rc;
    } else {
      TlGeom g;
      int rc = tl_shape(d.fmt, d.M, d.K, d.bk3, &g);
      if (rc) return rc;
    }
  }
  static const bool grouped = [] { const char* e = getenv("BITNET_GROUP"); return !(e && atoi(e) == 0); }();
  // 9 to 16 tokens: the grouped kernel's two-group form (every A register feeds an MMA per group of eight tokens;
  // the weights cross HBM once); BITNET_GROUP_WIDE=0 or a shape that form does not take: two items of the
  // one-group kernel (tokens 0..7, then the rest), which still beat the mid-batch kernel's launch per linear on
  // lists (5.5 against 8.4 ms on the 100B sweep at 16 tokens).  BITNET_GROUP_MAX_T lowers the limit.
  static const bool group_wide = [] { const char* e = getenv("BITNET_GROUP_WIDE"); return !(e && atoi(e) == 0); }();
  static const int group_max_t = [] { const char* e = getenv("BITNET_GROUP_MAX_T"); const int v = e ? atoi(e) : 16; return v < 8 ? 8 : (v > 16 ? 16 : v); }();
  auto takes = [&](const bitnet_group_item_t& d) {
    if (!grouped || d.fmt != BITNET_FMT_I2S || d.T > group_max_t) return false;
    if (d.T <= 8 || group_wide) {
      if (gemv_i2s_group_item_supported((int)d.T, d.M, d.K)) return true;
      if (d.T <= 8) return false;
    }
    return gemv_i2s_group_item_supported(8, d.M, d.K) && gemv_i2s_group_item_supported((int)d.T - 8, d.M, d.K);
  };
  // 17 to 128 tokens: the stand-alone quantiser per item, then the streaming tensor-core kernel over the run
  // (BITNET_I2S_STREAM_TC=0: every such item as bitnet_linear)
  static const bool stream_tc = [] { const char* e = getenv("BITNET_I2S_STREAM_TC"); return !(e && atoi(e) == 0); }();
  auto takes_tc = [&](const bitnet_group_item_t& d) {
    return grouped && stream_tc && d.fmt == BITNET_FMT_I2S && d.T > group_max_t && gemm_i2s_stream_tc_item_supported(d.T, d.M, d.K);
  };
  static thread_local std::vector<StreamTcLinear> run3;
  static thread_local std::vector<QuantListItem> qrun;
  static thread_local std::vector<GroupLinear> run;
  static thread_local std::vector<Tl2Linear> run2;
  auto takes2 = [&](const bitnet_group_item_t& d, TlGeom* g) {
    return grouped && d.fmt == BITNET_FMT_TL2 && tl_shape(d.fmt, d.M, d.K, d.bk3, g) == BITNET_OK &&
           tl2_scan_takes(d.fmt, d.T, d.M, d.K, *g);
  };
  auto takes1 = [&](const bitnet_group_item_t& d, TlGeom* pg) {
    TlGeom g;
    return grouped && d.fmt == BITNET_FMT_TL1 && tl_shape(d.fmt, d.M, d.K, d.bk3, &g) == BITNET_OK &&
           tl1_scan_takes(d.fmt, d.T, d.M, d.K, pg);
  };
  for (int64_t i = 0; i < n;) {
    TlGeom g2;
    if (takes2(items[i], &g2)) {
      run2.clear();
      for (; i < n && takes2(items[i], &g2); ++i) {
        const bitnet_group_item_t& d = items[i];
        run2.push_back(scan_item(d.packed, d.x, d.q, d.act_scale, d.y, d.acc_out, d.w_scale, d.T, d.M, d.K, 0, g2));
      }
      int rc = launch_gemv_tl2_scan(run2.data(), (int64_t)run2.size(), (cudaStream_t)stream);
      if (rc) return rc;
      continue;
    }
    if (takes1(items[i], &g2)) {
      run2.clear();
      for (; i < n && takes1(items[i], &g2); ++i) {
        const bitnet_group_item_t& d = items[i];
        run2.push_back(scan_item(d.packed, d.x, d.q, d.act_scale, d.y, d.acc_out, d.w_scale, d.T, d.M, d.K, 0, g2));
      }
      int rc = launch_gemv_elut_scan(run2.data(), (int64_t)run2.size(), 3, (cudaStream_t)stream);
      if (rc) return rc;
      continue;
    }
    if (takes_tc(items[i])) {
      run3.clear();
      qrun.clear();
      for (; i < n && takes_tc(items[i]); ++i) {
        const bitnet_group_item_t& d = items[i];
        if (qrun.empty() || qrun.back().x != d.x || qrun.back().q != d.q || qrun.back().act_scale != d.act_scale ||
            qrun.back().K != d.K || qrun.back().T != (int)d.T)
          qrun.push_back(QuantListItem{d.x, d.q, d.act_scale, d.K, (int)d.T});
        StreamTcLinear t;
        t.packed = (const uint8_t*)d.packed;
        t.q = d.q;
        t.act_scale = d.act_scale;
        t.y = d.y;
        t.acc_out = d.acc_out;
        t.w_scale = d.w_scale;
        t.T = (int)d.T;
        t.M = d.M;
        t.K = d.K;
        t.ldy = 0;
        run3.push_back(t);
      }
      int rc = 0;
      { const char* e = getenv("BITNET_STC_DBG"); if (!(e && (atoi(e) & 128))) rc = launch_quant_act_list(qrun.data(), (int64_t)qrun.size(), (cudaStream_t)stream); }
      if (rc) return rc;
      rc = launch_gemm_i2s_stream_tc(run3.data(), (int64_t)run3.size(), (cudaStream_t)stream);
      if (rc) return rc;
      continue;
    }
    if (!takes(items[i])) {
      const bitnet_group_item_t& d = items[i];
      int rc = bitnet_linear((bitnet_fmt_t)d.fmt, d.packed, d.w_scale, d.M, d.K, d.bk3, d.x, d.T, d.q, d.act_scale, d.y,
                             d.acc_out, d.workspace, d.workspace_bytes, stream);
      if (rc) return rc;
      ++i;
      continue;
    }
    run.clear();
    qrun.clear();
    for (; i < n && takes(items[i]); ++i) {
      const bitnet_group_item_t& d = items[i];
      GroupLinear gl;
      gl.packed = (const uint8_t*)d.packed;
      gl.x = d.x;
      gl.q = d.q;
      gl.act_scale = d.act_scale;
      gl.y = d.y;
      gl.acc_out = d.acc_out;
      gl.w_scale = d.w_scale;
      const bool split = d.T > 8 && !(group_wide && gemv_i2s_group_item_supported((int)d.T, d.M, d.K));
      gl.T = (int)(split ? 8 : d.T);
      gl.M = d.M;
      gl.K = d.K;
      gl.ldy = 0;
      if (d.T > 8 && !split) {
        // 9 to 16 tokens in one item: the codes come from one quantiser launch over all such items of the run (a CTA
        // of the grouped kernel would quantise 16 rows per linear it touches: more L2 reads than weight bytes)
        if (qrun.empty() || qrun.back().x != d.x || qrun.back().q != d.q || qrun.back().act_scale != d.act_scale ||
            qrun.back().K != d.K || qrun.back().T != (int)d.T)
          qrun.push_back(QuantListItem{d.x, d.q, d.act_scale, d.K, (int)d.T});
        gl.x = nullptr;
      }
      run.push_back(gl);
      if (split) {                         // the remaining tokens: a second item over the same weights
        gl.x = d.x + 8 * d.K;
        gl.q = d.q + 8 * d.K;
        gl.act_scale = d.act_scale + 8;
        gl.y = d.y + 8 * d.M;
        gl.acc_out = d.acc_out ? d.acc_out + 8 * d.M : nullptr;
        gl.T = (int)d.T - 8;
        run.push_back(gl);
      }
    }
    if (!qrun.empty()) {
      int rc = launch_quant_act_list(qrun.data(), (int64_t)qrun.size(), (cudaStream_t)stream);
      if (rc) return rc;
    }
    int rc = launch_gemv_i2s_group(run.data(), (int64_t)run.size(), (cudaStream_t)stream);
    if (rc) return rc;
  }
  return BITNET_OK;
}

int bitnet_linear_segments(bitnet_fmt_t fmt, const void* packed, int64_t M, int64_t K, int bk3, int64_t n_seg,
                           const int64_t* seg_end, const float* seg_scale, const float* x, int64_t T, int8_t* q,
                           float* act_scale, float* y, int32_t* acc_out, void* workspace, size_t workspace_bytes,
                           void* stream) {
  if (!packed || !x || !q || !act_scale || !y || !seg_end || !seg_scale || T < 1 || n_seg < 1 || n_seg > 16)
    return BITNET_ERR_INVALID_ARG;
  if (!aligned16(packed) || !aligned16(x) || !aligned16(q) || !aligned16(y) || (acc_out && !aligned16(acc_out)) ||
      (reinterpret_cast<uintptr_t>(act_scale) & 3u))
    return BITNET_ERR_INVALID_ARG;
  TlGeom g;
  int rc = fmt == BITNET_FMT_I2S ? i2s_shape(M, K) : tl_shape(fmt, M, K, bk3, &g);
  if (rc) return rc;
  // segments: ascending ends, the last one M; every segment but the last ends on a row block of the format
  // (16 rows for I2_S, 32 for TL), so that it is a contiguous piece of the blob
  const int64_t rows_per_block = fmt == BITNET_FMT_I2S ? 16 : 32;
  int64_t prev = 0;
  for (int64_t s = 0; s < n_seg; ++s) {
    if (seg_end[s] <= prev || seg_end[s] > M) return BITNET_ERR_INVALID_ARG;
    if (s + 1 < n_seg && (seg_end[s] % rows_per_block) != 0) return BITNET_ERR_UNSUPPORTED_SHAPE;
    prev = seg_end[s];
  }
  if (prev != M) return BITNET_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  static const bool grouped = [] { const char* e = getenv("BITNET_GROUP"); return !(e && atoi(e) == 0); }();
  // one grouped kernel: an item per segment, all sharing the input (quantised once per CTA), each writing its own
  // columns of y with its own scale
  if (grouped && fmt == BITNET_FMT_I2S && T <= 8) {
    bool ok = true;
    int64_t r0 = 0;
    for (int64_t s = 0; s < n_seg && ok; r0 = seg_end[s], ++s) ok = gemv_i2s_group_item_supported((int)T, seg_end[s] - r0, K);
    if (ok) {
      GroupLinear it[16];
      r0 = 0;
      for (int64_t s = 0; s < n_seg; r0 = seg_end[s], ++s) {
        it[s].packed = (const uint8_t*)packed + (size_t)(r0 / 16) * (size_t)(4 * i2s_kp(K));
        it[s].x = x;
        it[s].q = q;
        it[s].act_scale = act_scale;
        it[s].y = y + r0;
        it[s].acc_out = acc_out ? acc_out + r0 : nullptr;
        it[s].w_scale = seg_scale[s];
        it[s].T = (int)T;
        it[s].M = seg_end[s] - r0;
        it[s].K = K;
        it[s].ldy = M;
      }
      return launch_gemv_i2s_group(it, n_seg, st);
    }
  }
  if (grouped && fmt == BITNET_FMT_TL2 && T <= 8) {
    bool ok = true;
    int64_t r0 = 0;
    TlGeom gs[16];
    for (int64_t s = 0; s < n_seg && ok; r0 = seg_end[s], ++s)
      ok = tl_shape(fmt, seg_end[s] - r0, K, bk3, &gs[s]) == BITNET_OK && tl2_scan_takes(fmt, T, seg_end[s] - r0, K, gs[s]);
    if (ok) {
      Tl2Linear it[16];
      r0 = 0;
      for (int64_t s = 0; s < n_seg; r0 = seg_end[s], ++s)
        it[s] = scan_item((const uint8_t*)packed + (size_t)(r0 / 32) * (size_t)g.block_bytes, x, q, act_scale, y + r0,
                          acc_out ? acc_out + r0 : nullptr, seg_scale[s], T, seg_end[s] - r0, K, M, gs[s]);
      return launch_gemv_tl2_scan(it, n_seg, st);
    }
  }
  if (grouped && fmt == BITNET_FMT_TL1 && T <= 8) {
    bool ok = true;
    int64_t r0 = 0;
    TlGeom gs[16];
    for (int64_t s = 0; s < n_seg && ok; r0 = seg_end[s], ++s) ok = tl1_scan_takes(fmt, T, seg_end[s] - r0, K, &gs[s]);
    if (ok) {
      Tl2Linear it[16];
      r0 = 0;
      for (int64_t s = 0; s < n_seg; r0 = seg_end[s], ++s)
        it[s] = scan_item((const uint8_t*)packed + (size_t)(r0 / 32) * (size_t)g.block_bytes, x, q, act_scale, y + r0,
                          acc_out ? acc_out + r0 : nullptr, seg_scale[s], T, seg_end[s] - r0, K, M, gs[s]);
      return launch_gemv_elut_scan(it, n_seg, 3, st);
    }
  }
  // any other shape: the whole tensor with scale 1, then every segment's columns times its scale
  rc = bitnet_linear(fmt, packed, 1.0f, M, K, bk3, x, T, q, act_scale, y, acc_out, workspace, workspace_bytes, stream);
  if (rc) return rc;
  return launch_scale_segments(y, T, M, (int)n_seg, seg_end, seg_scale, st);
}

// ---- element-wise tables beyond ternary (App. A): g = 2, C = 3, 4, 5
static int elut_shape(int C, int g, int64_t M, int64_t K, TlGeom* geom) {
  if (C < 2 || g < 1 || M < 1 || K < 1 || M > 0x7fffffff) return BITNET_ERR_INVALID_ARG;
  if (g != 2 || !elut2_geom(C, M, K, geom)) return BITNET_ERR_UNSUPPORTED_SHAPE;
  return BITNET_OK;
}

size_t bitnet_elut_packed_bytes(int C, int g, int64_t M, int64_t K) {
  TlGeom geom;
  if (elut_shape(C, g, M, K, &geom)) return 0;
  return (size_t)(M / 32) * (size_t)geom.block_bytes;
}

int bitnet_pack_elut(int C, int g, const int8_t* w, int64_t M, int64_t K, void* packed, size_t packed_bytes,
                     int* dev_status, void* stream) {
  if (!w || !packed || !aligned16(packed)) return BITNET_ERR_INVALID_ARG;
  TlGeom geom;
  int rc = elut_shape(C, g, M, K, &geom);
  if (rc) return rc;
  if (packed_bytes < (size_t)(M / 32) * (size_t)geom.block_bytes) return BITNET_ERR_INVALID_ARG;
  return launch_pack_elut2(C, w, M, K, geom, (uint8_t*)packed, dev_status, (cudaStream_t)stream);
}

int bitnet_unpack_elut(int C, int g, const void* packed, int64_t M, int64_t K, int8_t* w, int* dev_status,
                       void* stream) {
  if (!w || !packed || !aligned16(packed)) return BITNET_ERR_INVALID_ARG;
  TlGeom geom;
  int rc = elut_shape(C, g, M, K, &geom);
  if (rc) return rc;
  return launch_unpack_elut2(C, (const uint8_t*)packed, M, K, geom, w, dev_status, (cudaStream_t)stream);
}

int bitnet_elut_linear_group(const bitnet_elut_item_t* items, int64_t n, void* stream) {
  if (n < 0 || (n > 0 && !items)) return BITNET_ERR_INVALID_ARG;
  static thread_local std::vector<Tl2Linear> run;
  run.clear();
  for (int64_t i = 0; i < n; ++i) {
    const bitnet_elut_item_t& d = items[i];
    if (!d.packed || !d.q || !d.act_scale || !d.y || d.T < 1 || d.T > 8) return BITNET_ERR_INVALID_ARG;
    if (!aligned16(d.packed) || (d.x && !aligned16(d.x)) || !aligned16(d.q) || !aligned16(d.y) ||
        (d.acc_out && !aligned16(d.acc_out)) || (reinterpret_cast<uintptr_t>(d.act_scale) & 3u))
      return BITNET_ERR_INVALID_ARG;
    Tl2Linear it;
    int rc = elut_shape(d.C, d.g, d.M, d.K, &it.g);
    if (rc) return rc;
    if (!gemv_elut_scan_item_supported((int)d.T, d.M, d.K, it.g)) return BITNET_ERR_UNSUPPORTED_SHAPE;
    run.push_back(scan_item(d.packed, d.x, d.q, d.act_scale, d.y, d.acc_out, d.w_scale, d.T, d.M, d.K, 0, it.g));
  }
  // one launch per run of items with the same cardinality (one decode table, one tile size per launch)
  for (int64_t i = 0; i < n;) {
    int64_t j = i + 1;
    while (j < n && items[j].C == items[i].C) ++j;
    int rc = launch_gemv_elut_scan(run.data() + i, j - i, items[i].C, (cudaStream_t)stream);
    if (rc) return rc;
    i = j;
  }
  return BITNET_OK;
}

}  // extern "C"

namespace {
// Side streams and events of bitnet_linear_host_batch, per device, created on first use and kept.  One mutex
// serialises the calls of all host threads: the call only queues work, and the events are shared.
struct HostPipe {
  cudaStream_t up = nullptr, down = nullptr;
  std::vector<cudaEvent_t> ev;
};
std::mutex g_host_pipe_mu;
HostPipe* host_pipe() {
  static HostPipe pipes[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return nullptr;
  HostPipe* p = &pipes[dev & 63];
  if (!p->up) {
    if (cudaStreamCreateWithFlags(&p->up, cudaStreamNonBlocking) != cudaSuccess) return nullptr;
    if (cudaStreamCreateWithFlags(&p->down, cudaStreamNonBlocking) != cudaSuccess) return nullptr;
  }
  return p;
}
bool grow_events(HostPipe* p, size_t n) {
  while (p->ev.size() < n) {
    cudaEvent_t e;
    if (cudaEventCreateWithFlags(&e, cudaEventDisableTiming) != cudaSuccess) return false;
    p->ev.push_back(e);
  }
  return true;
}
}  // namespace

extern "C" int bitnet_linear_host_batch(const bitnet_host_linear_t* items, int64_t n, void* stream) {
  if (n < 0 || (n > 0 && !items)) return BITNET_ERR_INVALID_ARG;
  if (n == 0) return BITNET_OK;
  for (int64_t i = 0; i < n; ++i) {
    const bitnet_host_linear_t& d = items[i];
    if (!d.packed || !d.x_host || !d.y_host || !d.x_dev || !d.q_dev || !d.scale_dev || !d.y_dev || d.T < 1 ||
        d.M < 1 || d.K < 1)
      return BITNET_ERR_INVALID_ARG;
  }
  std::lock_guard<std::mutex> lock(g_host_pipe_mu);
  // Items are handled in groups: one event after a group's uploads, one bitnet_linear_group call (for I2_S decode
  // items: one persistent kernel) per group, one event after it.  Five groups per batch, of 1, 4, 6, 4 and 1
  // sixteenths of the items: only the small first group's uploads and the small last group's downloads are not
  // hidden behind a kernel, a group's copies fit under its neighbour's kernel as long as they take no more than a
  // fifth of the kernel time per byte of activations (100B-shaped decode step: 0.3 ms up, 0.5 ms down, 2.5 ms of
  // kernels), and the fixed cost of a launch that waits for an event (no early start: ramp and drain) is paid
  // five times.  (Eight equal groups measured 2.99 ms per step against 2.52 for the kernels alone;
  // BITNET_HOST_GROUPS=n restores n equal groups.)
  static const int equal_groups = [] { const char* e = getenv("BITNET_HOST_GROUPS"); return e ? atoi(e) : 0; }();
  int64_t bounds[66];
  int64_t ngroups;
  if (equal_groups > 0 || n < 32) {
    ngroups = n < 32 ? 1 : (equal_groups > 64 ? 64 : equal_groups);
    if (ngroups > n) ngroups = n;
    for (int64_t g = 0; g <= ngroups; ++g) bounds[g] = n * g / ngroups;
  } else {
    ngroups = 5;
    bounds[0] = 0;
    bounds[1] = n / 16;
    bounds[2] = n * 5 / 16;
    bounds[3] = n - n * 5 / 16;
    bounds[4] = n - n / 16;
    bounds[5] = n;
  }
  HostPipe* p = host_pipe();
  if (!p || !grow_events(p, (size_t)(2 * ngroups + 2))) return note_cuda_error(cudaErrorUnknown);
  cudaStream_t st = (cudaStream_t)stream;
  cudaError_t e;
#define BN_TRY(call) do { e = (call); if (e != cudaSuccess) return note_cuda_error(e); } while (0)
  // the side streams start after whatever is already queued on `stream` (the staging buffers may be in use)
  cudaEvent_t e_in = p->ev[2 * ngroups], e_out = p->ev[2 * ngroups + 1];
  BN_TRY(cudaEventRecord(e_in, st));
  BN_TRY(cudaStreamWaitEvent(p->up, e_in, 0));
  BN_TRY(cudaStreamWaitEvent(p->down, e_in, 0));
  auto upload_group = [&](int64_t g) -> cudaError_t {
    const int64_t lo = bounds[g], hi = bounds[g + 1];
    // neighbouring items whose host and device buffers both continue where the previous item's end travel as
    // one copy (a caller that keeps its activations in one pinned block gets one copy per group)
    for (int64_t i = lo; i < hi;) {
      const char* src = reinterpret_cast<const char*>(items[i].x_host);
      char* dst = reinterpret_cast<char*>(items[i].x_dev);
      size_t bytes = (size_t)items[i].T * items[i].K * sizeof(float);
      int64_t j = i + 1;
      while (j < hi && reinterpret_cast<const char*>(items[j].x_host) == src + bytes &&
             reinterpret_cast<char*>(items[j].x_dev) == dst + bytes) {
        bytes += (size_t)items[j].T * items[j].K * sizeof(float);
        ++j;
      }
      cudaError_t er = cudaMemcpyAsync(dst, src, bytes, cudaMemcpyHostToDevice, p->up);
      if (er != cudaSuccess) return er;
      i = j;
    }
    return cudaEventRecord(p->ev[2 * g], p->up);
  };
  static thread_local std::vector<bitnet_group_item_t> grp;
  // uploads are queued one group ahead of the kernels, so that the first kernel does not wait for the host to
  // have queued every upload of the batch
  BN_TRY(upload_group(0));
  for (int64_t g = 0; g < ngroups; ++g) {
    if (g + 1 < ngroups) BN_TRY(upload_group(g + 1));
    const int64_t lo = bounds[g], hi = bounds[g + 1];
    BN_TRY(cudaStreamWaitEvent(st, p->ev[2 * g], 0));
    grp.clear();
    for (int64_t i = lo; i < hi; ++i) {
      const bitnet_host_linear_t& d = items[i];
      bitnet_group_item_t gi;
      gi.fmt = d.fmt;
      gi.bk3 = d.bk3;
      gi.packed = d.packed;
      gi.w_scale = d.w_scale;
      gi.M = d.M;
      gi.K = d.K;
      gi.T = d.T;
      gi.x = d.x_dev;
      gi.q = d.q_dev;
      gi.act_scale = d.scale_dev;
      gi.y = d.y_dev;
      gi.acc_out = nullptr;
      gi.workspace = d.workspace;
      gi.workspace_bytes = d.workspace_bytes;
      grp.push_back(gi);
    }
    int rc = bitnet_linear_group(grp.data(), (int64_t)grp.size(), stream);
    if (rc) {
      // join the side streams before reporting, so that nothing of this call is left dangling
      cudaEventRecord(e_out, p->down);
      cudaStreamWaitEvent(st, e_out, 0);
      cudaEventRecord(e_out, p->up);
      cudaStreamWaitEvent(st, e_out, 0);
      return rc;
    }
    BN_TRY(cudaEventRecord(p->ev[2 * g + 1], st));
    BN_TRY(cudaStreamWaitEvent(p->down, p->ev[2 * g + 1], 0));
    for (int64_t i = lo; i < hi;) {
      char* dst = reinterpret_cast<char*>(items[i].y_host);
      const char* src = reinterpret_cast<const char*>(items[i].y_dev);
      size_t bytes = (size_t)items[i].T * items[i].M * sizeof(float);
      int64_t j = i + 1;
      while (j < hi && reinterpret_cast<char*>(items[j].y_host) == dst + bytes &&
             reinterpret_cast<const char*>(items[j].y_dev) == src + bytes) {
        bytes += (size_t)items[j].T * items[j].M * sizeof(float);
        ++j;
      }
      BN_TRY(cudaMemcpyAsync(dst, src, bytes, cudaMemcpyDeviceToHost, p->down));
      i = j;
    }
  }
  BN_TRY(cudaEventRecord(e_out, p->down));
  BN_TRY(cudaStreamWaitEvent(st, e_out, 0));
#undef BN_TRY
  return BITNET_OK;
}
