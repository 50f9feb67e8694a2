/*
 * bitnet_b200 -- ternary-weight mixed-precision GEMV/GEMM (mpGEMM) for NVIDIA B200 (sm_100a).
 *
 * C ABI of libbitnet_b200.so.  The operation is the one the paper states in Alg. 1 / Eq. 1:
 *
 *     A_q      = Quantization(A)                      A: activations, T tokens x K features, fp32
 *     acc[t,m] = sum_k A_q[t,k] * W[m,k]              W: M x K ternary weights in {-1,0,+1}
 *     y[t,m]   = acc[t,m] * act_scale[t] * w_scale    ("Int2 with a Scale", Sec. 3.2.2)
 *
 * reached through three weight encodings: I2_S (2 bits per weight, multiply-add; Table 1,
 * Sec. 3.2.2), TL1 (pairs of weights -> 4-bit table index, Table 4 / Alg. 3) and TL2 (triples ->
 * 4-bit index + 1-bit sign, Table 5 / Alg. 4, Sec. 3.1).  All three give the same int32
 * accumulators as the definition (the lossless variants of Sec. 3.2).
 *
 * Naming: T = tokens (the paper's N), K = reduction length, M = output features; y and acc are
 * token-major [T][M].
 *
 * Conventions for every entry point unless stated otherwise:
 *   - pointers are DEVICE pointers owned by the caller; nothing is retained after the call;
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream); work is queued
 *     on it and the call returns without synchronising;
 *   - the library allocates no device memory and never throws; the return value is a status code
 *     below, and no kernel is launched when argument validation fails;
 *   - x, q, packed blobs, y, acc_out and workspaces must be 16-byte aligned.
 */
#ifndef BITNET_B200_H
#define BITNET_B200_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum { BITNET_FMT_I2S = 0, BITNET_FMT_TL1 = 1, BITNET_FMT_TL2 = 2 } bitnet_fmt_t;

enum {
  BITNET_OK = 0,
  BITNET_ERR_INVALID_ARG = 1,       /* null or misaligned pointer, bad enum, non-positive size       */
  BITNET_ERR_UNSUPPORTED_SHAPE = 2, /* K % 64 != 0 (I2_S); K odd or M % 32 != 0 (TL); bad bk3         */
  BITNET_ERR_WORKSPACE = 3,         /* workspace missing or smaller than *_workspace_bytes reports   */
  BITNET_ERR_BAD_WEIGHT = 4,        /* reserved: packers report bad weights through dev_status       */
  BITNET_ERR_CUDA = 5,              /* a CUDA call failed; see bitnet_last_cuda_error()              */
  BITNET_ERR_TIMEOUT = 6            /* a bounded device-side wait gave up (reported via dev_status)  */
};

/* Text for a status code (static storage). */
const char* bitnet_status_string(int status);
/* The cudaError_t of the most recent failing CUDA call made by this library on this thread. */
int bitnet_last_cuda_error(void);

/*
 * Device-side status: kernels that wait on asynchronous copies bound every wait; a wait that gave up
 * stores BITNET_ERR_TIMEOUT in a device flag.  This call synchronises the device and copies the flag
 * to *status_out (0 = no kernel ever gave up).  Not for the hot path.
 */
int bitnet_device_status(int* status_out);
/* Synchronises the device and clears the flag (after a reported time-out has been dealt with). */
int bitnet_device_status_clear(void);

/*
 * Early start (on by default).  The quantiser and the I2_S decode kernel are launched with
 * programmatic dependent launch: their prologue may run while the previous kernel queued on the same
 * stream is finishing, and the decode kernel starts copying the PACKED WEIGHTS into shared memory
 * before that kernel has finished (activations, scales and outputs are touched only after it has).
 * Packed weights are treated as read-only model state.  A blob written by this library's own packers is
 * safe to use at once: the first kernel the library launches on a stream after a packer was queued on it
 * starts in plain stream order (the library remembers such streams; a few words of host state).  If a
 * blob was written by other work queued earlier on the same stream (a copy, a kernel of the caller),
 * synchronise (or record/wait an event) before the first call that reads it, or switch early start off.
 * enable = 0 restores plain stream order for every later call.
 */
void bitnet_set_early_start(int enable);

/*
 * Which kernel serves TL1 and TL2 batches of up to 8 tokens (process-wide; also set by BITNET_TL2=lut in the
 * environment).
 *   0 (default): the scan kernel -- every packed index byte (TL2: plus its sign bits) is resolved by one
 *      shared-memory table lookup into the weights it stands for (Tables 4, 5), which go through the int8 tensor
 *      cores; 4 to 5 times the rate of the other form on a B200.  Shapes it does not take (K not a multiple of 4,
 *      fewer than three tiles per warp, more codes than fit beside its 128 KB table) fall back to the other form.
 *   1: the element-wise lookup-table kernel of Alg. 2 / Alg. 4 as the paper states it -- per-token tables of
 *      activation partial sums, one lookup, conditional negate and add per packed index.
 * Both give the same integers.
 */
void bitnet_set_tl2_lookup(int enable);

/*
 * Activation quantiser -- Alg. 1 Phase 1 ("Quantization"), Sec. 2.1 and 3.2.2: absmax int8.
 *   x[T][K] fp32 row-major (read)  ->  q[T][K] int8, act_scale[T] fp32, act_sum[T] int32 (nullable).
 * Per token t: amax = max(max_k |x[t,k]|, 1e-5); s = 127/amax (binary32); q = clamp(rint(x*s),
 * -128, 127), ties to even; act_scale[t] = amax/127; act_sum[t] = sum_k q[t,k].
 * per_tensor != 0 takes one amax over all T*K values (the paper's "per-tensor" wording); it equals
 * the per-token result at T = 1.
 */
int bitnet_quant_act(const float* x, int64_t T, int64_t K, int per_tensor, int8_t* q,
                     float* act_scale, int32_t* act_sum, void* stream);

/*
 * I2_S weight packer -- I2_S of Table 1 / Sec. 3.2.2 (2 bits per weight; the scale stays outside).
 *   w[M][K] int8 in {-1,0,+1}, row-major (read) -> packed, bitnet_i2s_packed_bytes(M,K) bytes.
 * Layout (code = w+1 in two bits; padding holds weight 0): rows in blocks of 16 (M padded to a
 * multiple of 16), K padded to a multiple of 256.  A block is contiguous: for each chunk c of 256
 * columns it holds 1024 bytes, of which row r of the block owns bytes [64r, 64r+64) = 16 little-endian
 * words.  Column kk = k % 256 of a chunk sits in word j = 2*(kk/32) + (kk%8)/4, byte b = kk%4, bits
 * [2s, 2s+1] with s = (kk%32)/8.  (Any K-slab of a 16-row block -- the tile of one int8 MMA -- is one
 * contiguous piece for a bulk copy; 32 lanes reading 16 bytes each cover 8 rows x 64 bytes without
 * bank conflicts; the two activation words an MMA needs for words 2h, 2h+1 are adjacent.)
 * dev_status (nullable device int): set to BITNET_ERR_BAD_WEIGHT if a non-ternary byte is met
 * (the blob is then undefined).  Requires K % 64 == 0.
 */
size_t bitnet_i2s_packed_bytes(int64_t M, int64_t K);
int bitnet_pack_i2s(const int8_t* w, int64_t M, int64_t K, void* packed, size_t packed_bytes,
                    int* dev_status, void* stream);

/*
 * TL weight packer -- Alg. 3 / Alg. 4 "PreprocessWeights" with the codes of Tables 4 and 5, the
 * signed-unsigned split and the block-fitting split ThreeK/TwoK of Sec. 3.1.2.
 *   fmt = BITNET_FMT_TL1 or BITNET_FMT_TL2; bk3 = BK3 (0 = 96; a positive multiple of 96).
 *   TL2: columns [0, ThreeK), ThreeK = floor(K/bk3)*bk3, are coded as triples
 *        (v = 9w0+3w1+w2, index |v|, sign [v<0]); the remaining TwoK columns as TL1 pairs
 *        (index 3(w0+1)+(w1+1)).  TL1: all columns as pairs.
 * Blob: for each block of 32 rows, ThreeK/96 tiles of 640 bytes then ceil(TwoK/64) tiles of 512
 * bytes.  A row of a tile has 16 index bytes, byte i = index of group 2i (low nibble) and 2i+1 (high
 * nibble).  Row r = g + 8u of the block (g = r % 8, u = r / 8) keeps byte i at 64g + 16(i/4) + 4u + i%4 of
 * the 512-byte index plane: every 16-byte piece holds one 32-bit word of the four rows g, g+8, g+16, g+24
 * (the rows one lane of a 16x8x32 tensor-core MMA owns in the two halves of the block).  A TL2 tile ends
 * with the 128-byte sign plane: row r's little-endian uint32 at 512 + 16g + 4u, the sign of group grp
 * (index byte i = grp/2) in its bit 8(i%4) + 2(i/4) + grp%2.  Pairs past K carry index 4 = (0,0).
 * Requires K even and M % 32 == 0.  dev_status as for bitnet_pack_i2s.
 */
size_t bitnet_tl_packed_bytes(bitnet_fmt_t fmt, int64_t M, int64_t K, int bk3);
int bitnet_pack_tl(bitnet_fmt_t fmt, const int8_t* w, int64_t M, int64_t K, int bk3, void* packed,
                   size_t packed_bytes, int* dev_status, void* stream);

/*
 * mpGEMM -- Alg. 1 Phase 2 (I2_S, multiply-add) or Alg. 2 / 3 / 4 (TL: per-token tables of group
 * partial sums built in shared memory, then one lookup per packed index; Eq. 3), followed by the
 * rescale y = acc * (act_scale[t] * w_scale).
 *   packed   blob from the packer of `fmt` for an M x K matrix (bk3 as given to the packer);
 *   q[T][K]  int8, act_scale[T] fp32 from bitnet_quant_act;
 *   y[T][M]  fp32 out; acc_out[T][M] int32 out, nullable (raw accumulators);
 *   workspace  bitnet_mpgemm_workspace_bytes(fmt,T,M,K) bytes (may be NULL when that is 0: I2_S with
 *              T <= 8 needs none except for extreme shapes; I2_S with 9 <= T <= 64, and with more tokens
 *              when the output has fewer 128 x 256 tiles than three quarters of the SMs, keeps the T*M
 *              int32 sums of its K-slices there; TL keeps its lookup tables and split-K sums there).
 *              TL calls clear what they rely on themselves: their workspace may hold anything.  For the
 *              I2_S kernels that keep sums there, the workspace must have been zeroed once with
 *              bitnet_workspace_init; its head (the sums) is left zeroed by every completed I2_S call, and a
 *              workspace last used by a TL call is initialised again before an I2_S call uses it.  Two
 *              calls sharing a workspace must not overlap on the GPU.
 * I2_S: T <= 8 runs the decode GEMV kernel; 9 <= T <= 64 a scan of the weights on mma.sync tensor-core
 * tiles over K-slices followed by a rescale kernel (when the workspace is missing or too small, the
 * prefill kernel takes the call instead) -- except that a tensor with many 128-row tiles (two thirds of a
 * tile per SM at 25..64 tokens, one tile per SM at 65..128) goes to the streaming tcgen05 kernel of
 * bitnet_linear_group, which needs no workspace; larger T the tcgen05 prefill kernel (whole tiles per CTA; parts
 * of a tile's K per CTA when there are few tiles and the workspace is there).  TL runs a decode kernel over
 * groups of 8 tokens (the scan kernel, see bitnet_set_tl2_lookup); from 128 tokens on, with K a multiple of
 * 64 and the workspace bitnet_mpgemm_workspace_bytes asks for, the TL blob is first turned into its I2_S form
 * inside the workspace (a device-side transcode of the packed codes) and the tcgen05 prefill kernel serves the
 * call, so that a model kept only in the 1.67-bit TL2 encoding has a tensor-core prefill too.  The integer
 * results do not depend on which kernel ran.
 */
size_t bitnet_mpgemm_workspace_bytes(bitnet_fmt_t fmt, int64_t T, int64_t M, int64_t K);
int bitnet_workspace_init(void* workspace, size_t workspace_bytes, void* stream);
int bitnet_mpgemm(bitnet_fmt_t fmt, const void* packed, float w_scale, int64_t M, int64_t K, int bk3,
                  const int8_t* q, const float* act_scale, int64_t T, float* y, int32_t* acc_out,
                  void* workspace, size_t workspace_bytes, void* stream);

/*
 * One linear layer from fp32 activations: Alg. 1 end to end -- Phase 1 (quantiser), Phase 2 (mpGEMM)
 * and the rescale -- with device buffers.
 *   x[T][K] fp32 in; q[T][K] int8 and act_scale[T] fp32 are OUTPUTS (the quantised activations, as
 *   bitnet_quant_act would give them); y[T][M] fp32 out; acc_out nullable; workspace as for
 *   bitnet_mpgemm.
 * For I2_S with T <= 8 (and T*(K+64) up to 144 KiB) this is ONE kernel: every CTA of the decode kernel
 * quantises the activation rows itself while its first weight tiles are in flight.  Exception: with 6 or
 * more tokens, or more than 96 KiB of codes (T * K padded to 256), and a workspace of the size
 * bitnet_mpgemm_workspace_bytes reports, the stand-alone quantiser and the mid-batch kernel run instead
 * (faster there).  Otherwise it is bitnet_quant_act followed by bitnet_mpgemm.  Results are identical
 * whichever kernels run.
 */
int bitnet_linear(bitnet_fmt_t fmt, const void* packed, float w_scale, int64_t M, int64_t K, int bk3,
                  const float* x, int64_t T, int8_t* q, float* act_scale, float* y, int32_t* acc_out,
                  void* workspace, size_t workspace_bytes, void* stream);

/*
 * One linear layer with HOST activations and HOST results: copies x_host[T][K] to x_dev, runs
 * bitnet_linear, and copies y_dev[T][M] to y_host, all queued on `stream`
 * (Alg. 1 end to end).  x_host / y_host should be pinned for the copies to be asynchronous; the
 * device buffers x_dev [T*K fp32], q_dev [T*K int8], scale_dev [T fp32], y_dev [T*M fp32] and the
 * workspace are caller-owned scratch.  The caller synchronises the stream before reading y_host.
 */
int bitnet_linear_host(bitnet_fmt_t fmt, const void* packed, float w_scale, int64_t M, int64_t K,
                       int bk3, const float* x_host, int64_t T, float* y_host, float* x_dev,
                       int8_t* q_dev, float* scale_dev, float* y_dev, void* workspace,
                       size_t workspace_bytes, void* stream);

/*
 * A batch of linear layers with HOST activations and HOST results (Alg. 1 end to end per item), with the
 * copies overlapped with the kernels.  The batch is cut into five groups of consecutive items, of 1, 4, 6, 4 and 1
 * sixteenths of the items (one group below 32 items): only the first group's uploads and the last group's
 * downloads are not hidden behind a kernel.  A group's x_host are uploaded on an internal stream, the group runs as one bitnet_linear_group
 * call on `stream` (one persistent kernel for I2_S decode items) once those uploads are complete, and its y_host
 * are downloaded on a second internal stream once the group is complete, while the next groups' uploads and
 * kernels proceed.  The items of a batch must therefore be independent of one another, as for
 * bitnet_linear_group.  When the call returns everything is queued, and `stream` has been made to wait for the
 * last download, so work queued on `stream` afterwards (or a synchronisation of `stream`) follows every copy of
 * the batch.
 *   - items[n]: plain structs in host memory, read during the call only.
 *   - x_host / y_host should be pinned.  The device buffers of different items must not overlap
 *     (uploads run ahead of the kernels); the workspace may be shared (the kernels are serial).
 *     Neighbouring items of a group whose x_host and x_dev (or y_dev and y_host) both start where the
 *     previous item's end are copied with one call: keeping the activations of a batch in one pinned
 *     block and one device block, in item order, saves a driver call per item and direction.
 *   - The internal streams and events are created on first use per device and kept for the life of the
 *     process; a mutex serialises concurrent calls from several host threads while they queue their work.
 *   - Errors: BITNET_ERR_INVALID_ARG for a null or malformed item (nothing of that item or later ones
 *     is queued); otherwise the status of the first failing call.
 */
typedef struct bitnet_host_linear {
  int32_t fmt;            /* bitnet_fmt_t */
  int32_t bk3;
  const void* packed;
  float w_scale;
  int64_t M, K, T;
  const float* x_host;    /* [T][K] */
  float* y_host;          /* [T][M] */
  float* x_dev;           /* scratch [T*K] fp32 */
  int8_t* q_dev;          /* scratch [T*K] int8 */
  float* scale_dev;       /* scratch [T] fp32 */
  float* y_dev;           /* scratch [T*M] fp32 */
  void* workspace;
  size_t workspace_bytes;
} bitnet_host_linear_t;
int bitnet_linear_host_batch(const bitnet_host_linear_t* items, int64_t n, void* stream);

/*
 * A list of linear layers on DEVICE buffers in one call (Alg. 1 end to end per item: Phase 1 quantiser,
 * Phase 2 mpGEMV, rescale), for linears whose inputs all exist when the call is queued: the Q/K/V or
 * gate/up projections of one decoder layer, or every linear of a benchmark sweep.  No item may read what
 * another item of the same call writes.
 *   - items[n]: plain structs in host memory, read during the call only.  Per item, as for bitnet_linear:
 *     x[T][K] fp32 in, q[T][K] int8 and act_scale[T] fp32 out, y[T][M] fp32 out, acc_out nullable.
 *     Items that share an input may share x, q and act_scale (neighbouring I2_S items with the same x, K and
 *     T are quantised once per CTA).
 *   - I2_S items with T <= 8 and K >= 1024 run in ONE persistent kernel per run of up to 409 consecutive
 *     such items: the packed weights of the whole run are one stream, cut into equal shares per SM at
 *     16-row borders; a CTA's asynchronous copies run on across the borders between linears, and each
 *     activation row is quantised by the two or three CTAs whose share touches its linear instead of by
 *     every CTA of a launch of its own (rows whose codes do not fit shared memory are walked in parts of K).
 *     The per-launch fixed cost of a decode GEMV (about 3 us of the 5-20 us a 100B-shaped linear takes) is
 *     paid once per run.  Items with 9 to 16 tokens run in launches of their own of the same kernel's
 *     two-group form (an MMA per group of eight tokens and weight register; the weights still cross HBM
 *     once), their codes coming from one quantiser launch over the run's activation matrices.
 *   - TL2 and TL1 items with T <= 8 (K a multiple of 4, at least three tiles per row) likewise run in one
 *     persistent kernel per run of up to 340 consecutive items of the same format (the scan kernel, see
 *     bitnet_set_tl2_lookup).
 *   - I2_S items with 17 to 128 tokens and 2048 <= K <= 131072: one quantiser launch over the run's
 *     activation matrices, then ONE persistent kernel per run of up to 160 such items of the same class (up to
 *     64 tokens, 65 to 128) that reads every blob once, unpacks the codes into tensor memory and multiplies on
 *     the tcgen05 tensor cores.
 *   - Every other item (more tokens, short K) is run by bitnet_linear in list order, with the item's
 *     workspace.
 * Results are identical to calling bitnet_linear per item.  Errors: BITNET_ERR_INVALID_ARG for a null or
 * malformed item (nothing is queued), otherwise the status of the first failing launch.
 */
typedef struct bitnet_group_item {
  int32_t fmt;            /* bitnet_fmt_t */
  int32_t bk3;
  const void* packed;
  float w_scale;
  int64_t M, K, T;
  const float* x;         /* [T][K] fp32, device */
  int8_t* q;              /* [T][K] int8, device, out */
  float* act_scale;       /* [T] fp32, device, out */
  float* y;               /* [T][M] fp32, device, out */
  int32_t* acc_out;       /* [T][M] int32, device, out, nullable */
  void* workspace;        /* only used by items the grouped kernel does not take */
  size_t workspace_bytes;
} bitnet_group_item_t;
int bitnet_linear_group(const bitnet_group_item_t* items, int64_t n, void* stream);

/*
 * One linear layer whose packed tensor is several matrices stacked by rows -- fused Q/K/V, gate and up -- each
 * quantised with its own scale: "Int2 with a Scale" (Sec. 3.2.2) per stacked matrix.  Same arguments and results
 * as bitnet_linear, except that rows [seg_end[s-1], seg_end[s]) of the output are rescaled with seg_scale[s]:
 *     y[t,m] = acc[t,m] * act_scale[t] * seg_scale[s(m)].
 *   - seg_end[n_seg], seg_scale[n_seg]: HOST arrays, read during the call; 1 <= n_seg <= 16; ends ascending, the
 *     last one M; every end but the last a multiple of the format's row block (16 for I2_S, 32 for TL), so that a
 *     segment is a contiguous piece of the blob packed from the stacked matrix.
 *   - I2_S and TL2 with T <= 8 (shapes the grouped kernels take): ONE persistent kernel, an item per segment, the
 *     shared input quantised once per CTA.  Otherwise the whole tensor runs with scale 1 and a small kernel
 *     multiplies every segment's columns by its scale (one more fp32 rounding, inside the 1e-6 relative bound).
 */
int bitnet_linear_segments(bitnet_fmt_t fmt, const void* packed, int64_t M, int64_t K, int bk3, int64_t n_seg,
                           const int64_t* seg_end, const float* seg_scale, const float* x, int64_t T, int8_t* q,
                           float* act_scale, float* y, int32_t* acc_out, void* workspace, size_t workspace_bytes,
                           void* stream);

/*
 * Element-wise tables beyond ternary (App. A, "ELUT mpGEMM"; Table 3).  Weights of cardinality C take the C
 * consecutive integers from -(C/2) (integer division): {-1,0,1} for C = 3, {-2,..,1} for C = 4, {-2,..,2} for
 * C = 5.  g weights form a group, stored as the group's index = its weights + C/2 read as a base-C number, first
 * weight most significant, in ceil(log2(C^g)) bits.  Built: g = 2 with C = 3, 4 (4 bits per pair: 2 bits per
 * weight) and C = 5 (5 bits per pair: 2.5 bits per weight, against 3 for bit-wise storage); other (C, g) return
 * BITNET_ERR_UNSUPPORTED_SHAPE.
 *
 * Blob (M a multiple of 32, K even; the kernels need K a multiple of 4): 32-row blocks, each a sequence of
 * ceil(K/64) tiles of 32 rows x 32 pairs.  A tile's first 512 bytes hold the low four bits of every index exactly
 * where a TL1 tile keeps its codes (see bitnet_pack_tl); for C = 5 another 128 bytes follow with the fifth bits,
 * placed where a TL2 tile keeps its signs.  Columns past K are zero weights.  For C = 3 the blob is the TL1 blob.
 *
 * bitnet_pack_elut: w[M][K] int8 in the alphabet -> packed; dev_status (nullable device int) is set to
 * BITNET_ERR_BAD_WEIGHT if a value outside the alphabet is met.  bitnet_unpack_elut is its inverse (a test hook).
 *
 * bitnet_elut_linear_group: a list of linear layers (as bitnet_linear_group: y = acc * act_scale[t] * w_scale,
 * acc[t,m] = sum_k q[t,k] w[m,k]) over such blobs, 1..8 tokens each, on DEVICE buffers.  Per item x[T][K] fp32 in and
 * q, act_scale out (Phase 1 runs inside the kernel) -- or x = NULL and q, act_scale are inputs.  Runs of items
 * with the same C are ONE persistent kernel that reads every blob once: an index byte plus its fifth bits selects
 * an entry of a shared-memory table that holds the four weights of the two pairs, which go to the int8 tensor cores
 * as they are (the table is indexed by the packed weights rather than filled from the activations: Phase 1 of the
 * algorithm then costs nothing per token and the lookups feed 4 weights x 8 tokens each).  At C = 4 the index is two
 * 2-bit codes side by side and is taken apart by masks instead (BITNET_ELUT4=table: through the table).  Integer results are
 * exact.  Errors: BITNET_ERR_INVALID_ARG (null or misaligned pointer, T outside 1..8), BITNET_ERR_UNSUPPORTED_SHAPE
 * ((C, g) not built, M % 32, K % 4, rows too short for the kernel's rings: K < 192); nothing is queued then.
 */
size_t bitnet_elut_packed_bytes(int C, int g, int64_t M, int64_t K);
int bitnet_pack_elut(int C, int g, const int8_t* w, int64_t M, int64_t K, void* packed, size_t packed_bytes,
                     int* dev_status, void* stream);
int bitnet_unpack_elut(int C, int g, const void* packed, int64_t M, int64_t K, int8_t* w, int* dev_status,
                       void* stream);
typedef struct bitnet_elut_item {
  int32_t C, g;
  const void* packed;
  float w_scale;
  int64_t M, K, T;
  const float* x;         /* [T][K] fp32, device; NULL: q and act_scale are inputs */
  int8_t* q;              /* [T][K] int8, device */
  float* act_scale;       /* [T] fp32, device */
  float* y;               /* [T][M] fp32, device, out */
  int32_t* acc_out;       /* [T][M] int32, device, out, nullable */
} bitnet_elut_item_t;
int bitnet_elut_linear_group(const bitnet_elut_item_t* items, int64_t n, void* stream);

/*
 * Table-lookup mpGEMV without a workspace argument (the paper has no counterpart: this entry point
 * exists for the sake of callers, not of the method).
 *
 * Same operation and arguments as bitnet_mpgemm for fmt = BITNET_FMT_TL1 / BITNET_FMT_TL2 and
 * T <= 8, but the scratch (the per-token lookup tables and the sums that join the K-slices) lives in
 * a fixed array inside the library (5.1 MiB, held by every GPU that loads the library until the
 * process exits).  It is meant for hosts that cannot call cudaMalloc or hand over a workspace:
 * code running while the device allocator is frozen or its pool is fully committed to weights,
 * latency-critical loops that must not make calls which can block or fail, and plug-ins that
 * receive input and output buffers only.  The call itself allocates nothing, on host or device.
 *   - M > BITNET_NOALLOC_MAX_M, K > BITNET_NOALLOC_MAX_K or T > 8 returns BITNET_ERR_WORKSPACE and
 *     launches nothing.
 *   - The first call on each device looks up the array's device address (a blocking runtime query);
 *     make that first call outside any stream capture.
 *   - Every call on a device shares the one array and clears the part it needs first, on `stream`;
 *     two calls that may run on the GPU at the same time (different streams) race on it.
 */
#define BITNET_NOALLOC_MAX_M 32768
#define BITNET_NOALLOC_MAX_K 32768
int bitnet_mpgemv_tl_noalloc(bitnet_fmt_t fmt, const void* packed, float w_scale, int64_t M, int64_t K,
                             int bk3, const int8_t* q, const float* act_scale, int64_t T, float* y,
                             int32_t* acc_out, void* stream);

/* ---- measurement hooks (not part of the path; the paper has no counterpart) ------------------- */
/*
 * The ceilings the decode kernels are judged against, measured rather than assumed (the host times the launches with
 * CUDA events).
 *   bitnet_microbench_read_stream: the grouped decode kernel's memory side alone -- persistent CTAs, per-warp rings of
 *     `depth` (4, 6 or 8) 1-KB chunks filled by 16-byte cp.async copies -- reads `bytes` bytes at buf (device, 16-byte
 *     aligned) once, no arithmetic.  sink: one device word the kernel may write.
 *   bitnet_microbench_issue: every warp of one 16-warp CTA per SM issues iters * 32 independent instructions of one
 *     kind: 0 dp4a, 1 lop3, 2 prmt, 3 32-bit multiply-add, 4 ld.shared.u32, 5 ld.shared.v4.u32,
 *     6 mma.sync.m16n8k32 (u8 x s8).
 */
int bitnet_microbench_read_stream(const void* buf, size_t bytes, int depth, unsigned* sink, void* stream);
int bitnet_microbench_issue(int kind, int iters, unsigned* sink, void* stream);

/* ---- test hooks (not part of the four operations) ------------------------------------------- */
/* Launches a one-CTA kernel whose bounded wait (the lookup-table kernel's own) is bound to run out: its barrier
 * expects bytes that no copy ever delivers.  Nothing is in flight, nothing faults; afterwards
 * bitnet_device_status reports BITNET_ERR_TIMEOUT until bitnet_device_status_clear. */
int bitnet_debug_wait_timeout_probe(void* stream);
/* Inverse of the packers: packed -> w[M][K] int8.  dev_status set if an invalid code is met. */
int bitnet_unpack_i2s(const void* packed, int64_t M, int64_t K, int8_t* w, int* dev_status,
                      void* stream);
int bitnet_unpack_tl(bitnet_fmt_t fmt, const void* packed, int64_t M, int64_t K, int bk3, int8_t* w,
                     int* dev_status, void* stream);
/* The tables of Alg. 3 / Alg. 4 "PreCompute" for one token, as the TL kernel builds them:
 * lut[group][16] int16, triples first (entry i = sum for the triple of value i, i = 0..13), then
 * pairs (entry i = sum for the pair of code i, i = 0..8); unused entries are zero.
 * bitnet_tl_num_groups gives the group count (32 per tile). */
int64_t bitnet_tl_num_groups(bitnet_fmt_t fmt, int64_t K, int bk3);
int bitnet_tl_build_lut_debug(bitnet_fmt_t fmt, const int8_t* q_row, int64_t K, int bk3, int16_t* lut,
                              void* stream);

#ifdef __cplusplus
}
#endif
#endif /* BITNET_B200_H */
