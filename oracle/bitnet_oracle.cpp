// CPU oracle for the ternary mixed-precision GEMM path (int8 activations x ternary weights).
//
// TEST INFRASTRUCTURE ONLY.  Plain, slow, scalar C++17 written from the paper's statement
// of the method; it shares no code, header, table or constant with the CUDA library and is
// never on the product path.  Only the tests, the smoke check and the benchmark's CPU
// baseline may call it.
//
// What each function follows:
//   oracle_quant_act      Alg. 1 Phase 1 ("Quantization"), Sec. 2.1 / Sec. 3.2.2 (int8 absmax
//                         activation quantisation); rounding and operation order: see below.
//   oracle_mpgemm_def     Alg. 1 Phase 2 / Eq. 1: R[n,m] = sum_k A_q[n,k] * W[m,k].
//   oracle_dequant        the "Scale" of I2_S (Sec. 3.2.2): y = acc * act_scale * w_scale.
//   oracle_dequant_segments  the same with one scale per stacked matrix of a fused tensor.
//   oracle_pack_i2s       I2_S, 2 bits per weight (Table 1); the byte layout is this build's.
//   oracle_pack_tl        TL1 codes of Table 4 (Alg. 3 PreprocessWeights); TL2 codes of
//                         Table 5 with the signed-unsigned split (Sec. 3.1.2, Alg. 4
//                         PreprocessWeights) and the block-fitting split ThreeK / TwoK.
//   oracle_tl_build_lut   Alg. 3 / Alg. 4 PreCompute (element-wise LUT, Eq. 3), int16 entries
//                         kept exact (Sec. 3.2.1, the lossless *_1 variants).
//   oracle_tl_mpgemm      Alg. 3 / Alg. 4 accumulation by table lookups from the packed blob,
//                         sign applied per group (caption of Fig. 5).
//   oracle_i2s_mpgemm     Alg. 1 Phase 2 evaluated straight from the I2_S blob.
//   oracle_elut_*         App. A: the element-wise table method for weights of any cardinality C in groups of
//                         g ("ELUT mpGEMM": Tbl-quantization, Table-setup, then one Lookup per group), the
//                         bits-per-weight figures of Table 3, and a packed form of the g = 2 case.
//
// Readings where the paper is silent (all listed in the design notes):
//   * activations are quantised per token (row of x); per_tensor != 0 gives the paper's
//     literal "per-tensor" wording (one absmax over all T*K values);
//   * amax is floored at 1e-5; s = 127 / amax in binary32; q = clamp(rint(x*s), -128, 127)
//     with round-half-to-even; act_scale = amax / 127 in binary32;
//   * TL2 code of a triple: v = 9*w0 + 3*w1 + w2, index = |v|, sign = [v < 0] -- this
//     reproduces every printed row of Table 5;
//   * TL1 code of a pair: 3*(w0+1) + (w1+1) -- Table 4;
//   * App. A gives weights "of cardinality C" without naming the values: here the C consecutive integers
//     from -(C/2) (integer division) upwards -- {-1,0,1} for C = 3 (the ternary case), {-2,..,1} for C = 4 (two's
//     complement int2), {-2,..,2} for C = 5; the index of a group is its weights read as a base-C number, first
//     weight most significant, each digit = weight + C/2 -- for C = 3, g = 2 exactly the codes of Table 4.
//
// Pins (tests/test_oracle_*.py): closed-form quantiser cases, brute-force enumeration on tiny
// shapes against numpy, one-hot position probes of every packed bit, Tables 4 and 5 as golden
// text fixtures, LUT identities, and I2_S == TL1 == TL2 == definition on random inputs.
// No function here is "parity unpinned".

#include <cmath>
#include <cstdint>
#include <cstdlib>
#include <cstring>
#include <vector>
#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

constexpr int FMT_I2S = 0;
constexpr int FMT_TL1 = 1;
constexpr int FMT_TL2 = 2;

inline int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }

// ---- TL geometry (Sec. 3.1.2).  A blob is a sequence of 32-row blocks; each block holds its triple-coded
// columns as tiles of 32 triples per row (96 weights, 640 bytes) followed by its pair-coded columns as tiles
// of 32 pairs per row (64 weights, 512 bytes).
struct TlGeom {
  int64_t three_k;      // ThreeK: columns coded as triples
  int64_t two_k;        // TwoK: columns coded as pairs
  int64_t tiles3;       // triple tiles per block
  int64_t tiles2;       // pair tiles per block
  int64_t block_bytes;  // bytes per block
};

bool tl_geom(int fmt, int64_t M, int64_t K, int bk3, TlGeom* g) {
  const int64_t BK3 = bk3 ? bk3 : 96;
  const bool shape_ok = M >= 32 && M % 32 == 0 && K >= 2 && K % 2 == 0 && BK3 > 0 && BK3 % 96 == 0;
  if (!shape_ok || (fmt != FMT_TL1 && fmt != FMT_TL2)) return false;
  // block-fitting split: ThreeK = floor(K / BK3) * BK3 columns as triples, the remaining TwoK as pairs;
  // TL1 codes every column as a pair
  const int64_t whole_blocks = (fmt == FMT_TL2) ? K / BK3 : 0;
  g->three_k = whole_blocks * BK3;
  g->two_k = K - g->three_k;
  g->tiles3 = g->three_k / 96;
  g->tiles2 = (g->two_k + 63) / 64;
  g->block_bytes = 640 * g->tiles3 + 512 * g->tiles2;
  return true;
}

// ---- positions inside a tile (this build's layout; the paper fixes only the codes and the split into an index
// plane and a sign plane).  Row r = g + 8u of the block (g = r % 8, u = r / 8); its 32 groups are 16 index bytes,
// byte i holding group 2i in the low nibble and group 2i+1 in the high nibble.
//   index plane (512 bytes): byte i of row r lies at 64g + 16(i/4) + 4u + i%4, i.e. the four rows g, g+8, g+16,
//     g+24 interleave word by word, each 16-byte piece holding word i/4 of those four rows;
//   sign plane of a triple tile (128 bytes at 512): row r owns the little-endian uint32 at 512 + 16g + 4u, and the
//     sign of group grp (index byte i = grp/2) is its bit 8(i%4) + 2(i/4) + grp%2.
inline int tl_idx_pos(int r, int grp) {
  const int i = grp / 2;
  return 64 * (r % 8) + 16 * (i / 4) + 4 * (r / 8) + (i % 4);
}
inline int tl_sign_pos(int r) { return 512 + 16 * (r % 8) + 4 * (r / 8); }
inline int tl_sign_bit(int grp) {
  const int i = grp / 2;
  return 8 * (i % 4) + 2 * (i / 4) + (grp % 2);
}

inline int tern_ok(int8_t w) { return w >= -1 && w <= 1; }

}  // namespace

extern "C" {

// ---------------------------------------------------------------------------------------------
// Quantiser.  x[T][K] fp32 -> q[T][K] int8, act_scale[T], act_sum[T] (nullable).
int oracle_quant_act(const float* x, int64_t T, int64_t K, int per_tensor, int8_t* q,
                     float* act_scale, int32_t* act_sum) {
  if (!x || !q || !act_scale || T < 1 || K < 1) return 1;
  float tensor_amax = 0.0f;
  if (per_tensor) {
    for (int64_t i = 0; i < T * K; ++i) tensor_amax = std::fmax(tensor_amax, std::fabs(x[i]));
  }
  for (int64_t t = 0; t < T; ++t) {
    const float* xr = x + t * K;
    float amax = 0.0f;
    if (per_tensor) {
      amax = tensor_amax;
    } else {
      for (int64_t k = 0; k < K; ++k) amax = std::fmax(amax, std::fabs(xr[k]));
    }
    const float amax_c = std::fmax(amax, 1e-5f);
    volatile float s = 127.0f / amax_c;        // one binary32 division
    volatile float inv = amax_c / 127.0f;      // one binary32 division
    act_scale[t] = inv;
    int64_t sum = 0;
    for (int64_t k = 0; k < K; ++k) {
      volatile float p = xr[k] * s;            // one binary32 product, no fused multiply-add
      float r = std::nearbyintf(p);            // round-half-to-even in the default mode
      if (r > 127.0f) r = 127.0f;
      if (r < -128.0f) r = -128.0f;
      const int v = (int)r;
      q[t * K + k] = (int8_t)v;
      sum += v;
    }
    if (act_sum) act_sum[t] = (int32_t)sum;
  }
  return 0;
}

// ---------------------------------------------------------------------------------------------
// Definition (Alg. 1 Phase 2).  acc[t][m] = sum_k q[t][k] * w[m][k].  Returns 2 on int32 overflow.
// The OpenMP pragma only spreads independent output rows over cores when the file is built with
// -fopenmp (the timed CPU baseline); the arithmetic is the same scalar loop either way.
int oracle_mpgemm_def(const int8_t* q, const int8_t* w, int64_t T, int64_t M, int64_t K,
                      int32_t* acc) {
  if (!q || !w || !acc || T < 1 || M < 1 || K < 1) return 1;
  int bad = 0;
#pragma omp parallel for schedule(static) reduction(| : bad)
  for (int64_t m = 0; m < M; ++m) {
    const int8_t* wr = w + m * K;
    for (int64_t t = 0; t < T; ++t) {
      const int8_t* qr = q + t * K;
      int64_t s = 0;
      for (int64_t k = 0; k < K; ++k) s += (int64_t)qr[k] * (int64_t)wr[k];
      if (s > INT32_MAX || s < INT32_MIN) bad |= 1;
      acc[t * M + m] = (int32_t)s;
    }
  }
  return bad ? 2 : 0;
}

// y[t][m] = acc * act_scale[t] * w_scale, evaluated in double.
void oracle_dequant(const int32_t* acc, const float* act_scale, float w_scale, int64_t T, int64_t M,
                    double* y) {
  for (int64_t t = 0; t < T; ++t)
    for (int64_t m = 0; m < M; ++m)
      y[t * M + m] = (double)acc[t * M + m] * (double)act_scale[t] * (double)w_scale;
}

// The same for a tensor made of several matrices stacked by rows (fused Q/K/V, gate and up), each with the scale it
// was quantised with: rows [seg_end[s-1], seg_end[s]) carry w_scale[s] (seg_end ascending, seg_end[n_seg-1] = M).
// "Int2 with a Scale" (Sec. 3.2.2) per stacked matrix.
int oracle_dequant_segments(const int32_t* acc, const float* act_scale, int64_t n_seg, const int64_t* seg_end,
                            const float* w_scale, int64_t T, int64_t M, double* y) {
  if (n_seg < 1 || seg_end[n_seg - 1] != M) return 1;
  for (int64_t t = 0; t < T; ++t) {
    int64_t row = 0;
    for (int64_t s = 0; s < n_seg; ++s) {
      if (seg_end[s] <= row) return 1;
      for (; row < seg_end[s]; ++row) y[t * M + row] = (double)acc[t * M + row] * (double)act_scale[t] * (double)w_scale[s];
    }
  }
  return 0;
}

// ---------------------------------------------------------------------------------------------
// I2_S.  code = w + 1 (0,1,2), two bits.  Rows are stored in blocks of 16 (M padded to a multiple of
// 16), K is padded to a multiple of 256; padding holds weight 0 (code 1).  A block is contiguous and
// holds, for each chunk c of 256 columns, 1024 bytes in which row r (0..15) owns bytes [64r, 64r+64).
// In those 64 bytes = 16 little-endian words, the weight at column kk = k % 256 of the chunk sits in
//   word j = 2*(kk/32) + (kk%8)/4,  byte b = kk%4 of that word,  bits [2s, 2s+1] with s = (kk%32)/8.
struct I2sPos {
  int64_t byte;
  int shift;
};
static I2sPos i2s_pos(int64_t m, int64_t k, int64_t kp) {
  const int64_t rb = m / 16, r = m % 16, c = k / 256, kk = k % 256;
  const int64_t j = 2 * (kk / 32) + (kk % 8) / 4, b = kk % 4, s = (kk % 32) / 8;
  return {rb * (4 * kp) + c * 1024 + r * 64 + 4 * j + b, (int)(2 * s)};
}

size_t oracle_i2s_packed_bytes(int64_t M, int64_t K) {
  if (M < 1 || K < 1) return 0;
  return (size_t)(ceil_div(M, 16) * 16) * (size_t)(ceil_div(K, 256) * 256) / 4;
}

int oracle_pack_i2s(const int8_t* w, int64_t M, int64_t K, uint8_t* packed) {
  if (!w || !packed || M < 1 || K < 1) return 1;
  const int64_t mp = ceil_div(M, 16) * 16, kp = ceil_div(K, 256) * 256;
  std::memset(packed, 0, (size_t)(mp * kp / 4));
  for (int64_t m = 0; m < mp; ++m)
    for (int64_t k = 0; k < kp; ++k) {
      const int8_t wk = (m < M && k < K) ? w[m * K + k] : (int8_t)0;
      if (!tern_ok(wk)) return 3;
      const I2sPos pos = i2s_pos(m, k, kp);
      packed[pos.byte] |= (uint8_t)((wk + 1) << pos.shift);
    }
  return 0;
}

int oracle_unpack_i2s(const uint8_t* packed, int64_t M, int64_t K, int8_t* w) {
  if (!w || !packed || M < 1 || K < 1) return 1;
  const int64_t kp = ceil_div(K, 256) * 256;
  for (int64_t m = 0; m < M; ++m)
    for (int64_t k = 0; k < K; ++k) {
      const I2sPos pos = i2s_pos(m, k, kp);
      const unsigned code = (packed[pos.byte] >> pos.shift) & 3u;
      if (code == 3u) return 3;
      w[m * K + k] = (int8_t)((int)code - 1);
    }
  return 0;
}

// Alg. 1 Phase 2 straight from the blob (decodes each weight where it is used).
int oracle_i2s_mpgemm(const uint8_t* packed, int64_t M, int64_t K, const int8_t* q, int64_t T,
                      int32_t* acc) {
  if (!packed || !q || !acc || M < 1 || K < 1 || T < 1) return 1;
  const int64_t kp = ceil_div(K, 256) * 256;
  for (int64_t m = 0; m < M; ++m)
    for (int64_t t = 0; t < T; ++t) {
      int64_t s = 0;
      for (int64_t k = 0; k < K; ++k) {
        const I2sPos pos = i2s_pos(m, k, kp);
        const int wv = (int)((packed[pos.byte] >> pos.shift) & 3u) - 1;
        s += (int64_t)q[t * K + k] * wv;
      }
      acc[t * M + m] = (int32_t)s;
    }
  return 0;
}

// ---------------------------------------------------------------------------------------------
// TL codes.
// Table 4: (w0, w1) -> 3*(w0+1) + (w1+1), 0..8.
int oracle_tl1_code(int w0, int w1) { return 3 * (w0 + 1) + (w1 + 1); }
// Table 5: v = 9 w0 + 3 w1 + w2; index |v| (0..13) in bits 0..3, sign [v<0] in bit 4.
int oracle_tl2_code(int w0, int w1, int w2) {
  const int v = 9 * w0 + 3 * w1 + w2;
  return (v < 0 ? 16 : 0) | (v < 0 ? -v : v);
}

size_t oracle_tl_packed_bytes(int fmt, int64_t M, int64_t K, int bk3) {
  TlGeom g;
  if (!tl_geom(fmt, M, K, bk3, &g)) return 0;
  return (size_t)(M / 32) * (size_t)g.block_bytes;
}

void oracle_tl_split(int fmt, int64_t K, int bk3, int64_t* three_k, int64_t* two_k) {
  TlGeom g;
  if (!tl_geom(fmt, 32, K, bk3, &g)) { *three_k = -1; *two_k = -1; return; }
  *three_k = g.three_k;
  *two_k = g.two_k;
}

// Blob = for each block of 32 rows: tiles3 TL2 tiles, then tiles2 TL1 tiles.
//  TL2 tile (640 B): 512-byte index plane (index of triple 2i in the low nibble of the row's byte i, of triple
//    2i+1 in the high nibble) then a 128-byte sign plane, one uint32 per row; positions as tl_idx_pos,
//    tl_sign_pos and tl_sign_bit above give them.
//  TL1 tile (512 B): the same index plane over 32 pairs; pairs past the end of K carry code 4 = (0,0).
int oracle_pack_tl(int fmt, const int8_t* w, int64_t M, int64_t K, int bk3, uint8_t* packed) {
  TlGeom g;
  if (!w || !packed || !tl_geom(fmt, M, K, bk3, &g)) return 1;
  std::memset(packed, 0, (size_t)(M / 32) * (size_t)g.block_bytes);
  for (int64_t m = 0; m < M; ++m) {
    const int64_t rb = m / 32, r = m % 32;
    uint8_t* blk = packed + rb * g.block_bytes;
    const int8_t* wr = w + m * K;
    for (int64_t k = 0; k < K; ++k)
      if (!tern_ok(wr[k])) return 3;
    for (int64_t t = 0; t < g.tiles3; ++t) {
      uint8_t* tile = blk + t * 640;
      uint32_t signs = 0;
      for (int grp = 0; grp < 32; ++grp) {
        const int64_t k = t * 96 + 3 * grp;
        const int code = oracle_tl2_code(wr[k], wr[k + 1], wr[k + 2]);
        const int idx = code & 15;
        if (code & 16) signs |= (1u << tl_sign_bit(grp));
        tile[tl_idx_pos((int)r, grp)] |= (uint8_t)((grp & 1) ? (idx << 4) : idx);
      }
      for (int b = 0; b < 4; ++b) tile[tl_sign_pos((int)r) + b] = (uint8_t)(signs >> (8 * b));
    }
    for (int64_t t = 0; t < g.tiles2; ++t) {
      uint8_t* tile = blk + g.tiles3 * 640 + t * 512;
      for (int grp = 0; grp < 32; ++grp) {
        const int64_t k = g.three_k + t * 64 + 2 * grp;
        const int idx = (k < K) ? oracle_tl1_code(wr[k], wr[k + 1]) : 4;
        tile[tl_idx_pos((int)r, grp)] |= (uint8_t)((grp & 1) ? (idx << 4) : idx);
      }
    }
  }
  return 0;
}

int oracle_unpack_tl(int fmt, const uint8_t* packed, int64_t M, int64_t K, int bk3, int8_t* w) {
  TlGeom g;
  if (!w || !packed || !tl_geom(fmt, M, K, bk3, &g)) return 1;
  for (int64_t m = 0; m < M; ++m) {
    const int64_t rb = m / 32, r = m % 32;
    const uint8_t* blk = packed + rb * g.block_bytes;
    int8_t* wr = w + m * K;
    for (int64_t t = 0; t < g.tiles3; ++t) {
      const uint8_t* tile = blk + t * 640;
      uint32_t signs = 0;
      for (int b = 0; b < 4; ++b) signs |= (uint32_t)tile[tl_sign_pos((int)r) + b] << (8 * b);
      for (int grp = 0; grp < 32; ++grp) {
        const uint8_t byte = tile[tl_idx_pos((int)r, grp)];
        const int idx = (grp & 1) ? (byte >> 4) : (byte & 15);
        if (idx > 13) return 3;
        const bool neg = ((signs >> tl_sign_bit(grp)) & 1u) != 0;
        int v = neg ? -idx : idx;
        if (idx == 0 && neg) return 3;
        // balanced-ternary digits of v in [-13, 13]
        int d[3];
        for (int i = 2; i >= 0; --i) {
          int rem = ((v % 3) + 3) % 3;  // 0,1,2
          if (rem == 2) rem = -1;
          d[i] = rem;
          v = (v - rem) / 3;
        }
        const int64_t k = t * 96 + 3 * grp;
        wr[k] = (int8_t)d[0];
        wr[k + 1] = (int8_t)d[1];
        wr[k + 2] = (int8_t)d[2];
      }
    }
    for (int64_t t = 0; t < g.tiles2; ++t) {
      const uint8_t* tile = blk + g.tiles3 * 640 + t * 512;
      for (int grp = 0; grp < 32; ++grp) {
        const uint8_t byte = tile[tl_idx_pos((int)r, grp)];
        const int idx = (grp & 1) ? (byte >> 4) : (byte & 15);
        if (idx > 8) return 3;
        const int64_t k = g.three_k + t * 64 + 2 * grp;
        if (k < K) {
          wr[k] = (int8_t)(idx / 3 - 1);
          wr[k + 1] = (int8_t)(idx % 3 - 1);
        } else if (idx != 4) {
          return 3;
        }
      }
    }
  }
  return 0;
}

// Number of 16-slot tables one token needs: ThreeK/3 triples followed by tiles2*32 pairs
// (pairs past the end of K are all-zero tables).
int64_t oracle_tl_num_groups(int fmt, int64_t K, int bk3) {
  TlGeom g;
  if (!tl_geom(fmt, 32, K, bk3, &g)) return -1;
  return g.tiles3 * 32 + g.tiles2 * 32;
}

// PreCompute of Alg. 3 / Alg. 4 for one token: lut[group][16] int16.
//  triple group: lut[i] = w0*a0 + w1*a1 + w2*a2 for the triple whose value 9w0+3w1+w2 equals i,
//    i = 0..13 (the non-negative half after mirror consolidation); slots 14, 15 are zero.
//  pair group: lut[i] = w0*a0 + w1*a1 with (w0, w1) = (i/3 - 1, i%3 - 1), i = 0..8; slots 9..15 zero.
int oracle_tl_build_lut(int fmt, const int8_t* q, int64_t K, int bk3, int16_t* lut) {
  TlGeom g;
  if (!q || !lut || !tl_geom(fmt, 32, K, bk3, &g)) return 1;
  const int64_t ng = g.tiles3 * 32 + g.tiles2 * 32;
  std::memset(lut, 0, (size_t)ng * 16 * sizeof(int16_t));
  for (int64_t grp = 0; grp < g.tiles3 * 32; ++grp) {
    const int a0 = q[3 * grp], a1 = q[3 * grp + 1], a2 = q[3 * grp + 2];
    for (int w0 = -1; w0 <= 1; ++w0)
      for (int w1 = -1; w1 <= 1; ++w1)
        for (int w2 = -1; w2 <= 1; ++w2) {
          const int v = 9 * w0 + 3 * w1 + w2;
          if (v < 0) continue;
          lut[grp * 16 + v] = (int16_t)(w0 * a0 + w1 * a1 + w2 * a2);
        }
  }
  for (int64_t p = 0; p < g.tiles2 * 32; ++p) {
    const int64_t k = g.three_k + 2 * p;
    if (k >= K) continue;
    const int a0 = q[k], a1 = q[k + 1];
    for (int w0 = -1; w0 <= 1; ++w0)
      for (int w1 = -1; w1 <= 1; ++w1)
        lut[(g.tiles3 * 32 + p) * 16 + 3 * (w0 + 1) + (w1 + 1)] = (int16_t)(w0 * a0 + w1 * a1);
  }
  return 0;
}

// Accumulation of Alg. 3 / Alg. 4: table lookups by the packed indices, the sign bit of a triple
// negating the looked-up value.
int oracle_tl_mpgemm(int fmt, const uint8_t* packed, int64_t M, int64_t K, int bk3, const int8_t* q,
                     int64_t T, int32_t* acc) {
  TlGeom g;
  if (!packed || !q || !acc || T < 1 || !tl_geom(fmt, M, K, bk3, &g)) return 1;
  const int64_t ng = g.tiles3 * 32 + g.tiles2 * 32;
  std::vector<int16_t> lut((size_t)ng * 16);
  for (int64_t t = 0; t < T; ++t) {
    if (oracle_tl_build_lut(fmt, q + t * K, K, bk3, lut.data())) return 1;
    for (int64_t m = 0; m < M; ++m) {
      const int64_t rb = m / 32, r = m % 32;
      const uint8_t* blk = packed + rb * g.block_bytes;
      int64_t s = 0;
      for (int64_t tile_i = 0; tile_i < g.tiles3; ++tile_i) {
        const uint8_t* tile = blk + tile_i * 640;
        uint32_t signs = 0;
        for (int b = 0; b < 4; ++b) signs |= (uint32_t)tile[tl_sign_pos((int)r) + b] << (8 * b);
        for (int grp = 0; grp < 32; ++grp) {
          const uint8_t byte = tile[tl_idx_pos((int)r, grp)];
          const int idx = (grp & 1) ? (byte >> 4) : (byte & 15);
          const int val = lut[(tile_i * 32 + grp) * 16 + idx];
          s += ((signs >> tl_sign_bit(grp)) & 1u) ? -val : val;
        }
      }
      for (int64_t tile_i = 0; tile_i < g.tiles2; ++tile_i) {
        const uint8_t* tile = blk + g.tiles3 * 640 + tile_i * 512;
        for (int grp = 0; grp < 32; ++grp) {
          const uint8_t byte = tile[tl_idx_pos((int)r, grp)];
          const int idx = (grp & 1) ? (byte >> 4) : (byte & 15);
          s += lut[(g.tiles3 * 32 + tile_i * 32 + grp) * 16 + idx];
        }
      }
      acc[t * M + m] = (int32_t)s;
    }
  }
  return 0;
}

// ---------------------------------------------------------------------------------------------
// ELUT beyond ternary (App. A).  Weights take C consecutive integer values from lo = -(C/2); g of them form a
// group; a group is stored as its index in [0, C^g) and costs ceil(log2(C^g)) bits (Table 3: bpw_e = that / g,
// against ceil(log2 C) bits per weight for bit-wise storage).
static int64_t ipow(int64_t c, int g) {
  int64_t p = 1;
  for (int i = 0; i < g; ++i) p *= c;
  return p;
}
static bool elut_ok(int C, int g) { return C >= 2 && C <= 16 && g >= 1 && g <= 8 && ipow(C, g) <= 65536; }

int oracle_elut_lo(int C) { return -(C / 2); }
// smallest b with 2^b >= n
static int bits_for(int64_t n) {
  int b = 0;
  while (((int64_t)1 << b) < n) ++b;
  return b;
}
int oracle_elut_index_bits(int C, int g) { return elut_ok(C, g) ? bits_for(ipow(C, g)) : -1; }   // bpw_e * g
int oracle_elut_bitwise_bits(int C) { return (C >= 2 && C <= 16) ? bits_for(C) : -1; }           // bpw_b

// Index of one group: digits w_i - lo, first weight most significant.  -1 if a weight lies outside the alphabet.
int oracle_elut_index(const int8_t* w, int C, int g) {
  if (!elut_ok(C, g)) return -1;
  const int lo = oracle_elut_lo(C);
  int idx = 0;
  for (int i = 0; i < g; ++i) {
    const int d = (int)w[i] - lo;
    if (d < 0 || d >= C) return -1;
    idx = idx * C + d;
  }
  return idx;
}

// Offline step: every group of every row -> its index.  idx[M][K/g].
int oracle_elut_encode(const int8_t* w, int64_t M, int64_t K, int C, int g, uint16_t* idx) {
  if (!w || !idx || M < 1 || K < 1 || !elut_ok(C, g) || K % g != 0) return 1;
  for (int64_t m = 0; m < M; ++m)
    for (int64_t k = 0; k < K / g; ++k) {
      const int v = oracle_elut_index(w + m * K + k * g, C, g);
      if (v < 0) return 3;
      idx[m * (K / g) + k] = (uint16_t)v;
    }
  return 0;
}

// Phase 1, "Table-setup": for one token, lut[k][i] = sum_j digit_j(i) * a[g k + j] for every group k and every one
// of the C^g weight combinations i (digit_j(i) = the j-th weight of the group whose index is i).
int oracle_elut_table_setup(const int8_t* q, int64_t K, int C, int g, int32_t* lut) {
  if (!q || !lut || K < 1 || !elut_ok(C, g) || K % g != 0) return 1;
  const int lo = oracle_elut_lo(C);
  const int64_t n = ipow(C, g);
  for (int64_t k = 0; k < K / g; ++k)
    for (int64_t i = 0; i < n; ++i) {
      int64_t rest = i, s = 0;
      for (int j = g - 1; j >= 0; --j) {      // least significant digit = last weight of the group
        const int wj = (int)(rest % C) + lo;
        rest /= C;
        s += (int64_t)wj * q[k * g + j];
      }
      lut[k * n + i] = (int32_t)s;
    }
  return 0;
}

// Phase 2, accumulation: R[n, m] = sum over groups k of Lookup(LUT[n, k], W[m, k]).
int oracle_elut_mpgemm(const uint16_t* idx, int64_t M, int64_t K, int C, int g, const int8_t* q, int64_t T,
                       int32_t* acc) {
  if (!idx || !q || !acc || M < 1 || T < 1 || K < 1 || !elut_ok(C, g) || K % g != 0) return 1;
  const int64_t n = ipow(C, g), ng = K / g;
  std::vector<int32_t> lut((size_t)(ng * n));
  for (int64_t t = 0; t < T; ++t) {
    if (oracle_elut_table_setup(q + t * K, K, C, g, lut.data())) return 1;
    for (int64_t m = 0; m < M; ++m) {
      int64_t s = 0;
      for (int64_t k = 0; k < ng; ++k) {
        const int64_t i = idx[m * ng + k];
        if (i >= n) return 3;
        s += lut[k * n + i];
      }
      acc[t * M + m] = (int32_t)s;
    }
  }
  return 0;
}

// Packed form of the g = 2 case for C = 3, 4, 5 (index of 4 bits for C <= 4, 5 bits for C = 5: Table 3's 2 and 2.5
// bits per weight).  Same 32-row blocks and tile geometry as the TL blobs: a tile covers 32 pairs (64 columns) of
// 32 rows; its first 512 bytes hold the low four bits of every index (pair 2i of a row in the low nibble of the
// row's byte i, pair 2i+1 in the high nibble; bytes placed as tl_idx_pos says); for C = 5 a 128-byte plane follows
// with the fifth bit (row r's uint32 at tl_sign_pos(r), pair grp at bit tl_sign_bit(grp)).  Columns past K are
// zero weights.  For C = 3 the blob equals the TL1 blob byte for byte.
static bool elut2_geom(int C, int64_t M, int64_t K, int64_t* tiles, int64_t* tile_bytes) {
  if (C < 3 || C > 5 || M < 32 || M % 32 != 0 || K < 2 || K % 2 != 0) return false;
  *tiles = (K + 63) / 64;
  *tile_bytes = (C == 5) ? 640 : 512;
  return true;
}

size_t oracle_elut2_packed_bytes(int C, int64_t M, int64_t K) {
  int64_t tiles, tb;
  if (!elut2_geom(C, M, K, &tiles, &tb)) return 0;
  return (size_t)(M / 32) * (size_t)(tiles * tb);
}

int oracle_pack_elut2(int C, const int8_t* w, int64_t M, int64_t K, uint8_t* packed) {
  int64_t tiles, tb;
  if (!w || !packed || !elut2_geom(C, M, K, &tiles, &tb)) return 1;
  std::memset(packed, 0, (size_t)(M / 32) * (size_t)(tiles * tb));
  const int8_t zero_pair[2] = {0, 0};
  for (int64_t m = 0; m < M; ++m) {
    const int64_t rb = m / 32, r = m % 32;
    for (int64_t t = 0; t < tiles; ++t) {
      uint8_t* tile = packed + (rb * tiles + t) * tb;
      uint32_t high = 0;
      for (int grp = 0; grp < 32; ++grp) {
        const int64_t k = t * 64 + 2 * grp;
        const int idx = oracle_elut_index(k < K ? w + m * K + k : zero_pair, C, 2);
        if (idx < 0) return 3;
        tile[tl_idx_pos((int)r, grp)] |= (uint8_t)((grp & 1) ? ((idx & 15) << 4) : (idx & 15));
        if (idx & 16) high |= 1u << tl_sign_bit(grp);
      }
      if (tb == 640)
        for (int b = 0; b < 4; ++b) tile[tl_sign_pos((int)r) + b] = (uint8_t)(high >> (8 * b));
    }
  }
  return 0;
}

// The index of pair grp of row r of a tile, read back.
static int elut2_read(const uint8_t* tile, int64_t tb, int r, int grp) {
  const uint8_t byte = tile[tl_idx_pos(r, grp)];
  int idx = (grp & 1) ? (byte >> 4) : (byte & 15);
  if (tb == 640) {
    uint32_t high = 0;
    for (int b = 0; b < 4; ++b) high |= (uint32_t)tile[tl_sign_pos(r) + b] << (8 * b);
    idx |= (int)((high >> tl_sign_bit(grp)) & 1u) << 4;
  }
  return idx;
}

int oracle_unpack_elut2(int C, const uint8_t* packed, int64_t M, int64_t K, int8_t* w) {
  int64_t tiles, tb;
  if (!w || !packed || !elut2_geom(C, M, K, &tiles, &tb)) return 1;
  const int lo = oracle_elut_lo(C);
  for (int64_t m = 0; m < M; ++m) {
    const int64_t rb = m / 32, r = m % 32;
    for (int64_t t = 0; t < tiles; ++t) {
      const uint8_t* tile = packed + (rb * tiles + t) * tb;
      for (int grp = 0; grp < 32; ++grp) {
        const int idx = elut2_read(tile, tb, (int)r, grp);
        if (idx >= C * C) return 3;
        const int w0 = idx / C + lo, w1 = idx % C + lo;
        const int64_t k = t * 64 + 2 * grp;
        if (k < K) {
          w[m * K + k] = (int8_t)w0;
          w[m * K + k + 1] = (int8_t)w1;
        } else if (w0 != 0 || w1 != 0) {
          return 3;
        }
      }
    }
  }
  return 0;
}

// "ELUT mpGEMM" straight from the packed blob: tables per token, one lookup per stored index.
int oracle_elut2_mpgemm(int C, const uint8_t* packed, int64_t M, int64_t K, const int8_t* q, int64_t T, int32_t* acc) {
  int64_t tiles, tb;
  if (!packed || !q || !acc || T < 1 || !elut2_geom(C, M, K, &tiles, &tb)) return 1;
  const int64_t n = (int64_t)C * C, kp = tiles * 64;
  std::vector<int8_t> qp((size_t)kp);
  std::vector<int32_t> lut((size_t)(kp / 2 * n));
  for (int64_t t = 0; t < T; ++t) {
    for (int64_t k = 0; k < kp; ++k) qp[k] = k < K ? q[t * K + k] : (int8_t)0;
    if (oracle_elut_table_setup(qp.data(), kp, C, 2, lut.data())) return 1;
    for (int64_t m = 0; m < M; ++m) {
      const int64_t rb = m / 32, r = m % 32;
      int64_t s = 0;
      for (int64_t ti = 0; ti < tiles; ++ti) {
        const uint8_t* tile = packed + (rb * tiles + ti) * tb;
        for (int grp = 0; grp < 32; ++grp) {
          const int idx = elut2_read(tile, tb, (int)r, grp);
          if (idx >= n) return 3;
          s += lut[(ti * 32 + grp) * n + idx];
        }
      }
      acc[t * M + m] = (int32_t)s;
    }
  }
  return 0;
}

int oracle_num_threads(void) {
#ifdef _OPENMP
  int n = 1;
#pragma omp parallel
  {
#pragma omp master
    n = omp_get_num_threads();
  }
  return n;
#else
  return 1;
#endif
}

}  // extern "C"
