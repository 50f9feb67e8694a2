// Weight packers (offline step of the path) and their inverses (test hooks).
//   I2_S : Table 1 / Sec. 3.2.2 -- code w+1 in two bits.
//   TL1  : Table 4 / Alg. 3 PreprocessWeights -- pair -> 3(w0+1)+(w1+1).
//   TL2  : Table 5 / Alg. 4 PreprocessWeights -- triple -> (|v|, [v<0]), v = 9w0+3w1+w2, index and
//          sign kept in separate planes (signed-unsigned weight splitting, Sec. 3.1.2).
// The byte layouts are documented in bitnet_b200.h.
#include "common.cuh"

namespace bitnet {
namespace {

__device__ __forceinline__ bool ternary(int w) { return w >= -1 && w <= 1; }

// One thread per 32-bit packed word of the blob (16 weights of one row, see common.cuh for the map).
__global__ void pack_i2s_kernel(const int8_t* __restrict__ w, int64_t M, int64_t K, int64_t kp, int64_t nwords,
                                uint32_t* __restrict__ packed, int* dev_status) {
  const int64_t gid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (gid >= nwords) return;
  const int64_t block_words = kp;            // 16 rows x kp / 16 words
  const int64_t rb = gid / block_words, rem = gid % block_words;
  const int64_t c = rem >> 8, r = (rem >> 4) & 15, j = rem & 15;
  const int64_t m = rb * 16 + r;
  uint32_t word = 0;
  bool bad = false;
#pragma unroll
  for (int s = 0; s < 4; ++s) {
#pragma unroll
    for (int b = 0; b < 4; ++b) {
      const int64_t k = c * 256 + 32 * (j >> 1) + 8 * s + 4 * (j & 1) + b;
      const int wk = (m < M && k < K) ? (int)w[m * K + k] : 0;
      bad |= !ternary(wk);
      word |= (uint32_t)((wk + 1) & 3) << (8 * b + 2 * s);
    }
  }
  packed[gid] = word;
  if (bad && dev_status) atomicExch(dev_status, BITNET_ERR_BAD_WEIGHT);
}

__global__ void unpack_i2s_kernel(const uint32_t* __restrict__ packed, int64_t M, int64_t K, int64_t kp,
                                  int64_t nwords, int8_t* __restrict__ w, int* dev_status) {
  const int64_t gid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (gid >= nwords) return;
  const int64_t block_words = kp;
  const int64_t rb = gid / block_words, rem = gid % block_words;
  const int64_t c = rem >> 8, r = (rem >> 4) & 15, j = rem & 15;
  const int64_t m = rb * 16 + r;
  const uint32_t word = packed[gid];
  bool bad = false;
#pragma unroll
  for (int s = 0; s < 4; ++s) {
#pragma unroll
    for (int b = 0; b < 4; ++b) {
      const int64_t k = c * 256 + 32 * (j >> 1) + 8 * s + 4 * (j & 1) + b;
      const int code = (word >> (8 * b + 2 * s)) & 3;
      bad |= (code == 3);
      if (m < M && k < K) w[m * K + k] = (int8_t)(code - 1);
    }
  }
  if (bad && dev_status) atomicExch(dev_status, BITNET_ERR_BAD_WEIGHT);
}

// One thread per (row, tile): emits the row's four index words (and the sign word of a TL2 tile) at the
// positions tl_word_off / tl_sign_off / tl_sign_bit give.
__global__ void pack_tl_kernel(const int8_t* __restrict__ w, int64_t M, int64_t K, TlGeom g,
                               uint8_t* __restrict__ packed, int* dev_status) {
  const int64_t tiles = g.tiles3 + g.tiles2;
  const int64_t gid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (gid >= M * tiles) return;
  // consecutive threads = consecutive rows of one tile: a warp's stores cover the tile's planes completely
  const int64_t r = gid % 32;
  const int64_t tile = (gid / 32) % tiles;
  const int64_t rb = gid / (32 * tiles);
  const int64_t m = rb * 32 + r;
  const int8_t* wr = w + m * K;
  uint8_t* blk = packed + rb * g.block_bytes;
  uint32_t idx_words[4] = {0, 0, 0, 0};
  bool bad = false;
  if (tile < g.tiles3) {
    uint32_t signs = 0;
    const int64_t k0 = tile * 96;
    for (int grp = 0; grp < 32; ++grp) {
      const int w0 = wr[k0 + 3 * grp], w1 = wr[k0 + 3 * grp + 1], w2 = wr[k0 + 3 * grp + 2];
      bad |= !(ternary(w0) && ternary(w1) && ternary(w2));
      const int v = 9 * w0 + 3 * w1 + w2;
      const uint32_t idx = (uint32_t)abs(v) & 15u;
      signs |= (v < 0 ? 1u : 0u) << tl_sign_bit(grp);
      idx_words[grp >> 3] |= idx << (4 * (grp & 7));
    }
    uint8_t* tp = blk + tile * 640;
#pragma unroll
    for (int t = 0; t < 4; ++t) *reinterpret_cast<uint32_t*>(tp + tl_word_off((int)r, t)) = idx_words[t];
    *reinterpret_cast<uint32_t*>(tp + tl_sign_off((int)r)) = signs;
  } else {
    const int64_t t2 = tile - g.tiles3;
    const int64_t k0 = g.three_k + t2 * 64;
    for (int grp = 0; grp < 32; ++grp) {
      const int64_t k = k0 + 2 * grp;
      uint32_t idx = 4;
      if (k < K) {
        const int w0 = wr[k], w1 = wr[k + 1];
        bad |= !(ternary(w0) && ternary(w1));
        idx = (uint32_t)(3 * (w0 + 1) + (w1 + 1)) & 15u;
      }
      idx_words[grp >> 3] |= idx << (4 * (grp & 7));
    }
    uint8_t* tp = blk + g.tiles3 * 640 + t2 * 512;
#pragma unroll
    for (int t = 0; t < 4; ++t) *reinterpret_cast<uint32_t*>(tp + tl_word_off((int)r, t)) = idx_words[t];
  }
  if (bad && dev_status) atomicExch(dev_status, BITNET_ERR_BAD_WEIGHT);
}

__global__ void unpack_tl_kernel(const uint8_t* __restrict__ packed, int64_t M, int64_t K, TlGeom g,
                                 int8_t* __restrict__ w, int* dev_status) {
  const int64_t tiles = g.tiles3 + g.tiles2;
  const int64_t gid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (gid >= M * tiles) return;
  const int64_t r = gid % 32;
  const int64_t tile = (gid / 32) % tiles;
  const int64_t rb = gid / (32 * tiles);
  const int64_t m = rb * 32 + r;
  int8_t* wr = w + m * K;
  const uint8_t* blk = packed + rb * g.block_bytes;
  bool bad = false;
  if (tile < g.tiles3) {
    const uint8_t* tp = blk + tile * 640;
    uint32_t words[4];
#pragma unroll
    for (int t = 0; t < 4; ++t) words[t] = *reinterpret_cast<const uint32_t*>(tp + tl_word_off((int)r, t));
    const uint32_t signs = *reinterpret_cast<const uint32_t*>(tp + tl_sign_off((int)r));
    for (int grp = 0; grp < 32; ++grp) {
      const int idx = (words[grp >> 3] >> (4 * (grp & 7))) & 15;
      const int neg = (signs >> tl_sign_bit(grp)) & 1;
      bad |= (idx > 13) || (idx == 0 && neg);
      // digits of idx in balanced ternary: idx = 9 d0 + 3 d1 + d2, digits in {-1,0,1}
      const int d0 = (idx + 4) / 9;                 // 0 for idx <= 4, 1 for 5..13
      const int rem = idx - 9 * d0;                 // -4..4
      const int d1 = (rem + 7) / 3 - 2;             // -1 for -4..-2, 0 for -1..1, 1 for 2..4
      const int d2 = rem - 3 * d1;
      const int sgn = neg ? -1 : 1;
      const int64_t k = tile * 96 + 3 * grp;
      wr[k] = (int8_t)(sgn * d0);
      wr[k + 1] = (int8_t)(sgn * d1);
      wr[k + 2] = (int8_t)(sgn * d2);
    }
  } else {
    const int64_t t2 = tile - g.tiles3;
    const uint8_t* tp = blk + g.tiles3 * 640 + t2 * 512;
    uint32_t words[4];
#pragma unroll
    for (int t = 0; t < 4; ++t) words[t] = *reinterpret_cast<const uint32_t*>(tp + tl_word_off((int)r, t));
    for (int grp = 0; grp < 32; ++grp) {
      const int idx = (words[grp >> 3] >> (4 * (grp & 7))) & 15;
      const int64_t k = g.three_k + t2 * 64 + 2 * grp;
      if (k < K) {
        bad |= idx > 8;
        wr[k] = (int8_t)(idx / 3 - 1);
        wr[k + 1] = (int8_t)(idx % 3 - 1);
      } else {
        bad |= idx != 4;
      }
    }
  }
  if (bad && dev_status) atomicExch(dev_status, BITNET_ERR_BAD_WEIGHT);
}

inline unsigned blocks_for(int64_t n, int threads) { return (unsigned)ceil_div(n, threads); }

}  // namespace

int launch_pack_i2s(const int8_t* w, int64_t M, int64_t K, uint8_t* packed, int* dev_status,
                    cudaStream_t st) {
  const int64_t kp = i2s_kp(K), nwords = i2s_mp(M) * kp / 16;
  pack_i2s_kernel<<<blocks_for(nwords, 256), 256, 0, st>>>(w, M, K, kp, nwords, reinterpret_cast<uint32_t*>(packed),
                                                         dev_status);
  return check_launch();
}

int launch_unpack_i2s(const uint8_t* packed, int64_t M, int64_t K, int8_t* w, int* dev_status,
                      cudaStream_t st) {
  const int64_t kp = i2s_kp(K), nwords = i2s_mp(M) * kp / 16;
  unpack_i2s_kernel<<<blocks_for(nwords, 256), 256, 0, st>>>(reinterpret_cast<const uint32_t*>(packed), M, K, kp,
                                                           nwords, w, dev_status);
  return check_launch();
}

int launch_pack_tl(int, const int8_t* w, int64_t M, int64_t K, const TlGeom& g, uint8_t* packed,
                   int* dev_status, cudaStream_t st) {
  pack_tl_kernel<<<blocks_for(M * (g.tiles3 + g.tiles2), 256), 256, 0, st>>>(w, M, K, g, packed, dev_status);
  return check_launch();
}

int launch_unpack_tl(int, const uint8_t* packed, int64_t M, int64_t K, const TlGeom& g, int8_t* w,
                     int* dev_status, cudaStream_t st) {
  unpack_tl_kernel<<<blocks_for(M * (g.tiles3 + g.tiles2), 256), 256, 0, st>>>(packed, M, K, g, w, dev_status);
  return check_launch();
}

}  // namespace bitnet
