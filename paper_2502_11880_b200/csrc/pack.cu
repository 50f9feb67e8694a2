// Weight packers (offline step of the path) and their inverses (test hooks).
//   I2_S : Table 1 / Sec. 3.2.2 -- code w+1 in two bits.
//   TL1  : Table 4 / Alg. 3 PreprocessWeights -- pair -> 3(w0+1)+(w1+1).
//   TL2  : Table 5 / Alg. 4 PreprocessWeights -- triple -> (|v|, [v<0]), v = 9w0+3w1+w2, index and
//          sign kept in separate planes (signed-unsigned weight splitting, Sec. 3.1.2).
//   ELUT : App. A -- weights of cardinality C in pairs, a pair stored as its index C (w0 + C/2) + (w1 + C/2).
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

// App. A, g = 2: one thread per (row, tile of 32 pairs).  The low four bits of a pair's index go where a TL1 tile
// keeps its codes; C = 5 adds the plane of fifth bits where a TL2 tile keeps its signs.
__global__ void pack_elut2_kernel(const int8_t* __restrict__ w, int64_t M, int64_t K, int C, int64_t tiles, int tile_bytes,
                                  uint8_t* __restrict__ packed, int* dev_status) {
  const int64_t gid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (gid >= M * tiles) return;
  const int64_t r = gid % 32, tile = (gid / 32) % tiles, rb = gid / (32 * tiles);
  const int8_t* wr = w + (rb * 32 + r) * K;
  const int z = C / 2;
  uint32_t idx_words[4] = {0, 0, 0, 0}, high = 0;
  bool bad = false;
  for (int grp = 0; grp < 32; ++grp) {
    const int64_t k = tile * 64 + 2 * grp;
    int d0 = z, d1 = z;                          // columns past K: zero weights
    if (k < K) {
      d0 = wr[k] + z;
      d1 = wr[k + 1] + z;
      if (d0 < 0 || d0 >= C || d1 < 0 || d1 >= C) {
        bad = true;
        d0 = d1 = z;
      }
    }
    const uint32_t idx = (uint32_t)(C * d0 + d1);
    idx_words[grp >> 3] |= (idx & 15u) << (4 * (grp & 7));
    high |= (idx >> 4) << tl_sign_bit(grp);
  }
  uint8_t* tp = packed + (rb * tiles + tile) * tile_bytes;
#pragma unroll
  for (int t = 0; t < 4; ++t) *reinterpret_cast<uint32_t*>(tp + tl_word_off((int)r, t)) = idx_words[t];
  if (tile_bytes == 640) *reinterpret_cast<uint32_t*>(tp + tl_sign_off((int)r)) = high;
  if (bad && dev_status) atomicExch(dev_status, BITNET_ERR_BAD_WEIGHT);
}

__global__ void unpack_elut2_kernel(const uint8_t* __restrict__ packed, int64_t M, int64_t K, int C, int64_t tiles,
                                    int tile_bytes, int8_t* __restrict__ w, int* dev_status) {
  const int64_t gid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (gid >= M * tiles) return;
  const int64_t r = gid % 32, tile = (gid / 32) % tiles, rb = gid / (32 * tiles);
  int8_t* wr = w + (rb * 32 + r) * K;
  const uint8_t* tp = packed + (rb * tiles + tile) * tile_bytes;
  const int z = C / 2;
  uint32_t words[4];
#pragma unroll
  for (int t = 0; t < 4; ++t) words[t] = *reinterpret_cast<const uint32_t*>(tp + tl_word_off((int)r, t));
  const uint32_t high = tile_bytes == 640 ? *reinterpret_cast<const uint32_t*>(tp + tl_sign_off((int)r)) : 0u;
  bool bad = false;
  for (int grp = 0; grp < 32; ++grp) {
    const int idx = (int)((words[grp >> 3] >> (4 * (grp & 7))) & 15u) | (int)(((high >> tl_sign_bit(grp)) & 1u) << 4);
    const int64_t k = tile * 64 + 2 * grp;
    if (idx >= C * C) {
      bad = true;
      continue;
    }
    if (k < K) {
      wr[k] = (int8_t)(idx / C - z);
      wr[k + 1] = (int8_t)(idx % C - z);
    } else {
      bad |= idx != C * z + z;
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
  note_blob_written(st);
  return check_launch();
}

int launch_unpack_i2s(const uint8_t* packed, int64_t M, int64_t K, int8_t* w, int* dev_status,
                      cudaStream_t st) {
  const int64_t kp = i2s_kp(K), nwords = i2s_mp(M) * kp / 16;
  unpack_i2s_kernel<<<blocks_for(nwords, 256), 256, 0, st>>>(reinterpret_cast<const uint32_t*>(packed), M, K, kp,
                                                           nwords, w, dev_status);
  return check_launch();
}

// TL blob -> I2_S blob of the same matrix, for batches large enough for the tensor-core prefill kernel (which reads
// I2_S): one thread per 32-bit word of the I2_S blob (16 weights = four runs of four consecutive columns).  A run of
// four triple-coded columns lies in two neighbouring triples: their (sign, index) pairs go through a 32-entry table
// to three 2-bit codes each, and a shift picks the run's four codes out of the six; a run of pair-coded columns is
// one index byte.  A 256-entry table spreads four codes over the four bytes of the word.
__global__ void __launch_bounds__(256) tl_to_i2s_kernel(const uint8_t* __restrict__ tl, int64_t M, int64_t K, TlGeom g,
                                                        uint32_t* __restrict__ out) {
  __shared__ unsigned short lut5[32];   // (sign << 4 | index) -> codes c0 | c1 << 2 | c2 << 4
  __shared__ unsigned spread[256];      // four 2-bit codes -> one per byte
  if (threadIdx.x < 32) {
    int idx = threadIdx.x & 15;
    const int neg = threadIdx.x >> 4;
    if (idx > 13) idx = 0;
    const int d0 = (idx + 4) / 9, rem = idx - 9 * d0, d1 = (rem + 7) / 3 - 2, d2 = rem - 3 * d1, sg = neg ? -1 : 1;
    lut5[threadIdx.x] = (unsigned short)((sg * d0 + 1) | ((sg * d1 + 1) << 2) | ((sg * d2 + 1) << 4));
  }
  {
    const unsigned x = threadIdx.x;
    spread[x] = (x & 3u) | (((x >> 2) & 3u) << 8) | (((x >> 4) & 3u) << 16) | (((x >> 6) & 3u) << 24);
  }
  __syncthreads();
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int64_t kp = i2s_kp(K), mp = i2s_mp(M);
  const int64_t nwords = mp * kp / 16;
  const int64_t wi = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (wi >= nwords) return;
  // word wi of the blob: 16-row unit, chunk, row in the unit, word j in the row's 64 bytes
  const int j = (int)(wi & 15), r16 = (int)((wi >> 4) & 15);
  const int64_t piece = wi >> 8, chunks = kp / 256;
  const int64_t unit = piece / chunks, chunk = piece - unit * chunks;
  const int64_t m = unit * 16 + r16;
  unsigned word = 0x55555555u;          // weight 0 everywhere (padding rows and columns)
  if (m < M) {
    const int r = (int)(m & 31);
    const uint8_t* blk = tl + (m >> 5) * g.block_bytes;
    word = 0;
#pragma unroll
    for (int s = 0; s < 4; ++s) {
      const int64_t k = chunk * 256 + 32 * (j >> 1) + 8 * s + 4 * (j & 1);      // the run's first column
      unsigned codes = 0x55u;                                                   // four zeros
      if (k < g.three_k) {
        const int tile = (int)(k / 96), c = (int)(k - 96 * (int64_t)tile);
        const int g0 = c / 3, d0 = c - 3 * g0;                                  // first triple of the run, digit offset
        const uint8_t* tp = blk + (int64_t)tile * 640;
        const unsigned signs = *reinterpret_cast<const unsigned*>(tp + tl_sign_off(r));
        unsigned six = 0;
#pragma unroll
        for (int q = 0; q < 2; ++q) {
          const int grp = g0 + q;                                               // (g0 + 1 <= 31: a run never leaves its tile)
          const unsigned byte = tp[tl_word_off(r, grp >> 3) + ((grp >> 1) & 3)];
          const unsigned idx = (grp & 1) ? (byte >> 4) : (byte & 15u);
          const unsigned neg = (signs >> tl_sign_bit(grp)) & 1u;
          six |= (unsigned)lut5[(neg << 4) | idx] << (6 * q);
        }
        codes = (six >> (2 * d0)) & 0xFFu;
      } else if (k < K) {
        const int64_t k2 = k - g.three_k;
        const int tile = (int)(k2 / 64), p = (int)((k2 - 64 * (int64_t)tile) >> 1);   // first pair of the run (even)
        const uint8_t* tp = blk + g.tiles3 * 640 + (int64_t)tile * 512;
        const unsigned byte = tp[tl_word_off(r, p >> 3) + ((p >> 1) & 3)];
        const unsigned lo = byte & 15u, hi = byte >> 4;
        // pair code i -> (i/3, i%3) as codes w+1; pairs beyond K carry code 4 = (0, 0)
        codes = (lo / 3) | ((lo % 3) << 2) | ((hi / 3) << 4) | ((hi % 3) << 6);
      }
      word |= spread[codes] << (2 * s);
    }
  }
  out[wi] = word;
}

int launch_tl_to_i2s(const uint8_t* tl, int64_t M, int64_t K, const TlGeom& g, uint8_t* i2s, cudaStream_t st) {
  const int64_t nwords = i2s_mp(M) * i2s_kp(K) / 16;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(blocks_for(nwords, 256));
  cfg.blockDim = dim3(256);
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = early_start_enabled(st) ? 1 : 0;
  cudaError_t e = cudaLaunchKernelEx(&cfg, tl_to_i2s_kernel, tl, M, K, g, reinterpret_cast<uint32_t*>(i2s));
  note_blob_written(st);     // the prefill kernel that follows reads this blob before it waits for earlier kernels
  return e == cudaSuccess ? BITNET_OK : note_cuda_error(e);
}

int launch_pack_elut2(int C, const int8_t* w, int64_t M, int64_t K, const TlGeom& g, uint8_t* packed, int* dev_status,
                      cudaStream_t st) {
  pack_elut2_kernel<<<blocks_for(M * g.tiles3, 256), 256, 0, st>>>(w, M, K, C, g.tiles3, (int)(g.block_bytes / g.tiles3),
                                                                 packed, dev_status);
  note_blob_written(st);
  return check_launch();
}

int launch_unpack_elut2(int C, const uint8_t* packed, int64_t M, int64_t K, const TlGeom& g, int8_t* w, int* dev_status,
                        cudaStream_t st) {
  unpack_elut2_kernel<<<blocks_for(M * g.tiles3, 256), 256, 0, st>>>(packed, M, K, C, g.tiles3,
                                                                   (int)(g.block_bytes / g.tiles3), w, dev_status);
  return check_launch();
}

int launch_pack_tl(int, const int8_t* w, int64_t M, int64_t K, const TlGeom& g, uint8_t* packed,
                   int* dev_status, cudaStream_t st) {
  pack_tl_kernel<<<blocks_for(M * (g.tiles3 + g.tiles2), 256), 256, 0, st>>>(w, M, K, g, packed, dev_status);
  note_blob_written(st);
  return check_launch();
}

int launch_unpack_tl(int, const uint8_t* packed, int64_t M, int64_t K, const TlGeom& g, int8_t* w,
                     int* dev_status, cudaStream_t st) {
  unpack_tl_kernel<<<blocks_for(M * (g.tiles3 + g.tiles2), 256), 256, 0, st>>>(packed, M, K, g, w, dev_status);
  return check_launch();
}

}  // namespace bitnet
