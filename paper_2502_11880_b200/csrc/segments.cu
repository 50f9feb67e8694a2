// Per-segment weight scales for a tensor made of several matrices stacked by rows ("Int2 with a Scale", Sec. 3.2.2,
// per stacked matrix): the fallback rescale used when a call cannot run as one grouped kernel with a scale per
// item -- the whole tensor is computed with scale 1 and the columns of every segment are multiplied afterwards.
#include "common.cuh"

namespace bitnet {
namespace {

constexpr int MAX_SEG = 16;
struct SegArgs {
  int n;
  int end[MAX_SEG];
  float scale[MAX_SEG];
};

__global__ void scale_segments_kernel(float* __restrict__ y, int64_t T, int64_t M, SegArgs a) {
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= T * M) return;
  const int m = (int)(i % M);
  int s = 0;
  while (s + 1 < a.n && m >= a.end[s]) ++s;
  y[i] = __fmul_rn(y[i], a.scale[s]);
}

}  // namespace

int launch_scale_segments(float* y, int64_t T, int64_t M, int n_seg, const int64_t* seg_end, const float* seg_scale,
                          cudaStream_t st) {
  if (n_seg < 1 || n_seg > MAX_SEG) return BITNET_ERR_INVALID_ARG;
  SegArgs a;
  a.n = n_seg;
  for (int s = 0; s < n_seg; ++s) {
    a.end[s] = (int)seg_end[s];
    a.scale[s] = seg_scale[s];
  }
  scale_segments_kernel<<<(unsigned)ceil_div(T * M, 256), 256, 0, st>>>(y, T, M, a);
  return check_launch();
}

}  // namespace bitnet
