// TL2 decode (1..8 tokens) through the scan kernel of scan_kernel.cuh: the 1.67-bit blob of Table 5 / Alg. 4 read
// once, every packed index resolved by one shared-memory table lookup, the weights it stands for multiplied on the
// int8 tensor cores.
#include "scan_kernel.cuh"

namespace bitnet {

bool gemv_tl2_scan_item_supported(int T, int64_t M, int64_t K, const TlGeom& g) {
  return scan::item_supported<0>(T, M, K, g);
}

int launch_gemv_tl2_scan(const Tl2Linear* items, int64_t n, cudaStream_t st) {
  return scan::launch_items<0>(items, n, 3, st);
}

}  // namespace bitnet
