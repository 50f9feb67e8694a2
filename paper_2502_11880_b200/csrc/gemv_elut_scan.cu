// Element-wise tables beyond ternary (App. A, Table 3) in their g = 2 form, 1..8 tokens: weights of cardinality
// C = 3, 4, 5 stored as pair indices (2 or 2.5 bits per weight), served by the scan kernel of scan_kernel.cuh in its
// pair mode -- an index byte and its fifth bits select a table entry holding the four weights of two pairs, which
// go to the int8 tensor cores as they are; C = 4, whose index is two 2-bit codes, is decoded by masks instead.
#include "scan_kernel.cuh"

namespace bitnet {

bool elut2_geom(int C, int64_t M, int64_t K, TlGeom* g) {
  if (C < 3 || C > 5 || M < 32 || (M % 32) != 0 || K < 2 || (K % 2) != 0) return false;
  g->three_k = K;                              // every column is pair coded; the kernel walks the tiles as its
  g->two_k = 0;                                // main (not its tail) tiles
  g->tiles3 = ceil_div(K, 64);
  g->tiles2 = 0;
  g->block_bytes = g->tiles3 * (C == 5 ? 640 : 512);
  return true;
}

bool gemv_elut_scan_item_supported(int T, int64_t M, int64_t K, const TlGeom& g) {
  return scan::item_supported<1>(T, M, K, g);
}

int launch_gemv_elut_scan(const Tl2Linear* items, int64_t n, int C, cudaStream_t st) {
  // Cardinality 4: the index is two 2-bit codes, decoded by masks; BITNET_ELUT4=table sends it through the decode
  // table like the other cardinalities.
  static const bool table4 = [] { const char* e = getenv("BITNET_ELUT4"); return e && strcmp(e, "table") == 0; }();
  if (C == 4 && !table4) return scan::launch_items<2>(items, n, C, st);
  // Cardinality 3 (TL1 blobs): the pair code 3 a + b is taken apart by byte-wise arithmetic; BITNET_TL1=table sends it
  // through the decode table.
  static const bool table3 = [] { const char* e = getenv("BITNET_TL1"); return e && strcmp(e, "table") == 0; }();
  if (C == 3 && !table3) return scan::launch_items<3>(items, n, C, st);
  return scan::launch_items<1>(items, n, C, st);
}

}  // namespace bitnet
