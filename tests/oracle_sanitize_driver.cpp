// Runs every entry point of the CPU oracle on small, odd shapes with exactly sized heap buffers.  The test
// that owns this file builds it with -fsanitize=address,undefined: an out-of-bounds access, a signed
// overflow or a misaligned load in the oracle ends the program with a report; wrong sums end it with code 2.
#include <cstdio>
#include <cstdlib>
#include <vector>

#include "../oracle/bitnet_oracle.cpp"

static unsigned lcg(unsigned& s) { return s = s * 1664525u + 1013904223u; }

static int run_case(int64_t M, int64_t K, int64_t T, unsigned seed) {
  unsigned s = seed;
  std::vector<int8_t> w((size_t)(M * K));
  for (auto& v : w) v = (int8_t)((int)(lcg(s) >> 16) % 3 - 1);
  std::vector<float> x((size_t)(T * K));
  for (auto& v : x) v = ((int)(lcg(s) >> 8) % 2001 - 1000) / 250.0f;
  std::vector<int8_t> q((size_t)(T * K));
  std::vector<float> sc((size_t)T);
  std::vector<int32_t> sm((size_t)T);
  if (oracle_quant_act(x.data(), T, K, 0, q.data(), sc.data(), sm.data())) return 1;
  if (oracle_quant_act(x.data(), T, K, 1, q.data(), sc.data(), nullptr)) return 1;
  if (oracle_quant_act(x.data(), T, K, 0, q.data(), sc.data(), sm.data())) return 1;
  std::vector<int32_t> ref((size_t)(T * M)), acc((size_t)(T * M));
  if (oracle_mpgemm_def(q.data(), w.data(), T, M, K, ref.data())) return 1;
  std::vector<double> y((size_t)(T * M));
  oracle_dequant(ref.data(), sc.data(), 0.5f, T, M, y.data());
  if (K % 64 == 0) {
    std::vector<uint8_t> blob(oracle_i2s_packed_bytes(M, K));
    std::vector<int8_t> back((size_t)(M * K));
    if (oracle_pack_i2s(w.data(), M, K, blob.data()) || oracle_unpack_i2s(blob.data(), M, K, back.data())) return 1;
    if (back != w) return 2;
    if (oracle_i2s_mpgemm(blob.data(), M, K, q.data(), T, acc.data())) return 1;
    if (acc != ref) return 2;
  }
  if (M % 32 == 0 && K % 2 == 0) {
    for (int fmt = 1; fmt <= 2; ++fmt) {
      std::vector<uint8_t> blob(oracle_tl_packed_bytes(fmt, M, K, 0));
      std::vector<int8_t> back((size_t)(M * K));
      if (oracle_pack_tl(fmt, w.data(), M, K, 0, blob.data()) || oracle_unpack_tl(fmt, blob.data(), M, K, 0, back.data()))
        return 1;
      if (back != w) return 2;
      std::vector<int16_t> lut((size_t)(oracle_tl_num_groups(fmt, K, 0) * 16));
      if (oracle_tl_build_lut(fmt, q.data(), K, 0, lut.data())) return 1;
      if (oracle_tl_mpgemm(fmt, blob.data(), M, K, 0, q.data(), T, acc.data())) return 1;
      if (acc != ref) return 2;
      int64_t three_k = -1, two_k = -1;
      oracle_tl_split(fmt, K, 0, &three_k, &two_k);
      if (three_k + two_k != K) return 2;
    }
  }
  return 0;
}

int main() {
  const int64_t shapes[][3] = {{5, 128, 3}, {33, 192, 1}, {32, 130, 2}, {64, 96 * 3 + 64, 3}, {32, 96, 1},
                               {1, 64, 1}, {96, 1536, 2}, {32, 2, 1}, {7, 70, 4}};
  unsigned seed = 1;
  for (const auto& sh : shapes) {
    const int rc = run_case(sh[0], sh[1], sh[2], seed++);
    if (rc) {
      std::printf("case M=%lld K=%lld T=%lld failed with %d\n", (long long)sh[0], (long long)sh[1], (long long)sh[2], rc);
      return rc;
    }
  }
  if (oracle_tl1_code(-1, -1) != 0 || oracle_tl1_code(1, 1) != 8 || oracle_num_threads() < 1) return 2;
  (void)oracle_tl2_code(1, 0, -1);
  std::printf("oracle sanitizer run ok\n");
  return 0;
}
