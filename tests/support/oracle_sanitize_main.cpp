// Drives the CPU checker over a few small arenas (short chunks, padding, tiles, every code width,
// non-finite values) so that AddressSanitizer / UndefinedBehaviorSanitizer can watch it.  Built and
// run by tests/test_oracle_sanitized.py; prints a checksum so the run cannot be optimised away.
#include <cmath>
#include <cstdint>
#include <cstdio>
#include <limits>
#include <vector>

extern "C" {
uint64_t slo_num_chunks_tiled(const uint64_t* offset, const uint64_t* cols, uint32_t n_tensors, int chunk);
uint64_t slo_codes_stride(int k, int bits);
int slo_compress_tiled(const float* theta_local, const float* theta_global, float* err, const uint64_t* offset,
                       const uint64_t* cols, uint32_t n_tensors, float beta, int chunk, int k, int bits,
                       uint16_t* idx, uint8_t* codes, float* scales, uint32_t* flags);
int slo_aggregate_tiled(int R, const uint16_t* const* idx, const uint8_t* const* codes, const float* const* scales,
                        const uint64_t* offset, const uint64_t* cols, uint32_t n_tensors, int chunk, int k, int bits,
                        float* update);
int slo_outer_apply(float* theta_global, const float* update, uint64_t n, float outer_lr);
int slo_chunk_lengths(const uint64_t* offset, const uint64_t* cols, uint32_t n_tensors, int chunk, uint32_t* len);
}

static uint64_t rng_state = 0x9E3779B97F4A7C15ull;
static float rnd() {   // xorshift, uniform in [-1, 1)
  rng_state ^= rng_state << 13; rng_state ^= rng_state >> 7; rng_state ^= rng_state << 17;
  return (float)((double)(rng_state >> 11) / 9007199254740992.0 * 2.0 - 1.0);
}

static bool failed = false;
static double run_checked(const std::vector<uint64_t>& off, const std::vector<uint64_t>& cols, int chunk, int k, int bits, int R,
                  bool poison) {
  const uint32_t nt = (uint32_t)off.size() - 1;
  const uint64_t n = off.back();
  const uint64_t* pc = cols.empty() ? nullptr : cols.data();
  const uint64_t nc = slo_num_chunks_tiled(off.data(), pc, nt, chunk);
  const uint64_t st = slo_codes_stride(k, bits);
  std::vector<float> tg(n), upd(n);
  for (auto& v : tg) v = 0.02f * rnd();
  std::vector<std::vector<float>> tl(R, std::vector<float>(n)), err(R, std::vector<float>(n, 0.0f)), sc(R, std::vector<float>(nc));
  std::vector<std::vector<uint16_t>> idx(R, std::vector<uint16_t>(nc * k));
  std::vector<std::vector<uint8_t>> codes(R, std::vector<uint8_t>(nc * st));
  std::vector<uint32_t> len(nc);
  if (slo_chunk_lengths(off.data(), pc, nt, chunk, len.data()) != 0) return -1.0;
  double sum = 0.0;
  for (int round = 0; round < 2; ++round) {
    std::vector<const uint16_t*> pi; std::vector<const uint8_t*> pcod; std::vector<const float*> ps;
    for (int r = 0; r < R; ++r) {
      for (uint64_t i = 0; i < n; ++i) tl[r][i] = tg[i] + 1e-3f * rnd();
      if (poison && n > 3) { tl[r][1] = std::numeric_limits<float>::infinity(); tl[r][2] = std::nanf(""); tl[r][3] = -0.0f; }
      uint32_t flags = 0;
      if (slo_compress_tiled(tl[r].data(), tg.data(), err[r].data(), off.data(), pc, nt, 0.95f, chunk, k, bits,
                             idx[r].data(), codes[r].data(), sc[r].data(), &flags) != 0) return -1.0;
      pi.push_back(idx[r].data()); pcod.push_back(codes[r].data()); ps.push_back(sc[r].data());
      sum += flags;
    }
    if (slo_aggregate_tiled(R, pi.data(), pcod.data(), ps.data(), off.data(), pc, nt, chunk, k, bits, upd.data()) != 0) return -1.0;
    if (slo_outer_apply(tg.data(), upd.data(), n, 0.8f) != 0) return -1.0;
  }
  for (uint64_t i = 0; i < n; ++i) if (std::isfinite(tg[i])) sum += tg[i];
  for (auto l : len) sum += l;
  return sum;
}

static double run(const std::vector<uint64_t>& off, const std::vector<uint64_t>& cols, int chunk, int k, int bits, int R,
                  bool poison) {
  const double v = run_checked(off, cols, chunk, k, bits, R, poison);
  if (v < 0.0) failed = true;     // the checksum of a good run is dominated by the chunk lengths: positive
  return v;
}

int main() {
  double s = 0.0;
  s += run({0, 4096 * 2 + 17, 4096 * 2 + 20, 4096 * 3 + 20}, {}, 4096, 64, 2, 3, false);
  s += run({0, 1000, 1003}, {}, 256, 8, 4, 2, false);
  s += run({0, 500}, {}, 100, 100, 8, 1, false);                 // k = chunk
  s += run({0, 300, 301}, {}, 64, 5, 32, 2, true);               // unquantised, non-finite values
  s += run({0, 100 * 70, 100 * 70 + 50}, {70, 0}, 4096, 64, 2, 2, false);   // edge tiles
  s += run({0, 16 * 16}, {16}, 64, 3, 2, 1, false);              // 8 x 8 tiles
  std::printf("checksum %.6f\n", s);
  return failed ? 1 : 0;
}
