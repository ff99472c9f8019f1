// Host-side check of the arithmetic that the checksumming kernel runs on the GPU. The helpers in
// topkv_crc.cuh are __host__ __device__, so the very same code is exercised here on the CPU:
//   - gf_mulmod_clmul (integer-multiplier carry-less product + sparse reduction) against the
//     bit-serial gf_mulmod,
//   - gf_fold64 (eight Horner steps with one reduction) against eight gf_mulx64 steps,
//   - the checksum of a message assembled the way the kernel and topkv_crc_finish assemble it
//     (runs folded from zero, aligned with x^(8 * bytes that follow), chained with the all-ones
//     initial value), printed for the caller to compare with an independent CRC-64.
// Built with nvcc and run by tests/test_crc_math_host.py; needs no GPU.
#include <cstdint>
#include <cstdio>
#include <cstring>
#include <vector>

#include "topkv_crc.cuh"

using namespace topkv;

static uint64_t splitmix(uint64_t& s) {
  uint64_t z = (s += 0x9E3779B97F4A7C15ull);
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}

static uint64_t fold_run(const uint8_t* p, int n) {  // n a multiple of 16, as in the kernel
  uint64_t rem = 0;
  int off = 0;
  for (; off + 64 <= n; off += 64) {
    uint32_t w[16];
    memcpy(w, p + off, 64);
    rem = gf_fold64(rem, w);
  }
  for (; off < n; off += 8) {
    uint64_t v;
    memcpy(&v, p + off, 8);
    rem = gf_mulx64(rem ^ v);
  }
  return rem;
}

int main(int argc, char** argv) {
  uint64_t seed = 42;
  int bad = 0;
  for (int i = 0; i < 100000; ++i) {
    uint64_t a = splitmix(seed), b = splitmix(seed);
    if (i < 64) a = 1ull << i;
    else if (i < 128) b = 1ull << (i - 64);
    else if (i % 9 == 0) a &= splitmix(seed) & splitmix(seed);
    if (gf_mulmod(a, b) != gf_mulmod_clmul(a, b)) ++bad;
  }
  for (int i = 0; i < 100000; ++i) {
    uint64_t s = splitmix(seed), w[8];
    for (auto& x : w) x = splitmix(seed);
    if (i % 5 == 0) { s = ~0ull; for (auto& x : w) x = ~0ull; }
    if (i % 7 == 0) { s = 0; for (auto& x : w) x = 0; w[i % 8] = 1ull << (i % 64); }
    uint64_t ref = s;
    for (int k = 0; k < 8; ++k) ref = gf_mulx64(ref ^ w[k]);
    uint32_t ww[16];
    memcpy(ww, w, 64);
    if (gf_fold64(s, ww) != ref) ++bad;
  }
  // x^n by repeated squaring with the carry-less product against the bit-serial definition
  for (int i = 0; i < 3000; ++i) {
    uint64_t n = splitmix(seed) >> (i % 64);
    if (i < 200) n = (uint64_t)i;
    if (i % 11 == 0) n = 8ull * 1024 * 32 * (uint64_t)(i + 1);
    if (gf_powx(n) != gf_powx_ref(n)) ++bad;
  }
  // a chain of affine steps composed pairwise (as the shuffle tree of topkv_crc_finish does it,
  // 32 steps at a time, identity padded) against the steps taken one after the other
  for (int i = 0; i < 200; ++i) {
    const int n = 1 + (int)(splitmix(seed) % 100);
    std::vector<GfAffine> f(n);
    for (auto& x : f) x = {splitmix(seed), splitmix(seed)};
    uint64_t seq = ~0ull, tree = ~0ull;
    for (int l = 0; l < n; ++l) seq = gf_mulmod(seq, f[l].A) ^ f[l].V;
    for (int base = 0; base < n; base += 32) {
      GfAffine lane[32];
      for (int q = 0; q < 32; ++q) lane[q] = base + q < n ? f[base + q] : GfAffine{kGfOne, 0ull};
      for (int o = 1; o < 32; o <<= 1)
        for (int q = 0; q + o < 32; q += 2 * o) lane[q] = gf_then(lane[q], lane[q + o]);
      tree = gf_mulmod_clmul(tree, lane[0].A) ^ lane[0].V;
    }
    if (seq != tree) ++bad;
  }
  if (bad) {
    printf("mismatches %d\n", bad);
    return 1;
  }
  // a message of `layers` slabs of `runs` runs of `run` bytes, bytes (7 i + 3) mod 256
  const int run = argc > 1 ? atoi(argv[1]) : 576, runs = argc > 2 ? atoi(argv[2]) : 45;
  const int layers = argc > 3 ? atoi(argv[3]) : 3;
  std::vector<uint8_t> msg((size_t)run * runs * layers);
  for (size_t i = 0; i < msg.size(); ++i) msg[i] = (uint8_t)(7 * i + 3);
  const uint64_t x_layer = gf_powx(8ull * run * runs);
  uint64_t state = ~0ull;
  for (int l = 0; l < layers; ++l) {
    uint64_t rem_l = 0;  // items of 32 runs counted from the end, as the kernel cuts them
    for (int g = 0; g < runs; ++g) {
      const uint64_t r = fold_run(msg.data() + ((size_t)l * runs + g) * run, run);
      rem_l ^= gf_mulmod_clmul(r, gf_powx(8ull * run * (uint64_t)(runs - 1 - g)));
    }
    state = gf_mulmod_clmul(state, x_layer) ^ rem_l;
  }
  printf("ok %d %d %d %016llx\n", run, runs, layers, (unsigned long long)~state);
  return 0;
}
