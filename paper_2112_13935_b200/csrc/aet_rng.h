// Counter-based integer generator shared by host scheduler and device kernels.
//
// The paper samples "uniformly at random xi from D_c" (Algorithm 3) and injects
// random compute / network delays (Section 3.3.2) without fixing a generator.
// Here every random quantity is a pure function of (seed, stream, client,
// counter): the SplitMix64 output function (Steele, Lea, Flood 2014) applied to
// golden-ratio-spaced inputs.  Delays are integer ticks computed without
// floating point, so the event order is identical on every machine.
#pragma once
#include <stdint.h>

#if defined(__CUDACC__)
#define AET_HD __host__ __device__ __forceinline__
#else
#define AET_HD inline
#endif

namespace aet {

constexpr uint64_t kGamma = 0x9E3779B97F4A7C15ull;
constexpr uint64_t kLn2Q32 = 2977044471ull;  // floor(ln 2 * 2^32)
enum Stream : uint32_t { kStreamSample = 0, kStreamCompute = 1, kStreamNetwork = 2, kStreamSetup = 3 };

AET_HD uint64_t mix64(uint64_t z) {
  z ^= z >> 30;
  z *= 0xBF58476D1CE4E5B9ull;
  z ^= z >> 27;
  z *= 0x94D049BB133111EBull;
  z ^= z >> 31;
  return z;
}

AET_HD uint64_t stream_key(uint64_t seed, uint32_t stream, uint32_t client) {
  uint64_t k = mix64(seed + kGamma * (uint64_t)(stream + 1));
  return mix64(k + kGamma * (uint64_t)(client + 1));
}

AET_HD uint64_t draw(uint64_t key, uint64_t counter) { return mix64(key + kGamma * (counter + 1)); }

// Uniform index in [0, n): high word of the draw times n, high word of that.
AET_HD uint32_t sample_index(uint64_t r, uint32_t n) {
  return (uint32_t)(((r >> 32) * (uint64_t)n) >> 32);
}

// Host only (the delay model is part of the host scheduler).
// -log2(x / 2^64) in Q32, x = r (1 when r == 0): integer part from the leading
// bit, 32 fraction bits by squaring the Q1.63 mantissa and watching for >= 2.
inline uint64_t neg_log2_q32(uint64_t r) {
  uint64_t x = r ? r : 1;
  int e = 63 - __builtin_clzll(x);
  uint64_t m = x << (63 - e);
  uint64_t f = 0;
  for (int it = 0; it < 32; ++it) {
    unsigned __int128 p = (unsigned __int128)m * m;
    if ((uint64_t)(p >> 127)) {
      f = (f << 1) | 1;
      m = (uint64_t)(p >> 64);
    } else {
      f <<= 1;
      m = (uint64_t)(p >> 63);
    }
  }
  return ((uint64_t)(64 - e) << 32) - f;
}

inline uint64_t exp_ticks(uint64_t r, uint64_t mean_ticks) {
  unsigned __int128 t = (unsigned __int128)neg_log2_q32(r) * kLn2Q32;
  t *= mean_ticks;
  uint64_t v = (uint64_t)(t >> 64);
  return v ? v : 1;
}

inline uint64_t uniform_ticks(uint64_t r, uint64_t lo, uint64_t hi) {
  uint64_t v = lo + (((r >> 32) * (hi - lo + 1)) >> 32);
  return v ? v : 1;
}

}  // namespace aet
