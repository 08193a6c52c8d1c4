/*
 * Seeded synthetic symbol generator (inputs only: none of the coder's or the
 * dequantiser's arithmetic lives here).
 *
 * Draw i of a stream with key `key` is the top 32 bits of the SplitMix64 output
 * function applied to key + (i + 1) * 0x9E3779B97F4A7C15 (a counter-based use of
 * the published SplitMix64 mixer), mapped to a symbol by inverse CDF over an
 * integer cumulative table cdf[0..A): symbol = smallest s with u < cdf[s],
 * cdf[A-1] = 2^32.
 */
#include <stdint.h>

static inline uint64_t splitmix64_at(uint64_t key, uint64_t i) {
  uint64_t z = key + (i + 1) * 0x9E3779B97F4A7C15ull;
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}

void synth_draw_symbols(uint64_t key, uint64_t first, uint64_t count,
                        const uint64_t* cdf, int A, uint8_t* out) {
  for (uint64_t t = 0; t < count; ++t) {
    const uint64_t u = splitmix64_at(key, first + t) >> 32;
    int s = 0;
    while (s < A - 1 && u >= cdf[s]) ++s;
    out[t] = (uint8_t)s;
  }
}

void synth_draw_u32(uint64_t key, uint64_t first, uint64_t count, uint32_t* out) {
  for (uint64_t t = 0; t < count; ++t) out[t] = (uint32_t)(splitmix64_at(key, first + t) >> 32);
}
