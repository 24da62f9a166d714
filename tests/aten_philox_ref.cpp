// Test helper: raw output of PyTorch's own Philox4x32-10 engine (header-only,
// CPU), used as an independent library reference for the oracle's generator.
// Engine(seed, subsequence, offset): key = seed, counter = (offset, subsequence);
// the first four draws are the four output words of that counter.
#include <ATen/core/PhiloxRNGEngine.h>
#include <cstdint>

extern "C" void aten_philox4x32_10(uint64_t seed, uint64_t subsequence, uint64_t offset,
                                   uint32_t out[4]) {
  at::Philox4_32 engine(seed, subsequence, offset);
  for (int i = 0; i < 4; ++i) out[i] = engine();
}

extern "C" void aten_philox4x32_10_batch(int64_t n, const uint64_t *seeds, const uint64_t *subsequences,
                                         const uint64_t *offsets, uint32_t *out) {
  for (int64_t i = 0; i < n; ++i) aten_philox4x32_10(seeds[i], subsequences[i], offsets[i], out + 4 * i);
}
