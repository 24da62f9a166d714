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
