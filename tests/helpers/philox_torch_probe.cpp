// Test-only probe: prints the four Philox words that the generator header
// shipped with PyTorch produces for (seed, subsequence, offset) triples read
// from the command line.  It is compiled by the test suite to pin the oracle's
// own generator against an implementation it did not come from.
#include <ATen/core/PhiloxRNGEngine.h>
#include <cstdint>
#include <cstdio>
#include <cstdlib>

int main(int argc, char** argv) {
  for (int i = 1; i + 2 < argc; i += 3) {
    uint64_t seed = strtoull(argv[i], nullptr, 0);
    uint64_t subseq = strtoull(argv[i + 1], nullptr, 0);
    uint64_t offset = strtoull(argv[i + 2], nullptr, 0);
    at::Philox4_32 eng(seed, subseq, offset);
    uint32_t w0 = eng(), w1 = eng(), w2 = eng(), w3 = eng();
    std::printf("%u %u %u %u\n", w0, w1, w2, w3);
  }
  return 0;
}
