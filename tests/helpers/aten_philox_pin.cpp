// Test helper: prints Philox4x32-10 blocks produced by ATen's host-side engine
// (an implementation independent of this repository's oracle).  Reads lines of
// "seed subsequence offset" (decimal, 64-bit) from stdin; for each prints the
// four 32-bit words of block `offset` of that (seed, subsequence) stream.
#include <ATen/core/PhiloxRNGEngine.h>

#include <cinttypes>
#include <cstdio>

int main() {
    unsigned long long seed, subseq, offset;
    while (std::scanf("%llu %llu %llu", &seed, &subseq, &offset) == 3) {
        at::Philox4_32 eng(seed, subseq, offset);
        uint32_t w0 = eng(), w1 = eng(), w2 = eng(), w3 = eng();
        std::printf("%" PRIu32 " %" PRIu32 " %" PRIu32 " %" PRIu32 "\n", w0, w1, w2, w3);
    }
    return 0;
}
