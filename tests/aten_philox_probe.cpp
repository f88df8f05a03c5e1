// Calls the Philox4_32 engine that ships in PyTorch's headers (ATen/core/PhiloxRNGEngine.h)
// through its documented constructor (seed, subsequence, offset) and prints the four
// 32-bit words of the first 128-bit block.  Used by the oracle's pin tests as an
// independently written implementation of Philox4x32-10; nothing of it is copied.
// stdin: lines "seed subsequence offset" (decimal, 64-bit); stdout: four hex words per line.
#include <ATen/core/PhiloxRNGEngine.h>
#include <cinttypes>
#include <cstdio>

int main() {
    unsigned long long seed, subseq, offset;
    while (std::scanf("%llu %llu %llu", &seed, &subseq, &offset) == 3) {
        at::Philox4_32 eng(seed, subseq, offset);
        uint32_t w0 = eng(), w1 = eng(), w2 = eng(), w3 = eng();
        std::printf("%08x %08x %08x %08x\n", w0, w1, w2, w3);
    }
    return 0;
}
