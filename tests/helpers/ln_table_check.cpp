// Host check of the logarithm's written-out constants: every entry of series_reciprocal
// must equal the pair that pair_reciprocal computes for the same odd integer.
#include <cstdio>

#include "ah_ln.cuh"

int main()
{
    int bad = 0;
    for (int k = 0; k <= 20; ++k) {
        const ah::Pair want = ah::pair_reciprocal((double)(2 * k + 3));
        const ah::Pair got = ah::series_reciprocal(k);
        if (want.hi != got.hi || want.lo != got.lo) {
            std::printf("entry %d (1/%d): %a %a, want %a %a\n", k, 2 * k + 3, got.hi, got.lo, want.hi, want.lo);
            ++bad;
        }
    }
    std::printf("checked 21 bad %d\n", bad);
    return bad != 0;
}
