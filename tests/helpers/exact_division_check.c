/*
 * Exhaustive host check of the constant-divisor shortcut the CUDA kernels use:
 *
 *     q  = RN(x * r)            r = RN(1 / b), rounded once on the host
 *     e  = RN(fma(-b, q, x))    the remainder x - b q, exact
 *     q' = RN(fma(e, r, q))
 *
 * Claim: q' == RN(x / b), the correctly rounded quotient, for every binary32 x whose
 * exponent keeps all intermediates in the normal range.  The sequence commutes with
 * scaling x by a power of two inside that range, so checking all 2^23 significands
 * of one binade per divisor covers every such x.  Divisors checked: the integers
 * 2..128 (spatial block sizes) and the bias-correction constants (float)(1 - beta^t).
 *
 * Usage: exact_division_check         -> prints "checked <n> mismatches <m>"
 * Built by the test with: gcc -O2 -mfma -ffp-contract=off -fopenmp ... -lm
 */
#include <math.h>
#include <stdint.h>
#include <stdio.h>
#include <string.h>

static float from_bits(uint32_t u) { float f; memcpy(&f, &u, 4); return f; }

static uint64_t check_divisor(float b)
{
    const float r = 1.0f / b;
    uint64_t bad = 0;
#pragma omp parallel for reduction(+ : bad) schedule(static)
    for (uint32_t mant = 0; mant < (1u << 23); ++mant) {
        const float x = from_bits(0x3f800000u | mant);          /* [1, 2) */
        const float q = x * r;
        const float e = fmaf(-b, q, x);
        const float q2 = fmaf(e, r, q);
        if (q2 != x / b) bad += 1;
    }
    return bad;
}

int main(void)
{
    uint64_t checked = 0, bad = 0;
    for (int b = 2; b <= 128; ++b) { bad += check_divisor((float)b); checked += 1; }
    const double betas[] = {0.9, 0.999, 0.99, 0.5, 0.95};
    for (unsigned k = 0; k < sizeof betas / sizeof betas[0]; ++k) {
        const float beta = (float)betas[k];
        float last = -1.0f;
        for (int t = 1; t <= 40; ++t) {
            /* t = 1..12 densely, then doubling up to about 2^28 steps */
            const double tt = t <= 12 ? (double)t : ldexp(1.0, t - 12 + 3) * 1.5;
            const float b = (float)(1.0 - pow((double)beta, tt));
            if (b == last || !(b > 0.0f)) continue;
            last = b;
            bad += check_divisor(b);
            checked += 1;
        }
    }
    printf("checked %llu mismatches %llu\n", (unsigned long long)checked, (unsigned long long)bad);
    return bad ? 1 : 0;
}
