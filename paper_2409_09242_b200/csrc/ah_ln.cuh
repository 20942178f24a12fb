// Natural logarithm in double-double arithmetic, identical on host and device.
//
// The dynamic weighting rule needs u = log ||x_i - c|| (Sec. V-B of the paper) on
// the host (dw_weights_next) and on the device (easgd_exchange_dynamic), and the
// weights derived from it must not depend on where it was evaluated or on the
// platform's math library.  So the logarithm is written out here as a fixed list of
// IEEE binary64 additions, multiplications, divisions and fused multiply-adds, none
// of which the compiler may regroup or contract:
//
//   x = m 2^e,  m in (sqrt(1/2), sqrt(2)];   s = (m - 1) / (m + 1);   z = s^2
//   ln m = 2 s (1 + z/3 + z^2/5 + ... + z^21/43)          Horner, highest term first
//   ln x = e ln 2 + ln m                                    ln 2 as a pair of doubles
//
// Every quantity is a pair (hi, lo) with about 100 significant bits; the result is
// the hi part after the last renormalisation, i.e. the correctly rounded logarithm
// except for inputs within 2^-98 of a rounding boundary.  Not installed.
#pragma once

#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>
#include <string.h>

namespace ah {

#ifdef __CUDA_ARCH__
#define AH_DADD(a, b) __dadd_rn((a), (b))
#define AH_DSUB(a, b) __dsub_rn((a), (b))
#define AH_DMUL(a, b) __dmul_rn((a), (b))
#define AH_DDIV(a, b) __ddiv_rn((a), (b))
#define AH_DFMA(a, b, c) __fma_rn((a), (b), (c))
#else
#define AH_DADD(a, b) ((a) + (b))
#define AH_DSUB(a, b) ((a) - (b))
#define AH_DMUL(a, b) ((a) * (b))
#define AH_DDIV(a, b) ((a) / (b))
#define AH_DFMA(a, b, c) fma((a), (b), (c))
#endif

struct Pair {
    double hi, lo;
};

// a + b exactly, as a pair (Knuth).
__host__ __device__ inline Pair sum_exact(double a, double b)
{
    Pair r;
    r.hi = AH_DADD(a, b);
    const double t = AH_DSUB(r.hi, a);
    r.lo = AH_DADD(AH_DSUB(a, AH_DSUB(r.hi, t)), AH_DSUB(b, t));
    return r;
}

// a + b exactly when |a| >= |b| (Dekker).
__host__ __device__ inline Pair sum_exact_ordered(double a, double b)
{
    Pair r;
    r.hi = AH_DADD(a, b);
    r.lo = AH_DSUB(b, AH_DSUB(r.hi, a));
    return r;
}

__host__ __device__ inline Pair pair_mul(Pair a, Pair b)
{
    const double p = AH_DMUL(a.hi, b.hi);
    double e = AH_DFMA(a.hi, b.hi, -p);
    e = AH_DFMA(a.hi, b.lo, e);
    e = AH_DFMA(a.lo, b.hi, e);
    return sum_exact_ordered(p, e);
}

__host__ __device__ inline Pair pair_add(Pair a, Pair b)
{
    const Pair s = sum_exact(a.hi, b.hi);
    const double e = AH_DADD(s.lo, AH_DADD(a.lo, b.lo));
    return sum_exact_ordered(s.hi, e);
}

// 1 / n for a small integer n: hi = RN(1 / n), lo = RN(fma(-hi, n, 1) / n).
__host__ __device__ inline Pair pair_reciprocal(double n)
{
    Pair r;
    r.hi = AH_DDIV(1.0, n);
    r.lo = AH_DDIV(AH_DFMA(-r.hi, n, 1.0), n);
    return r;
}

// The same pairs for the odd n = 3, 5, ..., 43 of the series, written out (entry k holds
// 1 / (2k + 3)), so that the series costs no divisions; a host test recomputes them with
// pair_reciprocal.  Kept as a table (constant memory on the device) so that the series
// can be a loop: the rule runs once per launch, where short code starts faster.
#define AH_SERIES_RECIPROCALS {                                              \
    {0x1.5555555555555p-2, 0x1.5555555555555p-56}  /* 1 / 3 */, \
    {0x1.999999999999ap-3, -0x1.999999999999ap-57}  /* 1 / 5 */, \
    {0x1.2492492492492p-3, 0x1.2492492492492p-57}  /* 1 / 7 */, \
    {0x1.c71c71c71c71cp-4, 0x1.c71c71c71c71cp-58}  /* 1 / 9 */, \
    {0x1.745d1745d1746p-4, -0x1.745d1745d1746p-59}  /* 1 / 11 */, \
    {0x1.3b13b13b13b14p-4, -0x1.3b13b13b13b14p-58}  /* 1 / 13 */, \
    {0x1.1111111111111p-4, 0x1.1111111111111p-60}  /* 1 / 15 */, \
    {0x1.e1e1e1e1e1e1ep-5, 0x1.e1e1e1e1e1e1ep-61}  /* 1 / 17 */, \
    {0x1.af286bca1af28p-5, 0x1.af286bca1af28p-59}  /* 1 / 19 */, \
    {0x1.8618618618618p-5, 0x1.8618618618618p-59}  /* 1 / 21 */, \
    {0x1.642c8590b2164p-5, 0x1.642c8590b2164p-60}  /* 1 / 23 */, \
    {0x1.47ae147ae147bp-5, -0x1.eb851eb851eb8p-61}  /* 1 / 25 */, \
    {0x1.2f684bda12f68p-5, 0x1.2f684bda12f68p-59}  /* 1 / 27 */, \
    {0x1.1a7b9611a7b96p-5, 0x1.1a7b9611a7b96p-61}  /* 1 / 29 */, \
    {0x1.0842108421084p-5, 0x1.0842108421084p-60}  /* 1 / 31 */, \
    {0x1.f07c1f07c1f08p-6, -0x1.f07c1f07c1f08p-61}  /* 1 / 33 */, \
    {0x1.d41d41d41d41dp-6, 0x1.0750750750750p-60}  /* 1 / 35 */, \
    {0x1.bacf914c1bad0p-6, -0x1.bacf914c1bad0p-60}  /* 1 / 37 */, \
    {0x1.a41a41a41a41ap-6, 0x1.0690690690690p-60}  /* 1 / 39 */, \
    {0x1.8f9c18f9c18fap-6, -0x1.f3831f3831f38p-61}  /* 1 / 41 */, \
    {0x1.7d05f417d05f4p-6, 0x1.7d05f417d05f4p-62}  /* 1 / 43 */ }
static const double kSeriesReciprocalHost[21][2] = AH_SERIES_RECIPROCALS;
#ifdef __CUDACC__
static __constant__ double kSeriesReciprocalDevice[21][2] = AH_SERIES_RECIPROCALS;
#endif
#undef AH_SERIES_RECIPROCALS

__host__ __device__ inline Pair series_reciprocal(int k)
{
#ifdef __CUDA_ARCH__
    return Pair{kSeriesReciprocalDevice[k][0], kSeriesReciprocalDevice[k][1]};
#else
    return Pair{kSeriesReciprocalHost[k][0], kSeriesReciprocalHost[k][1]};
#endif
}

// ln x for a positive, finite, normal x.
__host__ __device__ inline double ln_pairwise(double x)
{
    uint64_t bits;
#ifdef __CUDA_ARCH__
    bits = (uint64_t)__double_as_longlong(x);
#else
    memcpy(&bits, &x, sizeof bits);
#endif
    int e = (int)((bits >> 52) & 0x7ffu) - 1023;
    bits = (bits & 0x000fffffffffffffull) | 0x3ff0000000000000ull;
    double m;
#ifdef __CUDA_ARCH__
    m = __longlong_as_double((long long)bits);
#else
    memcpy(&m, &bits, sizeof m);
#endif
    if (m > 1.4142135623730951) {
        m = AH_DMUL(m, 0.5);
        e += 1;
    }
    // s = (m - 1) / (m + 1): quotient plus one correction from the exact remainder
    const double num = AH_DSUB(m, 1.0);
    const Pair den = sum_exact(m, 1.0);
    const double q = AH_DDIV(num, den.hi);
    double rem = AH_DFMA(-q, den.hi, num);
    rem = AH_DFMA(-q, den.lo, rem);
    const Pair s = sum_exact_ordered(q, AH_DDIV(rem, den.hi));

    const Pair z = pair_mul(s, s);
    Pair series = series_reciprocal(20);                       // 1 / 43
#pragma unroll 1
    for (int k = 20; k >= 1; --k)
        series = pair_add(pair_mul(series, z), series_reciprocal(k - 1));   // 1 / (2k + 1)
    const Pair unity = {1.0, 0.0};
    series = pair_add(pair_mul(series, z), unity);
    Pair ln_m = pair_mul(s, series);
    ln_m.hi = AH_DMUL(2.0, ln_m.hi);
    ln_m.lo = AH_DMUL(2.0, ln_m.lo);

    const Pair ln2 = {0x1.62e42fefa39efp-1, 0x1.abc9e3b39803fp-56};
    const Pair exponent = {(double)e, 0.0};
    return pair_add(pair_mul(ln2, exponent), ln_m).hi;
}

// u = log ||x_i - c|| from the squared distance, clamped away from zero (workers
// start as copies of the master, so the distance can be exactly 0).
// Out of line: one copy of the code per translation unit, so that on the device whoever
// runs it first has fetched it for everybody after it.
#ifdef __CUDACC__
#define AH_NOINLINE __noinline__
#else
#define AH_NOINLINE __attribute__((noinline))
#endif
static __host__ __device__ AH_NOINLINE double u_from_norm2(double n2)
{
    return AH_DMUL(0.5, ln_pairwise(n2 > 1e-300 ? n2 : 1e-300));
}

}  // namespace ah
