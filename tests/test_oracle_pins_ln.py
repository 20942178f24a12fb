"""Pins for the oracle's natural logarithm (the quad-precision library logarithm rounded
once to double, used for u = log ||x_i - c||, Sec. V-B): against arbitrary-precision
arithmetic, against the platform's libm, and at values that are known exactly."""
import math

import mpmath
import numpy as np


def _correctly_rounded_ln(x):
    mpmath.mp.prec = 300
    return float(mpmath.log(mpmath.mpf(x)))          # mpf -> float rounds to nearest


def test_ln_is_correctly_rounded_on_random_inputs(orc):
    rng = np.random.default_rng(50)
    xs = np.concatenate([
        np.exp(rng.uniform(-690, 700, 4000)),                      # the whole exponent range
        rng.uniform(0.5, 2.0, 4000),                               # around 1, where ln cancels
        1.0 + rng.uniform(-1, 1, 2000) * 1e-9,
        np.exp(2 * rng.normal(0, 3, 4000)),                        # squared distances of the method
        np.array([1e-300, 2.2250738585072014e-308, 1.7976931348623157e308, 0.7071067811865476,
                  1.4142135623730951, 1.4142135623730954, 2.0, 0.5, 3.0, 10.0, math.e]),
    ])
    bad = [(x, orc.ln(x), _correctly_rounded_ln(x)) for x in xs if orc.ln(x) != _correctly_rounded_ln(x)]
    assert not bad, bad[:5]


def test_ln_exact_values_and_identities(orc):
    assert orc.ln(1.0) == 0.0
    mpmath.mp.prec = 300
    for k in (-1022, -300, -1, 1, 2, 10, 52, 1023):
        assert orc.ln(math.ldexp(1.0, k)) == float(k * mpmath.log(2))
    xs = np.exp(np.linspace(-50, 50, 2001))
    vals = np.array([orc.ln(x) for x in xs])
    assert np.all(np.diff(vals) > 0)                               # monotone
    for x in (3.7, 1e-12, 8.25e40):                                # ln(1/x) = -ln(x) to an ulp
        assert abs(orc.ln(1 / x) + orc.ln(x)) <= 2 * np.spacing(abs(orc.ln(x)))


def test_ln_agrees_with_libm_within_one_ulp(orc):
    rng = np.random.default_rng(51)
    for x in np.exp(rng.uniform(-600, 600, 5000)):
        a, b = orc.ln(float(x)), math.log(float(x))
        assert abs(a - b) <= np.spacing(abs(b)), x


def test_u_is_half_the_log_of_the_squared_distance(orc):
    assert orc.u_from_norm2(0.0) == 0.5 * orc.ln(1e-300)           # clamp at the start (x_i = c)
    assert orc.u_from_norm2(math.e ** 2) == 0.5 * orc.ln(math.e ** 2)
    assert abs(orc.u_from_norm2(16.0) - math.log(4.0)) < 1e-15     # log of the 2-norm itself
