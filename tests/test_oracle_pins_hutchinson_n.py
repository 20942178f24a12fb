"""Pins for the oracle's Hutchinson estimate with n samples per step (Sec. IV-B:
diag(H) ~ (1/n) sum_s z_s (.) (H z_s))."""
import math

import numpy as np

from oracle import OracleState


def _second_moment_root(st, beta2=0.999):
    """|D| recovered from the second moment after one step from v = 0: v = (1 - beta2) D^2."""
    omb2 = float(np.float32(1) - np.float32(beta2))
    return np.sqrt(st.v.astype(np.float64) / omb2)


def test_sample_streams_are_distinct_and_sample_zero_is_the_single_stream(orc):
    K, P = 2, 512
    z0 = orc.sample_z_s(7, 3, 0, K, P)
    assert np.array_equal(z0, orc.sample_z(7, 3, K, P))
    z1, z2 = orc.sample_z_s(7, 3, 1, K, P), orc.sample_z_s(7, 3, 2, K, P)
    assert set(np.unique(z1)) == {-1.0, 1.0}
    for a, b in ((z0, z1), (z0, z2), (z1, z2)):
        assert abs((a.astype(np.float64) * b).mean()) < 5 / math.sqrt(K * P)
    # counter word by hand: sample s replaces the domain word 0 by 256 s
    j, i, t, seed = 300, 1, 3, 7
    w = orc.philox([j >> 7, i, t, 256 * 2], [seed & 0xffffffff, seed >> 32])
    assert z2[i, j] == (-1.0 if (w[(j >> 5) & 3] >> (j & 31)) & 1 else 1.0)


def test_n_samples_exact_on_diagonal_quadratic(orc):
    # every sample gives z (.) (h z) = h exactly, so the mean over n samples is h (the sum
    # of n equal binary32 values divided by n is exact for n = 2, 4) and v = (1 - beta2) h^2
    P, K = 500, 2
    rng = np.random.default_rng(40)
    h = rng.uniform(0.1, 10, P).astype(np.float32)
    for n in (2, 4):
        st = OracleState(rng.standard_normal(P).astype(np.float32), K, [(0, P, 1)])
        hvp = np.stack([(h[None] * orc.sample_z_s(5, 1, s, K, P)).astype(np.float32) for s in range(n)])
        g = (h[None] * st.x).astype(np.float32)
        st.local_step(g, hvp, 5, 1, lr=0.1)
        omb2 = np.float32(1) - np.float32(0.999)
        assert np.array_equal(st.v, np.broadcast_to((omb2 * h) * h, (K, P))), n


def test_n_samples_equal_the_mean_of_single_sample_estimates(orc):
    # dense symmetric H: the n-sample estimate is the mean of the n single-sample ones,
    # each formed outside the oracle from its own z_s
    P, n = 12, 3
    rng = np.random.default_rng(41)
    A = rng.standard_normal((P, P))
    H = (A @ A.T).astype(np.float32)
    zs = [orc.sample_z_s(9, 2, s, 1, P)[0] for s in range(n)]
    hvp = np.stack([(H @ z)[None].astype(np.float32) for z in zs])
    st = OracleState(np.zeros(P, np.float32), 1, [(0, P, 1)])
    st.local_step(np.zeros((1, P), np.float32), hvp, 9, 2, lr=0.0)
    want = np.mean([z.astype(np.float64) * hv[0].astype(np.float64) for z, hv in zip(zs, hvp)], axis=0)
    assert np.allclose(_second_moment_root(st)[0], np.abs(want), rtol=1e-5, atol=1e-6)


def test_more_samples_reduce_the_estimation_error(orc):
    # error of the estimate against diag(H) falls like 1 / sqrt(n)
    P, T = 8, 300
    rng = np.random.default_rng(42)
    A = rng.standard_normal((P, P))
    H = (A @ A.T + 20 * np.eye(P)).astype(np.float32)     # diagonal dominates: D stays positive
    err = {}
    for n in (1, 8):
        e = 0.0
        for t in range(1, T + 1):
            hvp = np.stack([(H @ orc.sample_z_s(3, t, s, 1, P)[0])[None].astype(np.float32)
                            for s in range(n)])
            st = OracleState(np.zeros(P, np.float32), 1, [(0, P, 1)])
            st.local_step(np.zeros((1, P), np.float32), hvp if n > 1 else hvp[0], 3, t, lr=0.0)
            e += np.mean((_second_moment_root(st)[0] - np.diag(H)) ** 2)
        err[n] = e / T
    assert 0.08 < err[8] / err[1] < 0.2                    # about 1 / 8


def test_single_sample_array_forms_agree(orc):
    # hvp given as [K, ld] and as [1, K, ld] are the same step, bit for bit
    K, P = 3, 100
    rng = np.random.default_rng(43)
    g = rng.standard_normal((K, P)).astype(np.float32)
    hv = rng.standard_normal((K, P)).astype(np.float32)
    a = OracleState(np.zeros(P, np.float32), K, [(0, 99, 9)])
    b = OracleState(np.zeros(P, np.float32), K, [(0, 99, 9)])
    a.local_step(g, hv, 1, 1, lr=0.01)
    b.local_step(g, hv[None].copy(), 1, 1, lr=0.01)
    assert np.array_equal(a.x, b.x) and np.array_equal(a.v, b.v)


def test_sum_then_divide_order_with_spatial_average(orc):
    # two samples, one block of 3: D = ((z0 h0 + z1 h1) / 2) per element, then the block mean
    P = 3
    z0, z1 = orc.sample_z_s(4, 1, 0, 1, P)[0], orc.sample_z_s(4, 1, 1, 1, P)[0]
    h0 = np.array([1.0, 2.0, 4.0], np.float32)
    h1 = np.array([8.0, -2.0, 0.5], np.float32)
    st = OracleState(np.zeros(P, np.float32), 1, [(0, 3, 3)])
    st.local_step(np.zeros((1, P), np.float32), np.stack([h0[None], h1[None]]), 4, 1, lr=0.0)
    per_elem = (z0 * h0 + z1 * h1) / 2.0                   # exact in binary32 for these values
    mean = np.float32((np.float32(per_elem[0] + per_elem[1]) + per_elem[2]) / np.float32(3))
    omb2 = np.float32(1) - np.float32(0.999)
    assert np.array_equal(st.v[0], np.full(3, (omb2 * mean) * mean, np.float32))
