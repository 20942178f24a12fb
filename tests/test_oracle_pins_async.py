"""Pins for the oracle's asynchronous exchange (workers reach the master one at a time,
Sec. II and Eqs. 12-13 taken per worker) and for the seeded arrival order.  Each pin is a
closed form, an invariant or a hand computation, not a second copy of the loop."""
import itertools
import math

import numpy as np

from oracle import OracleState


def _rand_state(K, P, seed):
    rng = np.random.default_rng(seed)
    st = OracleState(rng.standard_normal(P).astype(np.float32), K, [(0, P, 1)])
    st.x[:] = rng.standard_normal((K, P)).astype(np.float32)
    return st


def test_async_single_worker_is_eqs_12_13(orc):
    # one worker at 1, master at 0, h1 = 0.5, h2 = 0.25: Eq. 12 gives 1 - 0.5 (1 - 0) = 0.5,
    # Eq. 13 gives 0 + 0.25 (1 - 0) = 0.25 (all values exact in binary32)
    st = OracleState(np.zeros(3, np.float32), 1, [(0, 3, 1)])
    st.x[0] = 1.0
    st.exchange_async(h2=np.array([0.25], np.float32), h1=np.array([0.5], np.float32))
    assert np.array_equal(st.x[0], np.full(3, 0.5, np.float32))
    assert np.array_equal(st.center, np.full(3, 0.25, np.float32))


def test_async_with_one_arrival_equals_simultaneous_bit_for_bit(orc):
    # with a single worker arriving there is nobody whose move it could see
    for who in range(3):
        a, b = _rand_state(3, 257, 21), _rand_state(3, 257, 21)
        mask = np.zeros(3, np.uint8)
        mask[who] = 1
        h2 = np.array([0.07, 0.02, 0.1], np.float32)
        h1 = np.array([0.1, 0.6, 0.3], np.float32)
        a.exchange(mask, h2, h1)
        b.exchange_async(mask, h2, h1, order=np.array([2, 0, 1]))
        assert np.array_equal(a.x, b.x) and np.array_equal(a.center, b.center)


def test_async_identity_cases(orc):
    st = _rand_state(4, 100, 22)
    x0, c0 = st.x.copy(), st.center.copy()
    st.exchange_async(alpha=0.0, order=np.array([3, 1, 0, 2]))
    assert np.array_equal(st.x, x0) and np.array_equal(st.center, c0)
    st.exchange_async(mask=np.zeros(4, np.uint8), alpha=0.4)
    assert np.array_equal(st.x, x0) and np.array_equal(st.center, c0)


def test_async_full_swap_rotates_values_along_the_order(orc):
    # h1 = h2 = 1: every arriving worker takes the master's current value and leaves its
    # own there (x - 1 (x - c) and c + 1 (x - c) are exact for small integers).  Along the
    # arrival order pi the values rotate: first worker gets c0, each next one gets its
    # predecessor's value, and the master ends with the last arrival's value.
    K, P = 5, 16
    st = OracleState(np.zeros(P, np.float32), K, [(0, P, 1)])
    st.center[:] = 100.0
    for i in range(K):
        st.x[i] = float(i + 1)
    order = np.array([3, 0, 4, 1, 2])
    ones = np.ones(K, np.float32)
    st.exchange_async(h2=ones, h1=ones, order=order)
    assert np.all(st.x[3] == 100.0)
    assert np.all(st.x[0] == 4.0) and np.all(st.x[4] == 1.0)
    assert np.all(st.x[1] == 5.0) and np.all(st.x[2] == 2.0)
    assert np.all(st.center == 3.0)


def test_async_weights_belong_to_workers_not_to_arrival_slots(orc):
    # h1 = 0 (workers stay), h2_i = 1 / (arrival position of i): the master becomes the
    # running mean of the arrivals, so it ends at the plain mean of all workers and its
    # start value is forgotten.  Indexing h2 by slot instead of by worker breaks this.
    K, P = 4, 8
    st = _rand_state(K, P, 23)
    st.x[:] = np.array([[8.0], [-4.0], [16.0], [4.0]], np.float32)
    order = np.array([2, 0, 3, 1])
    h2 = np.empty(K, np.float32)
    for pos, i in enumerate(order):
        h2[i] = 1.0 / (pos + 1)
    st.exchange_async(h2=h2, h1=np.zeros(K, np.float32), order=order)
    assert np.allclose(st.center, 6.0, rtol=0, atol=1e-6)
    assert np.array_equal(st.x[:, 0], np.array([8.0, -4.0, 16.0, 4.0], np.float32))


def test_async_identical_workers_contract_geometrically(orc):
    # all workers at y, h2 = alpha, h1 = 0: c_K = y + (1 - alpha)^K (c_0 - y) for any K (the
    # simultaneous form would give c_0 + K alpha (y - c_0), which overshoots once K alpha > 1)
    K, P, al = 32, 10, 0.125
    st = OracleState(np.full(P, 3.0, np.float32), K, [(0, P, 1)])
    st.x[:] = -1.0
    st.exchange_async(h2=np.full(K, al, np.float32), h1=np.zeros(K, np.float32))
    assert np.allclose(st.center, -1.0 + (1 - al) ** K * 4.0, rtol=1e-6)
    sim = OracleState(np.full(P, 3.0, np.float32), K, [(0, P, 1)])
    sim.x[:] = -1.0
    sim.exchange(h2=np.full(K, al, np.float32), h1=np.zeros(K, np.float32))
    assert np.allclose(sim.center, 3.0 - K * al * 4.0)           # = -13: far past the workers


def test_async_equal_coefficients_conserve_the_sum(orc):
    K, P = 6, 300
    st = _rand_state(K, P, 24)
    tot = st.center.astype(np.float64) + st.x.astype(np.float64).sum(0)
    st.exchange_async(alpha=0.2, order=np.array([5, 2, 0, 3, 1, 4]))
    assert np.allclose(st.center.astype(np.float64) + st.x.astype(np.float64).sum(0), tot,
                       rtol=0, atol=2e-6)


def test_async_matches_exact_rational_arithmetic_on_dyadic_inputs(orc):
    # small integers and power-of-two coefficients keep every binary32 operation exact, so
    # the result must equal the exact composition of the affine maps of Eqs. 12-13, here
    # accumulated as a matrix product over the arrivals
    K = 3
    x = np.array([[8.0, -16.0], [4.0, 32.0], [-24.0, 0.0]])
    c = np.array([16.0, -8.0])
    h1 = np.array([0.5, 0.25, 1.0])
    h2 = np.array([0.25, 0.5, 0.125])
    order = [1, 2, 0]
    state = np.vstack([x, c[None]])                      # rows: workers, then master
    for i in order:
        T = np.eye(K + 1)
        T[i, i] -= h1[i]; T[i, K] += h1[i]               # x_i <- (1 - h1) x_i + h1 c
        T[K, K] -= h2[i]; T[K, i] += h2[i]               # c   <- (1 - h2) c   + h2 x_i  (old x_i)
        state = T @ state
    st = OracleState(c.astype(np.float32), K, [(0, 2, 1)])
    st.x[:] = x.astype(np.float32)
    st.exchange_async(h2=h2.astype(np.float32), h1=h1.astype(np.float32), order=np.array(order))
    assert np.array_equal(st.x.astype(np.float64), state[:K])
    assert np.array_equal(st.center.astype(np.float64), state[K])


def test_async_masked_worker_is_skipped_and_untouched(orc):
    a, b = _rand_state(4, 64, 25), _rand_state(4, 64, 25)
    mask = np.array([1, 0, 1, 1], np.uint8)
    x1 = a.x[1].copy()
    a.exchange_async(mask, alpha=0.1, order=np.array([3, 1, 0, 2]))
    b.exchange_async(np.array([1, 1, 1, 1], np.uint8), h2=np.array([.1, 0, .1, .1], np.float32),
                     h1=np.array([.1, 0, .1, .1], np.float32), order=np.array([3, 1, 0, 2]))
    assert np.array_equal(a.x[1], x1)
    assert np.array_equal(a.center, b.center) and np.array_equal(a.x, b.x)


def test_async_default_order_is_ascending(orc):
    a, b = _rand_state(5, 40, 26), _rand_state(5, 40, 26)
    a.exchange_async(alpha=0.3)
    b.exchange_async(alpha=0.3, order=np.arange(5))
    assert np.array_equal(a.x, b.x) and np.array_equal(a.center, b.center)
    c = _rand_state(5, 40, 26)
    c.exchange_async(alpha=0.3, order=np.arange(5)[::-1].copy())
    assert not np.array_equal(a.center, c.center)        # the order matters


# ------------------------------------------------------------------ arrival order
def test_order_is_a_permutation_and_deterministic(orc):
    for K in (1, 2, 3, 8, 64, 256):
        for t in (1, 2, 77):
            o = orc.order_next(K, 0x5EED0003, t)
            assert sorted(o.tolist()) == list(range(K))
            assert np.array_equal(o, orc.order_next(K, 0x5EED0003, t))
    assert not np.array_equal(orc.order_next(16, 1, 1), orc.order_next(16, 1, 2))
    assert not np.array_equal(orc.order_next(16, 1, 1), orc.order_next(16, 2, 1))


def test_order_by_hand_from_generator_words(orc):
    # K = 4: replay the three swaps from the raw generator output
    seed, t = 0xABCDEF0123456789, 9
    key = [seed & 0xffffffff, seed >> 32]
    want = [0, 1, 2, 3]
    r3 = orc.philox([3, 0, t, 3], key)[0] % 4
    want[3], want[r3] = want[r3], want[3]
    r2 = orc.philox([2, 0, t, 3], key)[0] % 3
    want[2], want[r2] = want[r2], want[2]
    r1 = orc.philox([1, 0, t, 3], key)[0] % 2
    want[1], want[r1] = want[r1], want[1]
    assert orc.order_next(4, seed, t).tolist() == want


def test_order_is_uniform_over_permutations(orc):
    # K = 4: all 24 permutations appear with equal frequency (chi-square, 23 d.o.f.)
    n = 24000
    counts = {p: 0 for p in itertools.permutations(range(4))}
    for t in range(n):
        counts[tuple(orc.order_next(4, 12345, t).tolist())] += 1
    chi2 = sum((v - n / 24) ** 2 / (n / 24) for v in counts.values())
    assert min(counts.values()) > 0 and chi2 < 60.0       # P(chi2_23 > 60) ~ 4e-5
    # K = 16: every worker lands on every position about equally often
    pos = np.zeros((16, 16))
    for t in range(8000):
        o = orc.order_next(16, 999, t)
        pos[o, np.arange(16)] += 1
    assert np.abs(pos - 500).max() < 5 * math.sqrt(500)


# ------------------------------------------------------------------ OpenMP build
def test_openmp_build_is_bit_identical_for_the_newer_steps():
    # the parity tests time-box themselves by using the OpenMP build of the oracle: it must
    # give the single-thread build's bits for the asynchronous exchange, the first-order
    # steps, several Hutchinson samples and the partition as well
    import oracle
    results = []
    for variant in ("fp32", "omp"):
        rng = np.random.default_rng(90)
        K, P, segs = 5, 700, [(0, 630, 9), (640, 49, 49)]
        st = OracleState(rng.standard_normal(P).astype(np.float32), K, segs, variant=variant)
        for t in range(1, 9):
            g = rng.standard_normal((K, P)).astype(np.float32)
            hv = rng.standard_normal((3, K, P)).astype(np.float32)
            if t % 2:
                st.local_step(g, hv, 11, t, lr=0.01, want_dist=True)
            else:
                st.sgd_step(g, 0.01, 0.5, active=(rng.random(K) > 0.3).astype(np.uint8), want_dist=True)
            h2, h1 = st.weights_next(0.1)
            st.exchange_async((rng.random(K) > 0.3).astype(np.uint8), h2, h1, order=st.order_next(3, t))
        perm, bounds = oracle.load(variant).partition(17, 5000, 7, 600)
        results.append((st.x.copy(), st.m.copy(), st.v.copy(), st.center.copy(), st.uhist.copy(), perm, bounds))
    for a, b in zip(*results):
        assert np.array_equal(a, b)
