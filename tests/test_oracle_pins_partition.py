"""Pins for the oracle's data-overlap partition (Sec. V-A): the set identities the paper
states, the sizes, a hand replay from raw generator words, and uniformity."""
import math

import numpy as np
import pytest


def _sets(perm, bounds, k):
    O = perm[:int(bounds[1])]
    S = [perm[int(bounds[j + 1]):int(bounds[j + 2])] for j in range(k)]
    return O, S


@pytest.mark.parametrize("n,k,o", [(60000, 8, 7500), (60000, 4, 15000), (1000, 4, 0), (1000, 8, 375),
                                   (17, 5, 3), (10, 3, 10), (1, 1, 0), (9, 4, 1)])
def test_partition_identities(orc, n, k, o):
    perm, bounds = orc.partition(0x5EED0004, n, k, o)
    assert sorted(perm.tolist()) == list(range(n))                # a permutation of the data set
    O, S = _sets(perm, bounds, k)
    assert len(O) == o                                              # |O| = o
    union = np.concatenate(S) if S else np.empty(0, np.uint32)
    assert len(set(union.tolist())) == len(union)                   # S_i and S_j disjoint
    assert set(union.tolist()) == set(range(n)) - set(O.tolist())   # union S_j = D - O
    sizes = [len(s) for s in S]
    base, extra = divmod(n - o, k)
    assert sizes == [base + (1 if j < extra else 0) for j in range(k)]
    if extra == 0:
        assert all(sz == (n - o) // k for sz in sizes)              # |S_j| = floor((n - o) / k)
    assert int(bounds[-1]) == n
    for j in range(k):                                               # D_j = O u S_j
        assert len(set(O.tolist()) | set(S[j].tolist())) == o + sizes[j]


def test_partition_paper_ratios(orc):
    # Sec. VII: overlap ratio 12.5% with 8 workers, 25% with 4 workers; MNIST has 60000
    # training points: 7500 shared + 6562 or 6563 own; 15000 shared + 11250 own
    _, b8 = orc.partition(1, 60000, 8, 60000 // 8)
    assert int(b8[1]) == 7500 and np.diff(b8[1:]).tolist() == [6563] * 4 + [6562] * 4
    _, b4 = orc.partition(1, 60000, 4, 60000 // 4)
    assert int(b4[1]) == 15000 and np.diff(b4[1:]).tolist() == [11250] * 4


def test_partition_by_hand_from_generator_words(orc):
    seed, n = 0x0123456789ABCDEF, 6
    key = [seed & 0xffffffff, seed >> 32]
    want = list(range(n))
    for q in range(n - 1, 0, -1):
        w = orc.philox([q, 0, 0, 4], key)
        pick = ((w[1] << 32) | w[0]) % (q + 1)
        want[q], want[pick] = want[pick], want[q]
    perm, bounds = orc.partition(seed, n, 2, 2)
    assert perm.tolist() == want
    assert bounds.tolist() == [0, 2, 4, 6]


def test_partition_determinism_and_seed(orc):
    a, _ = orc.partition(5, 5000, 4, 1000)
    b, _ = orc.partition(5, 5000, 4, 1000)
    c, _ = orc.partition(6, 5000, 4, 1000)
    assert np.array_equal(a, b) and not np.array_equal(a, c)
    with pytest.raises(ValueError):
        orc.partition(5, 10, 2, 11)


def test_partition_is_uniform(orc):
    # every data point is shared with probability o / n, and lands with each worker
    # equally often, over many seeds
    n, k, o, trials = 40, 4, 8, 6000
    shared = np.zeros(n)
    owner = np.zeros((n, k))
    for t in range(trials):
        perm, bounds = orc.partition(1000 + t, n, k, o)
        shared[perm[:o]] += 1
        for j in range(k):
            owner[perm[int(bounds[j + 1]):int(bounds[j + 2])], j] += 1
    p = o / n
    assert np.abs(shared - trials * p).max() < 5 * math.sqrt(trials * p * (1 - p))
    q = (1 - p) / k
    assert np.abs(owner - trials * q).max() < 5 * math.sqrt(trials * q * (1 - q))
    # position uniformity of the permutation itself (first slot)
    first = np.zeros(n)
    for t in range(trials):
        first[orc.partition(50000 + t, n, 1, 0)[0][0]] += 1
    assert np.abs(first - trials / n).max() < 5 * math.sqrt(trials / n)
