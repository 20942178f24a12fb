"""GPU parity tests: the CUDA library, called through its C ABI, against the CPU oracle
element by element on the same seeded inputs.  Bar: z, masks, weights bit-exact;
binary32 state within |gpu - oracle| <= 1e-6 + 1e-5 |oracle| (and, because the kernels
follow the oracle's operation order, in fact bit-identical for hessian power 1 and 1/2)."""
import ctypes as C

import numpy as np
import pytest

import oracle
from oracle import OracleState
from paper_2409_09242_b200 import workloads as W
from parity_driver import RunConfig, compare_state, run_gaussian, tolerance_violations, Z_SEED

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2409_09242_b200 import binding
    return binding


@pytest.fixture(scope="module")
def torch():
    import torch
    torch.cuda.set_device(0)
    return torch


ODD_SEGS = [(3, 18, 9), (21, 10, 1), (37, 4900, 49), (4940, 2505, 5), (9001, 4096, 128)]
ODD_P = 13_111


def _inputs(segs, P, K, n_pool, seed, scale=0.1):
    rng = np.random.default_rng(seed)
    ld = W.padded_ld(P)
    theta0 = (rng.standard_normal(P) * scale).astype(np.float32)
    pool = []
    for _ in range(n_pool):
        g = np.zeros((K, ld), np.float32)
        h = np.zeros((K, ld), np.float32)
        g[:, :P] = rng.standard_normal((K, P)).astype(np.float32) * np.float32(scale)
        h[:, :P] = rng.standard_normal((K, P)).astype(np.float32) * np.float32(scale)
        pool.append((g, h))
    return theta0, pool


# ------------------------------------------------------------------------- z
@pytest.mark.parametrize("K,P", [(4, 1 << 20), (3, 184_837), (2, 129), (1, 1), (5, 4097)])
def test_sample_z_bit_exact(B, torch, K, P):
    h = B.Handle(K, P, [])
    ld = W.padded_ld(P) + 8
    for seed, t in ((Z_SEED, 1), (0xDEADBEEFCAFEF00D, 77), (0, 0xFFFFFFFE)):
        dst = torch.full((K, ld), 7.0, dtype=torch.float32, device="cuda")
        h.ah_sample_z(seed, t, dst)
        got = dst.cpu().numpy()
        want = oracle.load("omp").sample_zbits(seed, t, K, P)
        assert np.array_equal(got[:, :P], np.where(want == 1, -1.0, 1.0).astype(np.float32))
        assert np.all(got[:, P:] == 7.0)                 # nothing written past P
    h.close()


# ------------------------------------------------- premises of the exact arithmetic
def test_branch_free_square_root_and_division_are_correctly_rounded(B, torch):
    # the local step's square root and division inside the usual operand range are branch-free
    # sequences built on hardware approximations; on this device: the square root equals the
    # IEEE one for every input of its range, the refined reciprocal equals the IEEE reciprocal
    # for every input of its range (the premise of Markstein's division), and the quotient
    # equals the IEEE one on 2^33 seeded pairs, half of them aimed at rounding boundaries
    assert B.ah_check_exact_arithmetic(1 << 33) == [0, 0, 0]


# ---------------------------------------------------------------- local step
@pytest.mark.parametrize("segs,P", [
    ([(0, 5000, 1)], 5000),                      # one unstructured tensor
    ([], 2048 * 3),                              # no table at all, exact tiles
    ([(0, 9 * 700, 9)], 6300),                   # blocks straddle tile edges
    (ODD_SEGS, ODD_P),                           # odd offsets, gaps, block 49/5/128
    ([(0, 1, 1)], 1), ([(0, 3, 3)], 3), ([(1, 4, 2)], 6),
])
@pytest.mark.parametrize("hp,wd", [(1.0, 0.0), (0.5, 0.01), (0.75, 0.0)])
def test_local_step_matches_oracle(B, torch, segs, P, hp, wd):
    K, R = 3, 4
    theta0, pool = _inputs(segs, P, K, 2, seed=P)
    cfg = RunConfig(K=K, segments=segs, P=P, rounds=R, tau=10 ** 6, lr=0.02, hessian_power=hp,
                    weight_decay=wd)
    h, ref, _ = run_gaussian(cfg, B, oracle, (theta0, pool), variant="fp32")
    viol, bits = compare_state(h, ref, B)
    assert sum(viol.values()) == 0, viol
    if hp in (1.0, 0.5):
        assert sum(bits.values()) == 0, bits           # same operation order => same bits
    assert np.array_equal(h.ah_state_get(B.AH_STEP), ref.step)
    h.close()


@pytest.mark.parametrize("seed", range(8))
def test_local_step_random_segment_tables(B, torch, seed):
    # irregular tensor tables: every block size up to 128, blocks across tile edges, many
    # tensors inside one tile, gaps, odd offsets, ragged ends; plain, distance, n-sample and
    # one-pass forms of the step
    segs, P = W.random_segment_table(100 + seed, B.AH_MAX_BLOCK)
    K, ld = 3, W.padded_ld(P)
    rng = np.random.default_rng(seed)
    theta0 = (rng.standard_normal(P) * 0.1).astype(np.float32)
    h = B.Handle(K, P, segs)
    ref = OracleState(theta0, K, segs)
    h.ah_state_set(B.AH_CENTER, theta0)
    h.ah_broadcast_center()
    for t in range(1, 7):
        n = 2 if t == 3 else 1
        g = np.zeros((K, ld), np.float32)
        hv = np.zeros((n, K, ld), np.float32)
        g[:, :P] = rng.standard_normal((K, P)).astype(np.float32) * np.float32(0.1)
        hv[:, :, :P] = rng.standard_normal((n, K, P)).astype(np.float32) * np.float32(0.1)
        gd = torch.from_numpy(g).cuda()
        hd = torch.from_numpy(hv if n > 1 else hv[0]).cuda()
        if t == 5:      # exchange, then this step, in one pass
            h.easgd_exchange_then_step(gd, hd, Z_SEED, lr=0.01, round_=t, alpha=0.2)
            ref.exchange(alpha=0.2)
            ref.local_step(g, hv[0], Z_SEED, t, lr=0.01)
        else:
            h.ah_local_step(gd, hd, Z_SEED, lr=0.01, round_=t, want_dist=t % 2 == 0)
            ref.local_step(g, hv if n > 1 else hv[0], Z_SEED, t, lr=0.01, want_dist=t % 2 == 0)
        if t % 2 == 0:
            assert np.array_equal(h.ah_state_get(B.AH_NORM2), ref.norm2), t
    for which, want in ((B.AH_X, ref.x), (B.AH_M, ref.m), (B.AH_V, ref.v), (B.AH_CENTER, ref.center)):
        assert np.array_equal(h.ah_state_get(which), want), which
    h.close()


def test_local_step_inactive_padding_and_auto_round(B, torch):
    segs, P, K = ODD_SEGS, ODD_P, 4
    theta0, pool = _inputs(segs, P, K, 1, seed=5)
    g = torch.from_numpy(pool[0][0]).cuda()
    hv = torch.from_numpy(pool[0][1]).cuda()
    # a wider row stride than P, with poison in the padding columns
    ld = W.padded_ld(P) + 64
    gw = torch.full((K, ld), float("nan"), device="cuda")
    hw = torch.full((K, ld), float("nan"), device="cuda")
    gw[:, :P] = g[:, :P]
    hw[:, :P] = hv[:, :P]
    h = B.Handle(K, P, segs)
    h.ah_state_set(B.AH_CENTER, theta0)
    h.ah_broadcast_center()
    ref = OracleState(theta0, K, segs)
    active = np.array([1, 0, 1, 1], np.uint8)
    for t in (1, 2, 3):
        act = active if t == 2 else None
        h.ah_local_step(gw, hw, Z_SEED, lr=0.01, active=act)          # round = call count
        ref.local_step(pool[0][0], pool[0][1], Z_SEED, t, lr=0.01, active=act)
    viol, bits = compare_state(h, ref, B)
    assert sum(viol.values()) == 0 and sum(bits.values()) == 0
    assert np.array_equal(h.ah_state_get(B.AH_STEP), np.array([3, 2, 3, 3], np.uint32))
    assert np.array_equal(h.ah_state_get(B.AH_ROUND), np.array([3, 0], np.uint32))
    h.close()


# ------------------------------------------------------------------ distances
@pytest.mark.parametrize("K,P", [(2, 1), (3, 5), (4, 2048), (2, 2049), (3, 300_001), (1, 1 << 20)])
def test_norm2_bit_exact(B, torch, K, P):
    rng = np.random.default_rng(P)
    theta0 = rng.standard_normal(P).astype(np.float32)
    x = (theta0[None] + rng.standard_normal((K, P)).astype(np.float32) * np.float32(0.01))
    h = B.Handle(K, P, [])
    h.ah_state_set(B.AH_CENTER, theta0)
    h.ah_state_set(B.AH_X, x)
    # a step in which nobody is active leaves x alone and still measures every distance
    z = torch.zeros((K, W.padded_ld(P)), device="cuda")
    h.ah_local_step(z, z, 1, lr=0.0, active=np.zeros(K, np.uint8), want_dist=True)
    got = h.ah_state_get(B.AH_NORM2)
    want = oracle.load("omp").norm2(np.ascontiguousarray(x), theta0)
    assert np.array_equal(got, want)
    assert np.array_equal(h.ah_state_get(B.AH_X), x)
    h.close()


# ------------------------------------------------------------------- exchange
@pytest.mark.parametrize("K,P", [(1, 7), (3, 1000), (4, 4099), (7, 2048), (16, 10_001), (64, 3001)])
def test_exchange_bit_exact(B, torch, K, P):
    rng = np.random.default_rng(K * 1000 + P)
    theta0 = rng.standard_normal(P).astype(np.float32)
    x = theta0[None] + rng.standard_normal((K, P)).astype(np.float32) * np.float32(0.05)
    h = B.Handle(K, P, [])
    ref = OracleState(theta0, K, [])
    h.ah_state_set(B.AH_CENTER, theta0)
    h.ah_state_set(B.AH_X, x)
    ref.x[:] = x
    for trial in range(4):
        mask = (rng.random(K) > 0.3).astype(np.uint8) if trial else None
        if trial == 3:
            mask[:] = 0                                    # nobody reaches the master
        if trial % 2 == 0:
            h2 = rng.uniform(0, 0.05, K).astype(np.float32)
            h1 = rng.uniform(0.05, 1, K).astype(np.float32)
            h.easgd_exchange(mask, np.concatenate([h2, h1]), 0.0)
            ref.exchange(mask, h2, h1)
        else:
            h.easgd_exchange(mask, None, 0.8 / K)
            ref.exchange(mask, alpha=0.8 / K)
        assert np.array_equal(h.ah_state_get(B.AH_X), ref.x), trial
        assert np.array_equal(h.ah_state_get(B.AH_CENTER), ref.center), trial
    h.close()


def test_exchange_alpha_zero_is_identity(B, torch):
    K, P = 4, 5000
    rng = np.random.default_rng(1)
    theta0 = rng.standard_normal(P).astype(np.float32)
    x = rng.standard_normal((K, P)).astype(np.float32)
    h = B.Handle(K, P, [])
    h.ah_state_set(B.AH_CENTER, theta0)
    h.ah_state_set(B.AH_X, x)
    h.easgd_exchange(None, None, 0.0)
    assert np.array_equal(h.ah_state_get(B.AH_X), x)
    assert np.array_equal(h.ah_state_get(B.AH_CENTER), theta0)
    h.close()


# ------------------------------------------- several Hutchinson samples per step
@pytest.mark.parametrize("sample", [0, 1, 7])
def test_sample_z_n_bit_exact(B, torch, sample):
    K, P = 3, 184_837
    h = B.Handle(K, P, [])
    dst = torch.empty(K, W.padded_ld(P), device="cuda")
    h.ah_sample_z_n(0xFEEDFACE12345678, 9, sample, dst)
    want = oracle.load("omp").sample_z_s(0xFEEDFACE12345678, 9, sample, K, P)
    assert np.array_equal(dst[:, :P].cpu().numpy(), want)
    h.close()


@pytest.mark.parametrize("n", [2, 3, 4, 8])
@pytest.mark.parametrize("layout", ["odd", "resnet18"])
def test_local_step_n_samples_matches_oracle(B, torch, n, layout):
    if layout == "odd":
        segs, P = ODD_SEGS, ODD_P
    else:
        lay = W.resnet18_layout(16)
        segs, P = W.segments(lay), W.total_params(lay)
    K, ld = 3, W.padded_ld(P)
    rng = np.random.default_rng(n * 100 + P)
    theta0 = (rng.standard_normal(P) * 0.1).astype(np.float32)
    h = B.Handle(K, P, segs)
    ref = OracleState(theta0, K, segs)
    h.ah_state_set(B.AH_CENTER, theta0)
    h.ah_broadcast_center()
    for t in range(1, 6):
        g = np.zeros((K, ld), np.float32)
        hv = np.zeros((n, K, ld), np.float32)
        g[:, :P] = rng.standard_normal((K, P)).astype(np.float32) * np.float32(0.1)
        hv[:, :, :P] = rng.standard_normal((n, K, P)).astype(np.float32) * np.float32(0.1)
        active = None if t != 3 else np.array([1, 0, 1], np.uint8)
        dist = t % 2 == 0
        h.ah_local_step(torch.from_numpy(g).cuda(), torch.from_numpy(hv).cuda(), Z_SEED, lr=0.01,
                        round_=t, active=active, want_dist=dist)
        ref.local_step(g, hv, Z_SEED, t, lr=0.01, active=active, want_dist=dist)
        if dist:
            assert np.array_equal(h.ah_state_get(B.AH_NORM2), ref.norm2), t
    for which, want in ((B.AH_X, ref.x), (B.AH_M, ref.m), (B.AH_V, ref.v)):
        assert np.array_equal(h.ah_state_get(which), want), which
    h.close()


def test_n_samples_argument_checks(B, torch):
    K, P = 2, 1000
    h = B.Handle(K, P, [])
    g = torch.zeros(K, P, device="cuda")
    with pytest.raises(B.AdaHessError) as e:
        h.ah_local_step(g, torch.zeros(B.AH_MAX_SAMPLES + 1, K, P, device="cuda"), 1, lr=0.1)
    assert e.value.status == B.AH_ERR_INVALID_ARG
    hy = B.ah_hyper(0.1, 0.9, 0.999, 1e-4, 1.0, 0.0, 1, None, 0, 2, P)     # samples would overlap
    hv = torch.zeros(2, K, P, device="cuda")
    assert B.raw().ah_local_step(h._h, g.data_ptr(), hv.data_ptr(), P, 1, C.byref(hy)) == B.AH_ERR_INVALID_ARG
    h.close()


# --------------------------------------------------- asynchronous exchange
@pytest.mark.parametrize("K,P", [(1, 7), (3, 1000), (4, 4099), (7, 2048), (16, 10_001), (64, 3001),
                                 (256, 1030)])
def test_exchange_async_bit_exact(B, torch, K, P):
    rng = np.random.default_rng(K * 1000 + P + 1)
    theta0 = rng.standard_normal(P).astype(np.float32)
    x = theta0[None] + rng.standard_normal((K, P)).astype(np.float32) * np.float32(0.05)
    h = B.Handle(K, P, [])
    ref = OracleState(theta0, K, [])
    h.ah_state_set(B.AH_CENTER, theta0)
    h.ah_state_set(B.AH_X, x)
    ref.x[:] = x
    for trial in range(5):
        mask = (rng.random(K) > 0.3).astype(np.uint8) if trial else None
        if trial == 3:
            mask[:] = 0                                    # nobody arrives
        order = None if trial == 4 else h.dw_order_next(77, trial)
        if trial != 4:
            assert np.array_equal(order, ref.order_next(77, trial))
        if trial % 2 == 0:
            h2 = rng.uniform(0, 0.3, K).astype(np.float32)   # sum far above 1: fine when sequential
            h1 = rng.uniform(0.05, 1, K).astype(np.float32)
            h.easgd_exchange_async(mask, np.concatenate([h2, h1]), 0.0, order)
            ref.exchange_async(mask, h2, h1, order=order)
        else:
            h.easgd_exchange_async(mask, None, 0.25, order)
            ref.exchange_async(mask, alpha=0.25, order=order)
        assert np.array_equal(h.ah_state_get(B.AH_X), ref.x), trial
        assert np.array_equal(h.ah_state_get(B.AH_CENTER), ref.center), trial
    # an order that is not a permutation is refused and nothing moves
    if K > 1:
        bad = np.arange(K, dtype=np.uint16)
        bad[0] = bad[1]
        with pytest.raises(B.AdaHessError) as e:
            h.easgd_exchange_async(None, None, 0.1, bad)
        assert e.value.status == B.AH_ERR_INVALID_ARG
        bad[0] = K
        with pytest.raises(B.AdaHessError):
            h.easgd_exchange_async(None, None, 0.1, bad)
        assert np.array_equal(h.ah_state_get(B.AH_X), ref.x)
    h.close()


def test_async_rounds_resnet18_shape_reduced(B, torch):
    # the whole round with the asynchronous exchange: dynamic weights, Bernoulli(1/3)
    # communication failures (Sec. VI), seeded arrival order, alpha = 0.1 (Sec. VII) for
    # K = 8, where the simultaneous form would sit at its stability limit
    layout = W.resnet18_layout(8)
    cfg = RunConfig(K=8, segments=W.segments(layout), P=W.total_params(layout), rounds=120, tau=2,
                    p_fail=1 / 3, alpha=0.1, asynchronous=True)
    h, ref, log = run_gaussian(cfg, B, oracle, _layout_inputs(layout, 8), variant="omp")
    viol, bits = compare_state(h, ref, B)
    assert log["masks_equal"] and log["weights_equal"] and log["norm2_equal"] and log["orders_equal"]
    assert sum(viol.values()) == 0 and sum(bits.values()) == 0, (viol, bits)
    h.close()


@pytest.mark.parametrize("K,width", [(40, 16), (256, 16)])
def test_many_workers_with_the_rule_inside_the_distance_round(B, torch, K, width):
    # more workers than consumer threads in a CTA (the rule takes several workers per thread), the
    # large per-worker launch tables, distances assembled and rule run at the head of the riding
    # exchange: the shape the benchmark times for its largest worker counts
    layout = W.resnet18_layout(width)
    cfg = RunConfig(K=K, segments=W.segments(layout), P=W.total_params(layout), rounds=12, tau=2,
                    p_fail=0.2, max_stale=3, frozen=True, fused="next")
    h, ref, log = run_gaussian(cfg, B, oracle, _layout_inputs(layout, K, n_pool=2), variant="omp")
    viol, bits = compare_state(h, ref, B)
    assert log["masks_equal"] and log["weights_equal"] and log["norm2_equal"], log
    assert sum(viol.values()) == 0 and sum(bits.values()) == 0, (viol, bits)
    assert np.array_equal(h.ah_state_get(B.AH_UHIST), ref.uhist)
    assert log["exchanges"] == 6
    h.close()


@pytest.mark.parametrize("polls,K,width", [(0, 8, 8), (1, 8, 8), (0, 40, 16), (0, 4, 32)])
def test_assembly_when_the_ctas_do_not_wait_for_one_another(B, torch, polls, K, width):
    # wait budget 0 (or one poll): every CTA of a launch that assembles the distances gives up on
    # the others at once and forms the whole tree by itself; same tree, same bits
    layout = W.resnet18_layout(width)
    cfg = RunConfig(K=K, segments=W.segments(layout), P=W.total_params(layout), rounds=24, tau=2,
                    p_fail=0.25, fused="next", wait_polls=polls)
    h, ref, log = run_gaussian(cfg, B, oracle, _layout_inputs(layout, K, n_pool=2), variant="omp")
    viol, bits = compare_state(h, ref, B)
    assert log["masks_equal"] and log["weights_equal"] and log["norm2_equal"], log
    assert sum(viol.values()) == 0 and sum(bits.values()) == 0, (viol, bits)
    assert np.array_equal(h.ah_state_get(B.AH_UHIST), ref.uhist)
    assert log["exchanges"] == 12
    h.close()


def test_riding_exchange_assembles_the_distances_without_a_launch_of_its_own(B, torch):
    # distance round, then the exchange riding on the next step: two launches, and the riding
    # one leaves the distances where a reader finds them; a twin that reads them at once (a
    # kernel of their own assembles them) sees the same bits and ends in the same state
    K, P = 4, 300_001
    rng = np.random.default_rng(7)
    theta0 = rng.standard_normal(P).astype(np.float32)
    ld = W.padded_ld(P)
    g = torch.from_numpy(rng.standard_normal((K, ld)).astype(np.float32)).cuda()
    hv = torch.from_numpy(rng.standard_normal((K, ld)).astype(np.float32)).cuda()
    mask = np.ones(K, np.uint8)
    seen = []
    for read_at_once in (False, True):
        h = B.Handle(K, P, [])
        h.ah_state_set(B.AH_CENTER, theta0)
        h.ah_broadcast_center()
        n0 = h.ah_launch_count()
        h.ah_local_step(g, hv, 1, round_=1, lr=0.01, want_dist=B.AH_DIST_AND_RULE, rule_alpha=0.05)
        first = h.ah_state_get(B.AH_NORM2).copy() if read_at_once else None
        h.easgd_exchange_then_step(g, hv, 1, round_=2, lr=0.01, worker_mask=mask, alpha=0.05, dynamic=True)
        assert h.ah_launch_count() - n0 == (3 if read_at_once else 2)
        n2 = h.ah_state_get(B.AH_NORM2).copy()
        assert h.ah_launch_count() - n0 == (3 if read_at_once else 2)
        if read_at_once:
            assert np.array_equal(first, n2)
        seen.append((n2, h.ah_state_get(B.AH_WEIGHTS).copy(), h.ah_state_get(B.AH_X).copy(),
                     h.ah_state_get(B.AH_CENTER).copy(), h.ah_state_get(B.AH_UHIST).copy()))
        h.close()
    for a, b in zip(*seen):
        assert np.array_equal(a, b)
    assert np.all(seen[0][0] > 0)


def test_a_rule_that_is_owed_runs_before_whatever_would_lose_it(B, torch):
    # Tile sums wait until somebody needs the distances.  If the weighting rule is owed on them
    # (AH_DIST_AND_RULE) and the next call would overwrite them (another distance round) or change
    # the rule's setting (dw_config), the rule runs first: the history advances once per such
    # round, exactly as when the host runs the rule after every distance round.
    K, P = 3, 70_001
    rng = np.random.default_rng(11)
    theta0 = rng.standard_normal(P).astype(np.float32)
    ld = W.padded_ld(P)
    pairs = [(torch.from_numpy(rng.standard_normal((K, ld)).astype(np.float32)).cuda(),
              torch.from_numpy(rng.standard_normal((K, ld)).astype(np.float32)).cuda()) for _ in range(3)]
    mask = np.ones(K, np.uint8)
    alpha = 0.07
    c_new, kappa_new = np.array([0.5, 0.3, 0.2]), -0.2

    def fresh():
        h = B.Handle(K, P, [])
        h.ah_state_set(B.AH_CENTER, theta0)
        h.ah_broadcast_center()
        return h

    lazy, eager = fresh(), fresh()
    # lazy: nobody looks at the distances between the rounds
    for t in (1, 2, 3):
        g, hv = pairs[t - 1]
        lazy.ah_local_step(g, hv, 5, round_=t, lr=0.01, want_dist=B.AH_DIST_AND_RULE, rule_alpha=alpha)
    lazy.dw_config(3, c_new, kappa_new)            # the rule owed on round 3 runs with the old setting
    # eager: the host runs the rule after every distance round
    for t in (1, 2, 3):
        g, hv = pairs[t - 1]
        eager.ah_local_step(g, hv, 5, round_=t, lr=0.01, want_dist=True)
        w_eager = eager.dw_weights_next(alpha)
    eager.dw_config(3, c_new, kappa_new)
    assert np.array_equal(lazy.ah_state_get(B.AH_NORM2), eager.ah_state_get(B.AH_NORM2))
    assert np.array_equal(lazy.ah_state_get(B.AH_UHIST, p_hist=3), eager.ah_state_get(B.AH_UHIST, p_hist=3))
    assert np.array_equal(lazy.ah_state_get(B.AH_WEIGHTS), w_eager)
    # one more period under the new setting, the exchange riding on the lazy side
    g, hv = pairs[0]
    lazy.ah_local_step(g, hv, 5, round_=4, lr=0.01, want_dist=B.AH_DIST_AND_RULE, rule_alpha=alpha)
    lazy.easgd_exchange_then_step(g, hv, 5, round_=5, lr=0.01, worker_mask=mask, alpha=alpha, dynamic=True)
    eager.ah_local_step(g, hv, 5, round_=4, lr=0.01, want_dist=True)
    w = eager.dw_weights_next(alpha)
    eager.easgd_exchange(mask, w, alpha)
    eager.ah_local_step(g, hv, 5, round_=5, lr=0.01)
    for which in (B.AH_X, B.AH_M, B.AH_V, B.AH_CENTER):
        assert np.array_equal(lazy.ah_state_get(which), eager.ah_state_get(which)), which
    assert np.array_equal(lazy.ah_state_get(B.AH_UHIST, p_hist=3), eager.ah_state_get(B.AH_UHIST, p_hist=3))
    assert np.array_equal(lazy.ah_state_get(B.AH_WEIGHTS), w)
    lazy.close(); eager.close()


# --------------------------------------- weights on the device, no host round trip
@pytest.mark.parametrize("asyn,mode", [(False, "yes"), (True, "yes"), (False, "mixed"), (True, "mixed")])
def test_dynamic_exchange_on_device_matches_oracle(B, torch, asyn, mode):
    layout = W.resnet18_layout(8)
    cfg = RunConfig(K=8, segments=W.segments(layout), P=W.total_params(layout), rounds=120, tau=2,
                    p_fail=0.3, alpha=0.1 if asyn else None, asynchronous=asyn, sync_free=mode)
    h, ref, log = run_gaussian(cfg, B, oracle, _layout_inputs(layout, 8), variant="omp")
    viol, bits = compare_state(h, ref, B)
    assert log["masks_equal"] and log["weights_equal"] and log["norm2_equal"] and log["orders_equal"], log
    assert sum(viol.values()) == 0 and sum(bits.values()) == 0, (viol, bits)
    assert np.array_equal(h.ah_state_get(B.AH_UHIST), ref.uhist)
    assert log["exchanges"] == 60
    h.close()


def test_dynamic_exchange_custom_rule_and_errors(B, torch):
    # a deeper history with other coefficients and threshold; K = 256 fills the weight kernel
    K, P, p_hist = 256, 1500, 7
    rng = np.random.default_rng(60)
    c = rng.dirichlet(np.ones(p_hist))
    theta0 = rng.standard_normal(P).astype(np.float32)
    h = B.Handle(K, P, [])
    h.dw_config(p_hist, c, -0.25)
    ref = OracleState(theta0, K, [], p_hist=p_hist, c=c, kappa=-0.25)
    h.ah_state_set(B.AH_CENTER, theta0)
    h.ah_broadcast_center()
    with pytest.raises(B.AdaHessError) as e:
        h.easgd_exchange_dynamic(None, 0.003)              # no distances yet
    assert e.value.status == B.AH_ERR_STATE
    zeros = torch.zeros(K, W.padded_ld(P), device="cuda")
    for t in range(1, 13):
        x = (theta0[None] + rng.standard_normal((K, P)).astype(np.float32) *
             rng.uniform(0.01, 1.0, (K, 1)).astype(np.float32))
        h.ah_state_set(B.AH_X, x)
        ref.x[:] = x
        h.ah_local_step(zeros, zeros, 1, lr=0.0, active=np.zeros(K, np.uint8), want_dist=True)
        ref.norm2 = oracle.load("omp").norm2(ref.x, ref.center)
        h.easgd_exchange_dynamic(None, 0.003)
        h2, h1 = ref.weights_next(0.003)
        ref.exchange(None, h2, h1)
        w = h.ah_state_get(B.AH_WEIGHTS)
        assert np.array_equal(w[:K], h2) and np.array_equal(w[K:], h1), t
    assert np.array_equal(h.ah_state_get(B.AH_UHIST, p_hist=p_hist), ref.uhist)
    assert np.array_equal(h.ah_state_get(B.AH_X), ref.x)
    assert np.array_equal(h.ah_state_get(B.AH_CENTER), ref.center)
    h.close()


# ------------------------------------------- exchange rounds in one pass (fused)
@pytest.mark.parametrize("layout", ["odd", "resnet18", "one", "ragged"])
@pytest.mark.parametrize("asyn", [False, True])
def test_fused_round_equals_step_then_exchange(B, torch, layout, asyn):
    K = 5
    if layout == "odd":
        segs, P = ODD_SEGS, ODD_P
    elif layout == "one":
        segs, P, K = [], 1, 1                                  # the smallest problem there is
    elif layout == "ragged":
        segs, P, K = [(0, 1026, 3)], 2051, 2                   # a block across the tile edge, odd tail
    else:
        lay = W.resnet18_layout(16)
        segs, P = W.segments(lay), W.total_params(lay)
    ld = W.padded_ld(P)
    rng = np.random.default_rng(70 + P)
    theta0 = (rng.standard_normal(P) * 0.1).astype(np.float32)
    h = B.Handle(K, P, segs)
    ref = OracleState(theta0, K, segs)
    h.ah_state_set(B.AH_CENTER, theta0)
    h.ah_broadcast_center()
    for t in range(1, 9):
        g = np.zeros((K, ld), np.float32)
        hv = np.zeros((K, ld), np.float32)
        g[:, :P] = rng.standard_normal((K, P)).astype(np.float32) * np.float32(0.1)
        hv[:, :P] = rng.standard_normal((K, P)).astype(np.float32) * np.float32(0.1)
        active = None if t % 3 else (rng.random(K) > 0.4).astype(np.uint8)
        mask = None if t % 4 == 1 else (rng.random(K) > 0.3).astype(np.uint8)
        if t == 6:
            mask = np.zeros(K, np.uint8)                      # nobody meets the master
        dist = t % 2 == 0
        order = h.dw_order_next(5, t) if asyn else None
        if t % 2:
            h2 = rng.uniform(0, 0.15, K).astype(np.float32)
            h1 = rng.uniform(0.05, 1, K).astype(np.float32)
            weights = np.concatenate([h2, h1])
        else:
            h2 = h1 = weights = None
        if t in (4, 7):                                          # two Hutchinson samples
            hv = np.stack([hv, np.roll(hv, 1, axis=0)])
        h.ah_local_step_exchange(torch.from_numpy(g).cuda(), torch.from_numpy(hv).cuda(), Z_SEED, lr=0.01,
                                 round_=t, active=active, want_dist=dist, worker_mask=mask,
                                 weights=weights, alpha=0.1, order=order, asynchronous=asyn)
        ref.local_step(g, hv, Z_SEED, t, lr=0.01, active=active, want_dist=dist)
        if asyn:
            ref.exchange_async(mask, h2, h1, alpha=0.1, order=order)
        else:
            ref.exchange(mask, h2, h1, alpha=0.1)
        if dist:
            assert np.array_equal(h.ah_state_get(B.AH_NORM2), ref.norm2), t
        for which, want in ((B.AH_X, ref.x), (B.AH_M, ref.m), (B.AH_V, ref.v), (B.AH_CENTER, ref.center)):
            assert np.array_equal(h.ah_state_get(which), want), (t, which)
    assert np.array_equal(h.ah_state_get(B.AH_STEP), ref.step)
    h.close()


@pytest.mark.parametrize("asyn,frozen", [(False, False), (True, False), (False, True)])
def test_fused_rounds_with_lagged_dynamic_weights(B, torch, asyn, frozen):
    # every exchange round in one pass, the rule's coefficients one period behind the
    # distances; the oracle takes the same schedule with its separate functions
    layout = W.resnet18_layout(8)
    cfg = RunConfig(K=8, segments=W.segments(layout), P=W.total_params(layout), rounds=100, tau=2,
                    p_fail=0.25, max_stale=4 if frozen else 1, frozen=frozen,
                    alpha=0.1 if asyn else None, asynchronous=asyn, fused="lagged")
    h, ref, log = run_gaussian(cfg, B, oracle, _layout_inputs(layout, 8), variant="omp")
    viol, bits = compare_state(h, ref, B)
    assert log["masks_equal"] and log["weights_equal"] and log["norm2_equal"] and log["orders_equal"], log
    assert sum(viol.values()) == 0 and sum(bits.values()) == 0, (viol, bits)
    assert np.array_equal(h.ah_state_get(B.AH_UHIST), ref.uhist)
    assert np.array_equal(h.ah_state_get(B.AH_STEP), ref.step)
    assert log["exchanges"] == 50
    h.close()


@pytest.mark.parametrize("asyn,frozen,dynamic", [(False, False, True), (True, False, True),
                                                 (False, True, True), (True, False, False)])
def test_exchange_riding_on_the_next_local_step(B, torch, asyn, frozen, dynamic):
    # every exchange is deferred to the next round's local step (one pass instead of two);
    # same coefficients, same bits as exchanging at once
    layout = W.resnet18_layout(8)
    cfg = RunConfig(K=8, segments=W.segments(layout), P=W.total_params(layout), rounds=100, tau=2,
                    p_fail=0.25, max_stale=4 if frozen else 1, frozen=frozen, dynamic=dynamic,
                    alpha=0.1 if asyn else None, asynchronous=asyn, fused="next")
    h, ref, log = run_gaussian(cfg, B, oracle, _layout_inputs(layout, 8), variant="omp")
    viol, bits = compare_state(h, ref, B)
    assert log["masks_equal"] and log["weights_equal"] and log["norm2_equal"] and log["orders_equal"], log
    assert sum(viol.values()) == 0 and sum(bits.values()) == 0, (viol, bits)
    assert np.array_equal(h.ah_state_get(B.AH_UHIST), ref.uhist)
    assert np.array_equal(h.ah_state_get(B.AH_STEP), ref.step)
    assert log["exchanges"] == 50
    h.close()


@pytest.mark.parametrize("layout", ["odd", "one", "ragged"])
def test_exchange_then_step_equals_the_two_calls(B, torch, layout):
    K = 4
    if layout == "odd":
        segs, P = ODD_SEGS, ODD_P
    elif layout == "one":
        segs, P, K = [], 1, 1
    else:
        segs, P, K = [(0, 1026, 3)], 2051, 2
    ld = W.padded_ld(P)
    rng = np.random.default_rng(80 + P)
    theta0 = (rng.standard_normal(P) * 0.1).astype(np.float32)
    x0 = theta0[None] + rng.standard_normal((K, P)).astype(np.float32) * np.float32(0.05)
    h = B.Handle(K, P, segs)
    ref = OracleState(theta0, K, segs)
    h.ah_state_set(B.AH_CENTER, theta0)
    h.ah_state_set(B.AH_X, x0)
    ref.x[:] = x0
    for t in range(1, 7):
        g = np.zeros((K, ld), np.float32)
        hv = np.zeros((K, ld), np.float32)
        g[:, :P] = rng.standard_normal((K, P)).astype(np.float32) * np.float32(0.1)
        hv[:, :P] = rng.standard_normal((K, P)).astype(np.float32) * np.float32(0.1)
        active = None if t % 3 else (rng.random(K) > 0.4).astype(np.uint8)
        mask = None if t % 4 == 1 else (rng.random(K) > 0.3).astype(np.uint8)
        asyn = t % 2 == 0
        order = h.dw_order_next(6, t) if asyn else None
        h2 = rng.uniform(0, 0.15, K).astype(np.float32)
        h1 = rng.uniform(0.05, 1, K).astype(np.float32)
        if t == 4:                                               # three Hutchinson samples
            hv = np.stack([hv, hv[::-1].copy(), -hv])
        h.easgd_exchange_then_step(torch.from_numpy(g).cuda(), torch.from_numpy(hv).cuda(), Z_SEED, lr=0.01,
                                   round_=t, active=active, worker_mask=mask,
                                   weights=np.concatenate([h2, h1]), order=order, asynchronous=asyn)
        if asyn:
            ref.exchange_async(mask, h2, h1, order=order)
        else:
            ref.exchange(mask, h2, h1)
        ref.local_step(g, hv, Z_SEED, t, lr=0.01, active=active)
        for which, want in ((B.AH_X, ref.x), (B.AH_M, ref.m), (B.AH_V, ref.v), (B.AH_CENTER, ref.center)):
            assert np.array_equal(h.ah_state_get(which), want), (t, which)
    g = torch.zeros(K, ld, device="cuda")
    with pytest.raises(B.AdaHessError) as e:                   # no distances pending for the rule
        h.easgd_exchange_then_step(g, g, 1, lr=0.1, alpha=0.1, dynamic=True)
    assert e.value.status == B.AH_ERR_STATE
    h.close()


def test_fused_round_argument_checks(B, torch):
    K, P = 2, 1000
    h = B.Handle(K, P, [])
    g = torch.zeros(K, P, device="cuda")
    with pytest.raises(B.AdaHessError) as e:          # lagged weights need this round's distances
        h.ah_local_step_exchange(g, g, 1, lr=0.1, lagged=True, want_dist=False)
    assert e.value.status == B.AH_ERR_INVALID_ARG
    with pytest.raises(B.AdaHessError) as e:
        h.ah_local_step_exchange(g, g, 1, lr=0.1, asynchronous=True, order=np.array([1, 1]))
    assert e.value.status == B.AH_ERR_INVALID_ARG
    h.close()


# ------------------------------------------- every form of the round, mixed at random
@pytest.mark.parametrize("seed", range(6))
def test_random_mix_of_round_forms(B, torch, seed):
    """Each exchange round picks one of the seven ways the library offers to take it (host
    or device rule, exchange kernel at once or riding on the next step, one pass with given
    or lagged coefficients, simultaneous or asynchronous), plain rounds take one or two
    Hutchinson samples; the oracle follows with its separate functions.  Checks that the
    forms compose: history ring on host and device, pending distances, lagged weights."""
    from parity_driver import MASK_SEED, ORDER_SEED
    rng = np.random.default_rng(1000 + seed)
    layout = W.resnet18_layout(16)
    segs, P, K, tau, R, alpha = W.segments(layout), W.total_params(layout), 5, 3, 36, 0.08
    ld = W.padded_ld(P)
    theta0 = W.theta0_np(layout, seed)
    h = B.Handle(K, P, segs)
    ref = OracleState(theta0, K, segs)
    h.ah_state_set(B.AH_CENTER, theta0)
    h.ah_broadcast_center()
    dev_w = None            # last output of the rule on the device (what a lagged round pulls with)
    pending = None          # an exchange deferred to the next round's step
    for t in range(1, R + 1):
        ex = t % tau == 0
        mask = h.dw_mask_next(MASK_SEED, t, 0.25)
        assert np.array_equal(mask, ref.mask_next(MASK_SEED, t, 0.25))
        n = 2 if rng.random() < 0.3 else 1
        g = np.zeros((K, ld), np.float32)
        hv = np.zeros((n, K, ld), np.float32)
        g[:, :P] = rng.standard_normal((K, P)).astype(np.float32) * np.float32(0.05)
        hv[:, :, :P] = rng.standard_normal((n, K, P)).astype(np.float32) * np.float32(0.05)
        hv_o = hv if n > 1 else hv[0]
        gd, hd = torch.from_numpy(g).cuda(), torch.from_numpy(hv_o).cuda()
        asyn = bool(rng.random() < 0.5)
        order = h.dw_order_next(ORDER_SEED, t) if asyn else None
        if asyn:
            assert np.array_equal(order, ref.order_next(ORDER_SEED, t))
        form = rng.choice(["host", "device", "defer", "given", "lagged"]) if ex else None

        def oracle_exchange(m, o, a, h2=None, h1=None):
            if a:
                ref.exchange_async(m, h2, h1, alpha=alpha, order=o)
            else:
                ref.exchange(m, h2, h1, alpha=alpha)

        if pending is not None:                 # last round's exchange rides on this step
            p_mask, p_order, p_asyn = pending
            h.easgd_exchange_then_step(gd, hd, Z_SEED, lr=0.01, round_=t, worker_mask=p_mask, alpha=alpha,
                                       order=p_order, asynchronous=p_asyn, dynamic=True)
            dev_w = ref.weights_next(alpha)
            w = h.ah_state_get(B.AH_WEIGHTS)
            assert np.array_equal(w[:K], dev_w[0]) and np.array_equal(w[K:], dev_w[1]), t
            oracle_exchange(p_mask, p_order, p_asyn, *dev_w)
            ref.local_step(g, hv_o, Z_SEED, t, lr=0.01)
            pending = None
        elif form in ("given", "lagged"):       # this round's step and exchange in one pass
            h.ah_local_step_exchange(gd, hd, Z_SEED, lr=0.01, round_=t, want_dist=True, worker_mask=mask,
                                     alpha=alpha, order=order, asynchronous=asyn, lagged=form == "lagged")
            ref.local_step(g, hv_o, Z_SEED, t, lr=0.01, want_dist=True)
            if form == "lagged":
                oracle_exchange(mask, order, asyn, *(dev_w if dev_w is not None else (None, None)))
                dev_w = ref.weights_next(alpha)
            else:
                oracle_exchange(mask, order, asyn)
            continue
        else:
            h.ah_local_step(gd, hd, Z_SEED, lr=0.01, round_=t, want_dist=ex)
            ref.local_step(g, hv_o, Z_SEED, t, lr=0.01, want_dist=ex)
        if form == "host":
            w = h.dw_weights_next(alpha)
            h2, h1 = ref.weights_next(alpha)
            assert np.array_equal(w[:K], h2) and np.array_equal(w[K:], h1), t
            if asyn:
                h.easgd_exchange_async(mask, w, alpha, order)
            else:
                h.easgd_exchange(mask, w, alpha)
            oracle_exchange(mask, order, asyn, h2, h1)
        elif form == "device":
            h.easgd_exchange_dynamic(mask, alpha, order, asyn)
            dev_w = ref.weights_next(alpha)
            oracle_exchange(mask, order, asyn, *dev_w)
        elif form == "defer":
            pending = (mask, order, asyn)
    if pending is not None:
        p_mask, p_order, p_asyn = pending
        h.easgd_exchange_dynamic(p_mask, alpha, p_order, p_asyn)
        oracle_exchange(p_mask, p_order, p_asyn, *ref.weights_next(alpha))
    for which, want in ((B.AH_X, ref.x), (B.AH_M, ref.m), (B.AH_V, ref.v), (B.AH_CENTER, ref.center)):
        assert np.array_equal(h.ah_state_get(which), want), which
    assert np.array_equal(h.ah_state_get(B.AH_UHIST), ref.uhist)
    h.close()


# ------------------------------------------- first-order local steps (EASGD / EAMSGD)
@pytest.mark.parametrize("K,P", [(1, 1), (2, 1023), (3, 4097), (4, 184_837), (8, 4 * 1024 * 5), (5, 8193)])
@pytest.mark.parametrize("delta", [0.0, 0.5])
def test_sgd_step_bit_exact(B, torch, K, P, delta):
    rng = np.random.default_rng(K * 7 + P)
    ld = W.padded_ld(P) + 8
    theta0 = rng.standard_normal(P).astype(np.float32)
    h = B.Handle(K, P, [])
    ref = OracleState(theta0, K, [])
    h.ah_state_set(B.AH_CENTER, theta0)
    h.ah_broadcast_center()
    for t in range(1, 7):
        g = np.full((K, ld), np.nan, np.float32)             # columns past P must never be used
        g[:, :P] = rng.standard_normal((K, P)).astype(np.float32)
        active = None if t % 3 else (rng.random(K) > 0.4).astype(np.uint8)
        dist = t % 2 == 0
        h.sgd_local_step(torch.from_numpy(g).cuda(), 0.01, delta, active=active, want_dist=dist)
        ref.sgd_step(g, 0.01, delta, active=active, want_dist=dist)
        if dist:
            assert np.array_equal(h.ah_state_get(B.AH_NORM2), ref.norm2), t
    assert np.array_equal(h.ah_state_get(B.AH_X), ref.x)
    assert np.array_equal(h.ah_state_get(B.AH_M), ref.m)
    assert not h.ah_state_get(B.AH_V).any()
    assert np.array_equal(h.ah_state_get(B.AH_STEP), ref.step)
    h.close()


@pytest.mark.parametrize("method,asyn", [("sgd", True), ("msgd", True), ("msgd", False)])
def test_easgd_eamsgd_rounds_reduced(B, torch, method, asyn):
    # the comparison methods of Sec. VI on the ResNet-18-shaped layout at 1/8 width: eta = 0.01,
    # delta = 0.5, fixed alpha, communication suppressed one third of the time, tau = 2
    layout = W.resnet18_layout(8)
    cfg = RunConfig(K=4, segments=W.segments(layout), P=W.total_params(layout), rounds=90, tau=2,
                    p_fail=1 / 3, alpha=0.1, dynamic=False, asynchronous=asyn, method=method)
    h, ref, log = run_gaussian(cfg, B, oracle, _layout_inputs(layout, 4), variant="omp")
    viol, bits = compare_state(h, ref, B)
    assert log["masks_equal"] and log["orders_equal"]
    assert sum(viol.values()) == 0 and sum(bits.values()) == 0, (viol, bits)
    h.close()


@pytest.mark.parametrize("K,P", [(1, 1), (2, 2051), (5, 13_111), (8, 184_837), (64, 3001)])
@pytest.mark.parametrize("delta", [0.0, 0.5])
def test_exchange_then_sgd_step_equals_the_two_calls(B, torch, K, P, delta):
    # EASGD / EAMSGD periods in one pass per exchange: pull, then the first-order step
    rng = np.random.default_rng(K * 11 + P)
    ld = W.padded_ld(P) + 4
    theta0 = rng.standard_normal(P).astype(np.float32)
    x0 = theta0[None] + rng.standard_normal((K, P)).astype(np.float32) * np.float32(0.05)
    h = B.Handle(K, P, [])
    ref = OracleState(theta0, K, [])
    h.ah_state_set(B.AH_CENTER, theta0)
    h.ah_state_set(B.AH_X, x0)
    ref.x[:] = x0
    for t in range(1, 8):
        g = np.full((K, ld), np.nan, np.float32)             # columns past P must never be used
        g[:, :P] = rng.standard_normal((K, P)).astype(np.float32)
        active = None if t % 3 else (rng.random(K) > 0.4).astype(np.uint8)
        mask = None if t % 4 == 1 else (rng.random(K) > 0.3).astype(np.uint8)
        if t == 6:
            mask = np.zeros(K, np.uint8)
        asyn = t % 2 == 0
        order = h.dw_order_next(8, t) if asyn else None
        if t % 3 == 1:
            h2 = rng.uniform(0, 0.1, K).astype(np.float32)
            h1 = rng.uniform(0.05, 1, K).astype(np.float32)
            weights = np.concatenate([h2, h1])
        else:
            h2 = h1 = weights = None
        h.easgd_exchange_then_sgd_step(torch.from_numpy(g).cuda(), 0.01, delta, active=active,
                                       worker_mask=mask, weights=weights, alpha=0.1, order=order,
                                       asynchronous=asyn)
        if asyn:
            ref.exchange_async(mask, h2, h1, alpha=0.1, order=order)
        else:
            ref.exchange(mask, h2, h1, alpha=0.1)
        ref.sgd_step(g, 0.01, delta, active=active)
        for which, want in ((B.AH_X, ref.x), (B.AH_M, ref.m), (B.AH_CENTER, ref.center)):
            assert np.array_equal(h.ah_state_get(which), want), (t, which)
    assert np.array_equal(h.ah_state_get(B.AH_STEP), ref.step)
    assert not h.ah_state_get(B.AH_V).any()
    h.close()


def test_sgd_argument_checks(B, torch):
    h = B.Handle(2, 100, [])
    g = torch.zeros(2, 100, device="cuda")
    with pytest.raises(B.AdaHessError) as e:
        h.sgd_local_step(g, 0.1, 1.0)                        # momentum must stay below 1
    assert e.value.status == B.AH_ERR_INVALID_ARG
    with pytest.raises(B.AdaHessError) as e:
        h.sgd_local_step(torch.zeros(2, 101, device="cuda")[:, 1:], 0.1)   # misaligned rows
    assert e.value.status in (B.AH_ERR_ALIGN, B.AH_ERR_INVALID_ARG)
    h.close()


# ---------------------------------------------------- whole configurations
def _check_run(B, cfg, inputs, bit_exact=True):
    h, ref, log = run_gaussian(cfg, B, oracle, inputs, variant="omp")
    viol, bits = compare_state(h, ref, B)
    assert log["masks_equal"] and log["weights_equal"] and log["norm2_equal"], log
    assert sum(viol.values()) == 0, viol
    if bit_exact:
        assert sum(bits.values()) == 0, bits
    assert np.array_equal(h.ah_state_get(B.AH_STEP), ref.step)
    assert np.array_equal(h.ah_state_get(B.AH_UHIST), ref.uhist)
    assert log["exchanges"] == cfg.rounds // cfg.tau
    h.close()


def _layout_inputs(layout, K, n_pool=3, seed=0):
    return W.theta0_np(layout, seed), W.gaussian_pool_np(layout, K, n_pool, seed + 1)


@pytest.mark.parametrize("K,tau", [(4, 1), (4, 4), (8, 2)])
def test_paper_setting_small_cnn(B, torch, K, tau):
    # the paper's own experiment shape (Sec. VI-VII): its two-convolution digit classifier
    # (1,199,882 parameters), 4 or 8 workers, tau in {1, 2, 4}, communication suppressed one
    # third of the time, alpha = 0.1, dynamic weights; 60 rounds at full size
    layout = W.mnist_cnn_layout()
    assert W.total_params(layout) == 1_199_882
    cfg = RunConfig(K=K, segments=W.segments(layout), P=W.total_params(layout), rounds=60, tau=tau,
                    p_fail=1 / 3, alpha=0.1)
    _check_run(B, cfg, _layout_inputs(layout, K))


def test_config_resnet18_shape_reduced(B, torch):
    # ResNet-18-shaped layout at 1/8 width (62 tensors, ragged tail), K=8, tau=4,
    # Bernoulli(0.1) communication failures, 200 rounds
    layout = W.resnet18_layout(8)
    cfg = RunConfig(K=8, segments=W.segments(layout), P=W.total_params(layout), rounds=200, tau=4,
                    p_fail=0.1)
    _check_run(B, cfg, _layout_inputs(layout, 8))


@pytest.mark.parametrize("tau", [1, 4, 16])
def test_config_resnet50_shape_reduced_stragglers(B, torch, tau):
    # ResNet-50-shaped layout at 1/8 width (161 tensors), K=16, failure 0.2 with
    # stragglers frozen for 1..8 rounds, 100 rounds per tau
    layout = W.resnet50_layout(8)
    cfg = RunConfig(K=16, segments=W.segments(layout), P=W.total_params(layout), rounds=100,
                    tau=tau, p_fail=0.2, max_stale=8, frozen=True)
    _check_run(B, cfg, _layout_inputs(layout, 16))


def test_config_vgg16_shape_reduced(B, torch):
    # VGG-16-shaped layout at 1/8 width (long dense tensors), K=4, tau=8, failure 0.25
    layout = W.vgg16_layout(8)
    cfg = RunConfig(K=4, segments=W.segments(layout), P=W.total_params(layout), rounds=50, tau=8,
                    p_fail=0.25)
    _check_run(B, cfg, _layout_inputs(layout, 4))


@pytest.mark.parametrize("K,p_fail", [(4, 0.0), (16, 0.1), (32, 0.3), (64, 0.1)])
def test_config_worker_sweep_reduced(B, torch, K, p_fail):
    layout = W.resnet50_layout(16)
    cfg = RunConfig(K=K, segments=W.segments(layout), P=W.total_params(layout), rounds=50, tau=4,
                    p_fail=p_fail)
    _check_run(B, cfg, _layout_inputs(layout, K, n_pool=2))


def test_config_diagonal_quadratic_full_size(B, torch):
    """f = 1/2 sum h theta^2, P = 2^20 in one tensor, K = 4, 100 rounds, tau = 4, worker 3
    cut off from the master in rounds 20..40; exact Hessian-vector products h * z with
    the z each side samples itself; gradients formed from each side's own x."""
    K, P, R, tau, alpha, lr = 4, 1 << 20, 100, 4, 0.05, 0.1
    hq, theta0 = W.quadratic_problem_np(P, 0)
    outages = [W.scripted_down(3, 20, 40)]
    segs = W.segments(W.single_segment_layout(P))
    h = B.Handle(K, P, segs)
    h.ah_state_set(B.AH_CENTER, theta0)
    h.ah_broadcast_center()
    ref = OracleState(theta0, K, segs, variant="omp")
    orc = oracle.load("omp")
    hq_dev = torch.from_numpy(hq).cuda()
    z_dev = torch.empty((K, P), device="cuda")
    masks_equal = weights_equal = True
    for t in range(1, R + 1):
        noise = W.quadratic_noise_np(K, P, 0, t)
        mask_g = W.apply_scripted(h.dw_mask_next(2, t, 0.0), t, outages)
        mask_o = ref.scripted_mask(ref.mask_next(2, t, 0.0), t, [(3, 20, 40)])
        masks_equal &= bool(np.array_equal(mask_g, mask_o))
        ex = t % tau == 0
        # device side: its own x, its own z
        g_dev = torch.from_numpy(W.quadratic_grad_np(hq, h.ah_state_get(B.AH_X), noise)).cuda()
        h.ah_sample_z(Z_SEED, t, z_dev)
        hv_dev = hq_dev[None, :] * z_dev
        h.ah_local_step(g_dev, hv_dev, Z_SEED, lr=lr, round_=t, want_dist=ex)
        # oracle side
        g = W.quadratic_grad_np(hq, ref.x, noise)
        hv = W.quadratic_hvp_np(hq, orc.sample_z(Z_SEED, t, K, P))
        ref.local_step(g, hv, Z_SEED, t, lr=lr, want_dist=ex)
        if ex:
            w = h.dw_weights_next(alpha)
            h2, h1 = ref.weights_next(alpha)
            weights_equal &= bool(np.array_equal(w[:K], h2) and np.array_equal(w[K:], h1))
            h.easgd_exchange(mask_g, w, alpha)
            ref.exchange(mask_o, h2, h1)
    assert masks_equal and weights_equal
    viol, bits = compare_state(h, ref, B)
    assert sum(viol.values()) == 0, viol
    assert sum(bits.values()) == 0, bits
    # Hutchinson is exact on a diagonal Hessian: v is an EMA of h^2 alone, noise-free
    v = h.ah_state_get(B.AH_V)
    bc2 = 1.0 - float(np.float32(0.999)) ** R
    assert np.allclose(v[0] / bc2, hq.astype(np.float64) ** 2, rtol=1e-4)
    h.close()


# ------------------------------------------------ checkpoint / resume, errors
def test_checkpoint_resume_is_bit_identical(B, torch):
    layout = W.resnet18_layout(16)
    segs, P, K = W.segments(layout), W.total_params(layout), 4
    inputs = _layout_inputs(layout, K)
    full = RunConfig(K=K, segments=segs, P=P, rounds=24, tau=4, p_fail=0.2, max_stale=4, frozen=True)
    half = RunConfig(K=K, segments=segs, P=P, rounds=12, tau=4, p_fail=0.2, max_stale=4, frozen=True)
    h_full, _, _ = run_gaussian(full, B, oracle, inputs, variant="omp")
    h_a, ref_a, _ = run_gaussian(half, B, oracle, inputs, variant="omp")
    # snapshot, restore into a fresh handle, continue rounds 13..24 by hand
    snap = {w: h_a.ah_state_get(w) for w in (B.AH_X, B.AH_M, B.AH_V, B.AH_CENTER, B.AH_STEP,
                                             B.AH_UHIST, B.AH_DOWN_UNTIL, B.AH_ROUND)}
    h_a.close()
    h_b = B.Handle(K, P, segs)
    for w, val in snap.items():
        h_b.ah_state_set(w, val)
    dev_pool = [(torch.from_numpy(g).cuda(), torch.from_numpy(hv).cuda()) for g, hv in inputs[1]]
    from parity_driver import MASK_SEED
    alpha = full.alpha_value()
    for t in range(13, 25):
        mask = h_b.dw_mask_next(MASK_SEED, t, 0.2, 4)
        ex = t % 4 == 0
        g, hv = dev_pool[t % len(dev_pool)]
        h_b.ah_local_step(g, hv, Z_SEED, lr=0.01, round_=t, active=mask, want_dist=ex)
        if ex:
            h_b.easgd_exchange(mask, h_b.dw_weights_next(alpha), alpha)
    for w in (B.AH_X, B.AH_M, B.AH_V, B.AH_CENTER):
        a, b = h_full.ah_state_get(w), h_b.ah_state_get(w)
        assert np.array_equal(a.view(np.uint32), b.view(np.uint32)), w
    assert np.array_equal(h_full.ah_state_get(B.AH_UHIST), h_b.ah_state_get(B.AH_UHIST))
    h_full.close()
    h_b.close()


def test_checkpoint_resume_with_the_rule_on_the_device(B, torch):
    # the same with lagged one-pass exchange rounds: the history ring lives on the device and
    # the coefficients waiting for the next exchange round are part of the snapshot
    layout = W.resnet18_layout(16)
    segs, P, K, tau = W.segments(layout), W.total_params(layout), 4, 2
    theta0, pool = _layout_inputs(layout, K)
    dev_pool = [(torch.from_numpy(g).cuda(), torch.from_numpy(hv).cuda()) for g, hv in pool]
    from parity_driver import MASK_SEED

    def rounds(h, first, last):
        for t in range(first, last + 1):
            mask = h.dw_mask_next(MASK_SEED, t, 0.2)
            g, hv = dev_pool[t % len(dev_pool)]
            if t % tau == 0:
                h.ah_local_step_exchange(g, hv, Z_SEED, lr=0.01, round_=t, want_dist=True,
                                         worker_mask=mask, alpha=0.05, lagged=True)
            else:
                h.ah_local_step(g, hv, Z_SEED, lr=0.01, round_=t)

    def fresh():
        h = B.Handle(K, P, segs)
        h.ah_state_set(B.AH_CENTER, theta0)
        h.ah_broadcast_center()
        return h

    h_full = fresh()
    rounds(h_full, 1, 20)
    h_a = fresh()
    rounds(h_a, 1, 10)
    snap = {w: h_a.ah_state_get(w) for w in (B.AH_X, B.AH_M, B.AH_V, B.AH_CENTER, B.AH_STEP, B.AH_UHIST,
                                             B.AH_DOWN_UNTIL, B.AH_ROUND, B.AH_WEIGHTS)}
    h_a.close()
    h_b = B.Handle(K, P, segs)
    for w, val in snap.items():
        h_b.ah_state_set(w, val)
    rounds(h_b, 11, 20)
    for w in (B.AH_X, B.AH_M, B.AH_V, B.AH_CENTER, B.AH_WEIGHTS):
        a, b = h_full.ah_state_get(w), h_b.ah_state_get(w)
        assert np.array_equal(a.view(np.uint32), b.view(np.uint32)), w
    assert np.array_equal(h_full.ah_state_get(B.AH_UHIST), h_b.ah_state_get(B.AH_UHIST))
    h_full.close()
    h_b.close()


def test_checkpoint_resume_with_an_exchange_pending(B, torch):
    # the bench's default shape: the exchange of a period rides on the first local step of the
    # next one, so at a period boundary something waits on the device: the distances (the rule
    # still to run), or the coefficients of a rule the distance round asked for (the snapshot
    # has them assembled and the rule run).  A snapshot taken there, restored into a fresh handle, must continue bit for bit:
    # in the first case the restored distances are pending again, in the second the restored
    # coefficients are handed to the exchange as caller weights.
    layout = W.resnet18_layout(16)
    segs, P, K, tau = W.segments(layout), W.total_params(layout), 4, 2
    theta0, pool = _layout_inputs(layout, K)
    dev_pool = [(torch.from_numpy(g).cuda(), torch.from_numpy(hv).cuda()) for g, hv in pool]
    from parity_driver import MASK_SEED

    def rounds(h, first, last, pending, rule_in_round, restored_weights=None):
        for t in range(first, last + 1):
            mask = h.dw_mask_next(MASK_SEED, t, 0.2)
            g, hv = dev_pool[t % len(dev_pool)]
            if pending is not None:
                if restored_weights is not None:
                    h.easgd_exchange_then_step(g, hv, Z_SEED, lr=0.01, round_=t, worker_mask=pending,
                                               weights=restored_weights, dynamic=False)
                    restored_weights = None
                else:
                    h.easgd_exchange_then_step(g, hv, Z_SEED, lr=0.01, round_=t, worker_mask=pending,
                                               alpha=0.05, dynamic=True)
                pending = None
            else:
                ex = t % tau == 0
                h.ah_local_step(g, hv, Z_SEED, lr=0.01, round_=t, rule_alpha=0.05,
                                want_dist=(B.AH_DIST_AND_RULE if rule_in_round else B.AH_DIST) if ex else 0)
                if ex:
                    pending = mask
        return pending

    def fresh():
        h = B.Handle(K, P, segs)
        h.ah_state_set(B.AH_CENTER, theta0)
        h.ah_broadcast_center()
        return h

    for rule_in_round in (False, True):
        h_full = fresh()
        rounds(h_full, 1, 20, None, rule_in_round)
        h_a = fresh()
        pending = rounds(h_a, 1, 10, None, rule_in_round)          # round 10 measured distances
        assert pending is not None
        sel = [B.AH_X, B.AH_M, B.AH_V, B.AH_CENTER, B.AH_STEP, B.AH_UHIST, B.AH_DOWN_UNTIL, B.AH_ROUND]
        sel.append(B.AH_WEIGHTS if rule_in_round else B.AH_NORM2)
        snap = {w: h_a.ah_state_get(w) for w in sel}
        h_a.close()
        h_b = B.Handle(K, P, segs)
        for w, val in snap.items():
            h_b.ah_state_set(w, val)
        rounds(h_b, 11, 20, pending, rule_in_round, snap[B.AH_WEIGHTS] if rule_in_round else None)
        for w in (B.AH_X, B.AH_M, B.AH_V, B.AH_CENTER, B.AH_WEIGHTS):
            a, b = h_full.ah_state_get(w), h_b.ah_state_get(w)
            assert np.array_equal(a.view(np.uint32), b.view(np.uint32)), (rule_in_round, w)
        assert np.array_equal(h_full.ah_state_get(B.AH_UHIST), h_b.ah_state_get(B.AH_UHIST))
        h_full.close()
        h_b.close()


def test_library_log_distance_on_the_device(B, torch):
    # u = log ||x_i - c|| as the device forms of the rule compute it (the rule as a launch of
    # its own, and the rule at the end of a distance round), against the definition in
    # 300-bit arithmetic: the natural logarithm rounded to the nearest double, halved
    import mpmath
    mpmath.mp.prec = 300
    rng = np.random.default_rng(78)
    K, P = 64, 2048
    n2 = np.concatenate([np.exp(rng.uniform(-680, 700, 4 * K)), rng.uniform(0.5, 2.0, 3 * K),
                         1.0 + rng.uniform(-1, 1, K) * 1e-9, np.exp(2 * rng.normal(0, 3, 4 * K))])
    h = B.Handle(K, P, [])
    h.dw_config(1, np.array([1.0]), -0.1)
    for lo in range(0, n2.size, K):
        chunk = n2[lo:lo + K]
        h.ah_state_set(B.AH_NORM2, chunk)                  # restored distances are pending
        h.easgd_exchange_dynamic(np.zeros(K, np.uint8), 0.05, None, False)   # the rule; nobody arrives
        u = h.ah_state_get(B.AH_UHIST, p_hist=1)[:, 0]
        want = np.array([float(mpmath.log(mpmath.mpf(float(v)))) * 0.5 for v in chunk])
        assert np.array_equal(u, want), (lo, chunk[u != want][:3])
    # the rule at the end of a distance round: x = c + d e_0 gives ||x_i - c||^2 = d_i^2 exactly
    d = np.exp(rng.uniform(-20, 20, K)).astype(np.float32)
    x = np.zeros((K, P), np.float32)
    x[:, 0] = d
    h.ah_state_set(B.AH_CENTER, np.zeros(P, np.float32))
    h.ah_state_set(B.AH_X, x)
    z = torch.zeros((K, P), device="cuda")
    h.ah_local_step(z, z, 1, lr=0.0, active=np.zeros(K, np.uint8), want_dist=B.AH_DIST_AND_RULE,
                    rule_alpha=0.05)
    u = h.ah_state_get(B.AH_UHIST, p_hist=1)[:, 0]
    n2d = d.astype(np.float64) ** 2
    assert np.array_equal(h.ah_state_get(B.AH_NORM2), n2d)
    want = np.array([float(mpmath.log(mpmath.mpf(float(v)))) * 0.5 for v in n2d])
    assert np.array_equal(u, want)
    h.close()


def test_error_paths_and_own_allocation(B, torch):
    K, P = 2, 1000
    h = B.Handle(K, P, [], own_alloc=True)           # cudaMalloc workspace, default stream
    g = torch.zeros((K, 1004), device="cuda")
    lib = B.raw()
    hy = B.ah_hyper(0.01, 0.9, 0.999, 1e-4, 1.0, 0.0, 1, None, 0)
    # misaligned base pointer, stride not a multiple of 4, stride below P, null pointer
    assert lib.ah_local_step(h._h, g.data_ptr() + 4, g.data_ptr(), 1004, 1, C.byref(hy)) == B.AH_ERR_ALIGN
    assert lib.ah_local_step(h._h, g.data_ptr(), g.data_ptr(), 1002, 1, C.byref(hy)) == B.AH_ERR_ALIGN
    assert lib.ah_local_step(h._h, g.data_ptr(), g.data_ptr(), 996, 1, C.byref(hy)) == B.AH_ERR_INVALID_ARG
    assert lib.ah_local_step(h._h, None, g.data_ptr(), 1004, 1, C.byref(hy)) == B.AH_ERR_INVALID_ARG
    bad = B.ah_hyper(0.01, 1.0, 0.999, 1e-4, 1.0, 0.0, 1, None, 0)      # beta1 = 1
    assert lib.ah_local_step(h._h, g.data_ptr(), g.data_ptr(), 1004, 1, C.byref(bad)) == B.AH_ERR_INVALID_ARG
    # weights before any distance has been measured
    w = (C.c_float * (2 * K))()
    assert lib.dw_weights_next(h._h, 0.1, w) == B.AH_ERR_STATE
    assert lib.ah_state_get(h._h, 99, 0, g.data_ptr(), 1) == B.AH_ERR_INVALID_ARG
    assert lib.ah_state_get(h._h, B.AH_X, K, g.data_ptr(), 1) == B.AH_ERR_INVALID_ARG
    # the handle still works after the refusals
    h.ah_local_step(g, g, 1, lr=0.01, want_dist=True)
    assert np.all(h.dw_weights_next(0.1) == np.float32(0.1))
    assert h.ah_launch_count() == 2                  # the step, and the assembly of its tile sums for the host
    # a refused call changes nothing: step counts and the call counter stay where they were
    steps, calls = h.ah_state_get(B.AH_STEP).copy(), h.ah_state_get(B.AH_ROUND).copy()
    assert lib.ah_local_step(h._h, g.data_ptr(), g.data_ptr(), 1002, 1, C.byref(hy)) == B.AH_ERR_ALIGN
    far = B.ah_hyper(0.01, 0.9, 0.999, 1e-4, 1.0, 0.0, 1, None, 3)       # want_dist out of range
    assert lib.ah_local_step(h._h, g.data_ptr(), g.data_ptr(), 1004, 1, C.byref(far)) == B.AH_ERR_INVALID_ARG
    order = (C.c_uint16 * K)(0, 0)                                       # names worker 0 twice
    assert lib.ah_local_step_exchange(h._h, g.data_ptr(), g.data_ptr(), 1004, 1, C.byref(hy), None, None,
                                      0.1, order, 1, 0) == B.AH_ERR_INVALID_ARG
    assert lib.easgd_exchange_then_step(h._h, g.data_ptr(), g.data_ptr(), 1004, 1, C.byref(hy), None, None,
                                        0.1, None, 0, 1) == B.AH_ERR_STATE  # no distances pending
    assert np.array_equal(h.ah_state_get(B.AH_STEP), steps)
    assert np.array_equal(h.ah_state_get(B.AH_ROUND), calls)
    assert h.ah_launch_count() == 2
    h.close()
    # a workspace that is too small is refused
    small = torch.empty(1024, dtype=torch.uint8, device="cuda")
    opt = B.ah_alloc((small.data_ptr() + 255) // 256 * 256, 512, None, 0)
    out = C.c_void_p(None)
    assert lib.ah_init(C.byref(out), 4, 10_000, None, 0, C.byref(opt)) == B.AH_ERR_ALLOC
    assert out.value is None


# ------------------------------------------- full-size configurations, short runs
def _full_size_run(B, kind, K, tau, rounds, p_fail, max_stale=1, frozen=False, n_pool=1):
    layout = W.LAYOUTS[kind]()
    cfg = RunConfig(K=K, segments=W.segments(layout), P=W.total_params(layout), rounds=rounds,
                    tau=tau, p_fail=p_fail, max_stale=max_stale, frozen=frozen)
    _check_run(B, cfg, _layout_inputs(layout, K, n_pool=n_pool))


@pytest.mark.parametrize("variant", ["async_device_weights", "fused_lagged", "fused_lagged_async", "eamsgd",
                                     "exchange_with_next_step"])
def test_full_size_resnet18_layout_variants(B, torch, variant):
    # config 2 at its full size with the other forms of the round, in the launch shapes the
    # bench times: two communication periods each, every element compared with the oracle
    layout = W.resnet18_layout()
    kw = dict(K=8, segments=W.segments(layout), P=W.total_params(layout), rounds=8, tau=4, p_fail=0.1)
    if variant == "async_device_weights":
        cfg = RunConfig(asynchronous=True, sync_free="yes", alpha=0.1, **kw)
    elif variant == "fused_lagged":
        cfg = RunConfig(fused="lagged", **kw)
    elif variant == "fused_lagged_async":
        cfg = RunConfig(fused="lagged", asynchronous=True, alpha=0.1, **kw)
    elif variant == "exchange_with_next_step":
        cfg = RunConfig(fused="next", **kw)
    else:
        cfg = RunConfig(method="msgd", dynamic=False, alpha=0.1, asynchronous=True, **kw)
    h, ref, log = run_gaussian(cfg, B, oracle, _layout_inputs(layout, 8, n_pool=2), variant="omp")
    viol, bits = compare_state(h, ref, B)
    assert log["masks_equal"] and log["weights_equal"] and log["norm2_equal"] and log["orders_equal"], log
    assert sum(viol.values()) == 0 and sum(bits.values()) == 0, (viol, bits)
    assert log["exchanges"] == 2
    h.close()


def test_full_size_resnet18_layout(B, torch):
    # config 2 at its full size (P = 11,689,512, K = 8): two communication periods
    _full_size_run(B, "resnet18", 8, 4, 8, 0.1, n_pool=2)


def test_full_size_resnet18_layout_all_200_rounds(B, torch):
    # config 2 exactly as stated: full size, K = 8, tau = 4, Bernoulli(0.1) failures, 200 rounds
    _full_size_run(B, "resnet18", 8, 4, 200, 0.1, n_pool=2)


def test_full_size_resnet50_layout_stragglers(B, torch):
    # config 3 at its full size (P = 25,557,032, K = 16), frozen stragglers
    _full_size_run(B, "resnet50", 16, 4, 4, 0.2, max_stale=8, frozen=True)


def test_full_size_vgg16_layout(B, torch):
    # config 4 at its full size (P = 138,357,544, K = 4, tau = 8): one period
    _full_size_run(B, "vgg16", 4, 8, 8, 0.25)


def test_full_size_k64_prefix_sample_and_distance_property(B, torch):
    """Config 5's largest case (ResNet-50-shaped layout, K = 64, 19.6 GB of state) in the
    launch shape the bench times.  The oracle recomputes a sample it can afford: every
    worker's leading tensors (columns are independent given the masks and a fixed alpha,
    and z is indexed by absolute position), compared element by element; the full-size
    distances are checked against a double-precision sum formed on the device."""
    layout = W.resnet50_layout()
    segs, P, K, tau, R = W.segments(layout), W.total_params(layout), 64, 4, 8
    ld = W.padded_ld(P)
    n_keep = next(k for k, tns in enumerate(layout) if tns.offset + tns.numel > 1_500_000)
    prefix = layout[:n_keep]
    Pp = W.total_params(prefix)
    gen = torch.Generator(device="cuda").manual_seed(7)
    g = torch.empty((K, ld), device="cuda").normal_(generator=gen).mul_(0.05)
    hv = torch.empty((K, ld), device="cuda").normal_(generator=gen).mul_(0.05)
    theta0 = torch.empty(P, device="cuda").normal_(generator=gen).mul_(0.05)
    h = B.Handle(K, P, segs)
    h.ah_state_set(B.AH_CENTER, theta0)
    h.ah_broadcast_center()
    gp = np.ascontiguousarray(g[:, :Pp].cpu().numpy())
    hp = np.ascontiguousarray(hv[:, :Pp].cpu().numpy())
    ref = OracleState(theta0[:Pp].cpu().numpy(), K, W.segments(prefix), variant="omp")
    alpha = 0.8 / K
    from parity_driver import MASK_SEED
    for t in range(1, R + 1):
        mask = h.dw_mask_next(MASK_SEED, t, 0.1)
        assert np.array_equal(mask, ref.mask_next(MASK_SEED, t, 0.1))
        ex = t % tau == 0
        h.ah_local_step(g, hv, Z_SEED, lr=0.01, round_=t, want_dist=ex)
        ref.local_step(gp, hp, Z_SEED, t, lr=0.01)
        if ex:
            # distances at full size: same value as a double-precision sum on the device
            xs = torch.empty((K, P), device="cuda")
            cs = torch.empty(P, device="cuda")
            h.ah_state_get(B.AH_X, out=xs)
            h.ah_state_get(B.AH_CENTER, out=cs)
            n2 = h.ah_state_get(B.AH_NORM2)
            for i in (0, 17, 63):
                want = float(((xs[i] - cs).double() ** 2).sum().item())
                assert abs(n2[i] - want) <= 1e-11 * want, (t, i)
            del xs, cs
            h.easgd_exchange(mask, None, alpha)
            ref.exchange(mask, alpha=alpha)
    row = torch.empty(P, device="cuda")
    for which, want in ((B.AH_X, ref.x), (B.AH_M, ref.m), (B.AH_V, ref.v)):
        for i in range(K):
            h.ah_state_get(which, worker=i, out=row)
            got = row[:Pp].cpu().numpy()
            assert np.array_equal(got.view(np.uint32), want[i].view(np.uint32)), (which, i)
    h.ah_state_get(B.AH_CENTER, out=row)
    assert np.array_equal(row[:Pp].cpu().numpy().view(np.uint32), ref.center.view(np.uint32))
    h.close()
