"""CPU-only tests: the C-ABI library loads and exports what include/adahess.h declares,
argument checks, and the host-side bookkeeping (failure mask, dynamic weights, tile
descriptors) against the oracle.  No compute call touches a GPU here."""
import ctypes as C
import os
import re

import numpy as np
import pytest

from oracle import OracleState
from paper_2409_09242_b200 import workloads as W


@pytest.fixture(scope="module")
def B():
    from paper_2409_09242_b200 import build
    build.build()
    from paper_2409_09242_b200 import binding
    return binding


def test_library_exports_every_declared_symbol(B):
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    declared = set()
    for fn in os.listdir(os.path.join(root, "include")):
        text = open(os.path.join(root, "include", fn)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        declared |= set(re.findall(r"\b((?:ah|dw|easgd|sgd)_[a-z0-9_]+)\s*\(", text))
    assert {"ah_init", "ah_local_step", "easgd_exchange", "ah_state_get"} <= declared
    lib = C.CDLL(B._build.LIB_PATH)
    for name in sorted(declared):
        assert hasattr(lib, name), name
    assert declared == set(B.EXPORTS)


def test_status_strings_and_argument_checks(B):
    assert B.ah_status_string(0) == "ok"
    assert "segment" in B.ah_status_string(B.AH_ERR_SEGMENTS)
    with pytest.raises(B.AdaHessError):
        B.ah_workspace_bytes(0, 10, 0)                     # K < 1
    with pytest.raises(B.AdaHessError):
        B.ah_workspace_bytes(B.AH_MAX_WORKERS + 1, 10, 0)  # K too large
    with pytest.raises(B.AdaHessError):
        B.ah_workspace_bytes(1, 1 << 31, 0)                # P too large
    assert B.ah_workspace_bytes(1, (1 << 31) - 1, 0) > 3 * 4 * ((1 << 31) - 1)
    # workspace covers x, m, v [K][P] plus the master row
    K, P = 16, 25_557_032
    assert B.ah_workspace_bytes(K, P, 161) >= (3 * K + 1) * P * 4


@pytest.mark.parametrize("segs,code", [
    ([(0, 10, 3)], "SEGMENTS"),            # length not a multiple of block
    ([(0, 9, 9), (5, 9, 9)], "SEGMENTS"),  # overlap
    ([(9, 9, 9), (0, 9, 9)], "SEGMENTS"),  # unsorted
    ([(0, 200, 1)], "SEGMENTS"),           # beyond P
    ([(0, 0, 0)], "SEGMENTS"),             # block 0
    ([(0, 258, 129)], "SEGMENTS"),         # block above the maximum
])
def test_bad_segment_tables_are_rejected(B, segs, code):
    with pytest.raises(B.AdaHessError) as e:
        B.Handle(2, 100 if segs[0][1] != 258 else 1000, segs, host_only=True)
    assert e.value.status == getattr(B, "AH_ERR_" + code)


def test_bookkeeping_handle_refuses_device_calls(B):
    h = B.Handle(2, 64, [(0, 64, 1)], host_only=True)
    assert B.raw().ah_broadcast_center(h._h) == B.AH_ERR_STATE
    assert B.raw().easgd_exchange(h._h, None, None, 0.1) == B.AH_ERR_STATE
    assert B.raw().easgd_exchange_async(h._h, None, None, 0.1, None) == B.AH_ERR_STATE
    w = (C.c_float * 4)()
    assert B.raw().dw_weights_next(h._h, 0.1, w) == B.AH_ERR_STATE
    h.close()


def test_refused_calls_leave_the_bookkeeping_untouched(B):
    # step counts, the call counter and the pending-distance state move only with a launch
    # that went in: a call that is refused (here: no device behind the handle, bad arguments)
    # leaves them exactly as they were
    K = 3
    h = B.Handle(K, 64, [(0, 64, 1)], host_only=True)
    lib = B.raw()
    steps0 = np.array([5, 0, 7], np.uint32)
    h.ah_state_set(B.AH_STEP, steps0)
    h.ah_state_set(B.AH_ROUND, np.array([9, 1], np.uint32))
    hy = B.ah_hyper(0.01, 0.9, 0.999, 1e-4, 1.0, 0.0, B.AH_ROUND_AUTO, None, 1)
    sg = B.sgd_hyper(0.01, 0.5, None, 0)
    fake = 0x1000                                   # never dereferenced: the calls are refused first
    order = (C.c_uint16 * K)(0, 1, 2)
    calls = [
        lambda: lib.ah_local_step(h._h, fake, fake, 64, 1, C.byref(hy)),
        lambda: lib.ah_local_step(h._h, None, fake, 64, 1, C.byref(hy)),
        lambda: lib.ah_local_step(h._h, fake, fake, 60, 1, C.byref(hy)),
        lambda: lib.ah_local_step_exchange(h._h, fake, fake, 64, 1, C.byref(hy), None, None, 0.1, order, 1, 0),
        lambda: lib.easgd_exchange_then_step(h._h, fake, fake, 64, 1, C.byref(hy), None, None, 0.1, None, 0, 0),
        lambda: lib.sgd_local_step(h._h, fake, 64, C.byref(sg)),
        lambda: lib.easgd_exchange_then_sgd_step(h._h, fake, 64, C.byref(sg), None, None, 0.1, None, 0),
        lambda: lib.easgd_exchange_dynamic(h._h, None, 0.1, None, 0),
        lambda: lib.ah_broadcast_center(h._h),
    ]
    for k, call in enumerate(calls):
        assert call() in (B.AH_ERR_STATE, B.AH_ERR_INVALID_ARG), k
        assert np.array_equal(h.ah_state_get(B.AH_STEP), steps0), k
        assert list(h.ah_state_get(B.AH_ROUND)) == [9, 1], k
        assert h.ah_launch_count() == 0
    # the host-side rule still runs after all the refusals, from the restored history flag
    w = h.dw_weights_from_norm2(np.array([1.0, 4.0, 9.0]), 0.05)
    assert w.shape == (2 * K,)
    h.close()


def test_mask_matches_oracle_bit_for_bit(B):
    for K, p, stale in ((4, 0.1, 1), (16, 0.2, 8), (64, 0.3, 1), (8, 1 / 3, 4), (3, 0.0, 1), (3, 1.0, 2)):
        h = B.Handle(K, 8, [], host_only=True)
        ref = OracleState(np.zeros(8, np.float32), K, [])
        for t in range(1, 400):
            assert np.array_equal(h.dw_mask_next(0x5EED0002, t, p, stale),
                                  ref.mask_next(0x5EED0002, t, p, stale)), (K, p, stale, t)
        assert np.array_equal(h.ah_state_get(B.AH_DOWN_UNTIL), ref.down_until)
        h.close()


def test_arrival_order_matches_oracle_bit_for_bit(B):
    for K in (1, 2, 3, 8, 64, 256):
        h = B.Handle(K, 8, [], host_only=True)
        ref = OracleState(np.zeros(8, np.float32), K, [])
        for t in (0, 1, 2, 3, 1000, 0xFFFFFFFE):
            for seed in (0x5EED0003, 0xFEDCBA9876543210):
                got = h.dw_order_next(seed, t)
                assert got.dtype == np.uint16 and np.array_equal(got, ref.order_next(seed, t)), (K, t)
        h.close()


def test_partition_matches_oracle_bit_for_bit(B, orc):
    for seed, n, k, o in ((0x5EED0004, 60000, 8, 7500), (1, 60000, 4, 15000), (2, 1000, 7, 0),
                          (3, 17, 5, 3), (4, 10, 3, 10), (5, 1, 1, 0), (1 << 40 | 9, 4097, 16, 512)):
        perm, bounds = B.dw_partition(seed, n, k, o)
        rperm, rbounds = orc.partition(seed, n, k, o)
        assert np.array_equal(perm, rperm) and np.array_equal(bounds, rbounds), (seed, n, k, o)
    with pytest.raises(B.AdaHessError):
        B.dw_partition(1, 10, 2, 11)
    with pytest.raises(B.AdaHessError):
        B.dw_partition(1, 10, 0, 1)


def test_weights_match_oracle_bit_for_bit_given_same_distances(B):
    rng = np.random.default_rng(0)
    for K, alpha, p_hist, kappa in ((4, 0.05, 4, -0.1), (16, 0.1, 2, -0.05), (64, 0.0125, 6, -0.3)):
        c = rng.dirichlet(np.ones(p_hist))
        h = B.Handle(K, 8, [], host_only=True)
        h.dw_config(p_hist, c, kappa)
        ref = OracleState(np.zeros(8, np.float32), K, [], p_hist=p_hist, c=c, kappa=kappa)
        u = rng.normal(0, 1, K)
        for s in range(60):
            u = u + rng.normal(0, 0.08, K) - (rng.random(K) < 0.1) * 0.3
            n2 = np.exp(2 * u)
            if s == 0:
                n2[:] = 0.0                      # workers start on top of the master
            w = h.dw_weights_from_norm2(n2, alpha)
            ref.norm2[:] = n2
            h2, h1 = ref.weights_next(alpha)
            assert np.array_equal(w[:K], h2) and np.array_equal(w[K:], h1), (K, s)
        assert np.array_equal(h.ah_state_get(B.AH_UHIST, p_hist=p_hist), ref.uhist)
        h.close()


def test_library_log_distance_is_the_correctly_rounded_value(B):
    # u = log ||x_i - c|| (Sec. V-B) as the library's own rule computes it from known squared
    # distances, against the definition evaluated in 300-bit arithmetic: the natural logarithm
    # rounded to the nearest double, halved.  Independent of the oracle.
    import mpmath
    mpmath.mp.prec = 300
    rng = np.random.default_rng(77)
    K = B.AH_MAX_WORKERS
    n2 = np.concatenate([
        np.exp(rng.uniform(-680, 700, 4 * K)),                  # the whole exponent range
        rng.uniform(0.5, 2.0, 4 * K),                           # around 1, where ln cancels
        1.0 + rng.uniform(-1, 1, 2 * K) * 1e-9,
        np.exp(2 * rng.normal(0, 3, 6 * K)),                    # squared distances of the method
    ])
    n2[:8] = [1.0, 2.0, 0.5, 1e-300, 0.0, 1.4142135623730951, 0.7071067811865476, 1.7976931348623157e308]
    h = B.Handle(K, 8, [], host_only=True)
    h.dw_config(1, np.array([1.0]), -0.1)
    for lo in range(0, n2.size, K):
        chunk = n2[lo:lo + K]
        h.dw_weights_from_norm2(chunk, 0.05)
        u = h.ah_state_get(B.AH_UHIST, p_hist=1)[:, 0]
        want = np.array([float(mpmath.log(mpmath.mpf(max(float(v), 1e-300)))) * 0.5 for v in chunk])
        assert np.array_equal(u, want), (lo, chunk[u != want][:3])
    h.close()


@pytest.mark.parametrize("name", ["resnet18", "resnet50", "vgg16", "odd"] + [f"random{k}" for k in range(12)])
def test_tile_descriptors_cover_whole_blocks(B, name):
    if name.startswith("random"):
        segs, P = W.random_segment_table(int(name[6:]), B.AH_MAX_BLOCK)
    elif name == "odd":
        segs = [(3, 18, 9), (21, 10, 1), (37, 4900, 49), (4940, 2505, 5), (9001, 4096, 128)]
        P = 13_111
    else:
        layout = W.LAYOUTS[name](8)
        segs, P = W.segments(layout), W.total_params(layout)
    h = B.Handle(2, P, segs, host_only=True)
    ntiles, nruns, T, lds = (int(v) for v in h.ah_state_get(B.AH_INFO))
    runs, tiles = h.ah_state_get(B.AH_RUNS), h.ah_state_get(B.AH_TILES)
    assert ntiles == (P + T - 1) // T and lds == (P + 3) // 4 * 4 and len(runs) == nruns
    # runs tile [0, P) exactly, and agree with the segment table element by element
    assert runs[0, 0] == 0 and runs[-1, 1] == P and np.array_equal(runs[1:, 0], runs[:-1, 1])
    block_of = np.ones(P, np.int64)
    for off, n, b in segs:
        block_of[off:off + n] = b
    for s, e, b, _ in runs:
        assert np.all(block_of[s:e] == b)
    for t in range(ntiles):
        run0, e0, e1, flags = (int(v) for v in tiles[t])
        t0, t1 = t * T, min(P, (t + 1) * T)
        assert runs[run0, 0] <= t0 < runs[run0, 1]
        assert e0 <= t0 and e1 >= t1 and e1 <= P
        assert t0 - e0 < B.AH_MAX_BLOCK and e1 - t1 < B.AH_MAX_BLOCK
        averaged = block_of[t0:t1][block_of[t0:t1] > 1]
        assert flags & 1 == int(averaged.size > 0)
        assert (flags >> 1) & 1 == int(averaged.size > 0 and np.all(averaged == 9))   # 3x3 kernels only
        assert flags >> 2 == 0
        # [e0, e1) ends on block boundaries of the runs they fall in
        for edge in (e0, e1):
            r = np.searchsorted(runs[:, 1], edge, side="right" if edge == e0 else "left")
            r = min(r, nruns - 1)
            s, e, b, _ = (int(v) for v in runs[r])
            assert (edge - s) % b == 0 or edge == e
    h.close()


def test_constant_divisor_shortcut_is_exact(tmp_path):
    # the kernels divide by per-launch constants (bias corrections, spatial block sizes)
    # with a reciprocal multiply plus one FMA correction; a C program checks on the host,
    # for every binary32 significand, that this equals the correctly rounded quotient
    import subprocess
    src = os.path.join(os.path.dirname(os.path.abspath(__file__)), "helpers", "exact_division_check.c")
    exe = str(tmp_path / "exact_division_check")
    subprocess.check_call(["gcc", "-O2", "-mfma", "-ffp-contract=off", "-fopenmp", src, "-o", exe, "-lm"])
    out = subprocess.run([exe], capture_output=True, text=True)
    assert out.returncode == 0, out.stdout
    checked, bad = (int(v) for v in out.stdout.split()[1::2])
    assert checked > 200 and bad == 0


def test_logarithm_constants_match_their_formula(tmp_path):
    # the series coefficients 1/3 ... 1/43 of the library's logarithm are written out as pairs
    # of doubles; a host program recomputes each from its defining formula
    import subprocess
    here = os.path.dirname(os.path.abspath(__file__))
    src = os.path.join(here, "helpers", "ln_table_check.cpp")
    csrc = os.path.join(os.path.dirname(here), "paper_2409_09242_b200", "csrc")
    cuda_inc = os.path.join(os.environ.get("CUDA_HOME", "/usr/local/cuda"), "include")
    exe = str(tmp_path / "ln_table_check")
    subprocess.check_call(["g++", "-O1", "-std=c++17", "-ffp-contract=off", "-I", csrc, "-I", cuda_inc,
                           src, "-o", exe])
    out = subprocess.run([exe], capture_output=True, text=True)
    assert out.returncode == 0, out.stdout
    assert out.stdout.strip().endswith("bad 0")
