"""Configurations 3, 4 and 5 at their full size for all their rounds: the CUDA library,
called through its C ABI, against the CPU oracle on the same seeded inputs; x, m, v and the
master compared element by element at the end, masks, distances and weights at every
exchange.  The oracle needs a minute or three per run, so one run per configuration is
always on; the remaining combinations of the configurations' sweeps (communication periods
1 and 16, every worker count and failure rate) run when AH_FULL_CONFIGS=1 is set:

    AH_FULL_CONFIGS=1 AH_PARITY_REPORT=report.txt python -m pytest tests/test_gpu_parity_full_configs.py -m gpu

AH_PARITY_REPORT names a text file that gets one line per run."""
import os
import time

import numpy as np
import pytest

import oracle
from paper_2409_09242_b200 import workloads as W
from parity_driver import RunConfig, compare_state, run_gaussian

pytestmark = pytest.mark.gpu

ALWAYS, SWEEP = True, False
# name, layout, always on, run parameters ("ride": every exchange is deferred to the next
# round's local step, the launch shape the benchmark times by default)
CASES = [
    ("c3-tau4-ride", "resnet50", ALWAYS,
     dict(K=16, rounds=100, tau=4, p_fail=0.2, max_stale=8, frozen=True, fused="next")),
    ("c4-ride", "vgg16", ALWAYS, dict(K=4, rounds=50, tau=8, p_fail=0.25, fused="next")),
    ("c5-K64-p0.1", "resnet50", ALWAYS, dict(K=64, rounds=50, tau=4, p_fail=0.1)),
]
for tau in (1, 4, 16):
    CASES.append((f"c3-tau{tau}", "resnet50", SWEEP,
                  dict(K=16, rounds=100, tau=tau, p_fail=0.2, max_stale=8, frozen=True)))
CASES.append(("c3-tau16-ride", "resnet50", SWEEP,
              dict(K=16, rounds=100, tau=16, p_fail=0.2, max_stale=8, frozen=True, fused="next")))
CASES.append(("c4", "vgg16", SWEEP, dict(K=4, rounds=50, tau=8, p_fail=0.25)))
for K in (4, 16, 32, 64):
    for p in (0.0, 0.1, 0.3):
        if (K, p) != (64, 0.1):
            CASES.append((f"c5-K{K}-p{p}", "resnet50", SWEEP, dict(K=K, rounds=50, tau=4, p_fail=p)))


@pytest.mark.parametrize("name,kind,always,kw", CASES, ids=[c[0] for c in CASES])
def test_config_full_size_all_rounds(name, kind, always, kw):
    if not always and os.environ.get("AH_FULL_CONFIGS") != "1":
        pytest.skip("part of the sweep: set AH_FULL_CONFIGS=1")
    import torch
    from paper_2409_09242_b200 import binding as B
    torch.cuda.set_device(0)
    layout = W.LAYOUTS[kind]()
    cfg = RunConfig(segments=W.segments(layout), P=W.total_params(layout), **kw)
    t0 = time.time()
    inputs = (W.theta0_np(layout, 0), W.gaussian_pool_np(layout, cfg.K, 1, 1))
    h, ref, log = run_gaussian(cfg, B, oracle, inputs, variant="omp")
    viol, bits = compare_state(h, ref, B)
    steps_equal = bool(np.array_equal(h.ah_state_get(B.AH_STEP), ref.step))
    ring_equal = bool(np.array_equal(h.ah_state_get(B.AH_UHIST), ref.uhist))
    h.close()
    del h, ref, inputs
    torch.cuda.empty_cache()
    report = os.environ.get("AH_PARITY_REPORT")
    if report:
        with open(report, "a") as f:
            f.write(f"{name}: {kind} layout {kw}: outside 1e-6 + 1e-5 rel. {sum(viol.values())}, bits differ "
                    f"{sum(bits.values())}, masks/distances/weights identical {log['masks_equal']}/"
                    f"{log['norm2_equal']}/{log['weights_equal']}, exchanges {log['exchanges']}, "
                    f"{time.time() - t0:.0f} s\n")
    assert log["masks_equal"] and log["weights_equal"] and log["norm2_equal"], log
    assert sum(viol.values()) == 0, viol
    assert sum(bits.values()) == 0, bits          # same operation order => same bits
    assert steps_equal and ring_equal
    assert log["exchanges"] == cfg.rounds // cfg.tau
