#!/usr/bin/env python
"""Every configuration at its full size for its full number of rounds, library against
oracle, element by element.  Too long for the test suite (the oracle needs minutes per
configuration): run by hand on a machine with a B200,

    python tests/run_full_configs.py [--ride] [c3 c4 c5 ...] > full_configs.txt

With --ride every exchange is deferred to the next round's local step
(easgd_exchange_then_step, the launch shape the benchmark times by default; runs with a
communication period of one round are skipped).

It prints one line per run: violations of |gpu - oracle| <= 1e-6 + 1e-5 |oracle| and the
number of elements whose bits differ, for x, m, v and the master, and whether masks,
distances and weights were bit-identical throughout.  The pytest suite covers the same
configurations at reduced width for all rounds and at full size for a few rounds.
"""
import os
import sys
import time

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
sys.path.insert(0, os.path.join(ROOT, "tests"))

import numpy as np  # noqa: E402

import oracle  # noqa: E402
from paper_2409_09242_b200 import binding, workloads as W  # noqa: E402
from parity_driver import RunConfig, compare_state, run_gaussian  # noqa: E402


def runs(which):
    if "c2" in which:
        yield "c2 resnet18 K=8 tau=4 p=0.1 R=200", "resnet18", dict(K=8, rounds=200, tau=4, p_fail=0.1)
    if "c3" in which:
        for tau in (1, 4, 16):
            yield (f"c3 resnet50 K=16 tau={tau} p=0.2 stale<=8 frozen R=100", "resnet50",
                   dict(K=16, rounds=100, tau=tau, p_fail=0.2, max_stale=8, frozen=True))
    if "c4" in which:
        yield "c4 vgg16 K=4 tau=8 p=0.25 R=50", "vgg16", dict(K=4, rounds=50, tau=8, p_fail=0.25)
    if "c5" in which:
        for K in (4, 16, 32, 64):
            for p in (0.0, 0.1, 0.3):
                yield (f"c5 resnet50 K={K} tau=4 p={p} R=50", "resnet50",
                       dict(K=K, rounds=50, tau=4, p_fail=p))


def main():
    import torch
    torch.cuda.set_device(0)
    args = sys.argv[1:]
    ride = "--ride" in args
    which = [a for a in args if a != "--ride"] or ["c2", "c3", "c4", "c5"]
    for name, kind, kw in runs(which):
        if ride:
            if kw["tau"] < 2:
                continue
            kw = dict(kw, fused="next")
            name += " (exchange riding on the next step)"
        layout = W.LAYOUTS[kind]()
        cfg = RunConfig(segments=W.segments(layout), P=W.total_params(layout), **kw)
        t0 = time.time()
        inputs = (W.theta0_np(layout, 0), W.gaussian_pool_np(layout, cfg.K, 1, 1))
        h, ref, log = run_gaussian(cfg, binding, oracle, inputs, variant="omp")
        viol, bits = compare_state(h, ref, binding)
        ok = (sum(viol.values()) == 0 and log["masks_equal"] and log["weights_equal"]
              and log["norm2_equal"] and np.array_equal(h.ah_state_get(binding.AH_STEP), ref.step))
        print(f"{'PASS' if ok else 'FAIL'}  {name}: out of tolerance {viol}, bits differ {bits}, "
              f"masks/distances/weights identical {log['masks_equal']}/{log['norm2_equal']}/"
              f"{log['weights_equal']}, exchanges {log['exchanges']}, {time.time() - t0:.0f} s", flush=True)
        h.close()
        del h, ref, inputs
        torch.cuda.empty_cache()


if __name__ == "__main__":
    main()
