#!/usr/bin/env python
"""Throughput of the AdaHessian + elastic-averaging round on B200.

One *step* is one communication period of the whole hot path: tau local steps of all K
workers (Rademacher signs, Hutchinson diagonal, spatial average, moments, update), and
on the last of them the distances to the master, the dynamic weights, the failure mask
and the weighted elastic exchange.  The metric is parameter updates per second,
K * P * tau * steps / time, with the time taken on the device (CUDA events on the
library's stream, maximum over ranks).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c2|c1|c3|c4|c5k64|...]
    python bench.py --impl reference ...      # the CPU oracle on the host cores

With N > 1 (launched by torchrun) every rank runs an independent replica on its own
GPU: the path has no inter-GPU exchange step, so scaling is weak by construction.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

Z_SEED, MASK_SEED, ORDER_SEED, DATA_SEED = 0x5EED0001, 0x5EED0002, 0x5EED0003, 0

# name -> (layout, K, tau, p_fail, max_stale, frozen stragglers)
WORKLOADS = {
    "c1": ("quadratic", 4, 4, 0.0, 1, False),
    "c2": ("resnet18", 8, 4, 0.1, 1, False),
    "c3": ("resnet50", 16, 4, 0.2, 8, True),
    "c3tau1": ("resnet50", 16, 1, 0.2, 8, True),
    "c3tau16": ("resnet50", 16, 16, 0.2, 8, True),
    "c4": ("vgg16", 4, 8, 0.25, 1, False),
    "c5k4": ("resnet50", 4, 4, 0.1, 1, False),
    "c5k16": ("resnet50", 16, 4, 0.1, 1, False),
    "c5k32": ("resnet50", 32, 4, 0.1, 1, False),
    "c5k64": ("resnet50", 64, 4, 0.1, 1, False),
    # the paper's own setting (Sec. VI-VII): its small CNN, 4 or 8 workers, tau in {1, 2, 4},
    # communication suppressed one third of the time
    "paper_k4_tau4": ("mnist_cnn", 4, 4, 1 / 3, 1, False),
    "paper_k8_tau2": ("mnist_cnn", 8, 2, 1 / 3, 1, False),
    "paper_k8_tau1": ("mnist_cnn", 8, 1, 1 / 3, 1, False),
    # small cases for profiler captures (about 1 GB on the device, still far above L2)
    "p18k4": ("resnet18", 4, 4, 0.1, 1, False),
    "pvggk1": ("vgg16", 1, 4, 0.1, 1, False),
}
SGD_LR, SGD_MOMENTUM = 0.01, 0.5          # Sec. VII: eta = 0.01, delta = 0.5
HYPER = dict(lr=0.01, beta1=0.9, beta2=0.999, eps=1e-4, hessian_power=1.0, weight_decay=0.0)

# DRAM bytes per parameter update of the fused local-step kernel, from one ncu capture
# (dram__bytes_read.sum + dram__bytes_write.sum over the launch / (K * P)), and the hash
# of the kernel sources it was taken on.  Reported only while the sources are unchanged.
NCU_TRAFFIC = {"sources_sha256": "21071469eb7f9ec7492ef6ad7b891cfb7db13d8c4eedcac99e44209bd09dbf6d",
               "dram_bytes_per_update": (935_952_896 + 506_401_536) / 46_758_048,
               "capture": "one ncu capture of the plain local step on workload p18k4 (ResNet-18-shaped "
                          "layout, K=4, 46,758,048 updates per launch), scaled by the updates of this "
                          "run's launch: traffic is proportional to updates"}


def kernel_sources_hash() -> str:
    h = hashlib.sha256()
    for fn in ("ah_local_step.cuh", "ah_step_inst.cu", "ah_tree.cuh", "ah_weights.cuh", "ah_ln.cuh",
               "ah_internal.h", "ah_device.cuh"):
        with open(os.path.join(ROOT, "paper_2409_09242_b200", "csrc", fn), "rb") as f:
            h.update(f.read())
    return h.hexdigest()


def measured_hbm_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


def make_layout(kind):
    from paper_2409_09242_b200 import workloads as W
    if kind == "quadratic":
        return W.single_segment_layout(1 << 20)
    return W.LAYOUTS[kind]()


def alpha_for(K):
    return min(0.05, 0.8 / K)


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the GPU runs the bench.
    A reader thread stamps every sample with the host time, so that the samples that fall
    inside the timed region can be told from those taken during warm-up."""
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap,power.draw")
    NAMES = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")

    def __init__(self, index):
        self.index, self.proc, self.samples, self.thread = index, None, [], None

    def start(self):
        import threading
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.FIELDS,
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True, bufsize=1)
        except Exception:
            self.proc = None
            return

        def reader():
            for line in self.proc.stdout:
                parts = [p.strip() for p in line.split(",")]
                if len(parts) < 6:
                    continue
                try:
                    watts = None
                    if len(parts) > 6:
                        try:
                            watts = float(parts[6])
                        except ValueError:
                            pass
                    self.samples.append((time.time(), float(parts[0]), float(parts[1]),
                                         [n for n, v in zip(self.NAMES, parts[2:6])
                                          if v.lower().startswith("active")], watts))
                except ValueError:
                    continue
        self.thread = threading.Thread(target=reader, daemon=True)
        self.thread.start()

    def count(self, since=0.0):
        return sum(1 for s in self.samples if s[0] >= since)

    def stop(self, t_from, t_to, window):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "samples": 0,
                    "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        if self.thread is not None:
            self.thread.join(timeout=2)
        inside = [s for s in self.samples if t_from <= s[0] <= t_to]
        clocks = [s[1] for s in inside]
        reasons = sorted({r for s in inside for r in s[3]})
        watts = [s[4] for s in inside if s[4] is not None]
        return {"sm_mhz": statistics.median(clocks) if clocks else None,
                "sm_mhz_min": min(clocks) if clocks else None,
                "sm_mhz_max_seen": max(clocks) if clocks else None,
                "sm_max_mhz": inside[-1][2] if inside else None, "samples": len(clocks),
                "power_w": round(statistics.median(watts), 1) if watts else None,
                "window": window, "reasons": reasons}


class InputStager:
    """End-to-end leg: the inputs of every round come from pinned host memory.  Two device
    buffers and a copy stream: while round t computes from one buffer, the inputs of round
    t + 1 are copied into the other."""

    def __init__(self, host_pool, like, with_hvp):
        import torch
        self.host_pool, self.with_hvp = host_pool, with_hvp
        self.bufs = [(torch.empty_like(like[0]), torch.empty_like(like[1])) for _ in range(2)]
        self.copy_stream = torch.cuda.Stream()
        self.ready = [torch.cuda.Event() for _ in range(2)]      # copy into buffer b finished
        self.done = [torch.cuda.Event() for _ in range(2)]       # compute from buffer b finished
        self.issued_for = None                                   # round whose copy is in flight

    def _issue(self, t):
        import torch
        b = t % 2
        hg, hh = self.host_pool[t % len(self.host_pool)]
        with torch.cuda.stream(self.copy_stream):
            self.copy_stream.wait_event(self.done[b])            # the buffer's last reader is through
            self.bufs[b][0].copy_(hg, non_blocking=True)
            if self.with_hvp:
                self.bufs[b][1].copy_(hh, non_blocking=True)
            self.ready[b].record(self.copy_stream)

    def inputs(self, t):
        """Device inputs of round t (the compute stream waits for their copy), and the copy
        of round t + 1 started behind them."""
        import torch
        if self.issued_for != t:
            self._issue(t)
        torch.cuda.current_stream().wait_event(self.ready[t % 2])
        self._issue(t + 1)
        self.issued_for = t + 1
        return self.bufs[t % 2]

    def release(self, t):
        self.done[t % 2].record()                                # on the compute stream


def _spread(vals, keep=48):
    """Summary of the per-repetition times: extremes, deciles, and an evenly spaced sample
    of the values in run order (all of them when there are few)."""
    srt = sorted(vals)
    pick = lambda q: round(srt[min(len(srt) - 1, int(q * len(srt)))], 4)
    stride = max(1, -(-len(vals) // keep))
    return {"min": pick(0.0), "p10": pick(0.1), "median": round(statistics.median(vals), 4),
            "p90": pick(0.9), "max": round(srt[-1], 4),
            "in_run_order": [round(v, 4) for v in vals[::stride]]}


def max_over_ranks(ms, dist, device):
    """The slowest rank's time: what a multi-GPU number is quoted on."""
    if dist is None:
        return float(ms)
    import torch
    t = torch.tensor([float(ms)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_updates_per_second(updates_per_rank, world, ms):
    """G parameter updates per second over all replicas (every rank does the same work)."""
    return updates_per_rank * world / (ms * 1e-3) / 1e9


def run_period(h, pool, t0, wl, events=None, stage=None, asynchronous=False, ex_events=None,
               method="adahessian", sync_free=False, fused=False, carry=None):
    """One communication period starting after round t0.  With `stage` (an InputStager)
    the inputs of every round are first copied from pinned host memory (the end-to-end
    leg).  With `carry` (a dict kept by the caller) the exchange
    of a period is not launched at its end but rides on the first local step of the next
    period (one pass over x instead of two, same result).  Returns (next t0, worker-steps
    taken, workers that exchanged)."""
    import torch
    _, K, tau, p_fail, max_stale, frozen = wl
    alpha = alpha_for(K)
    worker_steps = exchanged = 0
    for r in range(tau):
        t = t0 + r + 1
        mask = h.dw_mask_next(MASK_SEED, t, p_fail, max_stale)
        ex = r == tau - 1
        if stage is not None:
            g, hv = stage.inputs(t)
        else:
            g, hv = pool[t % len(pool)]
        if events is not None:
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
        first_order = method != "adahessian"     # EASGD / EAMSGD: fixed alpha, no distances
        rode = False
        if first_order and carry is not None and carry.get("pending") is not None:
            rode = True
            p_mask, p_order = carry.pop("pending")
            h.easgd_exchange_then_sgd_step(g, SGD_LR, SGD_MOMENTUM if method == "msgd" else 0.0,
                                           active=mask if frozen else None, worker_mask=p_mask,
                                           alpha=alpha, order=p_order, asynchronous=asynchronous)
        elif first_order:
            h.sgd_local_step(g, SGD_LR, SGD_MOMENTUM if method == "msgd" else 0.0,
                             active=mask if frozen else None)
        elif carry is not None and carry.get("pending") is not None:
            rode = True
            p_mask, p_order = carry.pop("pending")
            h.easgd_exchange_then_step(g, hv, Z_SEED, round_=t, active=mask if frozen else None,
                                       worker_mask=p_mask, alpha=alpha, order=p_order,
                                       asynchronous=asynchronous, dynamic=True, **HYPER)
        elif fused and ex:
            # the whole exchange round in one pass; the rule's coefficients lag one period
            h.ah_local_step_exchange(g, hv, Z_SEED, round_=t, active=mask if frozen else None,
                                     want_dist=True, worker_mask=mask, alpha=alpha,
                                     order=h.dw_order_next(ORDER_SEED, t) if asynchronous else None,
                                     asynchronous=asynchronous, lagged=True, **HYPER)
        else:
            # a distance round whose exchange will take its weights from the device also asks
            # for the weighting rule (it runs where the distances are assembled: at the head
            # of the riding exchange, or in a small kernel of its own)
            rule = ex and (carry is not None or sync_free)
            h.ah_local_step(g, hv, Z_SEED, round_=t, active=mask if frozen else None,
                            want_dist=2 if rule else ex, rule_alpha=alpha,
                            **HYPER)      # hv is [K, ld], or [n, K, ld] with --samples n
        if stage is not None:
            stage.release(t)
        n_act = int(mask.sum()) if frozen else K
        worker_steps += n_act
        if events is not None:
            e1.record()
            events.append((e0, e1, 2 if rode else int(ex), n_act))
        if ex and carry is not None:
            carry["pending"] = (mask, h.dw_order_next(ORDER_SEED, t) if asynchronous else None)
            exchanged += int(mask.sum())
        elif ex and fused and not first_order:
            exchanged += int(mask.sum())
        elif ex:
            on_device = sync_free and not first_order      # weights computed on the device
            w = None if (first_order or on_device) else h.dw_weights_next(alpha)
            if ex_events is not None:
                x0, x1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                x0.record()
            order = h.dw_order_next(ORDER_SEED, t) if asynchronous else None
            if on_device:
                h.easgd_exchange_dynamic(mask, alpha, order, asynchronous)
            elif asynchronous:
                h.easgd_exchange_async(mask, w, alpha, order)
            else:
                h.easgd_exchange(mask, w, alpha)
            if ex_events is not None:
                x1.record()
                ex_events.append((x0, x1, int(mask.sum())))
            exchanged += int(mask.sum())
    return t0 + tau, worker_steps, exchanged


def gpu_arm(args):
    import torch
    from paper_2409_09242_b200 import binding, workloads as W

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1 or "TORCHELASTIC_RUN_ID" in os.environ:     # launched by torchrun: use its rendezvous
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    wl = WORKLOADS[args.workload]
    kind, K, tau, p_fail, max_stale, frozen = wl
    layout = make_layout(kind)
    segs, P = W.segments(layout), W.total_params(layout)
    ld = W.padded_ld(P)
    dev = torch.device("cuda", local_rank)

    # synthetic inputs, resident in HBM before the timed region
    pair_bytes = (1 + args.samples) * K * ld * 4
    n_pool = max(1, min(args.pool, int(24e9 // pair_bytes)))
    pool = [W.gaussian_pair_torch(layout, K, DATA_SEED + 1 + 1000 * r + rank, dev) for r in range(n_pool)]
    if args.samples > 1:         # n Hutchinson samples per step: hvp becomes [n, K, ld]
        pool = [(g, torch.stack([hv] + [W.gaussian_pair_torch(layout, K, DATA_SEED + 7 + 1000 * r + 50 * q
                                                              + rank, dev)[1]
                                        for q in range(1, args.samples)]))
                for r, (g, hv) in enumerate(pool)]
    h = binding.Handle(K, P, segs)
    h.ah_state_set(binding.AH_CENTER, W.theta0_torch(layout, DATA_SEED + rank, dev))
    h.ah_broadcast_center()

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    t = 0
    asyn = args.exchange == "async"
    # with a period of one round every step also measures distances, which cannot ride along
    # (with several Hutchinson samples the one-pass form fits fewer CTAs per SM and was
    # measured slower than the separate exchange kernel)
    ride = (args.exchange_pass == "next-step" and not args.fused and tau >= 2
            and (args.samples == 1 or args.method != "adahessian"))
    carry = {} if ride else None
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    run_kw = dict(asynchronous=asyn, method=args.method, sync_free=args.sync_free, fused=args.fused)
    warm_until = time.time() + 2.0
    done = 0
    w0, w1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    while done < args.warmup or (world == 1 and rank == 0 and sampler.proc is not None
                                 and sampler.count() == 0 and time.time() < warm_until):
        # at least the asked warm-up periods; a little longer until the clock sampler is live
        if done == args.warmup - 1:
            w0.record()                           # the last asked warm-up period is also timed:
        t, _, _ = run_period(h, pool, t, wl, carry=carry, **run_kw)
        if done == args.warmup - 1:
            w1.record()                           # it sizes the number of repetitions below
        done += 1
        if done >= args.warmup:
            torch.cuda.synchronize()
    est_ms = max(w0.elapsed_time(w1), 1e-3)
    # Repetitions: each is `--steps` periods, timed by its own pair of events; at least
    # --reps of them and as many as it takes to keep the device busy for --min-seconds (so
    # that the clocks settle where a long job runs them); the line reports the median.
    # Every rank must run the same count: the slowest rank's estimate decides.
    est_ms = max_over_ranks(est_ms, dist, dev)
    reps = max(args.reps, int(args.min_seconds * 1e3 / (est_ms * args.steps)) + 1)
    reps = min(reps, max(args.reps, 20000 // max(1, args.steps)))
    # per-launch event pairs perturb very short kernels: every rep while that stays below a
    # few thousand pairs, else every n-th rep (the median rep is then one without them)
    launches_per_rep = args.steps * tau
    bracket_every = max(1, -(-reps * launches_per_rep // 6000))
    barrier()
    wall0 = time.time()
    launches0 = h.ah_launch_count()
    events, ex_events = [], []
    bounds = [torch.cuda.Event(enable_timing=True)]
    bounds[0].record()
    rep_ws, rep_exd = [], []
    for rep in range(reps):
        ws_r = exd_r = 0
        ev = events if rep % bracket_every == 0 else None
        for _ in range(args.steps):
            t, ws, exd = run_period(h, pool, t, wl, ev, ex_events=ex_events if ev is not None else None,
                                    carry=carry, **run_kw)
            ws_r += ws
            exd_r += exd
        bounds.append(torch.cuda.Event(enable_timing=True))
        bounds[-1].record()
        rep_ws.append(ws_r)
        rep_exd.append(exd_r)
    barrier()
    wall1 = time.time()
    rep_ms = [bounds[r].elapsed_time(bounds[r + 1]) for r in range(reps)]
    launches = h.ah_launch_count() - launches0
    if carry is not None and carry.get("pending") is not None:
        # the last timed period's exchange would ride on the next step; the first timed
        # period carried the one before it.  Launch it now, outside the timed region.
        p_mask, p_order = carry.pop("pending")
        if args.method != "adahessian":
            (h.easgd_exchange_async(p_mask, None, alpha_for(K), p_order) if asyn
             else h.easgd_exchange(p_mask, None, alpha_for(K)))
        else:
            h.easgd_exchange_dynamic(p_mask, alpha_for(K), p_order, asyn)
    clocks = None
    if rank == 0:
        clocks = sampler.stop(wall0, wall1, "timed region")
    # the slowest rank's time, repetition by repetition; parameter updates actually
    # performed (a frozen straggler takes no step); the median repetition is the line's value
    rep_ms = [max_over_ranks(m, dist, dev) for m in rep_ms]
    rep_value = [whole_job_updates_per_second(w * P, world, m) for w, m in zip(rep_ws, rep_ms)]
    value = statistics.median(rep_value)
    ms = statistics.median(rep_ms)
    worker_steps, exchanged = sum(rep_ws), sum(rep_exd)
    total_ms = sum(rep_ms)

    # per-launch duration of the fused local-step kernel (plain rounds; the rounds that
    # also measure distances are listed beside it)
    plain = [(a.elapsed_time(b), n) for a, b, ex, n in events if ex == 0]
    withd = [(a.elapsed_time(b), n) for a, b, ex, n in events if ex == 1]
    rides = [a.elapsed_time(b) for a, b, ex, n in events if ex == 2]
    # algorithmic bytes of a launch: 32 per update; a distance round also reads the
    # master row once and the x of every worker that sat the step out
    bpu = {"adahessian": 28 + 4 * args.samples, "sgd": 12, "msgd": 20}[args.method]
    if args.method != "adahessian":
        dom, dom_name = plain + withd, "sgd_step"       # no distance rounds with a fixed alpha
        dom_bytes = sum(bpu * P * n for _, n in dom) / len(dom)
    elif plain:
        dom, dom_name = plain, "local_step"
        dom_bytes = sum(bpu * P * n for _, n in dom) / len(dom)
    else:
        dom, dom_name = withd, "local_step+dist"
        dom_bytes = sum(bpu * P * n + 4 * P * (K - n) + 4 * P for _, n in dom) / len(dom)
    # a launch's bytes depend on how many workers stepped: the median launch duration goes
    # with the mean bytes of the launches at or next to the median
    dom_ms = statistics.median(d for d, _ in dom)
    peak, peak_kind = measured_hbm_peak()
    achieved = dom_bytes / (dom_ms * 1e-3) / 1e9
    traffic = traffic_note = None
    if (args.method == "adahessian" and NCU_TRAFFIC["sources_sha256"] == kernel_sources_hash()
            and NCU_TRAFFIC["dram_bytes_per_update"] and args.samples == 1):
        traffic = NCU_TRAFFIC["dram_bytes_per_update"] * dom_bytes / 32.0
        traffic_note = NCU_TRAFFIC["capture"]
    roofline = {"bound": "hbm", "kernel": dom_name, "achieved": round(achieved, 1), "peak": peak,
                "peak_kind": peak_kind, "unit": "GB/s", "frac": round(achieved / peak, 4),
                "frac_of_nominal_8000": round(achieved / 8000.0, 4), "traffic": traffic,
                "traffic_source": traffic_note,
                "achieved_dram": round(traffic / (dom_ms * 1e-3) / 1e9, 1) if traffic else None,
                "ms_per_launch": round(dom_ms, 4), "launches_bracketed": len(dom),
                "algorithmic_bytes_per_launch": int(dom_bytes),
                "dist_round_ms": round(statistics.median(d for d, _ in withd), 4) if withd else None,
                "exchange_plus_step_ms": round(statistics.median(rides), 4) if rides else None}
    # whole-run bytes: 32 per update + (8 P per exchanging worker + 12 P) per exchange
    if (args.fused and args.method == "adahessian") or ride:
        # fused exchange rounds: x crosses HBM once; the master row is read and written once
        run_bytes = bpu * P * worker_steps + 8 * P * args.steps * reps
    else:
        run_bytes = (bpu * P * worker_steps + 8 * P * exchanged +
                     (12 if args.method == "adahessian" else 8) * P * args.steps * reps)
    whole = {"algorithmic_GBps": round(run_bytes / (total_ms * 1e-3) / 1e9, 1)}
    whole["frac_of_measured_peak"] = round(whole["algorithmic_GBps"] / peak, 4)
    # the exchange kernel alone: 8 bytes per (arriving worker, parameter) + 8 per parameter
    exl = [(a.elapsed_time(b), n) for a, b, n in ex_events if n > 0]
    exchange = None
    if exl:
        ex_ms = sum(d for d, _ in exl) / len(exl)
        ex_bytes = sum(8 * P * n + 8 * P for _, n in exl) / len(exl)
        exchange = {"kernel": "exchange_async" if asyn else "exchange", "ms_per_launch": round(ex_ms, 4),
                    "algorithmic_GBps": round(ex_bytes / (ex_ms * 1e-3) / 1e9, 1),
                    "note": "x was just written by the local step, part of it is still in L2"}

    # end-to-end leg: same periods, inputs copied from pinned host memory every round,
    # the distances/weights read back every period
    e2e = None
    if not args.no_e2e:
        n_host = 1 if pair_bytes > 4e9 else 2
        host_pool = [(g.cpu().pin_memory(), hv.cpu().pin_memory()) for g, hv in pool[:n_host]]
        stager = InputStager(host_pool, pool[0], args.method == "adahessian")
        e2e_steps = max(1, min(args.steps, int(20e9 // (pair_bytes * tau)) or 1))
        t, _, _ = run_period(h, pool, t, wl, stage=stager, asynchronous=asyn,
                             method=args.method)      # the end-to-end leg reads the weights back
        start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e2e_vals = []
        for _ in range(3):
            barrier()
            start.record()
            e2e_ws = 0
            for _ in range(e2e_steps):
                t, ws, _ = run_period(h, pool, t, wl, stage=stager, asynchronous=asyn,
                                      method=args.method)
                e2e_ws += ws
            stop.record()
            barrier()
            ems = max_over_ranks(start.elapsed_time(stop), dist, dev)
            e2e_vals.append(whole_job_updates_per_second(e2e_ws * P, world, ems))
        e2e_value = statistics.median(e2e_vals)
        e2e = {"value": round(e2e_value, 3),
               "unit": "G param-updates/s", "steps": e2e_steps, "reps": 3,
               "h2d_bytes_per_step": (pair_bytes if args.method == "adahessian" else K * ld * 4) * tau,
               "d2h_bytes_per_step": 8 * K if args.method == "adahessian" else 0}

    out = {
        "metric": "AdaHessian+EASGD round: param-updates/s (K x P per round)",
        "value": round(value, 3), "unit": "G param-updates/s", "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(ms / args.steps, 4),
        "reps": reps, "timed_seconds": round(total_ms * 1e-3, 3),
        "ms_per_step_reps": _spread([m / args.steps for m in rep_ms]),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
        "data": "synthetic", "impl": "cuda",
        "config": {"workload": f"{args.workload}: {kind} layout, P={P}, K={K}, tau={tau}, "
                               f"p_fail={p_fail}, max_stale={max_stale}, frozen_stragglers={frozen}",
                   "step": f"one communication period = {tau} rounds + 1 exchange",
                   "exchange": "asynchronous, seeded arrival order" if asyn else "simultaneous",
                   "local_step": {"adahessian": "AdaHessian, dynamic weights",
                                  "sgd": "SGD, fixed alpha (EASGD)",
                                  "msgd": "SGD with momentum 0.5, fixed alpha (EAMSGD)"}[args.method],
                   "hutchinson_samples": args.samples,
                   "exchange_rounds": "one pass (step + pull), weights one period behind" if args.fused
                                      else "the exchange rides on the next round's local step" if ride
                                      else "local step, then exchange kernel",
                   "weights": "on the device, no host wait" if args.sync_free else "on the host, one wait per period",
                   "timing": f"median of {reps} repetitions of {args.steps} periods, back to back",
                   "rounds_timed": tau * args.steps * reps, "input_pool": n_pool,
                   "worker_steps_timed": worker_steps, "of_possible": K * tau * args.steps * reps,
                   "l2": "per-round working set %.2f GB exceeds the 126 MB L2, no flush needed"
                         % ((32 * K * P) / 1e9) if 32 * K * P > 4 * 126e6 else
                         "working set comparable to L2: partly L2-resident, reported as is",
                   "parallelism": "replicas only" if world > 1 else "single GPU"},
        "roofline": roofline, "whole_step": whole, "exchange_kernel": exchange, "e2e": e2e, "gpu_launches": int(launches),
        "clocks": clocks,
    }
    if clocks and clocks.get("sm_mhz"):
        # time x clock: what the period costs in SM cycles, to read the clock dependence
        # off runs that the power cap held at different clocks
        out["clocks"]["ms_per_step_x_mhz"] = round(ms / args.steps * clocks["sm_mhz"], 1)
    h.close()
    del pool
    torch.cuda.empty_cache()
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        out["cpu_baseline"] = cpu_baseline(args, budget_s=12.0)
    if rank == 0:
        print(json.dumps(out))
    if dist is not None:
        dist.destroy_process_group()


def oracle_sample(args, max_params):
    """The bounded sample of the workload the oracle is timed on: the same K, tau,
    failure model and hyper-parameters, on the leading whole tensors of the layout up
    to about max_params parameters (all of it when it is smaller)."""
    from paper_2409_09242_b200 import workloads as W
    kind, K, tau, p_fail, max_stale, frozen = WORKLOADS[args.workload]
    layout = make_layout(kind)
    keep = []
    for tns in layout:
        if keep and tns.offset + tns.numel > max_params:
            break
        keep.append(tns)
    if len(keep) == 1 and keep[0].numel > max_params and len(keep[0].shape) == 1:
        keep = W.single_segment_layout(max_params)
    return keep, f"first {len(keep)} of {len(layout)} tensors, P={W.total_params(keep)} of {W.total_params(layout)}"


def oracle_periods(args, layout, periods, warm):
    """Runs warm + periods communication periods of the oracle; returns (seconds, K, P, tau,
    threads, worker-steps taken in the timed periods)."""
    import numpy as np
    from paper_2409_09242_b200 import workloads as W
    kind, K, tau, p_fail, max_stale, frozen = WORKLOADS[args.workload]
    threads = max(1, min(K, len(os.sched_getaffinity(0))))
    os.environ["OMP_NUM_THREADS"] = str(threads)
    import oracle
    segs, P = W.segments(layout), W.total_params(layout)
    pool = W.gaussian_pool_np(layout, K, 2, DATA_SEED + 1)
    if args.samples > 1:
        more = [W.gaussian_pool_np(layout, K, 2, DATA_SEED + 7 + 50 * q) for q in range(1, args.samples)]
        pool = [(g, np.ascontiguousarray(np.stack([hv] + [m[r][1] for m in more])))
                for r, (g, hv) in enumerate(pool)]
    st = oracle.OracleState(W.theta0_np(layout, DATA_SEED), K, segs, variant="omp")
    alpha = alpha_for(K)
    t, t_start, worker_steps, lagged = 0, None, 0, None
    for period in range(warm + periods):
        if period == warm:
            t_start = time.perf_counter()
        for r in range(tau):
            t += 1
            mask = st.mask_next(MASK_SEED, t, p_fail, max_stale)
            if period >= warm:
                worker_steps += int(mask.sum()) if frozen else K
            ex = r == tau - 1
            g, hv = pool[t % 2]
            if args.method == "adahessian":
                st.local_step(g, hv, Z_SEED, t, active=mask if frozen else None, want_dist=ex, **HYPER)
            else:
                st.sgd_step(g, SGD_LR, SGD_MOMENTUM if args.method == "msgd" else 0.0,
                            active=mask if frozen else None)
            if ex:
                if args.method != "adahessian":
                    h2, h1 = None, None
                elif args.fused:     # coefficients one period behind the distances
                    h2, h1 = lagged if lagged is not None else (None, None)
                    lagged = st.weights_next(alpha)
                else:
                    h2, h1 = st.weights_next(alpha)
                if args.exchange == "async":
                    st.exchange_async(mask, h2, h1, alpha=alpha, order=st.order_next(ORDER_SEED, t))
                else:
                    st.exchange(mask, h2, h1, alpha=alpha)
    return time.perf_counter() - t_start, K, P, tau, min(threads, st.o.num_threads()), worker_steps


def cpu_baseline(args, budget_s):
    """The CPU oracle, as it stands, timed on this host on a bounded sample."""
    layout, what = oracle_sample(args, max_params=4_000_000)
    sec, K, P, tau, threads, _ = oracle_periods(args, layout, periods=1, warm=1)
    periods = max(1, min(200, int(budget_s / max(sec, 1e-3))))
    sec, K, P, tau, threads, ws = oracle_periods(args, layout, periods=periods, warm=1)
    return {"value": round(ws * P / sec / 1e9, 5), "unit": "G param-updates/s",
            "cores": threads, "kind": "oracle",
            "sample": f"{what}; {periods} periods of {tau} rounds, {sec:.1f} s; OpenMP build, "
                      f"local steps parallel over workers ({threads} threads)"}


def reference_arm(args):
    """--impl reference: the oracle on the host cores, same metric and config."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    layout, what = oracle_sample(args, max_params=1_000_000)
    sec, K, P, tau, threads, ws = oracle_periods(args, layout, periods=args.steps, warm=args.warmup)
    value = round(ws * P / sec / 1e9, 5)
    kind = WORKLOADS[args.workload][0]
    print(json.dumps({
        "metric": "AdaHessian+EASGD round: param-updates/s (K x P per round)",
        "value": value, "unit": "G param-updates/s", "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": round(sec / args.steps * 1e3, 3),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
        "data": "synthetic", "impl": "reference",
        "config": {"workload": f"{args.workload}: {kind} layout, K={K}, tau={tau} ({what})",
                   "step": f"one communication period = {tau} rounds + 1 exchange"},
        "cpu_baseline": {"value": value, "unit": "G param-updates/s", "cores": threads,
                         "kind": "oracle", "sample": what},
        "e2e": {"value": value, "unit": "G param-updates/s", "h2d_bytes_per_step": 0,
                "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20, help="communication periods per repetition")
    ap.add_argument("--reps", type=int, default=5, help="least number of timed repetitions")
    ap.add_argument("--min-seconds", type=float, default=2.0,
                    help="repeat until the device has been busy this long (0: --reps alone)")
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--workload", default="c2", choices=sorted(WORKLOADS))
    ap.add_argument("--pool", type=int, default=4, help="grad/hvp pairs kept in HBM")
    ap.add_argument("--exchange", default="simultaneous", choices=["simultaneous", "async"],
                    help="all workers against the same master value, or one at a time")
    ap.add_argument("--method", default="adahessian", choices=["adahessian", "sgd", "msgd"],
                    help="local step: the paper's method, or the EASGD / EAMSGD comparison methods")
    ap.add_argument("--host-weights", dest="sync_free", action="store_false",
                    help="dynamic weights computed on the host (one wait per period) instead of "
                         "on the device; same bits either way")
    ap.add_argument("--exchange-pass", default="next-step", choices=["next-step", "separate"],
                    help="the exchange rides on the next round's local step (one pass over x, same "
                         "bits), or runs as a kernel of its own")
    ap.add_argument("--fused", action="store_true",
                    help="exchange rounds in one pass (step + pull), dynamic weights one period behind")
    ap.add_argument("--samples", type=int, default=1, help="Hutchinson samples per step (paper: 1)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "cuda" else args.warmup
    if args.impl == "reference":
        reference_arm(args)
    else:
        gpu_arm(args)


if __name__ == "__main__":
    main()
