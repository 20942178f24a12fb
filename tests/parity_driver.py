"""Drives the CUDA library and the CPU oracle through the same rounds on the same
seeded inputs, for the parity tests.  Holds no arithmetic of the method itself."""
from dataclasses import dataclass, field

import numpy as np

Z_SEED = 0x5EED0001
MASK_SEED = 0x5EED0002
ORDER_SEED = 0x5EED0003


@dataclass
class RunConfig:
    K: int
    segments: list
    P: int
    rounds: int
    tau: int
    p_fail: float = 0.0
    max_stale: int = 1
    frozen: bool = False            # a worker that is down also skips its local steps
    lr: float = 0.01
    beta1: float = 0.9
    beta2: float = 0.999
    eps: float = 1e-4
    hessian_power: float = 1.0
    weight_decay: float = 0.0
    alpha: float | None = None      # None: min(0.05, 0.8 / K)
    dynamic: bool = True            # dynamic weights (else fixed alpha)
    asynchronous: bool = False      # workers reach the master one at a time, seeded order
    sync_free: str = "no"           # "yes": weights on the device (easgd_exchange_dynamic);
                                    # "mixed": device and host forms of the rule alternate
    fused: str = "no"               # "next": the exchange rides on the next round's local step
                                    # (easgd_exchange_then_step; needs tau >= 2); or the
                                    # exchange round in one pass: "given" (coefficients known
                                    # before the step: alpha) or "lagged" (the rule's output
                                    # of the previous exchange round, kept on the device)
    method: str = "adahessian"      # local step: "adahessian", "sgd" or "msgd" (momentum)
    momentum: float = 0.5
    scripted: list = field(default_factory=list)
    pool: int = 3
    data_seed: int = 0
    wait_polls: int | None = None   # library setting: how long the CTAs that assemble the
                                    # distances wait for one another (0: each works alone)

    def alpha_value(self):
        return min(0.05, 0.8 / self.K) if self.alpha is None else self.alpha


def tolerance_violations(got, want):
    """Count of elements outside |got - want| <= 1e-6 + 1e-5 |want| (the parity bar)."""
    got = np.asarray(got, np.float64)
    want = np.asarray(want, np.float64)
    return int(np.count_nonzero(np.abs(got - want) > 1e-6 + 1e-5 * np.abs(want)))


def run_gaussian(cfg: RunConfig, binding, oracle_mod, layout_inputs, variant="omp", check_every=0):
    """Gaussian grad/hvp pool (configs shaped like the CNN layouts).  layout_inputs =
    (theta0, [(grad, hvp), ...]) as numpy arrays.  Returns (handle, oracle_state, log)."""
    import torch
    from paper_2409_09242_b200 import workloads as W

    theta0, pool = layout_inputs
    dev_pool = [(torch.from_numpy(g).cuda(), torch.from_numpy(h).cuda()) for g, h in pool]
    h = binding.Handle(cfg.K, cfg.P, cfg.segments)
    h.ah_state_set(binding.AH_CENTER, theta0)
    h.ah_broadcast_center()
    if cfg.wait_polls is not None:
        h.ah_set_wait_polls(cfg.wait_polls)
    ref = oracle_mod.OracleState(theta0, cfg.K, cfg.segments, variant=variant)
    alpha = cfg.alpha_value()
    log = {"weights_equal": True, "masks_equal": True, "norm2_equal": True, "orders_equal": True,
           "exchanges": 0}
    lagged_weights = pending = None
    for t in range(1, cfg.rounds + 1):
        mask_g = h.dw_mask_next(MASK_SEED, t, cfg.p_fail, cfg.max_stale)
        mask_o = ref.mask_next(MASK_SEED, t, cfg.p_fail, cfg.max_stale)
        mask_g = W.apply_scripted(mask_g, t, cfg.scripted)
        mask_o = ref.scripted_mask(mask_o, t, [(o["worker"], o["first"], o["last"]) for o in cfg.scripted])
        log["masks_equal"] &= bool(np.array_equal(mask_g, mask_o))
        ex = t % cfg.tau == 0
        k = t % len(pool)
        common = dict(lr=cfg.lr, beta1=cfg.beta1, beta2=cfg.beta2, eps=cfg.eps,
                      hessian_power=cfg.hessian_power, weight_decay=cfg.weight_decay,
                      want_dist=ex)
        if cfg.fused == "next":
            # the library defers each exchange to the local step of the following round; the
            # oracle exchanges at once.  States agree whenever no exchange is pending.
            if pending is not None:
                p_mask, p_order, p_h2, p_h1, p_norm2 = pending
                h.easgd_exchange_then_step(dev_pool[k][0], dev_pool[k][1], Z_SEED, round_=t,
                                           active=mask_g if cfg.frozen else None, worker_mask=p_mask,
                                           alpha=alpha, order=p_order, asynchronous=cfg.asynchronous,
                                           dynamic=cfg.dynamic,
                                           **{q: v for q, v in common.items() if q != "want_dist"})
                if cfg.dynamic:
                    w = h.ah_state_get(binding.AH_WEIGHTS)
                    log["weights_equal"] &= bool(np.array_equal(w[:cfg.K], p_h2) and
                                                 np.array_equal(w[cfg.K:], p_h1))
                if p_norm2 is not None:      # assembled at the head of the riding launch
                    log["norm2_equal"] &= bool(np.array_equal(h.ah_state_get(binding.AH_NORM2), p_norm2))
                pending = None
                assert not ex, "tau >= 2"
            else:
                # every other distance round also asks for the weighting rule (AH_DIST_AND_RULE,
                # the shape the benchmark times); the others leave that to the call that makes
                # the exchange
                rule_now = ex and cfg.dynamic and log["exchanges"] % 2 == 0
                h.ah_local_step(dev_pool[k][0], dev_pool[k][1], Z_SEED, round_=t,
                                active=mask_g if cfg.frozen else None,
                                **dict(common, want_dist=binding.AH_DIST_AND_RULE if rule_now else ex,
                                       rule_alpha=alpha))
            ref.local_step(pool[k][0], pool[k][1], Z_SEED, t,
                           active=mask_o if cfg.frozen else None, **common)
            if ex:
                log["exchanges"] += 1
                # Reading the distances now has them assembled by a kernel of their own; left
                # alone, the riding launch assembles them at its head.  Both ways are taken.
                look_now = log["exchanges"] % 3 == 0 or t == cfg.rounds
                if look_now:
                    log["norm2_equal"] &= bool(np.array_equal(h.ah_state_get(binding.AH_NORM2), ref.norm2))
                order_g = order_o = None
                if cfg.asynchronous:
                    order_g = h.dw_order_next(ORDER_SEED, t)
                    order_o = ref.order_next(ORDER_SEED, t)
                    log["orders_equal"] &= bool(np.array_equal(order_g, order_o))
                h2, h1 = ref.weights_next(alpha) if cfg.dynamic else (None, None)
                if cfg.asynchronous:
                    ref.exchange_async(mask_o, h2, h1, alpha=alpha, order=order_o)
                else:
                    ref.exchange(mask_o, h2, h1, alpha=alpha)
                pending = (mask_g, order_g, h2, h1, None if look_now else ref.norm2.copy())
                if t == cfg.rounds:                                  # nothing follows: exchange now
                    if cfg.dynamic:
                        h.easgd_exchange_dynamic(mask_g, alpha, order_g, cfg.asynchronous)
                    elif cfg.asynchronous:
                        h.easgd_exchange_async(mask_g, None, alpha, order_g)
                    else:
                        h.easgd_exchange(mask_g, None, alpha)
                    pending = None
            continue
        if cfg.fused != "no" and ex:
            # one pass: step, distances, pull.  The oracle takes the same steps one by one.
            log["exchanges"] += 1
            lag = cfg.fused == "lagged"
            order_g = order_o = None
            if cfg.asynchronous:
                order_g = h.dw_order_next(ORDER_SEED, t)
                order_o = ref.order_next(ORDER_SEED, t)
                log["orders_equal"] &= bool(np.array_equal(order_g, order_o))
            h.ah_local_step_exchange(dev_pool[k][0], dev_pool[k][1], Z_SEED, round_=t,
                                     active=mask_g if cfg.frozen else None, worker_mask=mask_g,
                                     alpha=alpha, order=order_g, asynchronous=cfg.asynchronous,
                                     lagged=lag, **dict(common, want_dist=lag or ex))
            ref.local_step(pool[k][0], pool[k][1], Z_SEED, t,
                           active=mask_o if cfg.frozen else None, **common)
            h2, h1 = lagged_weights if (lag and lagged_weights is not None) else (None, None)
            if cfg.asynchronous:
                ref.exchange_async(mask_o, h2, h1, alpha=alpha, order=order_o)
            else:
                ref.exchange(mask_o, h2, h1, alpha=alpha)
            # Looking at the distances or the coefficients now has them assembled by a kernel
            # of their own; left alone, the next lagged round does it at its head (what it
            # used then shows in the state).  Both ways are taken.
            look_now = not lag or log["exchanges"] % 2 == 0 or t + cfg.tau > cfg.rounds
            if look_now:
                log["norm2_equal"] &= bool(np.array_equal(h.ah_state_get(binding.AH_NORM2), ref.norm2))
            if lag:
                lagged_weights = ref.weights_next(alpha)            # serves the next exchange round
                if look_now:
                    w = h.ah_state_get(binding.AH_WEIGHTS)
                    log["weights_equal"] &= bool(np.array_equal(w[:cfg.K], lagged_weights[0]) and
                                                 np.array_equal(w[cfg.K:], lagged_weights[1]))
            continue
        # where the weights of this exchange come from: the device (the rule either owed by
        # the distance round or asked for by the exchange) or the host
        ex_index = log["exchanges"] + 1
        on_device = ex and cfg.dynamic and (cfg.sync_free == "yes" or
                                            (cfg.sync_free == "mixed" and ex_index % 2 == 1))
        rule_now = on_device and ex_index % 3 != 0
        if cfg.method == "adahessian":
            h.ah_local_step(dev_pool[k][0], dev_pool[k][1], Z_SEED, round_=t,
                            active=mask_g if cfg.frozen else None,
                            **dict(common, want_dist=binding.AH_DIST_AND_RULE if rule_now else ex,
                                   rule_alpha=alpha))
            ref.local_step(pool[k][0], pool[k][1], Z_SEED, t,
                           active=mask_o if cfg.frozen else None, **common)
        else:
            delta = cfg.momentum if cfg.method == "msgd" else 0.0
            h.sgd_local_step(dev_pool[k][0], cfg.lr, delta,
                             active=mask_g if cfg.frozen else None, want_dist=ex)
            ref.sgd_step(pool[k][0], cfg.lr, delta,
                         active=mask_o if cfg.frozen else None, want_dist=ex)
        if ex:
            log["exchanges"] += 1
            w = h2 = h1 = None
            order_g = order_o = None
            if cfg.asynchronous:
                order_g = h.dw_order_next(ORDER_SEED, t)
                order_o = ref.order_next(ORDER_SEED, t)
                log["orders_equal"] &= bool(np.array_equal(order_g, order_o))
            if cfg.dynamic:
                h2, h1 = ref.weights_next(alpha)
            if on_device:
                h.easgd_exchange_dynamic(mask_g, alpha, order_g, cfg.asynchronous)
                w = h.ah_state_get(binding.AH_WEIGHTS)
            elif cfg.dynamic:
                w = h.dw_weights_next(alpha)
            if cfg.dynamic:
                log["norm2_equal"] &= bool(np.array_equal(h.ah_state_get(binding.AH_NORM2), ref.norm2))
                log["weights_equal"] &= bool(np.array_equal(w[:cfg.K], h2) and
                                             np.array_equal(w[cfg.K:], h1))
            if cfg.asynchronous:
                if not on_device:
                    h.easgd_exchange_async(mask_g, w, alpha, order_g)
                ref.exchange_async(mask_o, h2, h1, alpha=alpha, order=order_o)
            else:
                if not on_device:
                    h.easgd_exchange(mask_g, w, alpha)
                ref.exchange(mask_o, h2, h1, alpha=alpha)
        if check_every and t % check_every == 0:
            assert tolerance_violations(h.ah_state_get(binding.AH_X), ref.x) == 0, t
    return h, ref, log


def compare_state(h, ref, binding):
    """(violations of the parity bar, count of bit differences) over x, m, v, center."""
    viol, bits = {}, {}
    for name, which, want in (("x", binding.AH_X, ref.x), ("m", binding.AH_M, ref.m),
                              ("v", binding.AH_V, ref.v), ("center", binding.AH_CENTER, ref.center)):
        got = h.ah_state_get(which)
        viol[name] = tolerance_violations(got, want)
        bits[name] = int(np.count_nonzero(got.view(np.uint32) != want.view(np.uint32)))
    return viol, bits
