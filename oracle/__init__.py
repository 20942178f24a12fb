"""CPU oracle for the AdaHessian + elastic-averaging round: TEST INFRASTRUCTURE.

A ctypes loader around ``ah_oracle.c`` (plain C, built with gcc).  Nothing in the
product package may import this module; it exists so that the tests, the smoke
check and the benchmark's CPU-baseline leg can compare the CUDA library against an
independent, slow, obviously correct implementation of the paper's equations.

Three builds of the same source:
  ``fp32``   single thread, binary32 canonical order (the parity authority)
  ``omp``    the same arithmetic, loops over independent workers/columns in OpenMP
  ``fp64``   arithmetic in double, state still binary32 (measures the drift of fp32)
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ah_oracle.c")
_OUT = os.path.join(_HERE, "_build")
_FLAGS = ["-std=c11", "-O2", "-ffp-contract=off", "-fno-fast-math", "-fPIC", "-shared",
          "-Wno-unknown-pragmas"]
_VARIANTS = {
    "fp32": [],
    "omp": ["-fopenmp"],
    "fp64": ["-DORC_DOUBLE", "-fopenmp"],
}
_lock = threading.Lock()
_libs: dict[str, "Oracle"] = {}


def build(force: bool = False) -> dict[str, str]:
    """Compile every variant of the oracle with gcc; returns {variant: path}."""
    os.makedirs(_OUT, exist_ok=True)
    out = {}
    for name, extra in _VARIANTS.items():
        so = os.path.join(_OUT, f"libah_oracle_{name}.so")
        if force or not os.path.exists(so) or os.path.getmtime(so) < os.path.getmtime(_SRC):
            tmp = so + f".{os.getpid()}.tmp"
            subprocess.check_call(["gcc", *_FLAGS, *extra, "-o", tmp, _SRC, "-lquadmath", "-lm"])
            os.replace(tmp, so)
        out[name] = so
    return out


class Segment(C.Structure):
    _fields_ = [("offset", C.c_uint64), ("length", C.c_uint64),
                ("block", C.c_uint32), ("flags", C.c_uint32)]


def _segarray(segments):
    arr = (Segment * max(1, len(segments)))()
    for k, s in enumerate(segments):
        arr[k] = Segment(int(s[0]), int(s[1]), int(s[2]), 0)
    return arr


def _f32(a):
    assert isinstance(a, np.ndarray) and a.dtype == np.float32 and a.flags.c_contiguous
    return a.ctypes.data_as(C.POINTER(C.c_float))


def _u8(a):
    if a is None:
        return None
    assert a.dtype == np.uint8 and a.flags.c_contiguous
    return a.ctypes.data_as(C.POINTER(C.c_uint8))


class Oracle:
    """One loaded variant of the oracle library, with numpy-typed entry points."""

    def __init__(self, variant: str = "fp32"):
        path = build()[variant]
        self.variant = variant
        self.lib = L = C.CDLL(path)
        pf, pd, pu8, pu32 = (C.POINTER(C.c_float), C.POINTER(C.c_double),
                             C.POINTER(C.c_uint8), C.POINTER(C.c_uint32))
        ps = C.POINTER(Segment)
        L.orc_philox4x32_10.argtypes = [pu32, pu32, pu32]
        L.orc_philox4x32_10.restype = None
        L.orc_sample_z.argtypes = [C.c_uint64, C.c_uint32, C.c_int, C.c_uint64, pf, C.c_uint64]
        L.orc_sample_z.restype = None
        L.orc_sample_zbits.argtypes = [C.c_uint64, C.c_uint32, C.c_int, C.c_uint64, pu8]
        L.orc_sample_zbits.restype = None
        L.orc_spatial_average.argtypes = [pf, C.c_uint64, ps, C.c_int, pf]
        L.orc_spatial_average.restype = None
        L.orc_local_step.argtypes = [pf, pf, pf, pu32, pf, pf, C.c_int, C.c_uint64, C.c_uint64,
                                     ps, C.c_int, C.c_uint64, C.c_uint32,
                                     C.c_float, C.c_float, C.c_float, C.c_float, C.c_float,
                                     C.c_float, pu8]
        L.orc_local_step.restype = C.c_int
        L.orc_local_step_n.argtypes = [pf, pf, pf, pu32, pf, pf, C.c_int, C.c_uint64, C.c_int,
                                       C.c_uint64, C.c_uint64, ps, C.c_int, C.c_uint64, C.c_uint32,
                                       C.c_float, C.c_float, C.c_float, C.c_float, C.c_float,
                                       C.c_float, pu8]
        L.orc_local_step_n.restype = C.c_int
        L.orc_sample_z_s.argtypes = [C.c_uint64, C.c_uint32, C.c_uint32, C.c_int, C.c_uint64, pf,
                                     C.c_uint64]
        L.orc_sample_z_s.restype = None
        L.orc_norm2.argtypes = [pf, pf, C.c_int, C.c_uint64, pd]
        L.orc_norm2.restype = None
        L.orc_ln.argtypes = [C.c_double]
        L.orc_ln.restype = C.c_double
        L.orc_u_from_norm2.argtypes = [C.c_double]
        L.orc_u_from_norm2.restype = C.c_double
        for f in (L.orc_h1, L.orc_h2):
            f.argtypes = [C.c_double, C.c_double, C.c_double]
            f.restype = C.c_double
        L.orc_weights_next.argtypes = [pd, C.POINTER(C.c_int), C.c_int, C.c_int, pd, C.c_double,
                                       C.c_float, pd, pf, pf, pd]
        L.orc_weights_next.restype = None
        L.orc_mask_next.argtypes = [pu32, C.c_int, C.c_uint64, C.c_uint32, C.c_double, C.c_int, pu8]
        L.orc_mask_next.restype = None
        L.orc_exchange.argtypes = [pf, pf, C.c_int, C.c_uint64, pu8, pf, pf]
        L.orc_exchange.restype = None
        pu16 = C.POINTER(C.c_uint16)
        L.orc_exchange_async.argtypes = [pf, pf, C.c_int, C.c_uint64, pu8, pf, pf, pu16, C.c_int]
        L.orc_exchange_async.restype = None
        L.orc_order_next.argtypes = [C.c_int, C.c_uint64, C.c_uint32, pu16]
        L.orc_order_next.restype = None
        L.orc_sgd_step.argtypes = [pf, pf, pu32, pf, C.c_int, C.c_uint64, C.c_uint64, C.c_float,
                                   C.c_float, pu8]
        L.orc_sgd_step.restype = None
        L.orc_partition.argtypes = [C.c_uint64, C.c_uint64, C.c_uint32, C.c_uint64, pu32,
                                    C.POINTER(C.c_uint64)]
        L.orc_partition.restype = C.c_int
        L.orc_is_double.restype = C.c_int
        L.orc_num_threads.restype = C.c_int

    # ---- S1 ---------------------------------------------------------------
    def philox(self, ctr, key):
        c = (C.c_uint32 * 4)(*[int(v) & 0xffffffff for v in ctr])
        k = (C.c_uint32 * 2)(*[int(v) & 0xffffffff for v in key])
        o = (C.c_uint32 * 4)()
        self.lib.orc_philox4x32_10(c, k, o)
        return [int(v) for v in o]

    def sample_z(self, seed, t, K, P):
        z = np.empty((K, P), np.float32)
        self.lib.orc_sample_z(seed, t, K, P, _f32(z), P)
        return z

    def sample_z_s(self, seed, t, sample, K, P):
        z = np.empty((K, P), np.float32)
        self.lib.orc_sample_z_s(seed, t, sample, K, P, _f32(z), P)
        return z

    def sample_zbits(self, seed, t, K, P):
        b = np.empty((K, P), np.uint8)
        self.lib.orc_sample_zbits(seed, t, K, P, _u8(b))
        return b

    # ---- a3 ---------------------------------------------------------------
    def spatial_average(self, d, segments):
        d = np.ascontiguousarray(d, np.float32)
        out = np.empty_like(d)
        self.lib.orc_spatial_average(_f32(d), d.size, _segarray(segments), len(segments), _f32(out))
        return out

    # ---- S3 / S6 ------------------------------------------------------------
    def norm2(self, x, c):
        K, P = x.shape
        n2 = np.empty(K, np.float64)
        self.lib.orc_norm2(_f32(x), _f32(c), K, P, n2.ctypes.data_as(C.POINTER(C.c_double)))
        return n2

    def ln(self, x):
        return self.lib.orc_ln(float(x))

    def u_from_norm2(self, n2):
        return self.lib.orc_u_from_norm2(float(n2))

    def h1(self, a, alpha, kappa):
        return self.lib.orc_h1(a, alpha, kappa)

    def h2(self, a, alpha, kappa):
        return self.lib.orc_h2(a, alpha, kappa)

    def exchange(self, x, xc, mask, h2, h1):
        K, P = x.shape
        self.lib.orc_exchange(_f32(x), _f32(xc), K, P, _u8(mask), _f32(h2), _f32(h1))

    def exchange_async(self, x, xc, mask, h2, h1, order=None):
        K, P = x.shape
        n, po = 0, None
        if order is not None:
            order = np.ascontiguousarray(order, np.uint16)
            n, po = order.size, order.ctypes.data_as(C.POINTER(C.c_uint16))
        self.lib.orc_exchange_async(_f32(x), _f32(xc), K, P, _u8(mask), _f32(h2), _f32(h1), po, n)

    def order_next(self, K, seed, t):
        order = np.empty(K, np.uint16)
        self.lib.orc_order_next(K, int(seed), int(t), order.ctypes.data_as(C.POINTER(C.c_uint16)))
        return order

    def partition(self, seed, n, k, o):
        """Data-overlap partition: (perm[n], bounds[k + 2]); O = perm[:o],
        S_j = perm[bounds[j + 1]:bounds[j + 2]]."""
        perm = np.empty(max(n, 1), np.uint32)
        bounds = np.empty(k + 2, np.uint64)
        rc = self.lib.orc_partition(int(seed), int(n), int(k), int(o),
                                    perm.ctypes.data_as(C.POINTER(C.c_uint32)),
                                    bounds.ctypes.data_as(C.POINTER(C.c_uint64)))
        if rc != 0:
            raise ValueError("partition: need o <= n and k >= 1")
        return perm[:n], bounds

    def num_threads(self):
        return int(self.lib.orc_num_threads())


def load(variant: str = "fp32") -> Oracle:
    with _lock:
        if variant not in _libs:
            _libs[variant] = Oracle(variant)
        return _libs[variant]


DEFAULT_C = (0.4, 0.3, 0.2, 0.1)   # history coefficients: sum to 1, recent terms heavier
DEFAULT_KAPPA = -0.1               # threshold of h1/h2 (must be negative)


class OracleState:
    """State of K simulated workers plus the master, and the round driver.

    Follows the paper's set-up (Sec. II): one master, K workers that all start as
    copies of the master's parameters.  One *round* = one local AdaHessian step of
    every active worker; every tau-th round the workers also exchange with the
    master (Sec. VI, communication period tau).
    """

    def __init__(self, center0, K, segments, variant="fp32", p_hist=4, c=DEFAULT_C,
                 kappa=DEFAULT_KAPPA):
        self.o = load(variant)
        self.K = int(K)
        self.P = int(center0.size)
        self.segments = [tuple(int(v) for v in s) for s in segments]
        self._segs = _segarray(self.segments)
        self.center = np.ascontiguousarray(center0, np.float32).copy()
        self.x = np.ascontiguousarray(np.broadcast_to(self.center, (self.K, self.P))).copy()
        self.m = np.zeros((self.K, self.P), np.float32)
        self.v = np.zeros((self.K, self.P), np.float32)
        self.step = np.zeros(self.K, np.uint32)
        self.p_hist = int(p_hist)
        self.c = np.asarray(c, np.float64).copy()
        assert self.c.size == self.p_hist
        self.kappa = float(kappa)
        self.uhist = np.zeros((self.K, self.p_hist + 1), np.float64)
        self.filled = C.c_int(0)
        self.down_until = np.zeros(self.K, np.uint32)
        self.norm2 = np.zeros(self.K, np.float64)
        self.last_a = np.zeros(self.K, np.float64)

    # S2
    def local_step(self, grad, hvp, z_seed, t, lr, beta1=0.9, beta2=0.999, eps=1e-4,
                   hessian_power=1.0, weight_decay=0.0, active=None, want_dist=False):
        """hvp: [K, ld] for one Hutchinson sample, or [n, K, ld] for n samples."""
        assert grad.dtype == np.float32 and hvp.dtype == np.float32
        assert grad.shape[0] == self.K and grad.flags.c_contiguous and hvp.flags.c_contiguous
        ld = grad.shape[1]
        n = 1 if hvp.ndim == 2 else hvp.shape[0]
        assert hvp.shape[-2:] == grad.shape
        if active is not None:
            active = np.ascontiguousarray(active, np.uint8)
        rc = self.o.lib.orc_local_step_n(
            _f32(self.x), _f32(self.m), _f32(self.v),
            self.step.ctypes.data_as(C.POINTER(C.c_uint32)), _f32(grad), _f32(hvp),
            n, self.K * ld, self.K, self.P, ld, self._segs, len(self.segments), int(z_seed), int(t),
            lr, beta1, beta2, eps, hessian_power, weight_decay, _u8(active))
        if rc != 0:
            raise MemoryError("oracle scratch allocation failed")
        if want_dist:
            self.norm2 = self.o.norm2(self.x, self.center)

    # first-order local steps (EASGD / EAMSGD): the velocity lives in self.m
    def sgd_step(self, grad, lr, momentum=0.0, active=None, want_dist=False):
        assert grad.dtype == np.float32 and grad.shape[0] == self.K and grad.flags.c_contiguous
        if active is not None:
            active = np.ascontiguousarray(active, np.uint8)
        self.o.lib.orc_sgd_step(_f32(self.x), _f32(self.m),
                                self.step.ctypes.data_as(C.POINTER(C.c_uint32)), _f32(grad),
                                self.K, self.P, grad.shape[1], lr, momentum, _u8(active))
        if want_dist:
            self.norm2 = self.o.norm2(self.x, self.center)

    # S4
    def weights_next(self, alpha):
        h2 = np.empty(self.K, np.float32)
        h1 = np.empty(self.K, np.float32)
        pd = C.POINTER(C.c_double)
        self.o.lib.orc_weights_next(
            self.uhist.ctypes.data_as(pd), C.byref(self.filled), self.K, self.p_hist,
            self.c.ctypes.data_as(pd), self.kappa, alpha, self.norm2.ctypes.data_as(pd),
            _f32(h2), _f32(h1), self.last_a.ctypes.data_as(pd))
        return h2, h1

    # S5
    def mask_next(self, seed, t, p_fail, max_stale=1):
        mask = np.empty(self.K, np.uint8)
        self.o.lib.orc_mask_next(self.down_until.ctypes.data_as(C.POINTER(C.c_uint32)), self.K,
                                 int(seed), int(t), float(p_fail), int(max_stale), _u8(mask))
        return mask

    # scripted outages (the configuration with "worker 3 down in rounds 20 to 40"): a worker
    # listed as (worker, first, last) cannot reach the master in rounds first..last inclusive
    @staticmethod
    def scripted_mask(mask, t, outages):
        down = {w for w, first, last in outages if first <= t <= last}
        return np.array([0 if i in down else int(b) for i, b in enumerate(mask)], np.uint8)

    # S6
    def exchange(self, mask=None, h2=None, h1=None, alpha=0.0):
        if h2 is None:
            h2 = np.full(self.K, alpha, np.float32)
            h1 = np.full(self.K, alpha, np.float32)
        if mask is not None:
            mask = np.ascontiguousarray(mask, np.uint8)
        self.o.exchange(self.x, self.center, mask, np.ascontiguousarray(h2, np.float32),
                        np.ascontiguousarray(h1, np.float32))

    # asynchronous form of S6: workers arrive one at a time in `order`
    def exchange_async(self, mask=None, h2=None, h1=None, alpha=0.0, order=None):
        if h2 is None:
            h2 = np.full(self.K, alpha, np.float32)
            h1 = np.full(self.K, alpha, np.float32)
        if mask is not None:
            mask = np.ascontiguousarray(mask, np.uint8)
        self.o.exchange_async(self.x, self.center, mask, np.ascontiguousarray(h2, np.float32),
                              np.ascontiguousarray(h1, np.float32), order)

    def order_next(self, seed, t):
        return self.o.order_next(self.K, seed, t)
