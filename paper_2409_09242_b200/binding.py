"""ctypes binding of the C-ABI CUDA library declared in include/adahess.h.

Argument marshalling only: every step of the round runs in the library's kernels.
PyTorch supplies device memory (the workspace and the input tensors) and the
stream.  The module-level functions carry the C names; ``Handle`` wraps one
``ah_ctx`` with the same calls as methods.  Without the built library the import
fails: there is no fallback path.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

from . import build as _build

if not os.path.exists(_build.LIB_PATH):
    raise ImportError(
        f"{_build.LIB_PATH} is missing: build it with `python -m paper_2409_09242_b200.build` "
        "(nvcc, sm_100a); this package has no CPU fallback")

_lib = C.CDLL(_build.LIB_PATH)

AH_OK = 0
AH_ERR_INVALID_ARG, AH_ERR_ALIGN, AH_ERR_SEGMENTS, AH_ERR_ALLOC = -1, -2, -3, -4
AH_ERR_CUDA, AH_ERR_STATE, AH_ERR_INTERNAL, AH_ERR_TOO_LARGE = -5, -6, -7, -8
AH_STATIC_SCRATCH_ENTRIES = 1 << 17
AH_MAX_WORKERS, AH_MAX_BLOCK, AH_MAX_HIST, AH_MAX_SAMPLES = 256, 128, 32, 8
AH_ROUND_AUTO = 0xFFFFFFFF
AH_DEVICE_NONE = -2
AH_DIST_NONE, AH_DIST, AH_DIST_AND_RULE = 0, 1, 2
(AH_X, AH_M, AH_V, AH_CENTER, AH_NORM2, AH_STEP, AH_UHIST, AH_DOWN_UNTIL, AH_ROUND,
 AH_INFO, AH_RUNS, AH_TILES, AH_WEIGHTS) = range(13)

EXPORTS = ["ah_workspace_bytes", "ah_init", "ah_destroy", "ah_state_set", "ah_state_get",
           "ah_broadcast_center", "ah_sample_z", "ah_sample_z_n", "ah_local_step",
           "ah_local_step_exchange", "easgd_exchange_then_step", "dw_config",
           "dw_weights_next", "dw_weights_from_norm2", "dw_mask_next", "easgd_exchange",
           "dw_order_next", "easgd_exchange_async", "easgd_exchange_dynamic", "sgd_local_step", "easgd_exchange_then_sgd_step", "dw_partition", "ah_distances_static", "ah_check_exact_arithmetic", "ah_set_wait_polls", "ah_status_string",
           "ah_last_cuda_error", "ah_launch_count"]


class ah_segment(C.Structure):
    _fields_ = [("offset", C.c_uint64), ("length", C.c_uint64),
                ("block", C.c_uint32), ("flags", C.c_uint32)]


class ah_hyper(C.Structure):
    _fields_ = [("lr", C.c_float), ("beta1", C.c_float), ("beta2", C.c_float),
                ("eps", C.c_float), ("hessian_power", C.c_float), ("weight_decay", C.c_float),
                ("round", C.c_uint32), ("active", C.POINTER(C.c_uint8)), ("want_dist", C.c_int),
                ("n_samples", C.c_int), ("hvp_sample_stride", C.c_uint64), ("rule_alpha", C.c_float)]


class sgd_hyper(C.Structure):
    _fields_ = [("lr", C.c_float), ("momentum", C.c_float), ("active", C.POINTER(C.c_uint8)),
                ("want_dist", C.c_int)]


class ah_alloc(C.Structure):
    _fields_ = [("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t),
                ("cuda_stream", C.c_void_p), ("device", C.c_int)]


_vp = C.c_void_p
_lib.ah_workspace_bytes.argtypes = [C.c_int, C.c_uint64, C.c_int, C.POINTER(C.c_size_t)]
_lib.ah_init.argtypes = [C.POINTER(_vp), C.c_int, C.c_uint64, C.POINTER(ah_segment), C.c_int,
                         C.POINTER(ah_alloc)]
_lib.ah_destroy.argtypes = [_vp]
_lib.ah_state_set.argtypes = [_vp, C.c_int, C.c_int, _vp, C.c_int]
_lib.ah_state_get.argtypes = [_vp, C.c_int, C.c_int, _vp, C.c_int]
_lib.ah_broadcast_center.argtypes = [_vp]
_lib.ah_sample_z.argtypes = [_vp, C.c_uint64, C.c_uint32, _vp, C.c_uint64]
_lib.ah_local_step_exchange.argtypes = [_vp, _vp, _vp, C.c_uint64, C.c_uint64, C.POINTER(ah_hyper),
                                        C.POINTER(C.c_uint8), C.POINTER(C.c_float), C.c_float,
                                        C.POINTER(C.c_uint16), C.c_int, C.c_int]
_lib.easgd_exchange_then_step.argtypes = _lib.ah_local_step_exchange.argtypes
_lib.ah_sample_z_n.argtypes = [_vp, C.c_uint64, C.c_uint32, C.c_uint32, _vp, C.c_uint64]
_lib.ah_local_step.argtypes = [_vp, _vp, _vp, C.c_uint64, C.c_uint64, C.POINTER(ah_hyper)]
_lib.dw_config.argtypes = [_vp, C.c_int, C.POINTER(C.c_double), C.c_double]
_lib.dw_weights_next.argtypes = [_vp, C.c_float, C.POINTER(C.c_float)]
_lib.dw_weights_from_norm2.argtypes = [_vp, C.POINTER(C.c_double), C.c_float, C.POINTER(C.c_float)]
_lib.dw_mask_next.argtypes = [_vp, C.c_uint64, C.c_uint32, C.c_double, C.c_int,
                              C.POINTER(C.c_uint8)]
_lib.easgd_exchange.argtypes = [_vp, C.POINTER(C.c_uint8), C.POINTER(C.c_float), C.c_float]
_lib.sgd_local_step.argtypes = [_vp, _vp, C.c_uint64, C.POINTER(sgd_hyper)]
_lib.easgd_exchange_then_sgd_step.argtypes = [_vp, _vp, C.c_uint64, C.POINTER(sgd_hyper),
                                              C.POINTER(C.c_uint8), C.POINTER(C.c_float), C.c_float,
                                              C.POINTER(C.c_uint16), C.c_int]
_lib.dw_partition.argtypes = [C.c_uint64, C.c_uint64, C.c_uint32, C.c_uint64, C.POINTER(C.c_uint32),
                              C.POINTER(C.c_uint64)]
_lib.dw_order_next.argtypes = [_vp, C.c_uint64, C.c_uint32, C.POINTER(C.c_uint16)]
_lib.easgd_exchange_async.argtypes = [_vp, C.POINTER(C.c_uint8), C.POINTER(C.c_float), C.c_float,
                                      C.POINTER(C.c_uint16)]
_lib.easgd_exchange_dynamic.argtypes = [_vp, C.POINTER(C.c_uint8), C.c_float, C.POINTER(C.c_uint16),
                                        C.c_int]
_lib.ah_distances_static.argtypes = [_vp, C.c_uint64, _vp, C.c_int, C.c_uint64, _vp, _vp]
_lib.ah_check_exact_arithmetic.argtypes = [C.c_uint64, C.POINTER(C.c_uint64), _vp]
_lib.ah_set_wait_polls.argtypes = [_vp, C.c_uint32]
_lib.ah_status_string.argtypes = [C.c_int]
_lib.ah_status_string.restype = C.c_char_p
_lib.ah_last_cuda_error.argtypes = [_vp]
_lib.ah_launch_count.argtypes = [_vp]
_lib.ah_launch_count.restype = C.c_uint64
for _n in EXPORTS:
    if _n not in ("ah_status_string", "ah_launch_count"):
        getattr(_lib, _n).restype = C.c_int


class AdaHessError(RuntimeError):
    def __init__(self, status, where, cuda=0):
        self.status = status
        msg = f"{where}: {ah_status_string(status)} ({status})"
        if cuda:
            msg += f", cudaError {cuda}"
        super().__init__(msg)


# ---- the C names, unchanged ------------------------------------------------------
def ah_status_string(status: int) -> str:
    return _lib.ah_status_string(int(status)).decode()


def ah_workspace_bytes(K: int, P: int, nseg: int) -> int:
    out = C.c_size_t(0)
    rc = _lib.ah_workspace_bytes(K, P, nseg, C.byref(out))
    if rc != AH_OK:
        raise AdaHessError(rc, "ah_workspace_bytes")
    return int(out.value)


def _segments(segments):
    arr = (ah_segment * max(1, len(segments)))()
    for k, s in enumerate(segments):
        arr[k] = ah_segment(int(s[0]), int(s[1]), int(s[2]), 0)
    return arr


def ah_distances_static(x, c, norm2_out, stream=None):
    """||x_i - c||^2 for raw tensors, no handle, no allocation inside the library.

    x: float32 CUDA tensor [K, ld] (rows contiguous), c: float32 CUDA tensor with at
    least P = x.shape[1] entries (padded to a multiple of 4), norm2_out: float64 CUDA
    tensor [K], written asynchronously on `stream` (default: torch's current stream).
    The caller provides every buffer, the output included."""
    import torch
    K, P = x.shape
    if norm2_out.dtype != torch.float64 or not norm2_out.is_cuda or norm2_out.numel() < K:
        raise TypeError("norm2_out: float64 CUDA tensor of K entries")
    if stream is None:
        stream = torch.cuda.current_stream(x.device).cuda_stream
    rc = _lib.ah_distances_static(_dev_ptr(x, "x"), x.stride(0), _dev_ptr(c, "c"), int(K), int(P),
                                  norm2_out.data_ptr(), stream)
    if rc != AH_OK:
        raise AdaHessError(rc, "ah_distances_static")
    return norm2_out


def ah_check_exact_arithmetic(division_pairs=1 << 32, stream=None):
    """Mismatch counts (square root, refined reciprocal, quotient) of the kernels' branch-free
    exact routines against the IEEE routines on the current device; all must be zero."""
    import torch
    if stream is None:
        stream = torch.cuda.current_stream().cuda_stream
    out = (C.c_uint64 * 3)()
    rc = _lib.ah_check_exact_arithmetic(int(division_pairs), out, stream)
    if rc != AH_OK:
        raise AdaHessError(rc, "ah_check_exact_arithmetic")
    return [int(v) for v in out]


def dw_partition(seed, n, k, shared):
    """Data-overlap partition: returns (perm[n] uint32, bounds[k + 2] uint64); the shared
    subset is perm[:shared], worker j's own subset perm[bounds[j + 1]:bounds[j + 2]]."""
    perm = np.empty(max(int(n), 1), np.uint32)
    bounds = np.empty(int(k) + 2, np.uint64)
    rc = _lib.dw_partition(int(seed), int(n), int(k), int(shared),
                           perm.ctypes.data_as(C.POINTER(C.c_uint32)),
                           bounds.ctypes.data_as(C.POINTER(C.c_uint64)))
    if rc != AH_OK:
        raise AdaHessError(rc, "dw_partition")
    return perm[:int(n)], bounds


def raw():
    """The loaded ctypes library (for tests of the bare ABI)."""
    return _lib


def _dev_ptr(t, name):
    """Device pointer of a contiguous float32 CUDA tensor."""
    import torch
    if not (isinstance(t, torch.Tensor) and t.is_cuda and t.dtype == torch.float32):
        raise TypeError(f"{name}: expected a float32 CUDA tensor")
    if t.dim() == 2 and t.stride(1) != 1:
        raise ValueError(f"{name}: rows must be contiguous")
    return t.data_ptr()


def _hvp_samples(grad, hvp):
    """(n_samples, sample stride) of hvp given as [K, ld] or as [n, K, ld]."""
    if hvp.dim() == 3:
        if hvp.stride(2) != 1 or hvp.shape[1:] != grad.shape or hvp.stride(1) != grad.stride(0):
            raise ValueError("hvp: [n, K, ld] with the shape and row stride of grad")
        return int(hvp.shape[0]), int(hvp.stride(0))
    if grad.shape != hvp.shape or grad.stride(0) != hvp.stride(0):
        raise ValueError("grad and hvp must share shape and row stride")
    return 1, 0


class Handle:
    """One ``ah_ctx``: K workers of P parameters on the current CUDA device.

    The workspace is a torch uint8 tensor (so torch's allocator owns the memory)
    and kernels run on torch's current stream at construction time.
    """

    def __init__(self, K, P, segments=(), device=None, own_alloc=False, host_only=False):
        self.K, self.P = int(K), int(P)
        self._ws = None
        self._h = _vp(None)
        if host_only:
            # bookkeeping-only handle (AH_DEVICE_NONE): weights and masks, no GPU state
            self._opt = ah_alloc(None, 0, None, AH_DEVICE_NONE)
            rc = _lib.ah_init(C.byref(self._h), self.K, self.P, _segments(list(segments)),
                              len(segments), C.byref(self._opt))
            if rc != AH_OK:
                self._h = _vp(None)
                raise AdaHessError(rc, "ah_init")
            return
        import torch
        if not torch.cuda.is_available():
            raise RuntimeError("no CUDA device: this library has no CPU path")
        self.device = torch.device("cuda", torch.cuda.current_device()) if device is None \
            else torch.device(device)
        segs = _segments(list(segments))
        self._h = _vp(None)
        if own_alloc:
            self._ws = None
            opt = None
        else:
            nbytes = ah_workspace_bytes(self.K, self.P, len(segments))
            with torch.cuda.device(self.device):
                self._ws = torch.empty(nbytes + 256, dtype=torch.uint8, device=self.device)
                stream = torch.cuda.current_stream(self.device).cuda_stream
            base = (self._ws.data_ptr() + 255) // 256 * 256
            self._opt = ah_alloc(base, nbytes, stream, self.device.index or 0)
            opt = C.byref(self._opt)
        rc = _lib.ah_init(C.byref(self._h), self.K, self.P, segs, len(segments), opt)
        if rc != AH_OK:
            self._h = _vp(None)
            raise AdaHessError(rc, "ah_init")

    # -- helpers
    def _check(self, rc, where):
        if rc != AH_OK:
            raise AdaHessError(rc, where, _lib.ah_last_cuda_error(self._h))

    def close(self):
        if getattr(self, "_h", None) is not None and self._h.value:
            _lib.ah_destroy(self._h)
            self._h = _vp(None)
        self._ws = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- state
    def ah_state_set(self, which, src, worker=-1):
        import torch
        if isinstance(src, torch.Tensor) and src.is_cuda:
            self._check(_lib.ah_state_set(self._h, which, worker, _dev_ptr(src.contiguous(), "src"), 1),
                        "ah_state_set")
            return
        if isinstance(src, torch.Tensor):
            src = src.numpy()
        want = {AH_NORM2: np.float64, AH_UHIST: np.float64, AH_STEP: np.uint32,
                AH_DOWN_UNTIL: np.uint32, AH_ROUND: np.uint32}.get(which, np.float32)
        a = np.ascontiguousarray(src, want)
        self._check(_lib.ah_state_set(self._h, which, worker, a.ctypes.data, 0), "ah_state_set")

    def ah_state_get(self, which, worker=-1, out=None, p_hist=4):
        import torch
        if out is not None and isinstance(out, torch.Tensor) and out.is_cuda:
            self._check(_lib.ah_state_get(self._h, which, worker, _dev_ptr(out, "out"), 1),
                        "ah_state_get")
            return out
        if which in (AH_X, AH_M, AH_V):
            shape = (self.K, self.P) if worker < 0 else (self.P,)
            a = np.empty(shape, np.float32)
        elif which == AH_CENTER:
            a = np.empty(self.P, np.float32)
        elif which == AH_WEIGHTS:
            a = np.empty(2 * self.K, np.float32)
        elif which == AH_NORM2:
            a = np.empty(self.K, np.float64)
        elif which == AH_UHIST:
            a = np.empty((self.K, p_hist + 1), np.float64)
        elif which in (AH_STEP, AH_DOWN_UNTIL):
            a = np.empty(self.K, np.uint32)
        elif which == AH_ROUND:
            a = np.empty(2, np.uint32)
        elif which == AH_INFO:
            a = np.empty(4, np.uint32)
        elif which in (AH_RUNS, AH_TILES):
            info = self.ah_state_get(AH_INFO)
            a = np.empty((int(info[1 if which == AH_RUNS else 0]), 4), np.uint32)
        else:
            raise ValueError("which")
        self._check(_lib.ah_state_get(self._h, which, worker, a.ctypes.data, 0), "ah_state_get")
        return a

    def ah_broadcast_center(self):
        self._check(_lib.ah_broadcast_center(self._h), "ah_broadcast_center")

    # -- the round
    def ah_sample_z(self, z_seed, round_, dst):
        self._check(_lib.ah_sample_z(self._h, int(z_seed), int(round_), _dev_ptr(dst, "dst"),
                                     dst.stride(0)), "ah_sample_z")
        return dst

    def ah_sample_z_n(self, z_seed, round_, sample, dst):
        self._check(_lib.ah_sample_z_n(self._h, int(z_seed), int(round_), int(sample),
                                       _dev_ptr(dst, "dst"), dst.stride(0)), "ah_sample_z_n")
        return dst

    def ah_local_step(self, grad, hvp, z_seed, lr, beta1=0.9, beta2=0.999, eps=1e-4,
                      hessian_power=1.0, weight_decay=0.0, round_=AH_ROUND_AUTO, active=None,
                      want_dist=False, rule_alpha=0.0):
        """hvp: [K, ld] for one Hutchinson sample, or [n, K, ld] for n samples per step.
        want_dist: False / True, or AH_DIST_AND_RULE with rule_alpha."""
        n_samples, sample_stride = _hvp_samples(grad, hvp)
        act = None
        if active is not None:
            act = np.ascontiguousarray(active, np.uint8)
            if act.size != self.K:
                raise ValueError("active: K bytes")
        hy = ah_hyper(lr, beta1, beta2, eps, hessian_power, weight_decay, int(round_),
                      act.ctypes.data_as(C.POINTER(C.c_uint8)) if act is not None else None,
                      int(want_dist), int(n_samples), int(sample_stride), float(rule_alpha))
        self._check(_lib.ah_local_step(self._h, _dev_ptr(grad, "grad"), _dev_ptr(hvp, "hvp"),
                                       grad.stride(-2), int(z_seed), C.byref(hy)), "ah_local_step")

    def sgd_local_step(self, grad, lr, momentum=0.0, active=None, want_dist=False):
        act = None
        if active is not None:
            act = np.ascontiguousarray(active, np.uint8)
            if act.size != self.K:
                raise ValueError("active: K bytes")
        hy = sgd_hyper(lr, momentum,
                       act.ctypes.data_as(C.POINTER(C.c_uint8)) if act is not None else None,
                       1 if want_dist else 0)
        self._check(_lib.sgd_local_step(self._h, _dev_ptr(grad, "grad"), grad.stride(0), C.byref(hy)),
                    "sgd_local_step")

    def ah_local_step_exchange(self, grad, hvp, z_seed, lr, beta1=0.9, beta2=0.999, eps=1e-4,
                               hessian_power=1.0, weight_decay=0.0, round_=AH_ROUND_AUTO, active=None,
                               want_dist=False, worker_mask=None, weights=None, alpha=0.0, order=None,
                               asynchronous=False, lagged=False):
        n_samples, sample_stride = _hvp_samples(grad, hvp)
        act = m = w = o = None
        if active is not None:
            act = np.ascontiguousarray(active, np.uint8)
            if act.size != self.K:
                raise ValueError("active: K bytes")
        if worker_mask is not None:
            worker_mask = np.ascontiguousarray(worker_mask, np.uint8)
            m = worker_mask.ctypes.data_as(C.POINTER(C.c_uint8))
        if weights is not None:
            weights = np.ascontiguousarray(weights, np.float32)
            if weights.size != 2 * self.K:
                raise ValueError("weights: 2K floats (h2 then h1)")
            w = weights.ctypes.data_as(C.POINTER(C.c_float))
        if order is not None:
            order = np.ascontiguousarray(order, np.uint16)
            if order.size != self.K:
                raise ValueError("order: K entries")
            o = order.ctypes.data_as(C.POINTER(C.c_uint16))
        hy = ah_hyper(lr, beta1, beta2, eps, hessian_power, weight_decay, int(round_),
                      act.ctypes.data_as(C.POINTER(C.c_uint8)) if act is not None else None,
                      1 if want_dist else 0, n_samples, sample_stride)
        self._check(_lib.ah_local_step_exchange(self._h, _dev_ptr(grad, "grad"), _dev_ptr(hvp, "hvp"),
                                                grad.stride(-2), int(z_seed), C.byref(hy), m, w, alpha, o,
                                                1 if asynchronous else 0, 1 if lagged else 0),
                    "ah_local_step_exchange")

    def easgd_exchange_then_step(self, grad, hvp, z_seed, lr, beta1=0.9, beta2=0.999, eps=1e-4,
                                 hessian_power=1.0, weight_decay=0.0, round_=AH_ROUND_AUTO, active=None,
                                 worker_mask=None, weights=None, alpha=0.0, order=None,
                                 asynchronous=False, dynamic=False):
        n_samples, sample_stride = _hvp_samples(grad, hvp)
        act = m = w = o = None
        if active is not None:
            act = np.ascontiguousarray(active, np.uint8)
            if act.size != self.K:
                raise ValueError("active: K bytes")
        if worker_mask is not None:
            worker_mask = np.ascontiguousarray(worker_mask, np.uint8)
            m = worker_mask.ctypes.data_as(C.POINTER(C.c_uint8))
        if weights is not None:
            weights = np.ascontiguousarray(weights, np.float32)
            if weights.size != 2 * self.K:
                raise ValueError("weights: 2K floats (h2 then h1)")
            w = weights.ctypes.data_as(C.POINTER(C.c_float))
        if order is not None:
            order = np.ascontiguousarray(order, np.uint16)
            if order.size != self.K:
                raise ValueError("order: K entries")
            o = order.ctypes.data_as(C.POINTER(C.c_uint16))
        hy = ah_hyper(lr, beta1, beta2, eps, hessian_power, weight_decay, int(round_),
                      act.ctypes.data_as(C.POINTER(C.c_uint8)) if act is not None else None, 0,
                      n_samples, sample_stride)
        self._check(_lib.easgd_exchange_then_step(self._h, _dev_ptr(grad, "grad"), _dev_ptr(hvp, "hvp"),
                                                  grad.stride(-2), int(z_seed), C.byref(hy), m, w, alpha,
                                                  o, 1 if asynchronous else 0, 1 if dynamic else 0),
                    "easgd_exchange_then_step")

    def easgd_exchange_then_sgd_step(self, grad, lr, momentum=0.0, active=None, worker_mask=None,
                                     weights=None, alpha=0.0, order=None, asynchronous=False):
        act = m = w = o = None
        if active is not None:
            act = np.ascontiguousarray(active, np.uint8)
            if act.size != self.K:
                raise ValueError("active: K bytes")
        if worker_mask is not None:
            worker_mask = np.ascontiguousarray(worker_mask, np.uint8)
            m = worker_mask.ctypes.data_as(C.POINTER(C.c_uint8))
        if weights is not None:
            weights = np.ascontiguousarray(weights, np.float32)
            if weights.size != 2 * self.K:
                raise ValueError("weights: 2K floats (h2 then h1)")
            w = weights.ctypes.data_as(C.POINTER(C.c_float))
        if order is not None:
            order = np.ascontiguousarray(order, np.uint16)
            if order.size != self.K:
                raise ValueError("order: K entries")
            o = order.ctypes.data_as(C.POINTER(C.c_uint16))
        hy = sgd_hyper(lr, momentum,
                       act.ctypes.data_as(C.POINTER(C.c_uint8)) if act is not None else None, 0)
        self._check(_lib.easgd_exchange_then_sgd_step(self._h, _dev_ptr(grad, "grad"), grad.stride(0),
                                                      C.byref(hy), m, w, alpha, o,
                                                      1 if asynchronous else 0),
                    "easgd_exchange_then_sgd_step")

    def dw_config(self, p_hist, c, kappa):
        c = np.ascontiguousarray(c, np.float64)
        self._check(_lib.dw_config(self._h, int(p_hist), c.ctypes.data_as(C.POINTER(C.c_double)),
                                   float(kappa)), "dw_config")

    def dw_weights_next(self, alpha):
        w = np.empty(2 * self.K, np.float32)
        self._check(_lib.dw_weights_next(self._h, alpha, w.ctypes.data_as(C.POINTER(C.c_float))),
                    "dw_weights_next")
        return w

    def dw_weights_from_norm2(self, norm2, alpha):
        n2 = np.ascontiguousarray(norm2, np.float64)
        if n2.size != self.K:
            raise ValueError("norm2: K doubles")
        w = np.empty(2 * self.K, np.float32)
        self._check(_lib.dw_weights_from_norm2(self._h, n2.ctypes.data_as(C.POINTER(C.c_double)),
                                               alpha, w.ctypes.data_as(C.POINTER(C.c_float))),
                    "dw_weights_from_norm2")
        return w

    def dw_mask_next(self, seed, round_, p_fail, max_stale=1):
        mask = np.empty(self.K, np.uint8)
        self._check(_lib.dw_mask_next(self._h, int(seed), int(round_), float(p_fail), int(max_stale),
                                      mask.ctypes.data_as(C.POINTER(C.c_uint8))), "dw_mask_next")
        return mask

    def easgd_exchange(self, worker_mask=None, weights=None, alpha=0.0):
        m = w = None
        if worker_mask is not None:
            worker_mask = np.ascontiguousarray(worker_mask, np.uint8)
            m = worker_mask.ctypes.data_as(C.POINTER(C.c_uint8))
        if weights is not None:
            weights = np.ascontiguousarray(weights, np.float32)
            if weights.size != 2 * self.K:
                raise ValueError("weights: 2K floats (h2 then h1)")
            w = weights.ctypes.data_as(C.POINTER(C.c_float))
        self._check(_lib.easgd_exchange(self._h, m, w, alpha), "easgd_exchange")

    def dw_order_next(self, seed, round_):
        order = np.empty(self.K, np.uint16)
        self._check(_lib.dw_order_next(self._h, int(seed), int(round_),
                                       order.ctypes.data_as(C.POINTER(C.c_uint16))), "dw_order_next")
        return order

    def easgd_exchange_async(self, worker_mask=None, weights=None, alpha=0.0, order=None):
        m = w = o = None
        if worker_mask is not None:
            worker_mask = np.ascontiguousarray(worker_mask, np.uint8)
            m = worker_mask.ctypes.data_as(C.POINTER(C.c_uint8))
        if weights is not None:
            weights = np.ascontiguousarray(weights, np.float32)
            if weights.size != 2 * self.K:
                raise ValueError("weights: 2K floats (h2 then h1)")
            w = weights.ctypes.data_as(C.POINTER(C.c_float))
        if order is not None:
            order = np.ascontiguousarray(order, np.uint16)
            if order.size != self.K:
                raise ValueError("order: K entries")
            o = order.ctypes.data_as(C.POINTER(C.c_uint16))
        self._check(_lib.easgd_exchange_async(self._h, m, w, alpha, o), "easgd_exchange_async")

    def easgd_exchange_dynamic(self, worker_mask=None, alpha=0.0, order=None, asynchronous=False):
        m = o = None
        if worker_mask is not None:
            worker_mask = np.ascontiguousarray(worker_mask, np.uint8)
            m = worker_mask.ctypes.data_as(C.POINTER(C.c_uint8))
        if order is not None:
            order = np.ascontiguousarray(order, np.uint16)
            if order.size != self.K:
                raise ValueError("order: K entries")
            o = order.ctypes.data_as(C.POINTER(C.c_uint16))
        self._check(_lib.easgd_exchange_dynamic(self._h, m, alpha, o, 1 if asynchronous else 0),
                    "easgd_exchange_dynamic")

    def ah_set_wait_polls(self, polls):
        self._check(_lib.ah_set_wait_polls(self._h, int(polls)), "ah_set_wait_polls")

    def ah_launch_count(self):
        return int(_lib.ah_launch_count(self._h))
