"""Seeded synthetic workloads: flat parameter layouts and input buffers.

This module holds no arithmetic of the optimiser or of the elastic exchange.  It
only describes *shapes* (how a network's tensors tile the flat parameter row) and
draws seeded random input buffers, so that the CUDA library and an independent
checker can be handed the same bytes.

The paper trains a small CNN on MNIST (Sec. VI); neither is needed to exercise the
per-round update, so CNN-shaped layouts and Gaussian gradient / Hessian-vector
buffers stand in for them.  The layer tables are written out from the published
architectures (He et al. 2016 for the residual nets, Simonyan & Zisserman 2015 for
the 16-layer plain net); no third-party code or data is involved.

A layout is a list of ``Tensor`` records; ``segments(layout)`` turns it into the
``(offset, length, block)`` triples the library takes, where ``block = kh*kw`` for a
4-D convolution kernel (stored ``[c_out, c_in, kh, kw]``, so each (c_out, c_in)
filter is one contiguous run of kh*kw entries) and 1 for every other tensor.
"""
from __future__ import annotations

import math
from dataclasses import dataclass

import numpy as np


@dataclass(frozen=True)
class Tensor:
    name: str
    shape: tuple
    offset: int

    @property
    def numel(self) -> int:
        return int(np.prod(self.shape))

    @property
    def block(self) -> int:
        return int(self.shape[2] * self.shape[3]) if len(self.shape) == 4 else 1

    @property
    def fan_in(self) -> int:
        if len(self.shape) == 4:
            return int(self.shape[1] * self.shape[2] * self.shape[3])
        if len(self.shape) == 2:
            return int(self.shape[1])
        return int(self.shape[0])


class _Builder:
    def __init__(self):
        self.tensors: list[Tensor] = []
        self.off = 0

    def add(self, name, shape):
        t = Tensor(name, tuple(int(s) for s in shape), self.off)
        self.tensors.append(t)
        self.off += t.numel

    def conv(self, name, cin, cout, k, bias=False):
        self.add(name + ".weight", (cout, cin, k, k))
        if bias:
            self.add(name + ".bias", (cout,))

    def bn(self, name, c):
        self.add(name + ".weight", (c,))
        self.add(name + ".bias", (c,))

    def fc(self, name, fin, fout):
        self.add(name + ".weight", (fout, fin))
        self.add(name + ".bias", (fout,))


def _w(c, div):
    return max(1, c // div)


def resnet18_layout(width_div: int = 1, num_classes: int = 1000) -> list[Tensor]:
    """Basic-block residual net, stages of (2, 2, 2, 2) blocks: 62 tensors,
    11,689,512 parameters at full width."""
    b = _Builder()
    w = [_w(c, width_div) for c in (64, 128, 256, 512)]
    b.conv("conv1", 3, w[0], 7)
    b.bn("bn1", w[0])
    cin = w[0]
    for s, cout in enumerate(w):
        for blk in range(2):
            p = f"layer{s + 1}.{blk}"
            b.conv(p + ".conv1", cin, cout, 3)
            b.bn(p + ".bn1", cout)
            b.conv(p + ".conv2", cout, cout, 3)
            b.bn(p + ".bn2", cout)
            if blk == 0 and s > 0:
                b.conv(p + ".downsample.0", cin, cout, 1)
                b.bn(p + ".downsample.1", cout)
            cin = cout
    b.fc("fc", cin, _w(num_classes, width_div))
    return b.tensors


def resnet50_layout(width_div: int = 1, num_classes: int = 1000) -> list[Tensor]:
    """Bottleneck residual net, stages of (3, 4, 6, 3) blocks, expansion 4:
    161 tensors, 25,557,032 parameters at full width."""
    b = _Builder()
    w = [_w(c, width_div) for c in (64, 128, 256, 512)]
    b.conv("conv1", 3, w[0], 7)
    b.bn("bn1", w[0])
    cin = w[0]
    for s, (mid, nblk) in enumerate(zip(w, (3, 4, 6, 3))):
        cout = 4 * mid
        for blk in range(nblk):
            p = f"layer{s + 1}.{blk}"
            b.conv(p + ".conv1", cin, mid, 1)
            b.bn(p + ".bn1", mid)
            b.conv(p + ".conv2", mid, mid, 3)
            b.bn(p + ".bn2", mid)
            b.conv(p + ".conv3", mid, cout, 1)
            b.bn(p + ".bn3", cout)
            if blk == 0:
                b.conv(p + ".downsample.0", cin, cout, 1)
                b.bn(p + ".downsample.1", cout)
            cin = cout
    b.fc("fc", cin, _w(num_classes, width_div))
    return b.tensors


def vgg16_layout(width_div: int = 1, num_classes: int = 1000) -> list[Tensor]:
    """Plain 16-layer net: 13 3x3 convolutions with bias and three dense layers
    (7*7*512 -> 4096 -> 4096 -> classes): 32 tensors, 138,357,544 parameters."""
    b = _Builder()
    cfg = (64, 64, 128, 128, 256, 256, 256, 512, 512, 512, 512, 512, 512)
    cin = 3
    for k, c in enumerate(cfg):
        cout = _w(c, width_div)
        b.conv(f"features.{k}", cin, cout, 3, bias=True)
        cin = cout
    hidden = _w(4096, width_div)
    b.fc("classifier.0", cin * 49, hidden)
    b.fc("classifier.3", hidden, hidden)
    b.fc("classifier.6", hidden, _w(num_classes, width_div))
    return b.tensors


def single_segment_layout(P: int) -> list[Tensor]:
    """One unstructured tensor of P parameters (the diagonal quadratic problem)."""
    return [Tensor("theta", (int(P),), 0)]


def mnist_cnn_layout(width_div: int = 1) -> list[Tensor]:
    """The small two-convolution classifier for 28 x 28 digits that the paper trains
    (Sec. VI): conv 1->32 3x3, conv 32->64 3x3, dense 9216->128, dense 128->10, with
    biases: 8 tensors, 1,199,882 parameters, 98 % of them in the first dense layer."""
    assert width_div == 1
    b = _Builder()
    b.conv("conv1", 1, 32, 3, bias=True)
    b.conv("conv2", 32, 64, 3, bias=True)
    b.fc("fc1", 9216, 128)
    b.fc("fc2", 128, 10)
    return b.tensors


LAYOUTS = {
    "mnist_cnn": mnist_cnn_layout,
    "resnet18": resnet18_layout,
    "resnet50": resnet50_layout,
    "vgg16": vgg16_layout,
}


def random_segment_table(seed: int, max_block: int, target: int = 12_000):
    """A seeded, irregular tensor table for edge-case tests: (segments, P) with tensors of
    every size from one block to a few thousand elements, spatial blocks from 1 to
    max_block (3 x 3 kernels most often), occasional gaps, and a ragged end.  The caller
    states the largest block it wants drawn."""
    rng = np.random.default_rng(seed)
    segs, pos = [], int(rng.integers(0, 6))
    while pos < target:
        if rng.random() < 0.2:
            pos += int(rng.integers(1, 40))                        # a gap: behaves as block 1
        kind = rng.random()
        block = 9 if kind < 0.4 else 1 if kind < 0.65 else int(rng.integers(2, max_block + 1))
        length = block * int(rng.integers(1, max(2, min(400, 3000 // block))))
        segs.append((pos, length, block))
        pos += length
    return segs, pos + int(rng.integers(0, 7))


def total_params(layout) -> int:
    return layout[-1].offset + layout[-1].numel if layout else 0


def segments(layout) -> list[tuple[int, int, int]]:
    """(offset, length, block) per tensor, in offset order."""
    return [(t.offset, t.numel, t.block) for t in layout]


def sigma_per_tensor(layout) -> list[float]:
    """sigma_l = 1/sqrt(fan_in_l)."""
    return [1.0 / math.sqrt(t.fan_in) for t in layout]


# --------------------------------------------------------------------------
# Seeded buffers.  numpy versions serve small cases on the host; the torch
# versions draw directly in device memory for full-size runs.
# --------------------------------------------------------------------------

def padded_ld(P: int) -> int:
    """Row stride (elements) for a [K, P] input buffer: P rounded up to a multiple of 4."""
    return (int(P) + 3) // 4 * 4


def theta0_np(layout, seed: int) -> np.ndarray:
    """Initial parameters, N(0, sigma_l^2) per tensor, float32 [P]."""
    rng = np.random.Generator(np.random.PCG64(seed))
    P = total_params(layout)
    out = np.empty(P, np.float32)
    for t, s in zip(layout, sigma_per_tensor(layout)):
        out[t.offset:t.offset + t.numel] = rng.standard_normal(t.numel, np.float32) * np.float32(s)
    return out


def gaussian_pair_np(layout, K: int, seed: int, ld: int | None = None):
    """One (grad, hvp) pair, each float32 [K, ld], N(0, sigma_l^2) per tensor;
    padding columns (ld > P) are zero."""
    rng = np.random.Generator(np.random.PCG64(seed))
    P = total_params(layout)
    ld = padded_ld(P) if ld is None else int(ld)
    pair = []
    for _ in range(2):
        buf = np.zeros((K, ld), np.float32)
        for t, s in zip(layout, sigma_per_tensor(layout)):
            buf[:, t.offset:t.offset + t.numel] = (
                rng.standard_normal((K, t.numel), np.float32) * np.float32(s))
        pair.append(buf)
    return pair[0], pair[1]


def gaussian_pool_np(layout, K: int, n_pool: int, seed: int, ld: int | None = None):
    """A pool of n_pool (grad, hvp) pairs; round t uses pool[t % n_pool]."""
    return [gaussian_pair_np(layout, K, seed + 1000 * r, ld) for r in range(n_pool)]


def gaussian_pair_torch(layout, K: int, seed: int, device, ld: int | None = None):
    """Device-side version of gaussian_pair_np (different stream of numbers: use
    one or the other for both sides of a comparison, never a mix)."""
    import torch
    gen = torch.Generator(device=device)
    gen.manual_seed(int(seed))
    P = total_params(layout)
    ld = padded_ld(P) if ld is None else int(ld)
    pair = []
    for _ in range(2):
        buf = torch.empty((K, ld), dtype=torch.float32, device=device)
        buf.normal_(generator=gen)
        for t, s in zip(layout, sigma_per_tensor(layout)):
            buf[:, t.offset:t.offset + t.numel].mul_(s)
        if ld > P:
            buf[:, P:].zero_()
        pair.append(buf)
    return pair[0], pair[1]


def theta0_torch(layout, seed: int, device):
    import torch
    gen = torch.Generator(device=device)
    gen.manual_seed(int(seed))
    P = total_params(layout)
    out = torch.empty(P, dtype=torch.float32, device=device)
    out.normal_(generator=gen)
    for t, s in zip(layout, sigma_per_tensor(layout)):
        out[t.offset:t.offset + t.numel].mul_(s)
    return out


# --------------------------------------------------------------------------
# Diagonal quadratic problem f(theta) = 1/2 sum_j h_j theta_j^2.  Its Hessian is
# diag(h), so the exact Hessian-vector product with any z is h * z and the exact
# gradient at theta is h * theta.  These are properties of the *loss*, not of
# the optimiser under test.
# --------------------------------------------------------------------------

def quadratic_problem_np(P: int, seed: int):
    """h ~ U[0.1, 10], theta0 ~ N(0, 1); both float32 [P]."""
    rng = np.random.Generator(np.random.PCG64(seed))
    h = rng.uniform(0.1, 10.0, P).astype(np.float32)
    theta0 = rng.standard_normal(P, np.float32)
    return h, theta0


def quadratic_noise_np(K: int, P: int, seed: int, t: int, sigma: float = 0.01) -> np.ndarray:
    """Gradient noise of round t, N(0, sigma^2), float32 [K, P]."""
    rng = np.random.Generator(np.random.PCG64([int(seed), int(t), 0x6E6F6973]))
    return rng.standard_normal((K, P), np.float32) * np.float32(sigma)


def quadratic_grad_np(h: np.ndarray, x: np.ndarray, noise: np.ndarray | None) -> np.ndarray:
    """Stochastic gradient of the quadratic at each worker's x: h * x (+ noise)."""
    g = (h[None, :] * x).astype(np.float32)
    if noise is not None:
        g = (g + noise).astype(np.float32)
    return g


def quadratic_hvp_np(h: np.ndarray, z: np.ndarray) -> np.ndarray:
    """Exact Hessian-vector product of the quadratic: h * z, z given as +-1."""
    return (h[None, :] * z).astype(np.float32)


def scripted_down(worker: int, first: int, last: int):
    """A scripted outage: `worker` cannot reach the master in rounds first..last."""
    return {"worker": int(worker), "first": int(first), "last": int(last)}


def apply_scripted(mask: np.ndarray, t: int, outages) -> np.ndarray:
    """Force mask[worker] = 0 for every scripted outage that covers round t."""
    out = mask.copy()
    for o in outages:
        if o["first"] <= t <= o["last"]:
            out[o["worker"]] = 0
    return out
