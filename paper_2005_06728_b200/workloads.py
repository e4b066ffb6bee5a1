"""Seeded synthetic parameter sets and gradient streams.

This module only *describes shapes and draws random numbers*.  It holds none of
the update arithmetic: both the CUDA path and the CPU oracle are fed from here
so that they see identical inputs, and neither of them imports the other.

The paper trains real networks on MNIST / CIFAR-10 / ImageNet (Section 4.1).
None of that data is needed to exercise the parameter-update pass: what matters
is the number of tensors, their sizes, the number of workers and the value
distributions.  Each workload below is therefore a *shape* of a well-known
public architecture, filled with seeded random values.

Arena layout: tensors are concatenated in the listed order; every tensor starts
at an element offset that is a multiple of 4 (16 bytes); the padding between
tensors holds zeros in every arena (weights, momentum, gradients).
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import List, Optional, Sequence, Tuple

import torch

ALIGN_ELEMS = 4  # every tensor starts on a 16-byte boundary


@dataclass(frozen=True)
class TensorSpec:
    name: str
    shape: Tuple[int, ...]
    kind: str  # "weight" | "bias" | "bn_gamma" | "bn_beta"

    @property
    def numel(self) -> int:
        n = 1
        for s in self.shape:
            n *= s
        return n

    @property
    def fan_in(self) -> int:
        if len(self.shape) <= 1:
            return self.shape[0]
        n = 1
        for s in self.shape[1:]:
            n *= s
        return n


@dataclass
class Workload:
    """A synthetic parameter set plus the hyper-parameters it is run with."""

    name: str
    tensors: List[TensorSpec]
    n_workers: int
    lr: float
    local_lr: float
    momentum: float
    wd: float
    iterations: int
    seed: int
    grad_sigma: float = 1e-2
    # "fixed": every tensor uses grad_sigma; "log_uniform": one sigma per tensor,
    # 10**U(log10(lo), log10(hi)) drawn once from the seed.
    grad_sigma_mode: str = "fixed"
    grad_sigma_range: Tuple[float, float] = (1e-3, 1e-1)
    outlier_prob: float = 0.0
    outlier_scale: float = 1.0
    offsets: List[int] = field(default_factory=list)  # n_tensors + 1 entries
    arena_len: int = 0

    def __post_init__(self) -> None:
        off = 0
        self.offsets = []
        for t in self.tensors:
            self.offsets.append(off)
            off += t.numel
            off = (off + ALIGN_ELEMS - 1) // ALIGN_ELEMS * ALIGN_ELEMS
        self.offsets.append(off)
        self.arena_len = off

    @property
    def n_params(self) -> int:
        """True parameter count P (padding excluded)."""
        return sum(t.numel for t in self.tensors)

    @property
    def n_tensors(self) -> int:
        return len(self.tensors)

    def with_workers(self, n: int) -> "Workload":
        w = Workload(**{k: getattr(self, k) for k in (
            "name", "tensors", "lr", "local_lr", "momentum", "wd", "iterations", "seed",
            "grad_sigma", "grad_sigma_mode", "grad_sigma_range", "outlier_prob",
            "outlier_scale")}, n_workers=n)
        return w


# --------------------------------------------------------------------------- shapes

def _conv(name: str, cout: int, cin: int, k: int, bias: bool = False) -> List[TensorSpec]:
    out = [TensorSpec(f"{name}.weight", (cout, cin, k, k), "weight")]
    if bias:
        out.append(TensorSpec(f"{name}.bias", (cout,), "bias"))
    return out


def _fc(name: str, nout: int, nin: int) -> List[TensorSpec]:
    return [TensorSpec(f"{name}.weight", (nout, nin), "weight"),
            TensorSpec(f"{name}.bias", (nout,), "bias")]


def _bn(name: str, c: int) -> List[TensorSpec]:
    return [TensorSpec(f"{name}.gamma", (c,), "bn_gamma"),
            TensorSpec(f"{name}.beta", (c,), "bn_beta")]


def lenet5_tensors() -> List[TensorSpec]:
    t: List[TensorSpec] = []
    t += _conv("conv1", 20, 1, 5, bias=True)
    t += _conv("conv2", 50, 20, 5, bias=True)
    t += _fc("fc1", 500, 800)
    t += _fc("fc2", 10, 500)
    return t


def resnet56_cifar_tensors() -> List[TensorSpec]:
    t: List[TensorSpec] = []
    t += _conv("conv0", 16, 3, 3) + _bn("bn0", 16)
    cin = 16
    for s, width in enumerate((16, 32, 64)):
        for b in range(9):
            t += _conv(f"s{s}.b{b}.conv1", width, cin, 3) + _bn(f"s{s}.b{b}.bn1", width)
            t += _conv(f"s{s}.b{b}.conv2", width, width, 3) + _bn(f"s{s}.b{b}.bn2", width)
            cin = width
    t += _fc("fc", 10, 64)
    return t


def alexnet_tensors() -> List[TensorSpec]:
    # two-group original: conv2/4/5 see half of the previous layer's channels
    t: List[TensorSpec] = []
    t += _conv("conv1", 96, 3, 11, bias=True)
    t += _conv("conv2", 256, 48, 5, bias=True)
    t += _conv("conv3", 384, 256, 3, bias=True)
    t += _conv("conv4", 384, 192, 3, bias=True)
    t += _conv("conv5", 256, 192, 3, bias=True)
    t += _fc("fc6", 4096, 9216)
    t += _fc("fc7", 4096, 4096)
    t += _fc("fc8", 1000, 4096)
    return t


def resnet50_tensors() -> List[TensorSpec]:
    t: List[TensorSpec] = []
    t += _conv("conv1", 64, 3, 7) + _bn("bn1", 64)
    cin = 64
    for s, (blocks, width) in enumerate(zip((3, 4, 6, 3), (64, 128, 256, 512))):
        for b in range(blocks):
            p = f"layer{s + 1}.{b}"
            t += _conv(f"{p}.conv1", width, cin, 1) + _bn(f"{p}.bn1", width)
            t += _conv(f"{p}.conv2", width, width, 3) + _bn(f"{p}.bn2", width)
            t += _conv(f"{p}.conv3", 4 * width, width, 1) + _bn(f"{p}.bn3", 4 * width)
            if b == 0:
                t += _conv(f"{p}.down", 4 * width, cin, 1) + _bn(f"{p}.down_bn", 4 * width)
            cin = 4 * width
    t += _fc("fc", 1000, 2048)
    return t


def vgg16_tensors() -> List[TensorSpec]:
    t: List[TensorSpec] = []
    cin = 3
    for i, c in enumerate((64, 64, 128, 128, 256, 256, 256, 512, 512, 512, 512, 512, 512)):
        t += _conv(f"conv{i + 1}", c, cin, 3, bias=True)
        cin = c
    t += _fc("fc6", 4096, 25088)
    t += _fc("fc7", 4096, 4096)
    t += _fc("fc8", 1000, 4096)
    return t


def workload(name: str) -> Workload:
    """The five synthetic parameter sets, smallest first."""
    if name == "lenet5":
        return Workload("lenet5", lenet5_tensors(), n_workers=4, lr=0.01, local_lr=0.01,
                        momentum=0.9, wd=5e-4, iterations=50, seed=0, grad_sigma=1e-2)
    if name == "resnet56":
        return Workload("resnet56", resnet56_cifar_tensors(), n_workers=8, lr=0.1, local_lr=0.1,
                        momentum=0.9, wd=1e-4, iterations=100, seed=1,
                        grad_sigma_mode="log_uniform", grad_sigma_range=(1e-3, 1e-1))
    if name == "alexnet":
        return Workload("alexnet", alexnet_tensors(), n_workers=8, lr=0.01, local_lr=0.01,
                        momentum=0.9, wd=5e-4, iterations=20, seed=2, grad_sigma=1e-2,
                        outlier_prob=0.01, outlier_scale=100.0)
    if name == "resnet50":
        return Workload("resnet50", resnet50_tensors(), n_workers=16, lr=0.1, local_lr=0.1,
                        momentum=0.9, wd=1e-4, iterations=20, seed=3, grad_sigma=1e-2)
    if name == "vgg16":
        return Workload("vgg16", vgg16_tensors(), n_workers=32, lr=0.1, local_lr=0.1,
                        momentum=0.9, wd=1e-4, iterations=20, seed=4, grad_sigma=1e-2)
    raise KeyError(name)


WORKLOAD_NAMES = ("lenet5", "resnet56", "alexnet", "resnet50", "vgg16")


def ragged_workload(sizes: Sequence[int], n_workers: int, *, lr: float = 0.05,
                    local_lr: float = 0.02, momentum: float = 0.9, wd: float = 1e-3,
                    iterations: int = 3, seed: int = 7, name: str = "ragged") -> Workload:
    """A made-up parameter set with the given 1-D tensor sizes (for edge-case tests)."""
    tensors = [TensorSpec(f"t{i}", (int(s),), "weight") for i, s in enumerate(sizes)]
    return Workload(name, tensors, n_workers=n_workers, lr=lr, local_lr=local_lr,
                    momentum=momentum, wd=wd, iterations=iterations, seed=seed)


# --------------------------------------------------------------------------- values

def _gen(device: torch.device | str, *key: int) -> torch.Generator:
    """One generator per (seed, stream, worker, iteration, ...) key."""
    g = torch.Generator(device=device)
    s = 0x9E3779B97F4A7C15
    for k in key:
        s = (s ^ (int(k) + 0x632BE59BD9B4E019)) * 0xD6E8FEB86659FD93 % (1 << 64)
        s ^= s >> 32
    g.manual_seed(s % (1 << 63))
    return g


def pad_mask(wl: Workload, device: torch.device | str = "cpu") -> Optional[torch.Tensor]:
    """Indices of the padding elements of the arena (None when there are none)."""
    idx: List[int] = []
    for t, off, nxt in zip(wl.tensors, wl.offsets[:-1], wl.offsets[1:]):
        idx.extend(range(off + t.numel, nxt))
    if not idx:
        return None
    return torch.tensor(idx, dtype=torch.long, device=device)


def make_weights(wl: Workload, device: torch.device | str = "cpu") -> torch.Tensor:
    """Initial weights: normal(0, sqrt(2/fan_in)) for weight tensors, biases and BN beta 0,
    BN gamma 1.  Padding is zero."""
    arena = torch.zeros(wl.arena_len, dtype=torch.float32, device=device)
    g = _gen(device, wl.seed, 1)
    for t, off in zip(wl.tensors, wl.offsets):
        view = arena[off:off + t.numel]
        if t.kind == "weight":
            view.normal_(0.0, math.sqrt(2.0 / t.fan_in), generator=g)
        elif t.kind == "bn_gamma":
            view.fill_(1.0)
    return arena


def make_momentum(wl: Workload, device: torch.device | str = "cpu") -> torch.Tensor:
    """Momentum state starts at zero."""
    return torch.zeros(wl.arena_len, dtype=torch.float32, device=device)


def tensor_sigmas(wl: Workload) -> List[float]:
    """Per-tensor gradient standard deviation."""
    if wl.grad_sigma_mode == "fixed":
        return [wl.grad_sigma] * wl.n_tensors
    lo, hi = wl.grad_sigma_range
    g = _gen("cpu", wl.seed, 2)
    u = torch.rand(wl.n_tensors, generator=g, dtype=torch.float64)
    e = math.log10(lo) + u * (math.log10(hi) - math.log10(lo))
    return [float(10.0 ** x) for x in e.tolist()]


def sigma_arena(wl: Workload, device: torch.device | str = "cpu") -> Optional[torch.Tensor]:
    """Per-element sigma (only for the per-tensor mode; None for a fixed sigma)."""
    if wl.grad_sigma_mode == "fixed":
        return None
    s = torch.zeros(wl.arena_len, dtype=torch.float32, device=device)
    for t, off, sg in zip(wl.tensors, wl.offsets, tensor_sigmas(wl)):
        s[off:off + t.numel] = sg
    return s


def make_grad(wl: Workload, worker: int, iteration: int, device: torch.device | str = "cpu",
              out: Optional[torch.Tensor] = None, *, _sigma: Optional[torch.Tensor] = None,
              _pads: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Worker `worker`'s gradient arena for iteration `iteration` (fresh, seeded).

    normal(0, sigma) per element; with outlier_prob > 0 an independent Bernoulli mask
    multiplies the chosen entries by outlier_scale.  Padding is zero.
    """
    if out is None:
        out = torch.empty(wl.arena_len, dtype=torch.float32, device=device)
    g = _gen(device, wl.seed, 3, worker, iteration)
    out.normal_(0.0, 1.0, generator=g)
    if wl.grad_sigma_mode == "fixed":
        out.mul_(wl.grad_sigma)
    else:
        sg = _sigma if _sigma is not None else sigma_arena(wl, device)
        out.mul_(sg)
    if wl.outlier_prob > 0.0:
        chunk = 1 << 24
        for a in range(0, wl.arena_len, chunk):
            b = min(a + chunk, wl.arena_len)
            u = torch.rand(b - a, generator=g, device=device, dtype=torch.float32)
            sel = u < wl.outlier_prob
            out[a:b] = torch.where(sel, out[a:b] * wl.outlier_scale, out[a:b])
    pads = _pads if _pads is not None else pad_mask(wl, device)
    if pads is not None:
        out.index_fill_(0, pads, 0.0)
    return out


def make_grads(wl: Workload, iteration: int, device: torch.device | str = "cpu",
               n_workers: Optional[int] = None) -> List[torch.Tensor]:
    """All workers' gradient arenas for one iteration."""
    n = wl.n_workers if n_workers is None else n_workers
    sg = sigma_arena(wl, device)
    pads = pad_mask(wl, device)
    return [make_grad(wl, m, iteration, device, _sigma=sg, _pads=pads) for m in range(n)]


def special_values(n: int, seed: int = 11) -> torch.Tensor:
    """A float32 vector that mixes ordinary numbers with +-0, denormals, +-inf and NaN."""
    g = _gen("cpu", seed, 4)
    x = torch.randn(n, generator=g, dtype=torch.float32)
    pool = torch.tensor([0.0, -0.0, 1e-40, -1e-40, 1.1754944e-38, float("inf"), -float("inf"),
                         float("nan"), 3.4028235e38, -3.4028235e38, 1.0, -1.0],
                        dtype=torch.float32)
    pick = torch.randint(0, pool.numel() * 3, (n,), generator=g)
    special = pick < pool.numel()
    x[special] = pool[pick[special]]
    return x


def dyadic_values(n: int, seed: int, bits: int = 6, scale_pow: int = 3) -> torch.Tensor:
    """Multiples of 2**-bits in [-2**scale_pow, 2**scale_pow): short sums of these are exact."""
    g = _gen("cpu", seed, 5)
    q = torch.randint(-(1 << (bits + scale_pow)), 1 << (bits + scale_pow), (n,), generator=g)
    return (q.to(torch.float64) / float(1 << bits)).to(torch.float32)
