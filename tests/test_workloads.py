"""Shapes, sizes and determinism of the synthetic parameter sets (no GPU)."""
import math

import numpy as np
import pytest
import torch

from paper_2005_06728_b200 import workloads as W

EXPECT = {  # name: (tensors, parameters, workers)
    "lenet5": (8, 431_080, 4),
    "resnet56": (167, 853_018, 8),
    "alexnet": (16, 60_965_224, 8),
    "resnet50": (161, 25_557_032, 16),
    "vgg16": (32, 138_357_544, 32),
}


@pytest.mark.parametrize("name", W.WORKLOAD_NAMES)
def test_counts(name):
    wl = W.workload(name)
    assert (wl.n_tensors, wl.n_params, wl.n_workers) == EXPECT[name]
    assert len(wl.offsets) == wl.n_tensors + 1 and wl.offsets[-1] == wl.arena_len
    assert all(o % W.ALIGN_ELEMS == 0 for o in wl.offsets)
    assert all(b - a >= t.numel for a, b, t in zip(wl.offsets, wl.offsets[1:], wl.tensors))
    assert wl.arena_len - wl.n_params < W.ALIGN_ELEMS * wl.n_tensors


def test_values_lenet5():
    wl = W.workload("lenet5")
    w = W.make_weights(wl)
    assert torch.equal(w, W.make_weights(wl)), "seeded: same call, same numbers"
    pads = W.pad_mask(wl)
    assert pads is not None and torch.all(w[pads] == 0)
    fc1 = wl.tensors[4]
    off = wl.offsets[4]
    assert fc1.name == "fc1.weight" and fc1.fan_in == 800
    std = w[off:off + fc1.numel].std().item()
    assert abs(std - math.sqrt(2 / 800)) < 0.02 * math.sqrt(2 / 800)
    boff = wl.offsets[5]
    assert torch.all(w[boff:boff + 500] == 0), "biases start at zero"
    g0, g1 = W.make_grad(wl, 0, 0), W.make_grad(wl, 1, 0)
    assert not torch.equal(g0, g1) and torch.equal(g0, W.make_grad(wl, 0, 0))
    assert not torch.equal(g0, W.make_grad(wl, 0, 1))
    assert abs(g0.std().item() - 1e-2) < 2e-4 and torch.all(g0[pads] == 0)


def test_values_resnet56_per_tensor_sigma():
    wl = W.workload("resnet56")
    sig = W.tensor_sigmas(wl)
    assert len(sig) == 167 and min(sig) >= 1e-3 and max(sig) <= 1e-1
    assert max(sig) / min(sig) > 20
    g = W.make_grad(wl, 3, 5)
    big = max(range(167), key=lambda i: wl.tensors[i].numel)
    off, n = wl.offsets[big], wl.tensors[big].numel
    assert abs(g[off:off + n].std().item() / sig[big] - 1) < 0.03
    w = W.make_weights(wl)
    gam = [i for i, t in enumerate(wl.tensors) if t.kind == "bn_gamma"][0]
    assert torch.all(w[wl.offsets[gam]:wl.offsets[gam] + wl.tensors[gam].numel] == 1)


def test_outliers():
    wl = W.ragged_workload([200_000], 2)
    wl.outlier_prob, wl.outlier_scale, wl.grad_sigma = 0.01, 100.0, 1e-2
    g = W.make_grad(wl, 0, 0).numpy()
    frac = np.mean(np.abs(g) > 0.06)  # 6 sigma: essentially only the scaled entries
    assert 0.006 < frac < 0.012


def test_special_and_dyadic():
    s = W.special_values(4000)
    assert torch.isnan(s).any() and torch.isinf(s).any() and (s.abs() < 1e-38).any()
    d = W.dyadic_values(1000, seed=1)
    assert torch.equal(d * 64, (d * 64).round()) and d.abs().max() <= 8
