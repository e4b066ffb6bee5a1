"""Every rule on every element of the large parameter sets, bit for bit against the CPU oracle.

AlexNet-shaped (61 M parameters, 8 workers) and ResNet-50-shaped (25.6 M, 16 workers): the whole
run of 20 iterations with fresh seeded gradients each iteration.  VGG-16-shaped (138 M, 32
workers, 17.7 GB of gradients): two full iterations.  Four library contexts run side by side on
the same gradients, in the launch shape the benchmark times (default block and grid):

    fused     odsgd_fused_update, ping-pong weights, local weights of the last worker
    separate  odsgd_global_update then odsgd_local_update of workers 0 and M-1, in-place layout
              with a w_delayed arena
    ssgd      odsgd_ssgd_step
    asgd      one odsgd_asgd_step per worker, in a scrambled arrival order

The rules are element-wise, so the unchanged oracle walks the arena in chunks: each chunk of all
M gradients is copied to the host, the oracle advances its own copy of the state on that chunk,
and the library's result for the chunk is compared bit by bit.  The host never holds more than
one chunk of the gradients; the three independent oracle trajectories of a chunk run in three
threads (the oracle itself stays single-threaded code).
"""
from concurrent.futures import ThreadPoolExecutor

import numpy as np
import pytest
import torch

import oracle
from gpu_util import DEV, assert_bits
from paper_2005_06728_b200 import binding
from paper_2005_06728_b200 import workloads as W

pytestmark = pytest.mark.gpu

CHUNK = 1 << 22  # elements per chunk: 16 MB per arena, 512 MB of pinned staging at 32 workers


def _state(wl, n_locals_for=(), layout="pingpong"):
    w = W.make_weights(wl, DEV)
    v = W.make_momentum(wl, DEV)
    other = torch.zeros_like(w) if layout != "inplace" else None
    local = [torch.zeros_like(w) if m in n_locals_for else None for m in range(wl.n_workers)]
    ctx = binding.Odsgd(w, v, n_workers=wl.n_workers, lr=wl.lr, local_lr=wl.local_lr, momentum=wl.momentum,
                        wd=wl.wd, w_b=other if layout == "pingpong" else None,
                        w_delayed=other if layout == "delayed" else None, local=local,
                        tensor_offsets=wl.offsets)  # flags = 0: the default, exact flavour
    return ctx, w, v, local


def _arrival_order(n_workers, iteration):
    return np.random.default_rng(1000 + iteration).permutation(n_workers).tolist()


def _run_config(name, iterations, others_until):
    """`others_until`: the separate / ssgd / asgd contexts run for that many iterations."""
    wl = W.workload(name)
    n, M = wl.arena_len, wl.n_workers
    free, _ = torch.cuda.mem_get_info()
    need = (M + 16) * n * 4
    if free < need * 1.1:
        pytest.skip(f"needs {need / 2**30:.1f} GiB of device memory")
    last = M - 1
    fused, w_f, v_f, loc_f = _state(wl, (last,), "pingpong")
    sep, w_s, v_s, loc_s = _state(wl, (0, last), "delayed")
    ssgd, w_c, v_c, _ = _state(wl, (), "inplace")
    asgd, w_d, v_d, _ = _state(wl, (), "inplace")

    # the oracle's own copies of the three trajectories
    w0 = w_f.cpu().numpy()
    od_w, od_v = w0.copy(), np.zeros(n, np.float32)
    ss_w, ss_v = w0.copy(), np.zeros(n, np.float32)
    as_w, as_v = w0.copy(), np.zeros(n, np.float32)
    hp = dict(lr=wl.lr, momentum=wl.momentum, wd=wl.wd)

    grads = [torch.empty(n, dtype=torch.float32, device=DEV) for _ in range(M)]
    sg, pads = W.sigma_arena(wl, DEV), W.pad_mask(wl, DEV)
    stage = torch.empty((M, min(CHUNK, n)), dtype=torch.float32).pin_memory()
    pool = ThreadPoolExecutor(3)
    checked = 0
    for it in range(iterations):
        for m in range(M):  # fresh data every iteration
            W.make_grad(wl, m, it, DEV, out=grads[m], _sigma=sg, _pads=pads)
        others = it < others_until
        order = _arrival_order(M, it)
        fused.fused_update(grads, last)
        if others:
            sep.global_update(grads)
            sep.local_update(last)
            sep.local_update(0)
            ssgd.ssgd_step(grads)
            for m in order:
                asgd.asgd_step(m, grads[m])
        torch.cuda.synchronize()
        f_w, f_bak = fused.weights(), fused.delayed_weights()
        s_w, s_bak = sep.weights(), sep.delayed_weights()
        for a in range(0, n, CHUNK):
            b = min(a + CHUNK, n)
            for m in range(M):
                stage[m, :b - a].copy_(grads[m][a:b], non_blocking=True)
            torch.cuda.synchronize()
            gh = [stage[m, :b - a].numpy() for m in range(M)]
            bak = np.empty(b - a, np.float32)

            def od_job():
                oracle.global_update(gh, od_w[a:b], od_v[a:b], w_prev=bak, **hp)
                return (oracle.local_update(bak, gh[0], local_lr=wl.local_lr),
                        oracle.local_update(bak, gh[last], local_lr=wl.local_lr))

            def ss_job():
                oracle.ssgd_step(gh, ss_w[a:b], ss_v[a:b], **hp)

            def as_job():
                for m in order:
                    oracle.asgd_step(gh[m], as_w[a:b], as_v[a:b], **hp)

            jobs = [pool.submit(od_job)] + ([pool.submit(ss_job), pool.submit(as_job)] if others else [])
            x0, xl = jobs[0].result()
            for j in jobs[1:]:
                j.result()
            tag = f"{name} it {it} [{a}:{b}]"
            assert_bits(f_w[a:b].cpu().numpy(), od_w[a:b], f"fused w {tag}")
            assert_bits(v_f[a:b].cpu().numpy(), od_v[a:b], f"fused v {tag}")
            assert_bits(f_bak[a:b].cpu().numpy(), bak, f"fused backup {tag}")
            assert_bits(loc_f[last][a:b].cpu().numpy(), xl, f"fused x[{last}] {tag}")
            if others:
                assert_bits(s_w[a:b].cpu().numpy(), od_w[a:b], f"global w {tag}")
                assert_bits(v_s[a:b].cpu().numpy(), od_v[a:b], f"global v {tag}")
                assert_bits(s_bak[a:b].cpu().numpy(), bak, f"global backup {tag}")
                assert_bits(loc_s[0][a:b].cpu().numpy(), x0, f"local x[0] {tag}")
                assert_bits(loc_s[last][a:b].cpu().numpy(), xl, f"local x[{last}] {tag}")
                assert_bits(w_c[a:b].cpu().numpy(), ss_w[a:b], f"ssgd w {tag}")
                assert_bits(v_c[a:b].cpu().numpy(), ss_v[a:b], f"ssgd v {tag}")
                assert_bits(w_d[a:b].cpu().numpy(), as_w[a:b], f"asgd w {tag}")
                assert_bits(v_d[a:b].cpu().numpy(), as_v[a:b], f"asgd v {tag}")
            checked += b - a
    pool.shutdown()
    assert checked == n * iterations, "every element of every iteration was compared"
    assert fused.step == iterations and fused.launch_count == iterations
    assert asgd.step == others_until * M
    for c in (fused, sep, ssgd, asgd):
        c.close()
    del grads, stage
    torch.cuda.empty_cache()


def test_alexnet_every_rule_every_element_full_run(cuda_device):
    wl = W.workload("alexnet")
    _run_config("alexnet", wl.iterations, wl.iterations)


def test_resnet50_every_rule_every_element_full_run(cuda_device):
    wl = W.workload("resnet50")
    _run_config("resnet50", wl.iterations, wl.iterations)


def test_vgg16_every_rule_every_element(cuda_device):
    # two full iterations of the fused update; one of the separate calls, SSGD and an ASGD round
    _run_config("vgg16", 2, 1)


def test_resnet56_ssgd_and_asgd_full_run(cuda_device):
    """The comparison rules through the many-small-tensor set, whole run, all elements."""
    wl = W.workload("resnet56")
    _run_config("resnet56", wl.iterations, wl.iterations)


def test_lenet5_every_rule_full_run(cuda_device):
    wl = W.workload("lenet5")
    _run_config("lenet5", wl.iterations, wl.iterations)
