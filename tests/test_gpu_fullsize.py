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

The local rules with extra arenas (Eq. 4, Eq. 5-6, local momentum: the flavours the paper trained
its CIFAR-10 and ImageNet models with) get the same treatment on the AlexNet- and ResNet-50-shaped
sets: three iterations, every element, the update of one worker inside the server pass and the
update of three workers in the all-workers pass, each chained through its own arenas.
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


RULES = {"dc_c": binding.LOCAL_DC_C, "dc_a": binding.LOCAL_DC_A, "momentum": binding.LOCAL_MOMENTUM}
LAM, DECAY, EPS = 0.04, 0.95, 1e-7


def _oracle_local(rule, bak, g, x_prev, state, llr):
    """One worker's local update on a chunk; `state` (mean square or velocity) is updated in place."""
    if rule == "dc_c":
        return oracle.local_update_dc_c(bak, g, x_prev, local_lr=llr, lam=LAM)
    if rule == "dc_a":
        return oracle.local_update_dc_a(bak, g, x_prev, state, local_lr=llr, lam=LAM, m=DECAY, eps=EPS)
    return oracle.local_update_momentum(bak, g, state, local_lr=llr, momentum=DECAY, wd=LAM)


def _run_local_rules(name, iterations):
    wl = W.workload(name)
    n, M = wl.arena_len, wl.n_workers
    free, _ = torch.cuda.mem_get_info()
    if free < (M + 48) * n * 4 * 1.1:
        pytest.skip("not enough device memory")
    last, some = M - 1, (0, M // 2, M - 1)
    w0 = W.make_weights(wl, DEV)
    ctxs = {}
    for rule, rid in RULES.items():
        for kind, who in (("one", (last,)), ("some", some)):
            w, v, other = w0.clone(), torch.zeros_like(w0), torch.zeros_like(w0)
            local = [w0.clone() if m in who else None for m in range(M)]
            state = [torch.zeros_like(w0) if m in who else None for m in range(M)]
            c = binding.Odsgd(w, v, n_workers=M, lr=wl.lr, local_lr=wl.local_lr, momentum=wl.momentum, wd=wl.wd,
                              w_b=other, local=local, tensor_offsets=wl.offsets)
            c.set_local_rule(rid, LAM, DECAY, EPS, state if rule != "dc_c" else None)
            ctxs[rule, kind] = (c, v, local, state)
    # the oracle's copies: one server trajectory (it is the same in all six contexts), and per
    # rule and context the local weights and states of the workers that context updates
    od_w, od_v = w0.cpu().numpy().copy(), np.zeros(n, np.float32)
    hx = {(r, k, m): od_w.copy() for r in RULES for k, who in (("one", (last,)), ("some", some)) for m in who}
    hs = {key: np.zeros(n, np.float32) for key in hx}
    hp = dict(lr=wl.lr, momentum=wl.momentum, wd=wl.wd)
    grads = [torch.empty(n, dtype=torch.float32, device=DEV) for _ in range(M)]
    sg, pads = W.sigma_arena(wl, DEV), W.pad_mask(wl, DEV)
    stage = torch.empty((M, min(CHUNK, n)), dtype=torch.float32).pin_memory()
    pool = ThreadPoolExecutor(3)
    for it in range(iterations):
        for m in range(M):
            W.make_grad(wl, m, it, DEV, out=grads[m], _sigma=sg, _pads=pads)
        for (rule, kind), (c, _, _, _) in ctxs.items():
            c.fused_update(grads, last if kind == "one" else -1)
        torch.cuda.synchronize()
        for a in range(0, n, CHUNK):
            b = min(a + CHUNK, n)
            for m in range(M):
                stage[m, :b - a].copy_(grads[m][a:b], non_blocking=True)
            torch.cuda.synchronize()
            gh = [stage[m, :b - a].numpy() for m in range(M)]
            bak = np.empty(b - a, np.float32)
            oracle.global_update(gh, od_w[a:b], od_v[a:b], w_prev=bak, **hp)

            def rule_job(rule):
                for (r, k, m) in hx:
                    if r == rule:
                        hx[r, k, m][a:b] = _oracle_local(rule, bak, gh[m], hx[r, k, m][a:b].copy(), hs[r, k, m][a:b],
                                                         wl.local_lr)

            for j in [pool.submit(rule_job, r) for r in RULES]:
                j.result()
            for (rule, kind), (c, v, local, state) in ctxs.items():
                tag = f"{name} {rule}/{kind} it {it} [{a}:{b}]"
                assert_bits(c.weights()[a:b].cpu().numpy(), od_w[a:b], f"w {tag}")
                assert_bits(v[a:b].cpu().numpy(), od_v[a:b], f"v {tag}")
                for m in ((last,) if kind == "one" else some):
                    assert_bits(local[m][a:b].cpu().numpy(), hx[rule, kind, m][a:b], f"x[{m}] {tag}")
                    if rule != "dc_c":
                        assert_bits(state[m][a:b].cpu().numpy(), hs[rule, kind, m][a:b], f"state[{m}] {tag}")
    pool.shutdown()
    for c, _, _, _ in ctxs.values():
        assert c.launch_count == iterations
        c.close()
    del grads, stage, ctxs
    torch.cuda.empty_cache()


def test_alexnet_local_rules_with_extra_arenas_every_element(cuda_device):
    _run_local_rules("alexnet", 3)


def test_resnet50_local_rules_with_extra_arenas_every_element(cuda_device):
    _run_local_rules("resnet50", 3)
