"""GPU parity for the rules beyond the five core kernels: per-tensor multipliers, the
delay-compensated local updaters over several iterations, DC-ASGD at the server, and the
warm-up / switching state machine of Algorithm 2.  All through the C ABI, bit-exact in the
deterministic flavour."""
import numpy as np
import pytest
import torch

import oracle
import pins
from gpu_util import DEV, GpuImpl, assert_bits, assert_close_scaled, server_scales
from paper_2005_06728_b200 import binding
from paper_2005_06728_b200 import workloads as W

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("pingpong", [True, False], ids=["pingpong", "inplace"])
@pytest.mark.parametrize("pin", pins.EXT_PINS, ids=lambda f: f.__name__)
def test_ext_pins_on_gpu(cuda_device, pin, pingpong):
    pin(GpuImpl(deterministic=True, pingpong=pingpong))


def test_ext_pins_default_flavour_hand_examples(cuda_device):
    # dyadic hand examples hold with or without fused multiply-add
    impl = GpuImpl(deterministic=False)
    g = pins.read_golden("per_tensor_multipliers.txt")
    w1, v1, _ = impl.global_update_mult([pins.a32(g["g0"]), pins.a32(g["g1"])], pins.a32(g["w"]), pins.a32(g["v"]),
                                        0.5, 0.5, 0.25, [0, 4, 8], pins.a32(g["lr_mult"]), pins.a32(g["wd_mult"]))
    assert np.array_equal(w1, pins.a32(g["w1"])) and np.array_equal(v1, pins.a32(g["v1"]))


def _mults(wl, seed=3):
    rng = np.random.default_rng(seed)
    lr_mult = np.where(rng.random(wl.n_tensors) < 0.3, rng.choice([0.0, 0.1, 2.0, 10.0], wl.n_tensors), 1.0)
    wd_mult = np.array([1.0 if t.kind == "weight" else 0.0 for t in wl.tensors])
    return lr_mult.astype(np.float32), wd_mult.astype(np.float32)


@pytest.mark.parametrize("name", ["resnet56", "lenet5"])
def test_multipliers_on_many_small_tensors(cuda_device, name):
    """No decay on biases and batch-norm tensors, assorted learning-rate multipliers, 167 tensors
    from 10 to 36,864 elements in one launch; fused with every worker's local update."""
    wl = W.workload(name)
    M = wl.n_workers
    lr_mult, wd_mult = _mults(wl)
    for det in (True, False):
        w = W.make_weights(wl, DEV)
        v = W.make_momentum(wl, DEV)
        local = [torch.zeros_like(w) for _ in range(M)]
        ctx = binding.Odsgd(w, v, n_workers=M, lr=wl.lr, local_lr=wl.local_lr, momentum=wl.momentum, wd=wl.wd,
                            w_b=torch.zeros_like(w), local=local, tensor_offsets=wl.offsets,
                            flags=binding.FLAG_DETERMINISTIC if det else binding.FLAG_ALLOW_FMA)
        ctx.set_tensor_multipliers(lr_mult.tolist(), wd_mult.tolist())
        w_ref, v_ref = w.cpu().numpy().copy(), v.cpu().numpy().copy()
        for it in range(4):
            grads = W.make_grads(wl, it, DEV)
            gh = [g.cpu().numpy() for g in grads]
            w0, v0 = w_ref.copy(), v_ref.copy()
            ctx.fused_update(grads, -1)
            wp = np.empty_like(w_ref)
            oracle.global_update_mult(gh, w_ref, v_ref, lr=wl.lr, momentum=wl.momentum, wd=wl.wd,
                                      offsets=wl.offsets, lr_mult=lr_mult, wd_mult=wd_mult, w_prev=wp)
            torch.cuda.synchronize()
            if det:
                assert_bits(ctx.weights().cpu().numpy(), w_ref, f"{name} w it {it}")
                assert_bits(v.cpu().numpy(), v_ref, f"{name} v it {it}")
                for m in (0, M - 1):
                    assert_bits(local[m].cpu().numpy(), oracle.local_update(wp, gh[m], local_lr=wl.local_lr), "x")
            else:
                sw, sv = server_scales(gh, w0, v0, wl.lr * float(lr_mult.max()), wl.momentum, wl.wd)
                assert_close_scaled(ctx.weights().cpu().numpy(), w_ref, sw, "w")
                assert_close_scaled(v.cpu().numpy(), v_ref, sv, "v")
                ctx.weights().copy_(torch.from_numpy(w_ref))
                v.copy_(torch.from_numpy(v_ref))
        assert ctx.launch_count == 4
        # switching the feature off restores the plain rule
        ctx.set_tensor_multipliers(None, None)
        grads = W.make_grads(wl, 9, DEV)
        ctx.ssgd_step(grads)
        oracle.ssgd_step([g.cpu().numpy() for g in grads], w_ref, v_ref, lr=wl.lr, momentum=wl.momentum, wd=wl.wd)
        torch.cuda.synchronize()
        if det:
            assert_bits(ctx.weights().cpu().numpy(), w_ref, "plain rule after switching multipliers off")
        ctx.close()


def test_multipliers_with_offsets_that_split_vectors(cuda_device):
    """Tensor boundaries that are not multiples of 4 elements: refused on the 128-bit path,
    exact on the scalar path."""
    sizes = [5, 1, 1022, 3, 70_001, 2]
    offs = np.concatenate([[0], np.cumsum(sizes)]).tolist()
    n = offs[-1]
    rng = np.random.default_rng(0)
    w, v = rng.normal(0, 1, n).astype(np.float32), rng.normal(0, 0.1, n).astype(np.float32)
    grads = [rng.normal(0, 0.1, n).astype(np.float32) for _ in range(3)]
    lm = np.array([1, 0.5, 2, 0, 1.5, 3], np.float32)
    wm = np.array([1, 0, 1, 0, 0.5, 1], np.float32)
    wd_, vd = torch.from_numpy(w).to(DEV), torch.from_numpy(v).to(DEV)
    kw = dict(n_workers=3, lr=0.1, local_lr=0.1, momentum=0.9, wd=1e-2, tensor_offsets=offs)
    strict = binding.Odsgd(wd_, vd, flags=binding.FLAG_DETERMINISTIC, **kw)
    with pytest.raises(binding.OdsgdError) as e:
        strict.set_tensor_multipliers(lm.tolist(), wm.tolist())
    assert e.value.code == binding.ERR_ALIGN
    strict.close()
    ctx = binding.Odsgd(wd_, vd, flags=binding.FLAG_DETERMINISTIC | binding.FLAG_ALLOW_UNALIGNED, **kw)
    ctx.set_tensor_multipliers(lm.tolist(), wm.tolist())
    ctx.ssgd_step([torch.from_numpy(g).to(DEV) for g in grads])
    oracle.global_update_mult(grads, w, v, lr=0.1, momentum=0.9, wd=1e-2, offsets=offs, lr_mult=lm, wd_mult=wm)
    torch.cuda.synchronize()
    assert_bits(wd_.cpu().numpy(), w, "w")
    assert_bits(vd.cpu().numpy(), v, "v")


def _dc_oracle_local(rule, wp, g, x_prev, ms, llr, lam, m, eps):
    if rule == binding.LOCAL_SGD:
        return oracle.local_update(wp, g, local_lr=llr)
    if rule == binding.LOCAL_DC_C:
        return oracle.local_update_dc_c(wp, g, x_prev, local_lr=llr, lam=lam)
    if rule == binding.LOCAL_MOMENTUM:
        return oracle.local_update_momentum(wp, g, ms, local_lr=llr, momentum=m, wd=lam)
    return oracle.local_update_dc_a(wp, g, x_prev, ms, local_lr=llr, lam=lam, m=m, eps=eps)


@pytest.mark.parametrize("rule", [binding.LOCAL_SGD, binding.LOCAL_DC_C, binding.LOCAL_DC_A, binding.LOCAL_MOMENTUM],
                         ids=["sgd", "dc_c", "dc_a", "momentum"])
@pytest.mark.parametrize("wp", [0, 1, 3])
@pytest.mark.parametrize("layout", ["pingpong", "inplace"])
def test_algorithm2_state_machine(cuda_device, rule, wp, layout):
    """odsgd_step: wp SSGD iterations, then fused global + local updates; the first local
    update (iteration wp) sees no delay; the chain x_prev -> x runs through the local arenas.
    In the in-place layout the weights are overwritten by the same pass that, at iteration wp,
    reads them a second time as x_prev."""
    wl = W.ragged_workload([3000, 17, 40_004, 5], n_workers=3, lr=0.05, local_lr=0.04, momentum=0.9, wd=1e-3)
    M, n = 3, wl.arena_len
    lam, m_, eps = 0.5, 0.95, 1e-7
    w = W.make_weights(wl, DEV)
    v = W.make_momentum(wl, DEV)
    w_b = torch.zeros_like(w)
    local = [torch.full_like(w, 777.0) for _ in range(M)]  # junk: must never be read as x_prev at iteration wp
    msq = [torch.zeros_like(w) for _ in range(M)]
    ctx = binding.Odsgd(w, v, n_workers=M, lr=wl.lr, local_lr=wl.local_lr, momentum=wl.momentum, wd=wl.wd,
                        w_b=w_b if layout == "pingpong" else None, w_delayed=None if layout == "pingpong" else w_b,
                        local=local, tensor_offsets=wl.offsets, flags=binding.FLAG_DETERMINISTIC)
    has_state = rule in (binding.LOCAL_DC_A, binding.LOCAL_MOMENTUM)
    ctx.set_local_rule(rule, lam, m_, eps, msq if has_state else None)
    ctx.set_warmup(wp)
    w_ref, v_ref = w.cpu().numpy().copy(), v.cpu().numpy().copy()
    x_ref = [None] * M
    ms_ref = [np.zeros(n, np.float32) for _ in range(M)]
    for k in range(wp + 4):
        # the arena each worker trains on
        for mm in range(M):
            t = ctx.train_weights(mm)
            if k <= wp:
                assert t.data_ptr() == ctx.weights().data_ptr(), f"iteration {k}: workers train on the global weights"
            else:
                assert t.data_ptr() == local[mm].data_ptr(), f"iteration {k}: workers train on their local weights"
        grads = W.make_grads(wl, k, DEV)
        gh = [g.cpu().numpy() for g in grads]
        ctx.step_update(grads)
        wprev = np.empty_like(w_ref)
        if k < wp:
            oracle.ssgd_step(gh, w_ref, v_ref, lr=wl.lr, momentum=wl.momentum, wd=wl.wd)
        else:
            oracle.global_update(gh, w_ref, v_ref, lr=wl.lr, momentum=wl.momentum, wd=wl.wd, w_prev=wprev)
            for mm in range(M):
                xp = wprev if k == wp else x_ref[mm]
                x_ref[mm] = _dc_oracle_local(rule, wprev, gh[mm], xp, ms_ref[mm], wl.local_lr, lam, m_, eps)
        torch.cuda.synchronize()
        assert_bits(ctx.weights().cpu().numpy(), w_ref, f"w at iteration {k}")
        assert_bits(v.cpu().numpy(), v_ref, f"v at iteration {k}")
        if k >= wp:
            for mm in range(M):
                assert_bits(local[mm].cpu().numpy(), x_ref[mm], f"x[{mm}] at iteration {k}")
                if has_state:
                    assert_bits(msq[mm].cpu().numpy(), ms_ref[mm], f"state arena [{mm}] at iteration {k}")
    with pytest.raises(binding.OdsgdError) as e:
        ctx.set_warmup(5)
    assert e.value.code == binding.ERR_STATE


@pytest.mark.parametrize("rule", [binding.LOCAL_DC_C, binding.LOCAL_DC_A, binding.LOCAL_MOMENTUM],
                         ids=["dc_c", "dc_a", "momentum"])
@pytest.mark.parametrize("M", [1, 2, 3, 4, 5, 8, 12, 13, 16, 33, 64])
@pytest.mark.parametrize("layout", ["pingpong", "inplace"])
def test_fused_one_worker_with_extra_arenas_over_worker_counts(cuda_device, rule, M, layout):
    """One worker's Eq. 4 / Eq. 5-6 / momentum update inside the server pass, for every launch
    shape of the kernel (the worker counts), for the first, a middle and the last worker (the
    update is computed where that worker's gradient comes by in the sum), on a ragged arena of
    several tiles, with per-tensor multipliers on the server rule in one of the steps.  The
    chain x_prev -> x and the state arenas run through three calls; bit for bit against the
    oracle."""
    wl = W.ragged_workload([9_001, 7, 11_000, 3], n_workers=M, lr=0.05, local_lr=0.04, momentum=0.9, wd=1e-3, seed=M)
    n = wl.arena_len
    lam, m_, eps = 0.5, 0.95, 1e-7
    has_state = rule in (binding.LOCAL_DC_A, binding.LOCAL_MOMENTUM)
    workers = sorted({0, M // 2, M - 1})
    w = W.make_weights(wl, DEV)
    v = W.make_momentum(wl, DEV)
    other = torch.zeros_like(w)
    local = [w.clone() + 0.01 * (i + 1) if i in workers else None for i in range(M)]
    msq = [torch.zeros_like(w) if i in workers else None for i in range(M)]
    ctx = binding.Odsgd(w, v, n_workers=M, lr=wl.lr, local_lr=wl.local_lr, momentum=wl.momentum, wd=wl.wd,
                        w_b=other if layout == "pingpong" else None, w_delayed=None if layout == "pingpong" else other,
                        local=local, tensor_offsets=wl.offsets)
    ctx.set_local_rule(rule, lam, m_, eps, msq if has_state else None)
    w_ref, v_ref = w.cpu().numpy().copy(), v.cpu().numpy().copy()
    x_ref = {i: local[i].cpu().numpy().copy() for i in workers}
    ms_ref = {i: np.zeros(n, np.float32) for i in workers}
    lr_mult = np.asarray([1.0, 0.0, 2.0, 0.5], np.float32)
    wd_mult = np.asarray([1.0, 0.0, 1.0, 0.0], np.float32)
    hp = dict(lr=wl.lr, momentum=wl.momentum, wd=wl.wd)
    for it, wk in enumerate(workers + [workers[0]]):
        grads = W.make_grads(wl, it, DEV)
        gh = [g.cpu().numpy() for g in grads]
        mult = it == 1
        ctx.set_tensor_multipliers(lr_mult.tolist() if mult else None, wd_mult.tolist() if mult else None)
        ctx.fused_update(grads, wk)
        wprev = np.empty_like(w_ref)
        if mult:
            oracle.global_update_mult(gh, w_ref, v_ref, offsets=wl.offsets, lr_mult=lr_mult, wd_mult=wd_mult,
                                      w_prev=wprev, **hp)
        else:
            oracle.global_update(gh, w_ref, v_ref, w_prev=wprev, **hp)
        x_ref[wk] = _dc_oracle_local(rule, wprev, gh[wk], x_ref[wk], ms_ref[wk], wl.local_lr, lam, m_, eps)
        torch.cuda.synchronize()
        assert_bits(ctx.weights().cpu().numpy(), w_ref, f"w, call {it}")
        assert_bits(v.cpu().numpy(), v_ref, f"v, call {it}")
        for i in workers:  # the updated worker's arenas moved on, the others' are untouched
            assert_bits(local[i].cpu().numpy(), x_ref[i], f"x[{i}], call {it} (updated worker {wk})")
            if has_state:
                assert_bits(msq[i].cpu().numpy(), ms_ref[i], f"state[{i}], call {it}")
    ctx.close()


@pytest.mark.parametrize("rule", [binding.LOCAL_DC_C, binding.LOCAL_DC_A, binding.LOCAL_MOMENTUM],
                         ids=["dc_c", "dc_a", "momentum"])
def test_separate_dc_local_update_equals_fused(cuda_device, rule):
    wl = W.ragged_workload([10_000, 33], n_workers=2)
    ctxs = []
    for _ in range(2):
        w = W.make_weights(wl, DEV)
        v = W.make_momentum(wl, DEV)
        local = [w.clone(), w.clone()]
        ms = [torch.zeros_like(w), torch.zeros_like(w)]
        c = binding.Odsgd(w, v, n_workers=2, lr=wl.lr, local_lr=wl.local_lr, momentum=wl.momentum, wd=wl.wd,
                          w_b=torch.zeros_like(w), local=local, flags=binding.FLAG_DETERMINISTIC)
        c.set_local_rule(rule, 0.3, 0.9, 1e-6, ms if rule != binding.LOCAL_DC_C else None)
        ctxs.append((c, v, local, ms))
    for it in range(3):
        grads = W.make_grads(wl, it, DEV)
        ctxs[0][0].fused_update(grads, -1)
        ctxs[1][0].global_update(grads)
        ctxs[1][0].local_update(1)
        ctxs[1][0].local_update(0)
        torch.cuda.synchronize()
        for m in range(2):
            assert torch.equal(ctxs[0][2][m], ctxs[1][2][m]) and torch.equal(ctxs[0][3][m], ctxs[1][3][m])
        assert torch.equal(ctxs[0][0].weights(), ctxs[1][0].weights())
    # a worker without its mean-square arena cannot be updated under DC_A
    if rule != binding.LOCAL_DC_C:
        c = ctxs[0][0]
        c.set_local_rule(rule, 0.3, 0.9, 1e-6, [ctxs[0][3][0], None])
        with pytest.raises(binding.OdsgdError) as e:
            c.fused_update(W.make_grads(wl, 5, DEV), 1)
        assert e.value.code == binding.ERR_STATE


@pytest.mark.parametrize("rule", [binding.LOCAL_DC_C, binding.LOCAL_DC_A], ids=["dc_c", "dc_a"])
def test_dcasgd_server_sequence(cuda_device, rule):
    """Three workers deliver gradients in a scrambled order; each keeps the copy it pulled last."""
    wl = W.ragged_workload([50_001, 7], n_workers=3, lr=0.05)
    n = wl.arena_len
    lam, m_, eps = 0.4, 0.9, 1e-6
    for det in (True, False):
        w = W.make_weights(wl, DEV)
        v = W.make_momentum(wl, DEV)
        local = [w.clone() for _ in range(3)]
        ms = torch.zeros_like(w)
        ctx = binding.Odsgd(w, v, n_workers=3, lr=wl.lr, local_lr=9.0, momentum=0.9, wd=0.5, local=local,
                            flags=binding.FLAG_DETERMINISTIC if det else binding.FLAG_ALLOW_FMA)
        with pytest.raises(binding.OdsgdError) as e:
            ctx.dcasgd_step(0, W.make_grad(wl, 0, 0, DEV))
        assert e.value.code == binding.ERR_STATE  # rule still SGD
        ctx.set_local_rule(rule, lam, m_, eps, None)
        if rule == binding.LOCAL_DC_A:
            with pytest.raises(binding.OdsgdError) as e:
                ctx.dcasgd_step(0, W.make_grad(wl, 0, 0, DEV))
            assert e.value.code == binding.ERR_STATE  # no server mean-square arena yet
            ctx.set_server_mean_square(ms)
        w_ref = w.cpu().numpy().copy()
        bak = [w_ref.copy() for _ in range(3)]
        ms_ref = np.zeros(n, np.float32)
        for it, worker in enumerate([0, 1, 1, 2, 0, 2, 2, 1]):
            g = W.make_grad(wl, worker, it, DEV)
            gh = g.cpu().numpy()
            w_before = w_ref.copy()
            ctx.dcasgd_step(worker, g)
            if rule == binding.LOCAL_DC_C:
                oracle.dcasgd_step_c(gh, w_ref, bak[worker], lr=wl.lr, lam=lam)
            else:
                oracle.dcasgd_step_a(gh, w_ref, bak[worker], ms_ref, lr=wl.lr, lam=lam, m=m_, eps=eps)
            torch.cuda.synchronize()
            if det:
                assert_bits(w.cpu().numpy(), w_ref, f"w after gradient {it}")
                assert_bits(local[worker].cpu().numpy(), bak[worker], f"backup of worker {worker}")
                if rule == binding.LOCAL_DC_A:
                    assert_bits(ms.cpu().numpy(), ms_ref, "server mean square")
            else:
                scale = np.abs(w_before.astype(np.float64)) + wl.lr * np.abs(gh.astype(np.float64)) * (1 + 4.0)
                assert_close_scaled(w.cpu().numpy(), w_ref, scale, "w", tol=2e-6)
                w.copy_(torch.from_numpy(w_ref))
                local[worker].copy_(torch.from_numpy(bak[worker]))
                ms.copy_(torch.from_numpy(ms_ref))
        assert torch.all(v == 0), "Eq. 4/5 carry no momentum: v is untouched"
        ctx.close()


def test_checkpoint_resume_reproduces_the_run(cuda_device):
    """Stop after iteration 4 of a run with wp = 2 and the Eq. 5-6 local rule, rebuild a context
    from the saved arenas and the saved iteration index, and finish: same bits as the
    uninterrupted run."""
    wl = W.ragged_workload([20_000, 9, 4_001], n_workers=2, lr=0.05, local_lr=0.04)
    total, stop = 7, 4

    def make(state=None):
        if state is None:
            w = W.make_weights(wl, DEV)
            v = W.make_momentum(wl, DEV)
            local = [torch.zeros_like(w) for _ in range(2)]
            ms = [torch.zeros_like(w) for _ in range(2)]
        else:
            w, v, local, ms = state
        ctx = binding.Odsgd(w, v, n_workers=2, lr=wl.lr, local_lr=wl.local_lr, momentum=wl.momentum, wd=wl.wd,
                            w_b=torch.zeros_like(w), local=local, tensor_offsets=wl.offsets,
                            flags=binding.FLAG_DETERMINISTIC)
        ctx.set_local_rule(binding.LOCAL_DC_A, 0.5, 0.9, 1e-6, ms)
        ctx.set_warmup(2)
        return ctx, v, local, ms

    ref, v_ref, loc_ref, ms_ref = make()
    for k in range(total):
        ref.step_update(W.make_grads(wl, k, DEV))
    a, v_a, loc_a, ms_a = make()
    for k in range(stop):
        a.step_update(W.make_grads(wl, k, DEV))
    torch.cuda.synchronize()
    saved = (a.weights().clone(), v_a.clone(), [t.clone() for t in loc_a], [t.clone() for t in ms_a])
    saved_iter = a.iteration
    assert saved_iter == stop
    a.close()
    b, v_b, loc_b, ms_b = make(saved)
    b.iteration = saved_iter
    for k in range(stop, total):
        for m in range(2):
            assert b.train_weights(m).data_ptr() == loc_b[m].data_ptr()
        b.step_update(W.make_grads(wl, k, DEV))
    torch.cuda.synchronize()
    assert torch.equal(b.weights(), ref.weights()) and torch.equal(v_b, v_ref)
    for m in range(2):
        assert torch.equal(loc_b[m], loc_ref[m]) and torch.equal(ms_b[m], ms_ref[m])
