"""Gradient tables bound once (odsgd_bind_grads), the worker-role local update on explicit
inputs (odsgd_worker_local_update), and the ordering guarantees of the host-buffer call.
All through the C ABI on a live device."""
import numpy as np
import pytest
import torch

import oracle
from gpu_util import DEV, assert_bits
from paper_2005_06728_b200 import binding
from paper_2005_06728_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _ctx(wl, locals_for=(0,), pingpong=True, flags=0):
    w = W.make_weights(wl, DEV)
    v = W.make_momentum(wl, DEV)
    other = torch.zeros_like(w)
    local = [torch.zeros_like(w) if m in locals_for else None for m in range(wl.n_workers)]
    ctx = binding.Odsgd(w, v, n_workers=wl.n_workers, lr=wl.lr, local_lr=wl.local_lr, momentum=wl.momentum,
                        wd=wl.wd, w_b=other if pingpong else None, w_delayed=None if pingpong else other,
                        local=local, tensor_offsets=wl.offsets, flags=flags)
    return ctx, w, v, local


def test_bound_calls_match_unbound_calls_and_the_oracle(cuda_device):
    wl = W.ragged_workload([30_000, 11, 4_001], n_workers=5)
    a, wa, va, la = _ctx(wl, (0, 3))
    b, wb, vb, lb = _ctx(wl, (0, 3))
    w_ref, v_ref = wa.cpu().numpy().copy(), va.cpu().numpy().copy()
    grads = W.make_grads(wl, 0, DEV)
    gh = [g.cpu().numpy() for g in grads]
    bound = a.bind_grads(grads)
    assert 0 <= bound.slot < binding.MAX_BINDINGS
    hp = dict(lr=wl.lr, momentum=wl.momentum, wd=wl.wd)
    for it in range(4):  # the same buffers every iteration, new contents
        for m, g in enumerate(grads):
            W.make_grad(wl, m, it, DEV, out=g)
        gh = [g.cpu().numpy() for g in grads]
        if it == 0:
            a.global_update(bound), b.global_update(grads)
            a.local_update(3), b.local_update(3)
        elif it == 1:
            a.fused_update(bound, 3), b.fused_update(grads, 3)
        elif it == 2:
            a.fused_update(bound, -1), b.fused_update(grads, -1)
        else:
            a.ssgd_step(bound), b.ssgd_step(grads)
        if it < 3:
            wp = np.empty_like(w_ref)
            oracle.global_update(gh, w_ref, v_ref, w_prev=wp, **hp)
            x3 = oracle.local_update(wp, gh[3], local_lr=wl.local_lr)
        else:
            oracle.ssgd_step(gh, w_ref, v_ref, **hp)
        torch.cuda.synchronize()
        assert torch.equal(a.weights(), b.weights()) and torch.equal(va, vb)
        assert torch.equal(la[3], lb[3]) and torch.equal(la[0], lb[0])
        assert_bits(a.weights().cpu().numpy(), w_ref, f"w it {it}")
        assert_bits(va.cpu().numpy(), v_ref, f"v it {it}")
        if it < 3:
            assert_bits(la[3].cpu().numpy(), x3, f"x[3] it {it}")
    assert a.step == b.step == 4 and a.launch_count == b.launch_count
    # the raw form used by tight loops: slot and stream handle, error code back
    rc = a.fused_update_bound_raw(bound.slot, 0, torch.cuda.current_stream().cuda_stream)
    b.fused_update(grads, 0)
    torch.cuda.synchronize()
    assert rc == binding.OK and torch.equal(a.weights(), b.weights()) and torch.equal(la[0], lb[0])
    bound.unbind()
    with pytest.raises(ValueError):
        a.fused_update(bound, 0)
    rc = a.fused_update_bound_raw(0, 0, torch.cuda.current_stream().cuda_stream)
    assert rc == binding.ERR_ARG, "the slot is empty again"


def test_state_machine_on_a_bound_table(cuda_device):
    wl = W.ragged_workload([9_000, 5], n_workers=3)
    a, _, va, la = _ctx(wl, (0, 1, 2))
    b, _, vb, lb = _ctx(wl, (0, 1, 2))
    a.set_warmup(2), b.set_warmup(2)
    grads = W.make_grads(wl, 0, DEV)
    bound = a.bind_grads(grads)
    for it in range(5):
        for m, g in enumerate(grads):
            W.make_grad(wl, m, it, DEV, out=g)
        a.step_update(bound), b.step_update(grads)
    torch.cuda.synchronize()
    assert a.iteration == b.iteration == 5
    assert torch.equal(a.weights(), b.weights()) and torch.equal(va, vb)
    assert all(torch.equal(x, y) for x, y in zip(la, lb))


def test_binding_is_refused_or_invalidated_when_buffers_overlap_state(cuda_device):
    wl = W.ragged_workload([8_192], n_workers=2)
    ctx, w, v, local = _ctx(wl, (0,))
    g = [torch.zeros(wl.arena_len, device=DEV) for _ in range(2)]
    # a table that overlaps a state buffer is refused when it is bound, not at the first call
    with pytest.raises(binding.OdsgdError) as e:
        ctx.bind_grads([g[0], v])
    assert e.value.code == binding.ERR_OVERLAP
    with pytest.raises(binding.OdsgdError) as e:
        ctx.bind_grads([g[0], torch.zeros(wl.arena_len + 1, device=DEV)[1:]])
    assert e.value.code == binding.ERR_ALIGN
    before = ctx.launch_count
    bound = ctx.bind_grads(g)
    ctx.fused_update(bound, 0)
    # the set of state buffers changes: a gradient buffer of the bound table becomes a state
    # arena.  The stale binding must not be used; binding again repeats the overlap check.
    ctx.set_local_rule(binding.LOCAL_MOMENTUM, 0.0, 0.9, 0.0, [g[1], None])
    with pytest.raises(binding.OdsgdError) as e:
        ctx.fused_update(bound, 0)
    assert e.value.code == binding.ERR_STATE
    with pytest.raises(binding.OdsgdError) as e:
        ctx.bind_grads(g)
    assert e.value.code == binding.ERR_OVERLAP, "worker_grads[1] is now the velocity arena of worker 0"
    torch.cuda.synchronize()
    assert ctx.launch_count == before + 1, "none of the refused calls launched anything"
    # all slots taken
    ctx.set_local_rule(binding.LOCAL_SGD)
    tables = [ctx.bind_grads(g) for _ in range(binding.MAX_BINDINGS - 1)]  # one slot is still held by `bound`
    with pytest.raises(binding.OdsgdError) as e:
        ctx.bind_grads(g)
    assert e.value.code == binding.ERR_UNSUPPORTED
    tables[3].unbind()
    again = ctx.bind_grads(g)
    assert again.slot == tables[3].slot or again.slot >= 0
    ctx.fused_update(again, 0)
    torch.cuda.synchronize()


@pytest.mark.parametrize("rule", ["sgd", "dc_c", "dc_a", "momentum"])
def test_worker_local_update_on_explicit_inputs(cuda_device, rule):
    """A worker-only context (no momentum arena) reproduces the oracle's local rules on explicit
    (w_bak, grad) inputs, and the local update of a full context's fused call."""
    n = 50_003
    rng = np.random.default_rng(12)
    w_bak = rng.normal(0, 1, n).astype(np.float32)
    g = rng.normal(0, 0.1, n).astype(np.float32)
    x_prev = (w_bak + rng.normal(0, 0.01, n)).astype(np.float32)
    state = np.abs(rng.normal(0, 0.01, n)).astype(np.float32)
    wd_, gd_ = torch.from_numpy(w_bak).to(DEV), torch.from_numpy(g).to(DEV)
    x = torch.from_numpy(x_prev).to(DEV)
    st = torch.from_numpy(state).to(DEV)
    ctx = binding.Odsgd(torch.zeros(n, device=DEV), None, n_workers=4, lr=0.0, local_lr=0.05, momentum=0.0, wd=0.0,
                        local=[None, None, x, None], flags=binding.FLAG_WORKER_ONLY)
    llr, lam, m, eps = 0.05, 0.04, 0.95, 1e-7
    if rule == "sgd":
        want = oracle.local_update(w_bak, g, local_lr=llr)
    elif rule == "dc_c":
        ctx.set_local_rule(binding.LOCAL_DC_C, lam)
        want = oracle.local_update_dc_c(w_bak, g, x_prev, local_lr=llr, lam=lam)
    elif rule == "dc_a":
        ctx.set_local_rule(binding.LOCAL_DC_A, lam, m, eps, [None, None, st, None])
        ms = state.copy()
        want = oracle.local_update_dc_a(w_bak, g, x_prev, ms, local_lr=llr, lam=lam, m=m, eps=eps)
    else:
        ctx.set_local_rule(binding.LOCAL_MOMENTUM, 1e-3, 0.9, 0.0, [None, None, st, None])
        ms = state.copy()
        want = oracle.local_update_momentum(w_bak, g, ms, local_lr=llr, momentum=0.9, wd=1e-3)
    ctx.worker_local_update(2, wd_, gd_)
    torch.cuda.synchronize()
    assert_bits(x.cpu().numpy(), want, f"x ({rule})")
    if rule in ("dc_a", "momentum"):
        assert_bits(st.cpu().numpy(), ms, f"state ({rule})")
    # no_delay: the gradient was taken on w_bak itself, so Eq. 4 / Eq. 5 see a zero difference
    if rule == "dc_c":
        x.copy_(torch.from_numpy(x_prev))
        ctx.worker_local_update(2, wd_, gd_, no_delay=True)
        torch.cuda.synchronize()
        assert_bits(x.cpu().numpy(), oracle.local_update_dc_c(w_bak, g, w_bak, local_lr=llr, lam=lam), "no delay")
    # a worker-only context has no server state to update
    for call in (lambda: ctx.global_update([gd_] * 4), lambda: ctx.asgd_step(0, gd_)):
        with pytest.raises(binding.OdsgdError) as e:
            call()
        assert e.value.code == binding.ERR_STATE
    with pytest.raises(binding.OdsgdError) as e:
        ctx.worker_local_update(2, x, gd_)  # the backup is the arena the call writes
    assert e.value.code == binding.ERR_OVERLAP
    with pytest.raises(binding.OdsgdError) as e:
        ctx.worker_local_update(1, wd_, gd_)  # worker 1 has no local arena
    assert e.value.code == binding.ERR_ARG


def test_host_call_validates_before_it_copies(cuda_device):
    """A refused odsgd_fused_update_host leaves the staging arenas untouched."""
    wl = W.ragged_workload([20_000], n_workers=2)
    ctx, w, v, local = _ctx(wl, (0,))
    staging = [torch.full((wl.arena_len,), 7.0, device=DEV) for _ in range(2)]
    hg = [torch.ones(wl.arena_len).pin_memory() for _ in range(2)]
    out = torch.empty(wl.arena_len).pin_memory()
    ctx.set_launch_config(1024, 0)  # too wide for the server kernel's register use
    with pytest.raises(binding.OdsgdError) as e:
        ctx.fused_update_host(hg, staging, 0, out)
    assert e.value.code == binding.ERR_UNSUPPORTED
    with pytest.raises(binding.OdsgdError) as e:
        ctx.fused_update_host(hg, staging, 1, None)  # worker 1 has no local buffer
    assert e.value.code == binding.ERR_ARG
    torch.cuda.synchronize()
    assert all(bool(torch.all(s == 7.0)) for s in staging), "no copy was enqueued by the refused calls"
    assert ctx.step == 0 and ctx.launch_count == 0
    ctx.set_launch_config(0, 0)
    ctx.fused_update_host(hg, staging, 0, out)
    torch.cuda.synchronize()
    assert all(bool(torch.all(s == 1.0)) for s in staging) and ctx.step == 1


def test_pending_copy_back_is_respected_by_every_stream(cuda_device):
    """After a host-buffer call with a separate copy stream, kernels on two other streams both
    wait for the copy-back: the first one to come by must not lift the guard for the second,
    which is the one that overwrites the local arena."""
    wl = W.ragged_workload([6_000_000], n_workers=2)
    ctx, w, v, local = _ctx(wl, (1,))
    ref, wr, vr, lr_ = _ctx(wl, (1,))
    staging = [torch.empty_like(w) for _ in range(2)]
    hg = [W.make_grad(wl, m, 0).pin_memory() for m in range(2)]
    out = torch.empty(wl.arena_len).pin_memory()
    main = torch.cuda.current_stream()
    side, s1, s2 = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream()
    g2 = W.make_grads(wl, 1, DEV)
    torch.cuda.synchronize()
    ctx.fused_update_host(hg, staging, 1, out, None, side)  # copy-back of local[1] pending on `side`
    s1.wait_stream(main)
    s2.wait_stream(main)
    ctx.global_update(g2, s1)   # first stream to come by (does not touch local[1])
    ctx.local_update(1, s2)     # second stream, independent of the first: rewrites local[1]
    ref.fused_update([g.to(DEV) for g in hg], 1)
    want_out = lr_[1].clone()
    ref.global_update(g2)
    ref.local_update(1)
    torch.cuda.synchronize()
    assert torch.equal(out, want_out.cpu()), "the copy-back saw the local weights of its own step"
    assert torch.equal(local[1], lr_[1]) and torch.equal(ctx.weights(), ref.weights())


def test_multiplier_setter_refuses_stream_capture(cuda_device):
    """The table upload (and a possible allocation) does not belong in a graph; update calls that
    use a table set beforehand can be captured."""
    wl = W.ragged_workload([4_096, 4_096], n_workers=2)
    a, _, va, la = _ctx(wl, (0,))
    b, _, vb, lb = _ctx(wl, (0,))
    grads = W.make_grads(wl, 0, DEV)
    for c in (a, b):
        c.set_tensor_multipliers([1.0, 0.5], [1.0, 0.0])
        c.fused_update(grads, 0), c.fused_update(grads, 0)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        with pytest.raises(binding.OdsgdError) as e:
            a.set_tensor_multipliers([2.0, 2.0], None)
        a.fused_update(grads, 0), a.fused_update(grads, 0)
    assert e.value.code == binding.ERR_STATE
    graph.replay()
    b.fused_update(grads, 0), b.fused_update(grads, 0)
    torch.cuda.synchronize()
    assert torch.equal(a.weights(), b.weights()) and torch.equal(va, vb) and torch.equal(la[0], lb[0])


def test_other_device_is_refused_without_a_launch(cuda_device):
    """With a second device current, every launching or allocating call answers ERR_STATE."""
    if torch.cuda.device_count() < 2:
        pytest.skip("needs two visible devices")
    wl = W.ragged_workload([4_096], n_workers=1)
    ctx, w, v, local = _ctx(wl, (0,))
    g = [torch.zeros(wl.arena_len, device=DEV)]
    with torch.cuda.device(1):
        for call in (lambda: ctx.set_tensor_multipliers([1.0], [1.0]), lambda: ctx.fused_update(g, 0),
                     lambda: ctx.asgd_step(0, g[0])):
            with pytest.raises(binding.OdsgdError) as e:
                call()
            assert e.value.code == binding.ERR_STATE
    assert ctx.launch_count == 0
