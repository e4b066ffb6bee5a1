"""Weight mirrors (odsgd_set_weight_mirrors): the server pass stores every new weight into further
buffers as well - the other ranks' replicas when the server role is sharded.  Here the mirrors are
ordinary buffers of the one device; the kernel cannot tell the difference.  Through the C ABI,
against the CPU oracle, bit for bit."""
import numpy as np
import pytest
import torch

import oracle
from gpu_util import DEV, GUARD, POISON, assert_bits
from paper_2005_06728_b200 import binding
from paper_2005_06728_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _guarded(n, fill=POISON):
    """A buffer of n floats inside a poisoned guard band, itself poisoned: a mirror is write-only,
    so whatever survives a call was not written."""
    pad = (-n) % 4
    whole = torch.full((GUARD + n + pad + GUARD,), POISON, dtype=torch.float32, device=DEV)
    view = whole[GUARD:GUARD + n]
    view.fill_(fill)
    return view, whole


def _guards_ok(whole, n):
    return bool(torch.all(whole[:GUARD] == POISON)) and bool(torch.all(whole[GUARD + n:] == POISON))


@pytest.mark.parametrize("n,M,n_mirrors", [(1, 1, 1), (7, 2, 3), (4_099, 3, 2), (100_003, 4, 7), (65_536, 8, 15),
                                           (300_001, 17, 1), (33_333, 5, 4)])
@pytest.mark.parametrize("pingpong", [True, False])
def test_mirrors_receive_the_new_weights_bit_for_bit(cuda_device, n, M, n_mirrors, pingpong):
    """Global updates and an SSGD step with mirrors set: every mirror of the half that was written
    equals that half; the mirrors of the other half are untouched; results equal the oracle's.
    The worker counts cover every launch shape of the server kernel, the sizes a ragged tail."""
    wl = W.ragged_workload([n], n_workers=M, lr=0.1, local_lr=0.05, momentum=0.9, wd=1e-3, seed=11)
    w = W.make_weights(wl, DEV)[:n].clone()
    v = torch.zeros(n, device=DEV)
    other = torch.zeros(n, device=DEV)
    ctx = binding.Odsgd(w, v, n_workers=M, lr=wl.lr, local_lr=wl.local_lr, momentum=wl.momentum, wd=wl.wd,
                        w_b=other if pingpong else None, w_delayed=None if pingpong else other)
    ma = [_guarded(n) for _ in range(n_mirrors)]
    mb = [_guarded(n) for _ in range(n_mirrors)] if pingpong else None
    ctx.set_weight_mirrors([t for t, _ in ma], [t for t, _ in mb] if pingpong else None)
    w_ref, v_ref = w.cpu().numpy().copy(), v.cpu().numpy().copy()
    hp = dict(lr=wl.lr, momentum=wl.momentum, wd=wl.wd)
    grads = [torch.empty(n, device=DEV) for _ in range(M)]
    bound = ctx.bind_grads(grads)
    written = {0: False, 1: False}
    for it in range(4):
        for m, g in enumerate(grads):
            g.copy_(W.make_grad(wl, m, it, DEV)[:n])
        gh = [g.cpu().numpy() for g in grads]
        if it == 3:
            ctx.ssgd_step(bound)
            oracle.ssgd_step(gh, w_ref, v_ref, **hp)
        else:
            ctx.global_update(bound if it else grads)  # the unbound call takes the same path
            oracle.global_update(gh, w_ref, v_ref, **hp)
        torch.cuda.synchronize()
        cur = ctx.weights()
        half = 1 if (pingpong and cur.data_ptr() == other.data_ptr()) else 0
        written[half] = True
        assert_bits(cur.cpu().numpy(), w_ref, f"weights, iteration {it}")
        assert_bits(v.cpu().numpy(), v_ref, f"momentum, iteration {it}")
        for i, (t, whole) in enumerate(mb if half else ma):
            assert torch.equal(t.view(torch.int32), cur.view(torch.int32)), f"mirror {i} of half {half}, iteration {it}"
            assert _guards_ok(whole, n), "a store went outside a mirror"
        for h, tab in ((0, ma), (1, mb)):
            if tab is not None and not written[h]:
                assert all(bool(torch.all(t == POISON)) for t, _ in tab), "mirrors of the half not written stay as they were"
    assert written[0] and (written[1] or not pingpong)
    # switched off: the next update leaves the mirrors alone
    ctx.set_weight_mirrors(None)
    snap = [t.clone() for t, _ in ma]
    for _ in range(2):
        ctx.global_update(grads)
    torch.cuda.synchronize()
    assert all(torch.equal(a, t) for a, (t, _) in zip(snap, ma))
    ctx.close()


def test_mirrors_with_per_tensor_multipliers_and_the_scalar_path(cuda_device):
    """The mirrored pass also exists with per-tensor multipliers and on 4-byte-aligned pointers."""
    wl = W.ragged_workload([1000, 12, 5_003, 4], n_workers=3, lr=0.1, momentum=0.9, wd=1e-2)
    n = wl.arena_len
    lr_mult, wd_mult = [1.0, 0.5, 2.0, 0.0], [1.0, 0.0, 1.0, 0.0]
    for shift in (0, 1):  # shift 1: every pointer 4 bytes off a 16-byte boundary
        flags = binding.FLAG_ALLOW_UNALIGNED if shift else 0
        buf = lambda: torch.zeros(n + 4, device=DEV)[shift:shift + n]
        w = buf()
        w.copy_(W.make_weights(wl, DEV))
        v, wb = buf(), buf()
        ctx = binding.Odsgd(w, v, n_workers=3, lr=wl.lr, local_lr=wl.local_lr, momentum=wl.momentum, wd=wl.wd,
                            w_b=wb, tensor_offsets=wl.offsets, flags=flags)
        ctx.set_tensor_multipliers(lr_mult, wd_mult)
        ma, mb = [buf(), buf()], [buf(), buf()]
        ctx.set_weight_mirrors(ma, mb)
        w_ref, v_ref = w.cpu().numpy().copy(), v.cpu().numpy().copy()
        for it in range(2):
            grads = [W.make_grad(wl, m, it, DEV) for m in range(3)]
            if shift:
                gs = [buf() for _ in range(3)]
                for a, g in zip(gs, grads):
                    a.copy_(g)
                grads = gs
            ctx.global_update(grads)
            oracle.global_update_mult([np.ascontiguousarray(g.cpu().numpy()) for g in grads], w_ref, v_ref,
                                      lr=wl.lr, momentum=wl.momentum, wd=wl.wd, offsets=wl.offsets,
                                      lr_mult=np.asarray(lr_mult, np.float32), wd_mult=np.asarray(wd_mult, np.float32))
            torch.cuda.synchronize()
            assert_bits(ctx.weights().cpu().numpy(), w_ref, f"shift {shift}, iteration {it}")
            for t in (mb if it == 0 else ma):
                assert torch.equal(t.view(torch.int32), ctx.weights().view(torch.int32))
        ctx.close()


def test_mirror_tables_are_validated(cuda_device):
    n = 4096
    mk = lambda: torch.zeros(n, device=DEV)
    w, v, wb, loc = mk(), mk(), mk(), mk()
    ctx = binding.Odsgd(w, v, n_workers=2, lr=0.1, local_lr=0.1, momentum=0.9, wd=0.0, w_b=wb, local=[loc, None])
    grads = [mk(), mk()]
    bound = ctx.bind_grads(grads)

    def refused(code, *args):
        with pytest.raises(binding.OdsgdError) as e:
            ctx.set_weight_mirrors(*args)
        assert e.value.code == code, str(e.value)

    refused(binding.ERR_ARG, [mk()], None)                        # ping-pong layout needs both tables
    refused(binding.ERR_ARG, [mk()] * 16, [mk()] * 16)            # more than ODSGD_MAX_MIRRORS
    refused(binding.ERR_OVERLAP, [w], [mk()])                     # a mirror that is a state arena
    refused(binding.ERR_OVERLAP, [mk()], [loc])
    m = mk()
    refused(binding.ERR_OVERLAP, [m], [m])                        # two mirrors on the same memory
    big = torch.zeros(n + 4, device=DEV)
    refused(binding.ERR_ALIGN, [big[1:n + 1]], [mk()])
    # nothing above took effect: the fused call still runs, and the bound table is still valid
    ctx.fused_update(bound, 0)
    ma, mb = [mk()], [mk()]
    ctx.set_weight_mirrors(ma, mb)
    # setting mirrors changes the set of state buffers: the table has to be bound again ...
    with pytest.raises(binding.OdsgdError) as e:
        ctx.global_update(bound)
    assert e.value.code == binding.ERR_STATE
    # ... a gradient buffer that is a mirror is refused ...
    with pytest.raises(binding.OdsgdError) as e:
        ctx.global_update([grads[0], ma[0]])
    assert e.value.code == binding.ERR_OVERLAP
    # ... and the calls that would leave the mirrors stale are refused, with nothing launched
    launches = ctx.launch_count
    for call in (lambda: ctx.fused_update(grads, 0), lambda: ctx.fused_update(grads, -1),
                 lambda: ctx.step_update(grads), lambda: ctx.asgd_step(0, grads[0]),
                 lambda: ctx.fused_update_mult_static(grads, 0, None, None)):
        with pytest.raises(binding.OdsgdError) as e:
            call()
        assert e.value.code == binding.ERR_STATE, str(e.value)
    assert ctx.launch_count == launches
    ctx.global_update(grads)
    torch.cuda.synchronize()
    assert ctx.launch_count == launches + 1
    ctx.close()
    # in-place layout: mirrors_b must be NULL; a worker-only context has nothing to mirror
    c2 = binding.Odsgd(mk(), mk(), n_workers=1, lr=0.1, local_lr=0.1, momentum=0.0, wd=0.0)
    with pytest.raises(binding.OdsgdError) as e:
        c2.set_weight_mirrors([mk()], [mk()])
    assert e.value.code == binding.ERR_ARG
    c2.close()
    c3 = binding.Odsgd(mk(), None, n_workers=1, lr=0.1, local_lr=0.1, momentum=0.0, wd=0.0, local=[mk()],
                       flags=binding.FLAG_WORKER_ONLY)
    with pytest.raises(binding.OdsgdError) as e:
        c3.set_weight_mirrors([mk()], None)
    assert e.value.code == binding.ERR_STATE
    c3.close()


def test_gradients_and_mirrors_outside_device_memory(cuda_device):
    """The kernel reaches memory that is not this GPU's own with the same plain loads and stores:
    here page-locked host memory, which the device addresses over the bus under the process's
    unified addressing - the one kind of non-local memory a single-GPU machine offers.  One
    gradient is read from there and one mirror per weight half is written there.  Raw pointers,
    so this goes through the C entry points directly."""
    n, M = 50_003, 3
    wl = W.ragged_workload([n], n_workers=M, lr=0.1, local_lr=0.05, momentum=0.9, wd=1e-3, seed=21)
    w = W.make_weights(wl, DEV)[:n].clone()
    v, wb = torch.zeros(n, device=DEV), torch.zeros(n, device=DEV)
    ctx = binding.Odsgd(w, v, n_workers=M, lr=wl.lr, local_lr=wl.local_lr, momentum=wl.momentum, wd=wl.wd, w_b=wb)
    lib, h = binding.load_library(), ctx._h
    host_g = torch.empty(n, dtype=torch.float32).pin_memory()
    host_ma = torch.full((n,), POISON, dtype=torch.float32).pin_memory()
    host_mb = torch.full((n,), POISON, dtype=torch.float32).pin_memory()
    dev_ma, dev_mb = torch.zeros(n, device=DEV), torch.zeros(n, device=DEV)
    assert all(t.data_ptr() % 16 == 0 for t in (host_g, host_ma, host_mb))
    ta = binding._ptr_table([dev_ma.data_ptr(), host_ma.data_ptr()])
    tb = binding._ptr_table([dev_mb.data_ptr(), host_mb.data_ptr()])
    ctx.check(lib.odsgd_set_weight_mirrors(h, ta, tb, 2))
    dev_g = [torch.empty(n, device=DEV) for _ in range(M)]
    table = binding._ptr_table([dev_g[0].data_ptr(), host_g.data_ptr(), dev_g[2].data_ptr()])
    w_ref, v_ref = w.cpu().numpy().copy(), v.cpu().numpy().copy()
    stream = torch.cuda.current_stream().cuda_stream
    for it in range(3):
        gh = []
        for m in range(M):
            g = W.make_grad(wl, m, it, DEV)[:n]
            if m == 1:
                host_g.copy_(g)
            else:
                dev_g[m].copy_(g)
            gh.append(g.cpu().numpy())
        torch.cuda.synchronize()
        ctx.check(lib.odsgd_global_update(h, table, stream))
        torch.cuda.synchronize()
        oracle.global_update(gh, w_ref, v_ref, lr=wl.lr, momentum=wl.momentum, wd=wl.wd)
        cur = w if it % 2 else wb
        assert_bits(cur.cpu().numpy(), w_ref, f"weights, iteration {it}")
        host_m, dev_m = (host_ma, dev_ma) if it % 2 else (host_mb, dev_mb)
        assert_bits(host_m.numpy(), w_ref, f"mirror in host memory, iteration {it}")
        assert_bits(dev_m.cpu().numpy(), w_ref, f"mirror in device memory, iteration {it}")
    ctx.close()
