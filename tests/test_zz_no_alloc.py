"""The allocation-free fused update (odsgd_fused_update_mult_static) against the regular path.

Some users of this library run where a cudaMalloc is off limits: a parameter-server loop
sharing the GPU with training streams (cudaMalloc synchronises the whole device), or a process
whose device memory was handed to a framework's pool.  For them the per-tensor multiplier
table lives in a fixed array inside the library.  This test drives that entry point through the
C ABI and checks that it produces exactly what odsgd_set_tensor_multipliers + odsgd_fused_update
produce, twice in a row with different multipliers (the shared array keeps the previous call's
table, which must not leak into the next call), that both agree with the CPU oracle, that the
amount of free device memory does not move across the calls, and that the call refuses to be
recorded into a stream capture.

Collected last on purpose (file name), so a failure here cannot hide the other tests.  It must
pass alone in a fresh process and after the rest of the suite.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2005_06728_b200 import binding
from paper_2005_06728_b200 import workloads as W

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _pair(wl, flags):
    """Two contexts over identical, independent copies of the state."""
    out = []
    for _ in range(2):
        w = W.make_weights(wl, DEV)
        v = W.make_momentum(wl, DEV)
        v.normal_(0, 0.01, generator=torch.Generator(device=DEV).manual_seed(5))
        local = [None] * wl.n_workers
        local[1] = torch.zeros_like(w)
        ctx = binding.Odsgd(w, v, n_workers=wl.n_workers, lr=wl.lr, local_lr=wl.local_lr, momentum=wl.momentum,
                            wd=wl.wd, w_b=torch.zeros_like(w), local=local, tensor_offsets=wl.offsets, flags=flags)
        out.append((ctx, v, local[1]))
    return out


@pytest.mark.parametrize("flags", [0, binding.FLAG_ALLOW_FMA], ids=["default", "fma"])
def test_static_table_call_matches_allocating_path_twice(cuda_device, flags):
    wl = W.workload("resnet56")  # 167 tensors in one launch
    (ref, v_ref, x_ref), (sta, v_sta, x_sta) = _pair(wl, flags)
    rng = np.random.default_rng(1)
    tables = []
    for _ in range(2):
        lr_mult = rng.choice([0.0, 0.5, 1.0, 2.0], wl.n_tensors).astype(np.float32)
        wd_mult = np.array([1.0 if t.kind == "weight" else 0.0 for t in wl.tensors], np.float32)
        tables.append((lr_mult.tolist(), (wd_mult * rng.choice([1.0, 3.0])).tolist()))
    w_or, v_or = sta.weights().cpu().numpy().copy(), v_sta.cpu().numpy().copy()
    all_grads = [W.make_grads(wl, it, DEV) for it in range(2)]  # made up front: no allocation between the calls
    torch.cuda.synchronize()
    free_before = None
    for it, (lr_mult, wd_mult) in enumerate(tables):  # two calls in a row, different tables
        grads = all_grads[it]
        ref.set_tensor_multipliers(lr_mult, wd_mult)
        ref.fused_update(grads, 1)
        torch.cuda.synchronize()
        if free_before is None:
            free_before = torch.cuda.mem_get_info()[0]
        sta.fused_update_mult_static(grads, 1, lr_mult, wd_mult)
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] == free_before, "the static call took or returned device memory"
        # same kernel, same table contents: equal to the last bit in both flavours
        assert torch.equal(ref.weights(), sta.weights()), f"weights differ after call {it}"
        assert torch.equal(v_ref, v_sta), f"momentum differs after call {it}"
        assert torch.equal(x_ref, x_sta), f"local weights differ after call {it}"
        assert torch.equal(ref.delayed_weights(), sta.delayed_weights())
        # and against the oracle itself: bit for bit in the default flavour
        gh = [g.cpu().numpy() for g in grads]
        bak = np.empty_like(w_or)
        oracle.global_update_mult(gh, w_or, v_or, lr=wl.lr, momentum=wl.momentum, wd=wl.wd, offsets=wl.offsets,
                                  lr_mult=np.asarray(lr_mult, np.float32), wd_mult=np.asarray(wd_mult, np.float32),
                                  w_prev=bak)
        x_or = oracle.local_update(bak, gh[1], local_lr=wl.local_lr)
        if flags == 0:
            same = lambda t, a: np.array_equal(t.cpu().numpy().view(np.uint32), a.view(np.uint32))
            assert same(sta.weights(), w_or) and same(v_sta, v_or), f"static call differs from the oracle (call {it})"
            assert same(x_sta, x_or) and same(sta.delayed_weights(), bak)
        else:  # multiply-add pairs may fuse: follow the library, compare within the arithmetic's bound
            got_w, got_v = sta.weights().cpu().numpy(), v_sta.cpu().numpy()
            scale = np.abs(w_or) + np.abs(v_or) + wl.lr * 2.0 * (sum(np.abs(g) for g in gh) / len(gh) + 1e-3)
            assert np.max(np.abs(got_w - w_or) / np.maximum(scale, 1e-30)) <= 1e-6
            assert np.max(np.abs(x_sta.cpu().numpy() - x_or) / (np.abs(bak) + wl.local_lr * np.abs(gh[1]) + 1e-30)) <= 1e-6
            w_or, v_or = got_w.copy(), got_v.copy()
    assert sta.step == 2 and sta.launch_count == 2
    # the static call left the allocating path's own table alone: NULL multipliers = all ones
    grads = W.make_grads(wl, 7, DEV)
    ref.set_tensor_multipliers(None, None)
    ref.fused_update(grads, 1)
    sta.fused_update_mult_static(grads, 1, None, None)
    torch.cuda.synchronize()
    assert torch.equal(ref.weights(), sta.weights()) and torch.equal(x_ref, x_sta)
    sta.local_update(1)  # the separate local update can follow, as after odsgd_fused_update
    torch.cuda.synchronize()
    assert torch.equal(x_ref, x_sta)


def test_static_table_call_refuses_stream_capture(cuda_device):
    """Recorded into a graph, the table upload would replay whatever the shared host staging
    array holds at that time; the call answers ERR_STATE instead and records nothing."""
    wl = W.workload("lenet5")
    (ref, v_ref, x_ref), (sta, v_sta, x_sta) = _pair(wl, 0)
    grads = W.make_grads(wl, 0, DEV)
    ref.fused_update_mult_static(grads, 1, None, None)
    sta.fused_update_mult_static(grads, 1, None, None)  # eager calls work ...
    ref.fused_update(grads, 1)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        with pytest.raises(binding.OdsgdError) as e:
            sta.fused_update_mult_static(grads, 1, None, None)  # ... a captured one is refused
        sta.fused_update(grads, 1)  # the capture itself stays usable
    assert e.value.code == binding.ERR_STATE
    assert sta.step == 2 and sta.launch_count == 2, "the refused call neither launched nor counted"
    graph.replay()
    torch.cuda.synchronize()
    assert torch.equal(sta.weights(), ref.weights()) and torch.equal(v_sta, v_ref) and torch.equal(x_sta, x_ref)


def test_static_table_limits_are_reported(cuda_device):
    n_t = 4097  # one more than ODSGD_STATIC_MAX_TENSORS
    offs = [4 * i for i in range(n_t + 1)]
    n = offs[-1]
    w, v = torch.zeros(n, device=DEV), torch.zeros(n, device=DEV)
    g = [torch.zeros(n, device=DEV)]
    ctx = binding.Odsgd(w, v, n_workers=1, lr=0.1, local_lr=0.1, momentum=0.9, wd=0.0,
                        local=[torch.zeros(n, device=DEV)], tensor_offsets=offs)
    with pytest.raises(binding.OdsgdError) as e:
        ctx.fused_update_mult_static(g, 0, None, None)
    assert e.value.code == binding.ERR_UNSUPPORTED and "4096" in str(e.value)
    assert ctx.launch_count == 0 and ctx.step == 0, "nothing was launched"
    ctx.set_tensor_multipliers([1.0] * n_t, None)  # the allocating path has no such limit
    ctx.fused_update(g, 0)
    torch.cuda.synchronize()
    ctx.close()
    # other rules are refused too
    ctx = binding.Odsgd(w, v, n_workers=1, lr=0.1, local_lr=0.1, momentum=0.9, wd=0.0,
                        local=[torch.zeros(n, device=DEV)])
    ctx.set_local_rule(binding.LOCAL_DC_C, 0.1)
    with pytest.raises(binding.OdsgdError) as e:
        ctx.fused_update_mult_static(g, 0, None, None)
    assert e.value.code == binding.ERR_UNSUPPORTED
    ctx.close()
