"""The sharded exchange around the update pass.

On CPU (world size 2 and 3 over gloo): the package's push / pull move the right slices to the
right owners in worker order, and an update applied slice by slice between them gathers to
exactly what the oracle computes on the whole arena.  On one GPU: R emulated ranks of
ShardedOdsgd, driven phase by phase through an in-process stand-in for the collectives,
reproduce the unsharded library bit for bit - with the slices moved around the kernel, and with
the kernel itself reading the other ranks' gradient arenas and writing their replicas."""
import json
import os
import socket
import subprocess
import sys

import numpy as np
import pytest
import torch

from paper_2005_06728_b200 import binding, shard
from paper_2005_06728_b200 import workloads as W

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_layout_agrees_with_the_library_partition():
    for n in (1, 7, 8, 1000, 10_003, 25_557_032, 138_357_544):
        for R in (1, 2, 3, 8):
            lay = shard.ShardLayout(n, R, 2)
            S = lay.shard_len
            assert S % 4 == 0 and lay.padded_len == R * S >= n and lay.n_workers == 2 * R
            for r in range(R):
                assert lay.owned(r) == (min(r * S, n), min((r + 1) * S, n)) == binding.shard_range(n, R, r)
            assert lay.worker_id(R - 1, 1) == 2 * R - 1


def test_shard_views_are_in_worker_order():
    lay = shard.ShardLayout(22, 3, 2)  # S = 8; rank 2 owns [16, 22)
    recv = [torch.arange(lay.padded_len, dtype=torch.float32) + 100 * j for j in range(2)]
    views = shard.shard_views(lay, 2, recv)
    assert [v.numel() for v in views] == [6] * 6
    # worker m = q * 2 + j sits at recv[j][q * S ...]
    assert [float(v[0]) for v in views] == [0.0, 100.0, 8.0, 108.0, 16.0, 116.0]


@pytest.mark.parametrize("world", [2, 3])
def test_exchange_over_gloo_matches_the_unsharded_oracle(world):
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={world}",
           "--master-addr", "127.0.0.1", "--master-port", str(_free_port()), os.path.join("tests", "_shard_worker.py")]
    env = dict(os.environ, CUDA_VISIBLE_DEVICES="", OMP_NUM_THREADS="1")
    res = subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=300)
    assert res.returncode == 0, res.stderr[-3000:]
    lines = [json.loads(x) for x in res.stdout.splitlines() if x.strip().startswith("{")]
    assert len(lines) == 1 and lines[0]["world_size"] == world
    assert len(lines[0]["cases"]) == 4
    for case in lines[0]["cases"]:
        assert case["ok"], case


def test_sharded_update_needs_a_cuda_device():
    lay = shard.ShardLayout(16, 1, 1)
    with pytest.raises(RuntimeError, match="CUDA"):
        shard.ShardedOdsgd(lay, 0, torch.zeros(16), lr=0.1, local_lr=0.1, momentum=0.9, wd=0.0, exchange=None)


# ------------------------------------------------------------------ one GPU, R emulated ranks

class _Loopback:
    """Stands in for the collectives when several ranks are emulated in one process: the ranks'
    phases are run in lockstep and the slices are moved with plain device copies."""

    def __init__(self, layout):
        self.layout, self.sent, self.recv, self.pulled = layout, {}, {}, {}

    def port(self, rank):
        hub = self

        class Port:
            def push(self, grads, recv):
                hub.sent[rank], hub.recv[rank] = list(grads), list(recv)

            def pull(self, w_full):
                hub.pulled[rank] = w_full

        return Port()

    def deliver_push(self):
        S, R = self.layout.shard_len, self.layout.n_ranks
        for dst in range(R):
            for j, r in enumerate(self.recv[dst]):
                for q in range(R):
                    r[q * S:(q + 1) * S].copy_(self.sent[q][j][dst * S:(dst + 1) * S])

    def deliver_pull(self):
        S, R = self.layout.shard_len, self.layout.n_ranks
        for src in range(R):
            piece = self.pulled[src][src * S:(src + 1) * S]
            for dst in range(R):
                if dst != src:
                    self.pulled[dst][src * S:(src + 1) * S].copy_(piece)


class _PeerHub:
    """Stands in for symmetric memory when several ranks are emulated in one process: every rank's
    gradient arenas and replicas are ordinary tensors of this device, and a "peer's" buffer is
    simply the other emulated rank's tensor.  The ranks run in lockstep on one stream, so the
    fences have nothing to do."""

    def __init__(self, layout, dev):
        k, L, R = layout.workers_per_rank, layout.padded_len, layout.n_ranks
        self.layout = layout
        self.grads = [[torch.zeros(L, dtype=torch.float32, device=dev) for _ in range(k)] for _ in range(R)]
        self.reps = [[torch.zeros(L, dtype=torch.float32, device=dev) for _ in range(2)] for _ in range(R)]
        self.fences = 0

    def port(self, rank):
        hub = self

        class Port:
            direct = True
            grad_arenas = hub.grads[rank]
            replicas = hub.reps[rank]

            def peer_grad(self, q, j):
                return hub.grads[q][j]

            def peer_replica(self, q, half):
                return hub.reps[q][half]

            def fence(self):
                hub.fences += 1

        return Port()

    # the collectives of the other exchange have no counterpart here
    def deliver_push(self):
        pass

    def deliver_pull(self):
        pass


@pytest.mark.gpu
@pytest.mark.parametrize("R,k,n", [(2, 1, 100_003), (3, 2, 50_001), (8, 1, 200_000), (8, 2, 37), (2, 4, 8)])
@pytest.mark.parametrize("rule", ["sgd", "dc_c"])
@pytest.mark.parametrize("exchange", ["collectives", "direct"])
def test_emulated_ranks_reproduce_the_unsharded_library(cuda_device, R, k, n, rule, exchange):
    dev = torch.device("cuda:0")
    lay = shard.ShardLayout(n, R, k)
    N, L = lay.n_workers, lay.padded_len
    wl = W.ragged_workload([n], n_workers=N, lr=0.1, local_lr=0.05, momentum=0.9, wd=1e-3, seed=5)
    w0 = W.make_weights(wl, dev)[:n].clone()
    lrule = binding.LOCAL_SGD if rule == "sgd" else binding.LOCAL_DC_C
    warmup = 2
    # the unsharded library: one context over the whole arena, all N workers local
    w, v = w0.clone(), torch.zeros(n, device=dev)
    local = [torch.zeros(n, device=dev) for _ in range(N)]
    ref = binding.Odsgd(w, v, n_workers=N, lr=wl.lr, local_lr=wl.local_lr, momentum=wl.momentum, wd=wl.wd,
                        w_b=torch.zeros(n, device=dev), local=local)
    ref.set_local_rule(lrule, 0.04)
    ref.set_warmup(warmup)
    direct = exchange == "direct"
    hub = _PeerHub(lay, dev) if direct else _Loopback(lay)
    ranks = [shard.ShardedOdsgd(lay, r, w0, lr=wl.lr, local_lr=wl.local_lr, momentum=wl.momentum, wd=wl.wd,
                                exchange=hub.port(r), local_rule=lrule, rule_lambda=0.04, warmup=warmup)
             for r in range(R)]
    for it in range(6):
        grads = [W.make_grad(wl, m, it, dev)[:n] for m in range(N)]
        padded = []
        for m in range(N):
            # direct exchange: the gradient is produced in the arena the other ranks have mapped
            g = hub.grads[m // k][m % k] if direct else torch.zeros(L, device=dev)
            g[:n].copy_(grads[m])
            padded.append(g)
        ref.step_update(grads)
        for r, sh in enumerate(ranks):
            sh.phase_local_and_push([padded[lay.worker_id(r, j)] for j in range(k)])
        hub.deliver_push()
        for sh in ranks:
            sh.phase_server()
        for sh in ranks:
            sh.phase_pull()
        hub.deliver_pull()
        torch.cuda.synchronize()
        for r, sh in enumerate(ranks):
            assert sh.iteration == it + 1
            assert torch.equal(sh.weights(), ref.weights()), f"replica of rank {r} after iteration {it}"
            assert bool(torch.all(sh.w_full[sh.cur][n:] == 0)), "padding stays zero"
            b, e = lay.owned(r)
            assert torch.equal(sh.v[:e - b], v[b:e]), f"momentum slice of rank {r}"
            for j in range(k):
                m = lay.worker_id(r, j)
                want = ref.train_weights(m)
                assert torch.equal(sh.train_weights(j), want), f"train weights of worker {m}, iteration {it}"
        if direct:
            assert hub.fences == 2 * R * (it + 1), "one fence before and one after the server kernel, per rank"
            for r in range(R):
                assert all(bool(torch.all(g[n:] == 0)) for g in hub.grads[r]), "gradient padding untouched"
    if direct:
        with pytest.raises(ValueError, match="grad_arenas"):
            ranks[0].phase_local_and_push([torch.zeros(L, device=dev) for _ in range(k)])
    for sh in ranks:
        sh.close()
    ref.close()


@pytest.mark.gpu
@pytest.mark.parametrize("R", [1, 3, 8])
def test_emulated_ranks_with_per_tensor_multipliers(cuda_device, R):
    """Tensor boundaries cut by slice boundaries: each rank's server context gets the offsets and
    multipliers of the (parts of) tensors in its slice, and the result equals the unsharded one."""
    dev = torch.device("cuda:0")
    wl = W.ragged_workload([1000, 12, 20_000, 4, 7_777, 3], n_workers=R, lr=0.1, local_lr=0.05, momentum=0.9, wd=1e-2)
    n = wl.arena_len
    lay = shard.ShardLayout(n, R, 1)
    rng = np.random.default_rng(R)
    lr_mult = rng.choice([0.0, 0.5, 1.0, 2.0], wl.n_tensors).tolist()
    wd_mult = rng.choice([0.0, 1.0], wl.n_tensors).tolist()
    w0 = W.make_weights(wl, dev)
    w, v = w0.clone(), torch.zeros(n, device=dev)
    local = [torch.zeros(n, device=dev) for _ in range(R)]
    ref = binding.Odsgd(w, v, n_workers=R, lr=wl.lr, local_lr=wl.local_lr, momentum=wl.momentum, wd=wl.wd,
                        w_b=torch.zeros(n, device=dev), local=local, tensor_offsets=wl.offsets)
    ref.set_tensor_multipliers(lr_mult, wd_mult)
    hub = _Loopback(lay)
    ranks = [shard.ShardedOdsgd(lay, r, w0, lr=wl.lr, local_lr=wl.local_lr, momentum=wl.momentum, wd=wl.wd,
                                exchange=hub.port(r), tensor_offsets=wl.offsets) for r in range(R)]
    for sh in ranks:
        sh.set_tensor_multipliers(lr_mult, wd_mult)
    assert sum(len(sh.slice_tensors) for sh in ranks) >= wl.n_tensors, "every tensor is owned by some rank"
    for it in range(3):
        grads = [W.make_grad(wl, m, it, dev) for m in range(R)]
        padded = []
        for g in grads:
            p = torch.zeros(lay.padded_len, device=dev)
            p[:n].copy_(g)
            padded.append(p)
        ref.step_update(grads)
        for r, sh in enumerate(ranks):
            sh.phase_local_and_push([padded[r]])
        hub.deliver_push()
        for sh in ranks:
            sh.phase_server()
        for sh in ranks:
            sh.phase_pull()
        hub.deliver_pull()
        torch.cuda.synchronize()
        for r, sh in enumerate(ranks):
            assert torch.equal(sh.weights(), ref.weights()), f"rank {r}, iteration {it}"
            assert torch.equal(sh.train_weights(0), ref.train_weights(r))
    for sh in ranks:
        sh.close()
    ref.close()


@pytest.mark.gpu
def test_single_rank_process_group_runs_the_real_exchange(cuda_device):
    """World size 1 over NCCL: the real collectives (degenerate: one rank) inside ShardedOdsgd.step."""
    import torch.distributed as dist

    dev = torch.device("cuda:0")
    torch.cuda.set_device(dev)
    created = False
    if not dist.is_initialized():
        dist.init_process_group("nccl", init_method=f"tcp://127.0.0.1:{_free_port()}", rank=0, world_size=1)
        created = True
    try:
        n = 300_001
        lay = shard.ShardLayout(n, 1, 3)
        wl = W.ragged_workload([n], n_workers=3, lr=0.1, local_lr=0.05, momentum=0.9, wd=1e-3, seed=9)
        w0 = W.make_weights(wl, dev)[:n].clone()
        w, v = w0.clone(), torch.zeros(n, device=dev)
        local = [torch.zeros(n, device=dev) for _ in range(3)]
        ref = binding.Odsgd(w, v, n_workers=3, lr=wl.lr, local_lr=wl.local_lr, momentum=wl.momentum, wd=wl.wd,
                            w_b=torch.zeros(n, device=dev), local=local)
        sh = shard.ShardedOdsgd(lay, 0, w0, lr=wl.lr, local_lr=wl.local_lr, momentum=wl.momentum, wd=wl.wd,
                                exchange=shard.ShardExchange(lay, 0))
        for it in range(3):
            grads = [W.make_grad(wl, m, it, dev)[:n] for m in range(3)]
            padded = []
            for g in grads:
                p = torch.zeros(lay.padded_len, device=dev)
                p[:n].copy_(g)
                padded.append(p)
            ref.step_update(grads)
            sh.step(padded)
            torch.cuda.synchronize()
            assert torch.equal(sh.weights(), ref.weights()) and torch.equal(sh.v[:n], v)
            for j in range(3):
                assert torch.equal(sh.train_weights(j), ref.train_weights(j))
        sh.close()
        ref.close()
    finally:
        if created:
            dist.destroy_process_group()


@pytest.mark.gpu
def test_single_rank_symmetric_memory_runs_the_direct_exchange(cuda_device):
    """World size 1: PeerExchange's real symmetric-memory allocation, rendezvous, views and fences
    inside ShardedOdsgd.step (degenerate: no other rank to map, no mirror)."""
    import torch.distributed as dist

    dev = torch.device("cuda:0")
    torch.cuda.set_device(dev)
    created = False
    if not dist.is_initialized():
        dist.init_process_group("nccl", init_method=f"tcp://127.0.0.1:{_free_port()}", rank=0, world_size=1)
        created = True
    try:
        n = 300_001
        lay = shard.ShardLayout(n, 1, 3)
        wl = W.ragged_workload([n], n_workers=3, lr=0.1, local_lr=0.05, momentum=0.9, wd=1e-3, seed=9)
        w0 = W.make_weights(wl, dev)[:n].clone()
        w, v = w0.clone(), torch.zeros(n, device=dev)
        local = [torch.zeros(n, device=dev) for _ in range(3)]
        ref = binding.Odsgd(w, v, n_workers=3, lr=wl.lr, local_lr=wl.local_lr, momentum=wl.momentum, wd=wl.wd,
                            w_b=torch.zeros(n, device=dev), local=local)
        ref.set_warmup(1)
        ex = shard.PeerExchange(lay, 0, dev)
        assert len(ex.grad_arenas) == 3 and all(g.numel() == lay.padded_len for g in ex.grad_arenas)
        assert ex.peer_grad(0, 2).data_ptr() == ex.grad_arenas[2].data_ptr()
        assert ex.peer_replica(0, 1).data_ptr() == ex.replicas[1].data_ptr()
        assert all(g.data_ptr() % 16 == 0 for g in ex.grad_arenas + ex.replicas)
        sh = shard.ShardedOdsgd(lay, 0, w0, lr=wl.lr, local_lr=wl.local_lr, momentum=wl.momentum, wd=wl.wd,
                                exchange=ex, warmup=1)
        assert sh.w_full[0].data_ptr() == ex.replicas[0].data_ptr()
        for it in range(4):
            grads = [W.make_grad(wl, m, it, dev)[:n] for m in range(3)]
            for a, g in zip(ex.grad_arenas, grads):
                a[:n].copy_(g)
            ref.step_update(grads)
            sh.step(ex.grad_arenas)
            torch.cuda.synchronize()
            assert torch.equal(sh.weights(), ref.weights()) and torch.equal(sh.v[:n], v)
            for j in range(3):
                assert torch.equal(sh.train_weights(j), ref.train_weights(j))
        ex.quiesce()
        sh.close()
        ref.close()
    finally:
        if created:
            dist.destroy_process_group()
