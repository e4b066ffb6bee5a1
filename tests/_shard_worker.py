"""Child process of tests/test_shard.py: one gloo rank of the sharded exchange on CPU tensors.

The exchange (push = all-to-all of gradient slices, pull = all-gather of weight slices) is the
package's; the arithmetic between the two is the CPU oracle applied to this rank's slice, so
that the gathered result can be compared with the oracle applied to the whole arena."""
import json
import os
import sys

import numpy as np
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import oracle  # noqa: E402
from paper_2005_06728_b200 import benchutil, shard  # noqa: E402
from paper_2005_06728_b200 import workloads as W  # noqa: E402


def run_case(dist, rank, R, n, k, iterations):
    lay = shard.ShardLayout(n, R, k)
    N, S, L = lay.n_workers, lay.shard_len, lay.padded_len
    ex = shard.ShardExchange(lay, rank)
    wl = W.ragged_workload([n], n_workers=N, lr=0.1, local_lr=0.05, momentum=0.9, wd=1e-3, seed=21)
    hp = dict(lr=wl.lr, momentum=wl.momentum, wd=wl.wd)
    w0 = W.make_weights(wl).numpy()[:n].copy()
    # unsharded oracle trajectory, computed by every rank for itself
    w_ref, v_ref = w0.copy(), np.zeros(n, np.float32)
    # this rank's state: a replica of the weights (padded) and the momentum of its slice
    b, e = lay.owned(rank)
    w_full = torch.zeros(L)
    w_full[:n] = torch.from_numpy(w0)
    v_shard = np.zeros(e - b, np.float32)
    recv = [torch.zeros(L) for _ in range(k)]
    ok = True
    for it in range(iterations):
        all_g = [W.make_grad(wl, m, it).numpy()[:n].copy() for m in range(N)]
        mine = []
        for j in range(k):
            g = torch.zeros(L)
            g[:n] = torch.from_numpy(all_g[lay.worker_id(rank, j)])
            mine.append(g)
        # worker role: local update from the replica this rank holds and its own gradient
        xs = [oracle.local_update(w_full[:n].numpy().copy(), all_g[lay.worker_id(rank, j)], local_lr=wl.local_lr)
              for j in range(k)]
        ex.push(mine, recv)
        views = shard.shard_views(lay, rank, recv)
        assert len(views) == N
        for m, view in enumerate(views):  # worker order, each view = worker m's slice [b, e)
            ok &= bool(np.array_equal(view.numpy(), all_g[m][b:e]))
        if e > b:
            w_slice = w_full[b:e].numpy()  # shares memory with the replica
            oracle.global_update([np.ascontiguousarray(x.numpy()) for x in views], w_slice, v_shard, **hp)
        ex.pull(w_full)
        bak = np.empty(n, np.float32)
        oracle.global_update(all_g, w_ref, v_ref, w_prev=bak, **hp)
        ok &= bool(np.array_equal(w_full[:n].numpy().view(np.uint32), w_ref.view(np.uint32)))
        ok &= bool(np.array_equal(v_shard.view(np.uint32), v_ref[b:e].view(np.uint32)))
        ok &= bool(torch.all(w_full[n:] == 0))
        for j in range(k):
            want = oracle.local_update(bak, all_g[lay.worker_id(rank, j)], local_lr=wl.local_lr)
            ok &= bool(np.array_equal(xs[j].view(np.uint32), want.view(np.uint32)))
    flag = torch.tensor([1.0 if ok else 0.0])
    dist.all_reduce(flag, op=dist.ReduceOp.MIN)
    return bool(flag.item() == 1.0), (b, e), S


def main():
    dist = benchutil.init_process_group("gloo")
    ri = benchutil.rank_info()
    rank, R = ri["rank"], ri["world_size"]
    out = []
    for n, k, its in ((10_000, 1, 3), (10_003, 2, 3), (7, 1, 2), (4 * R, 3, 2)):
        good, owned, S = run_case(dist, rank, R, n, k, its)
        out.append({"n": n, "k": k, "ok": good, "owned": owned, "shard_len": S})
    benchutil.barrier()
    if rank == 0:
        print(json.dumps({"world_size": R, "cases": out}), flush=True)
    dist.destroy_process_group()


if __name__ == "__main__":
    main()
