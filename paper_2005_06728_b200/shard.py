"""The exchange steps either side of the update pass when the server role is spread over R GPUs.

In the paper a worker reduces its gradient inside the node, pushes it to the parameter server
and pulls the new weights back (Section 2.2, Fig. 3); OD-SGD overlaps the push with the local
update and the pull with the next iteration's broadcast and compute (Section 3.1; Algorithm 2,
repeat-loop).  Every element of the server's update is independent of the others, so on a
multi-GPU node the server role shards by index: rank r of R owns the slice of every arena that
odsgd_shard_range gives it.  One iteration is then

    push          every worker sends slice s of its gradient to rank s.  The owner ends up with
                  N separate shard buffers in its own memory, one per worker, in worker order.
                  This is an all-to-all, not a reduce-scatter: a reduction inside the collective
                  would add the workers in the collective's order, and the server rule adds them
                  in worker order 0..N-1 (which is what makes results reproducible bit for bit).
    server step   the library's global-update (or SSGD) kernel on the shard, summing the N
                  buffers in worker order: the same kernel, the same arithmetic, on a slice.
    pull          all-gather of the updated slices into every rank's replica of the weights.
    local update  meanwhile, on a second stream, each worker compensates the weights it already
                  has with its own gradient (odsgd_worker_local_update); it reads only the
                  gradient and the old replica, so it overlaps the push.

Two ways to move the slices:

    ShardExchange   torch.distributed collectives into this GPU's own memory (NCCL on GPUs, gloo
                    on CPU tensors in the tests): all-to-all before the kernel, all-gather after.
    PeerExchange    no collective on the data path.  Gradient arenas and weight replicas live in
                    symmetric memory, so every rank has every other rank's buffers mapped.  The
                    server kernel reads the N gradient slices where they are (its own workers'
                    locally, the others' over NVLink) and stores each new weight into the owned
                    slice of all R replicas (odsgd_set_weight_mirrors): push, update and pull are
                    one pass, the transfers overlap the arithmetic element by element, and the
                    staging copies of the all-to-all (one extra write and read of N slices per
                    rank) disappear.  Plain 128-bit loads and stores only: no bulk-copy engine and
                    no multicast touch a peer's memory.  What remains between ranks is ordering: a
                    stream-ordered fence before the kernel (every rank's gradients are complete)
                    and one after it (every rank's slice has landed in this replica).

Nothing here computes an update: the arithmetic stays in the CUDA library; this module moves
slices, maps buffers and orders streams.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Optional, Sequence, Tuple

import torch

from . import binding


@dataclass(frozen=True)
class ShardLayout:
    """How an arena of `n_params` elements is spread over `n_ranks` ranks, each hosting
    `workers_per_rank` workers.  Worker ids are global: worker j of rank q is q * k + j."""

    n_params: int
    n_ranks: int
    workers_per_rank: int = 1

    @property
    def n_workers(self) -> int:
        return self.n_ranks * self.workers_per_rank

    @property
    def shard_len(self) -> int:
        """Nominal slice length: ceil(n_params / n_ranks) rounded up to 4 elements, the same for
        every rank (odsgd_shard_range cuts the same slices and clips them to n_params)."""
        per = -(-self.n_params // self.n_ranks)
        return -(-per // 4) * 4

    @property
    def padded_len(self) -> int:
        """Length of the arenas the exchange works on: n_ranks equal slices (zero padding at the end)."""
        return self.shard_len * self.n_ranks

    def owned(self, rank: int) -> Tuple[int, int]:
        """[begin, end) of the elements rank `rank` owns (odsgd_shard_range)."""
        return binding.shard_range(self.n_params, self.n_ranks, rank)

    def worker_id(self, rank: int, j: int) -> int:
        return rank * self.workers_per_rank + j


class ShardExchange:
    """push / pull over a torch.distributed process group.  Works on tensors of any device the
    group's backend supports (CUDA with NCCL; CPU with gloo, which is how the tests run it)."""

    def __init__(self, layout: ShardLayout, rank: int, group=None):
        import torch.distributed as dist

        self.layout, self.rank, self.group, self._dist = layout, rank, group, dist
        if dist.get_world_size(group) != layout.n_ranks:
            raise ValueError(f"process group has {dist.get_world_size(group)} ranks, layout has {layout.n_ranks}")

    def push(self, grads: Sequence[torch.Tensor], recv: Sequence[torch.Tensor]) -> None:
        """grads[j]: worker j of this rank, `padded_len` elements.  recv[j] (same length) receives,
        at [q * S, (q + 1) * S), slice `rank` of the gradient of worker j of rank q."""
        for g, r in zip(grads, recv):
            self._dist.all_to_all_single(r, g, group=self.group)

    def pull(self, w_full: torch.Tensor) -> None:
        """All-gather, in place: every rank contributes its own slice of `w_full`."""
        S = self.layout.shard_len
        self._dist.all_gather_into_tensor(w_full, w_full[self.rank * S:(self.rank + 1) * S], group=self.group)


class PeerExchange:
    """Buffers of the sharded update in symmetric memory, and the fences between ranks.

    One symmetric allocation per rank holds its k gradient arenas and its two weight replicas
    (`padded_len` floats each); after the rendezvous every rank can address every other rank's
    copy of it.  The caller writes worker j's gradient into `grad_arenas[j]`; ShardedOdsgd takes
    the replicas, the gradient table of its server kernel (`peer_grad`) and the mirrors of its
    weight stores (`peer_replica`) from here.  `fence()` is a one-element all-reduce on the
    current stream: it completes on a rank only once every rank has reached it in stream order,
    which is all the ordering the kernels need (they never wait on one another themselves).
    """

    direct = True

    def __init__(self, layout: ShardLayout, rank: int, device: torch.device, group=None):
        import os

        import torch.distributed as dist

        # nothing here uses the NVSwitch multicast mapping symmetric memory would otherwise set up
        os.environ.setdefault("TORCH_SYMM_MEM_DISABLE_MULTICAST", "1")
        import torch.distributed._symmetric_memory as symm_mem

        if dist.get_world_size(group) != layout.n_ranks:
            raise ValueError(f"process group has {dist.get_world_size(group)} ranks, layout has {layout.n_ranks}")
        if layout.n_ranks - 1 > binding.MAX_MIRRORS:
            raise ValueError(f"at most {binding.MAX_MIRRORS + 1} ranks (one weight mirror per other rank)")
        self.layout, self.rank, self.group, self._dist = layout, rank, group, dist
        k, L = layout.workers_per_rank, layout.padded_len
        self._total = (k + 2) * L
        self._own = symm_mem.empty(self._total, dtype=torch.float32, device=device)
        self._own.zero_()
        self._hdl = symm_mem.rendezvous(self._own, dist.group.WORLD if group is None else group)
        self._whole = [self._own if q == rank else self._hdl.get_buffer(q, (self._total,), torch.float32)
                       for q in range(layout.n_ranks)]
        self._token = torch.zeros(1, dtype=torch.float32, device=device)
        self.grad_arenas = [self.peer_grad(rank, j) for j in range(k)]
        self.replicas = [self.peer_replica(rank, h) for h in range(2)]

    def peer_grad(self, q: int, j: int) -> torch.Tensor:
        """Gradient arena of worker j of rank q, as mapped into this process."""
        L = self.layout.padded_len
        return self._whole[q][j * L:(j + 1) * L]

    def peer_replica(self, q: int, half: int) -> torch.Tensor:
        """Weight replica `half` (0 / 1) of rank q, as mapped into this process."""
        k, L = self.layout.workers_per_rank, self.layout.padded_len
        return self._whole[q][(k + half) * L:(k + half + 1) * L]

    def fence(self) -> None:
        self._dist.all_reduce(self._token, group=self.group)

    def quiesce(self) -> None:
        """Call on every rank before the buffers are dropped: once it returns, no rank has a
        kernel in flight that reads or writes another rank's memory."""
        self.fence()
        torch.cuda.current_stream().synchronize()


def shard_views(layout: ShardLayout, rank: int, recv: Sequence[torch.Tensor]) -> List[torch.Tensor]:
    """The N per-worker shard buffers of rank `rank`, as views into its receive buffers, in worker
    order m = q * k + j; each has the length of the slice the rank owns."""
    S = layout.shard_len
    b, e = layout.owned(rank)
    own = e - b
    return [recv[j][q * S:q * S + own] for q in range(layout.n_ranks) for j in range(layout.workers_per_rank)]


class ShardedOdsgd:
    """One rank of the sharded update: the server role on the slice it owns, the worker role for
    the workers it hosts.  CUDA only (the kernels are the library's).

    The three phases of an iteration are separate methods so that a test can run several
    emulated ranks in lockstep on one device; `step` runs them in order with the real exchange.

    `exchange` is a ShardExchange (collectives around the kernel) or anything with
    `direct = True` and PeerExchange's members (`replicas`, `grad_arenas`, `peer_grad`,
    `peer_replica`, `fence`): then the server kernel itself reads the peers' gradient slices and
    writes the peers' replicas, the gradients passed to `phase_local_and_push` must be the
    exchange's own `grad_arenas`, and `w0` has to be the same on every rank (each fills its own
    replicas with it).
    """

    def __init__(self, layout: ShardLayout, rank: int, w0: torch.Tensor, *, lr: float, local_lr: float,
                 momentum: float, wd: float, exchange, device: Optional[torch.device] = None, flags: int = 0,
                 local_rule: int = binding.LOCAL_SGD, rule_lambda: float = 0.0, rule_m: float = 0.0,
                 rule_eps: float = 0.0, warmup: int = 0, tensor_offsets: Optional[Sequence[int]] = None):
        dev = w0.device if device is None else device
        if dev.type != "cuda":
            raise RuntimeError("ShardedOdsgd runs the CUDA library: it needs a CUDA device (there is no CPU path)")
        if w0.numel() != layout.n_params:
            raise ValueError(f"w0 has {w0.numel()} elements, layout has {layout.n_params}")
        self.layout, self.rank, self.exchange, self.device = layout, rank, exchange, dev
        n, k, N = layout.n_params, layout.workers_per_rank, layout.n_workers
        L, S = layout.padded_len, layout.shard_len
        self.direct = bool(getattr(exchange, "direct", False))
        if self.direct:
            self.w_full = list(exchange.replicas)
            for h in range(2):  # the mirrors are never read, but a replica is: both start as w_0
                self.w_full[h].zero_()
                self.w_full[h][:n].copy_(w0)
            self.recv = []
        else:
            self.w_full = [torch.zeros(L, dtype=torch.float32, device=dev) for _ in range(2)]
            self.w_full[0][:n].copy_(w0)
            self.recv = [torch.zeros(L, dtype=torch.float32, device=dev) for _ in range(k)]
        self.cur = 0
        self.local = [torch.zeros(L, dtype=torch.float32, device=dev) for _ in range(k)]
        self.begin, self.end = layout.owned(rank)
        own = self.end - self.begin
        self.warmup, self.iteration = int(warmup), 0
        self.side = torch.cuda.Stream(device=dev)
        self.local_done = torch.cuda.Event()
        # server role: a context over the slices of the two weight replicas this rank owns
        self.server = None
        self.v = torch.zeros(max(own, 4), dtype=torch.float32, device=dev)
        # the tensors (or parts of tensors) that fall into the owned slice, as offsets relative to it
        offs = list(tensor_offsets) if tensor_offsets is not None else [0, n]
        if offs[0] != 0 or offs[-1] != n:
            raise ValueError("tensor_offsets must start at 0 and end at n_params")
        self.slice_tensors = [t for t in range(len(offs) - 1) if offs[t] < self.end and offs[t + 1] > self.begin]
        self.slice_offsets = [max(offs[t], self.begin) - self.begin for t in self.slice_tensors] + [own]
        self.n_tensors = len(offs) - 1
        if own > 0:
            b, e = self.begin, self.end
            self.server = binding.Odsgd(self.w_full[0][b:e], self.v[:own], n_workers=N, lr=lr, local_lr=local_lr,
                                        momentum=momentum, wd=wd, w_b=self.w_full[1][b:e], flags=flags,
                                        tensor_offsets=self.slice_offsets)
            if self.direct:
                R = layout.n_ranks
                others = [q for q in range(R) if q != rank]
                if others:
                    self.server.set_weight_mirrors([exchange.peer_replica(q, 0)[b:e] for q in others],
                                                   [exchange.peer_replica(q, 1)[b:e] for q in others])
                # the N gradient slices where they are, in worker order m = q * k + j
                self.shard_grads = self.server.bind_grads(
                    [exchange.peer_grad(q, j)[b:e] for q in range(R) for j in range(k)])
            else:
                self.shard_grads = self.server.bind_grads(shard_views(layout, rank, self.recv))
        # worker role: a worker-only context over the whole arena
        slots: List[Optional[torch.Tensor]] = [None] * N
        for j in range(k):
            slots[layout.worker_id(rank, j)] = self.local[j][:n]
        self.worker = binding.Odsgd(self.w_full[0][:n], None, n_workers=N, lr=lr, local_lr=local_lr,
                                    momentum=momentum, wd=wd, w_b=self.w_full[1][:n], local=slots,
                                    flags=flags | binding.FLAG_WORKER_ONLY)
        self.state = None
        if local_rule != binding.LOCAL_SGD:
            tab = None
            if local_rule in (binding.LOCAL_DC_A, binding.LOCAL_MOMENTUM):
                self.state = [torch.zeros(n, dtype=torch.float32, device=dev) for _ in range(k)]
                tab = [None] * N
                for j in range(k):
                    tab[layout.worker_id(rank, j)] = self.state[j]
            self.worker.set_local_rule(local_rule, rule_lambda, rule_m, rule_eps, tab)

    # -- queries
    def weights(self) -> torch.Tensor:
        """This rank's replica of the current global weights (valid once the pull has completed)."""
        return self.w_full[self.cur][:self.layout.n_params]

    def train_weights(self, j: int) -> torch.Tensor:
        """What hosted worker j computes its next gradient on (Algorithm 2): the global weights
        while the next iteration index is <= warmup, its local weights afterwards."""
        if self.iteration <= self.warmup:
            return self.weights()
        return self.local[j][:self.layout.n_params]

    def set_lr(self, lr: float) -> None:
        if self.server is not None:
            self.server.set_lr(lr)

    def set_local_lr(self, local_lr: float) -> None:
        self.worker.set_local_lr(local_lr)

    def set_tensor_multipliers(self, lr_mult: Optional[Sequence[float]], wd_mult: Optional[Sequence[float]]) -> None:
        """Per-tensor multipliers of the whole parameter set (one entry per tensor of
        `tensor_offsets`); each rank keeps the entries of the tensors its slice touches."""
        if self.server is None:
            return
        if lr_mult is None and wd_mult is None:
            self.server.set_tensor_multipliers(None, None)
            return
        for m in (lr_mult, wd_mult):
            if m is not None and len(m) != self.n_tensors:
                raise ValueError(f"need {self.n_tensors} multipliers, got {len(m)}")
        pick = lambda m: None if m is None else [float(m[t]) for t in self.slice_tensors]
        self.server.set_tensor_multipliers(pick(lr_mult), pick(wd_mult))

    def set_momentum(self, momentum: float) -> None:
        if self.server is not None:
            self.server.set_momentum(momentum)

    def set_wd(self, wd: float) -> None:
        if self.server is not None:
            self.server.set_wd(wd)

    # -- the phases of one iteration
    def phase_local_and_push(self, grads: Sequence[torch.Tensor]) -> None:
        """grads[j]: gradient of hosted worker j, `padded_len` elements on this device (zeros
        beyond n_params).  Starts the local updates on the side stream and pushes the slices."""
        lay, n = self.layout, self.layout.n_params
        if len(grads) != lay.workers_per_rank or any(g.numel() != lay.padded_len for g in grads):
            raise ValueError(f"need {lay.workers_per_rank} gradients of {lay.padded_len} elements")
        self._delayed = self.iteration >= self.warmup
        if self._delayed:
            main = torch.cuda.current_stream(self.device)
            self.side.wait_stream(main)  # the gradients and the replica are ready
            for j, g in enumerate(grads):
                self.worker.worker_local_update(lay.worker_id(self.rank, j), self.w_full[self.cur][:n], g[:n],
                                                no_delay=self.iteration == self.warmup, stream=self.side)
            self.local_done.record(self.side)
        if self.direct:
            if any(g.data_ptr() != a.data_ptr() for g, a in zip(grads, self.exchange.grad_arenas)):
                raise ValueError("with a direct exchange the gradients must be written into exchange.grad_arenas")
            # every rank's gradients are complete, and every rank is done with the replica half
            # and the gradient arenas of the previous iteration, before any server kernel starts
            self.exchange.fence()
        else:
            self.exchange.push(grads, self.recv)

    def phase_server(self) -> None:
        """The server rule on the slice this rank owns, over the N received shard buffers."""
        if self.server is None:
            return
        if self._delayed:
            self.server.global_update(self.shard_grads)  # reads replica `cur`, writes replica `cur ^ 1`
        else:
            self.server.ssgd_step(self.shard_grads)      # warm-up: in place

    def phase_pull(self) -> None:
        """All-gather of the updated slices; afterwards the replica holds the new global weights."""
        if self._delayed:
            self.cur ^= 1
        if self.direct:
            self.exchange.fence()  # every rank's kernel has finished: all slices of the replica are in
        else:
            self.exchange.pull(self.w_full[self.cur])
        if self._delayed:
            # the next iteration's local update reads the replica the pull just filled and writes
            # the local arenas: both are ordered behind this iteration's local updates
            torch.cuda.current_stream(self.device).wait_stream(self.side)
        self.iteration += 1

    def step(self, grads: Sequence[torch.Tensor]) -> None:
        self.phase_local_and_push(grads)
        self.phase_server()
        self.phase_pull()

    def close(self) -> None:
        if self.server is not None:
            self.server.close()
        self.worker.close()
