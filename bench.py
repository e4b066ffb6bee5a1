#!/usr/bin/env python
"""Benchmark of the OD-SGD parameter-update pass.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--workers M]
    python bench.py --impl reference ...      # the CPU oracle on a bounded sample

A step is one OD-SGD iteration of the update pass on one synthetic parameter set: the fused
global + local update (server step over M gradient buffers plus one worker's local weights)
in a single kernel launch.  `value` is algorithmic bytes per second, (M + 5) * 4 * P bytes per
step, with every buffer resident in HBM; `e2e` is the same figure when the M gradients start
in pinned host memory and the worker's new weights are copied back, all inside the timed
region, through the host-buffer entry point of the C ABI.  One JSON line goes to stdout.

Besides the headline workload (VGG-16-shaped, M = 32) the default run times, and reports under
`configs`, the other parameter sets: every rule on the AlexNet- and ResNet-50-shaped sets, the
worker-count sweep on the VGG-16-shaped set, and the two small cache-resident sets (eager
launches and CUDA-graph replay; effective figures, not HBM ones).

With --gpus N > 1 every rank updates its own full parameter set on its own GPU: the ranks share
no data, so nothing but a barrier and the final max/sum of two scalars crosses between them.
Started without torchrun, `--gpus N` launches its N ranks itself.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "OD-SGD update throughput: HBM GB/s & % of B200 peak; params/sec at N workers"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
L2_BYTES = 126e6
ORACLE_CHUNK = 1 << 22  # elements per chunk when the oracle walks a whole arena


def hbm_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as fh:
            return float(json.load(fh)["hbm_gbs"]), "measured"
    except (OSError, KeyError, ValueError):
        return FALLBACK_HBM_GBS, "fallback"


# DRAM traffic of the fused kernel, from its ncu capture (two launches of the M = 32 instantiation
# on the 25.6 M-parameter arena; figures and command in profiles/server_kernel_fused_m32_resnet50_arena.md):
# dram__bytes_read.sum + dram__bytes_write.sum over the algorithmic bytes of that launch, and the
# digest of csrc/odsgd_kernels.cuh (kernels and launch shapes) at the time of the capture.
PROFILED_TRAFFIC_RATIO = 0.998
PROFILED_KERNEL_DIGEST = "29d418ddb2084b4c21b8f33a6d9a255c4ca09cf5975ade67586460aa972cdd87"
KERNEL_SOURCE = os.path.join(ROOT, "paper_2005_06728_b200", "csrc", "odsgd_kernels.cuh")


def kernel_source_digest(path=KERNEL_SOURCE):
    """SHA-256 of the kernel source as the compiler sees it: `//` comments, trailing blanks and
    empty lines removed first, so that rewording a comment does not orphan the capture."""
    import hashlib
    import re

    with open(path, encoding="utf-8") as fh:
        lines = [re.sub(r"\s*//.*$", "", ln.rstrip()) for ln in fh]
    return hashlib.sha256("\n".join(ln for ln in lines if ln.strip()).encode()).hexdigest()


def measured_traffic(step_bytes):
    """DRAM bytes per launch: the profiled traffic ratio scaled by this workload's algorithmic
    bytes (traffic grows in proportion: every stream is touched once).  None when the kernel
    source has changed since the counters were taken."""
    try:
        if kernel_source_digest() != PROFILED_KERNEL_DIGEST:
            return None
    except OSError:
        return None
    return PROFILED_TRAFFIC_RATIO * step_bytes


def workload_label(wl, n_workers):
    return f"{wl.name}-shaped parameter set, M={n_workers} workers, fused global+local update"


def parse_args(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=400)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", choices=["cuda", "reference"], default="cuda")
    ap.add_argument("--workload", default="vgg16", help="lenet5 | resnet56 | alexnet | resnet50 | vgg16")
    ap.add_argument("--workers", type=int, default=0, help="override the workload's worker count")
    ap.add_argument("--allow-fma", action="store_true",
                    help="time the flavour in which multiply-add pairs may fuse (default: one rounding per operator)")
    ap.add_argument("--block", type=int, default=0)
    ap.add_argument("--ctas-per-sm", type=int, default=0)
    ap.add_argument("--multipliers", action="store_true", help="per-tensor lr/wd multipliers (no decay off the weight tensors)")
    ap.add_argument("--local-rule", choices=["sgd", "dc_c", "dc_a", "momentum"], default="sgd")
    ap.add_argument("--all-locals", action="store_true", help="update every worker's local weights in the fused pass")
    ap.add_argument("--sweep-workers", default="", help="comma list of worker counts (<= the workload's) to time as well")
    ap.add_argument("--graph", type=int, default=0,
                    help="capture this many steps (even) in one CUDA graph and replay it; for the small, launch-bound sets")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extra-kernels", action="store_true")
    ap.add_argument("--no-configs", action="store_true", help="skip the other parameter sets (only the headline workload)")
    ap.add_argument("--sharded", action="store_true",
                    help="spread the server role over the N ranks (all-to-all of gradient slices, update of the owned "
                         "slice, all-gather of the weights) instead of N independent replicas")
    ap.add_argument("--peer", action="store_true",
                    help="with --sharded: no collective on the data path; the server kernel reads the other ranks' "
                         "gradient slices and writes their weight replicas through symmetric memory")
    ap.add_argument("--cpu-sample", type=int, default=1 << 22, help="elements in the reference arm's sample")
    return ap.parse_args(argv)


# ----------------------------------------------------------------------------- CPU oracle arm
class _OneCore:
    """Pins the process to one core while the single-threaded oracle is timed."""

    def __enter__(self):
        self.old = None
        try:
            self.old = os.sched_getaffinity(0)
            os.sched_setaffinity(0, {sorted(self.old)[-1]})
        except (AttributeError, OSError):
            self.old = None
        return self

    def __exit__(self, *exc):
        if self.old:
            try:
                os.sched_setaffinity(0, self.old)
            except OSError:
                pass


def oracle_sample(wl, n_workers, sample_elems):
    """Inputs for the oracle: the workload's hyper-parameters and value distributions on an
    arena cut down to `sample_elems` elements."""
    import numpy as np

    from paper_2005_06728_b200 import workloads as W

    s = min(sample_elems, wl.arena_len)
    cut = W.ragged_workload([s], n_workers, lr=wl.lr, local_lr=wl.local_lr, momentum=wl.momentum,
                            wd=wl.wd, seed=wl.seed, name=wl.name + "-sample")
    cut.grad_sigma = wl.grad_sigma
    rng_w = W.make_weights(wl if wl.arena_len <= (1 << 24) else cut)
    w = rng_w[:s].numpy().copy()
    v = np.zeros(s, np.float32)
    grads = [W.make_grad(cut, m, 0).numpy() for m in range(n_workers)]
    return cut, w, v, grads


def time_oracle(wl, n_workers, sample_elems, steps, warmup, budget_s=25.0):
    """Times the oracle as it stands (single thread) on a sample made on the host."""
    import numpy as np

    import oracle
    from paper_2005_06728_b200.benchutil import algorithmic_bytes, host_info

    cut, w, v, grads = oracle_sample(wl, n_workers, sample_elems)
    s = w.size
    wp = np.empty_like(w)
    x = np.empty_like(w)
    times = []
    with _OneCore():
        t_start = time.perf_counter()
        for it in range(warmup + steps):
            t0 = time.perf_counter()
            oracle.global_update(grads, w, v, lr=wl.lr, momentum=wl.momentum, wd=wl.wd, w_prev=wp)
            oracle.local_update(wp, grads[0], local_lr=wl.local_lr, out=x)
            dt = time.perf_counter() - t0
            if it >= warmup:
                times.append(dt)
            if it >= warmup + 2 and time.perf_counter() - t_start > budget_s:
                break
    sec = statistics.median(times)
    nbytes = algorithmic_bytes("fused", s, n_workers)
    info = {"value": nbytes / sec / 1e9, "unit": "GB/s", "cores": 1, "kind": "oracle",
            "sample": f"first {s} of {wl.arena_len} elements of {wl.name}, all {n_workers} workers, "
                      f"{len(times)} calls of global+local update, single thread",
            "ms_per_call": sec * 1e3, "params_per_s": s / sec, "host": host_info()}
    return info, len(times), sec


def time_oracle_full(wl, n_workers, w_dev, grads_dev, passes=3):
    """Times the oracle as it stands (single thread) on the WHOLE arena of the workload: the
    benchmark's own device-resident inputs are brought to the host chunk by chunk (outside the
    timed sections; the rules are element-wise, so the oracle's loops are unchanged) and a pass
    is the sum of the oracle's time over all chunks.  Median of `passes` passes after a warm-up
    on the first chunk."""
    import numpy as np
    import torch

    import oracle
    from paper_2005_06728_b200.benchutil import algorithmic_bytes, host_info

    n = wl.arena_len
    ch = min(ORACLE_CHUNK, n)
    stage = torch.empty((n_workers, ch), dtype=torch.float32).pin_memory()
    w = w_dev.cpu().numpy().copy()
    v = np.zeros(n, np.float32)
    wp = np.empty(ch, np.float32)
    x = np.empty(ch, np.float32)
    hp = dict(lr=wl.lr, momentum=wl.momentum, wd=wl.wd)
    totals = []
    with _OneCore():
        for p in range(passes + 1):
            total = 0.0
            for a in range(0, n, ch):
                b = min(a + ch, n)
                for m in range(n_workers):
                    stage[m, :b - a].copy_(grads_dev[m][a:b], non_blocking=True)
                torch.cuda.synchronize()
                gh = [stage[m, :b - a].numpy() for m in range(n_workers)]
                t0 = time.perf_counter()
                oracle.global_update(gh, w[a:b], v[a:b], w_prev=wp[:b - a], **hp)
                oracle.local_update(wp[:b - a], gh[0], local_lr=wl.local_lr, out=x[:b - a])
                total += time.perf_counter() - t0
                if p == 0:
                    break  # warm-up: one chunk touches every buffer the later passes use
            if p > 0:
                totals.append(total)
    sec = statistics.median(totals)
    nbytes = algorithmic_bytes("fused", wl.n_params, n_workers)
    return {"value": nbytes / sec / 1e9, "unit": "GB/s", "cores": 1, "kind": "oracle",
            "sample": f"the whole {wl.name} arena ({n} elements, all {n_workers} workers), walked in chunks of "
                      f"{ch} elements; median of {passes} passes of global+local update, single thread",
            "ms_per_call": sec * 1e3, "params_per_s": wl.n_params / sec, "host": host_info()}


def run_reference(args):
    from paper_2005_06728_b200 import workloads as W
    from paper_2005_06728_b200.benchutil import rank_info

    if rank_info()["rank"] != 0:
        return 0
    wl = W.workload(args.workload)
    n_workers = args.workers or wl.n_workers
    info, done, sec = time_oracle(wl, n_workers, args.cpu_sample, args.steps, args.warmup, budget_s=150.0)
    line = {
        "impl": "reference", "metric": METRIC, "value": info["value"], "unit": "GB/s", "n_gpus": args.gpus,
        "steps": done, "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": workload_label(wl, n_workers), "n_params": wl.n_params, "n_tensors": wl.n_tensors,
                   "n_workers": n_workers, "sample_elems": min(args.cpu_sample, wl.arena_len),
                   "note": "CPU oracle, single thread, on a bounded sample of the workload"},
        "cpu_baseline": {k: info[k] for k in ("value", "unit", "cores", "kind", "sample")},
        "e2e": {"value": info["value"], "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0, "params_per_s": info["params_per_s"], "host": info["host"],
    }
    print(json.dumps(line), flush=True)
    return 0


# ----------------------------------------------------------------------------- CUDA arm
def _timed(fn, reps, stream, warm=3):
    """ms per call: CUDA events on the launching stream around `reps` back-to-back calls."""
    import torch

    for _ in range(warm):
        fn()
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record(stream)
    for _ in range(reps):
        fn()
    b.record(stream)
    torch.cuda.synchronize()
    return a.elapsed_time(b) / reps


def _rate(nbytes, ms, peak, hbm_bound=True):
    gbps = nbytes / ms / 1e6
    return {"ms": ms, "GBps": gbps, "frac": gbps / peak if hbm_bound else None,
            "frac_of_nominal_8000": gbps / NOMINAL_HBM_GBS if hbm_bound else None}


class _Set:
    """One parameter set resident on the device, with a context over it."""

    def __init__(self, wl, M, dev, flags=0, n_locals=1):
        import torch

        from paper_2005_06728_b200 import binding
        from paper_2005_06728_b200 import workloads as W

        self.wl, self.M, self.dev = wl, M, dev
        self.w_a = W.make_weights(wl, dev)
        self.w_b = torch.zeros_like(self.w_a)
        self.v = W.make_momentum(wl, dev)
        self.local = [self.w_a.clone() for _ in range(n_locals)] + [None] * (M - n_locals)
        self.sg, self.pads = W.sigma_arena(wl, dev), W.pad_mask(wl, dev)
        self.grads = [W.make_grad(wl, m, 0, dev, _sigma=self.sg, _pads=self.pads) for m in range(M)]
        self.flags = flags
        self.ctx = binding.Odsgd(self.w_a, self.v, n_workers=M, lr=wl.lr, local_lr=wl.local_lr, momentum=wl.momentum,
                                 wd=wl.wd, w_b=self.w_b, local=self.local, tensor_offsets=wl.offsets, flags=flags)

    def sub_context(self, m):
        """A context over the first m gradient buffers of the same arenas (worker sweep)."""
        from paper_2005_06728_b200 import binding

        wl = self.wl
        return binding.Odsgd(self.w_a, self.v, n_workers=m, lr=wl.lr, local_lr=wl.local_lr, momentum=wl.momentum,
                             wd=wl.wd, w_b=self.w_b, local=[self.local[0]] + [None] * (m - 1),
                             tensor_offsets=wl.offsets, flags=self.flags)


def _all_rules(s, reps, stream, peak, hbm_bound=True):
    """ms and GB/s of every rule on one resident set (bound gradient table, back-to-back calls)."""
    from paper_2005_06728_b200.benchutil import algorithmic_bytes

    ctx, P, M = s.ctx, s.wl.n_params, s.M
    bound = ctx.bind_grads(s.grads)
    out = {}
    calls = (("fused", lambda: ctx.fused_update(bound, 0, stream)),
             ("global", lambda: ctx.global_update(bound, stream)),
             ("local", lambda: ctx.local_update(0, stream)),
             ("ssgd", lambda: ctx.ssgd_step(bound, stream)),
             ("asgd", lambda: ctx.asgd_step(0, s.grads[0], stream)))
    for name, fn in calls:
        if name == "local":
            ctx.global_update(bound, stream)
        out[name] = _rate(algorithmic_bytes(name, P, M), _timed(fn, reps, stream), peak, hbm_bound)
    bound.unbind()
    return out


def _sweep(s, worker_counts, reps, stream, peak):
    from paper_2005_06728_b200.benchutil import algorithmic_bytes

    rows = []
    for m in worker_counts:
        if m < 1 or m > s.M:
            continue
        c2 = s.sub_context(m)
        bound = c2.bind_grads(s.grads[:m])
        ms = _timed(lambda: c2.fused_update(bound, 0, stream), reps, stream)
        nb = algorithmic_bytes("fused", s.wl.n_params, m)
        row = {"workers": m, "bytes_per_step": nb, "params_per_s": s.wl.n_params / (ms * 1e-3),
               "grad_elems_per_s": m * s.wl.n_params / (ms * 1e-3)}
        row.update(_rate(nb, ms, peak))
        rows.append(row)
        c2.close()
    return rows


def _end_to_end(s, step_bytes, steps, stream, dev, world=1):
    """The fused update through the host-buffer entry point: every step copies the M gradients
    from pinned host memory, runs the kernel and copies the worker's new weights back, all
    inside the timed region.  The set's gradient arenas serve as the device staging buffers."""
    import torch

    from paper_2005_06728_b200 import workloads as W
    from paper_2005_06728_b200.benchutil import aggregate, barrier

    wl, M, ctx, n = s.wl, s.M, s.ctx, s.wl.arena_len
    pool = [W.make_grad(wl, m, 1, dev, _sigma=s.sg, _pads=s.pads).cpu().pin_memory() for m in range(min(M, 4))]
    host_grads = [pool[m % len(pool)] for m in range(M)]
    host_out = torch.empty(n, dtype=torch.float32).pin_memory()
    # copy-back on a second stream overlaps the next step's uploads; for small arenas the
    # cross-stream hand-over costs more than it hides, so they keep a single stream
    copy_stream = torch.cuda.Stream(device=dev) if n * 4 >= (1 << 26) else None
    ctx.fused_update_host(host_grads, s.grads, 0, host_out, stream, copy_stream)
    torch.cuda.synchronize()
    barrier(dev)
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0 = time.perf_counter()
    a.record(stream)
    for _ in range(steps):
        ctx.fused_update_host(host_grads, s.grads, 0, host_out, stream, copy_stream)
    if copy_stream is not None:
        stream.wait_stream(copy_stream)  # the last copy-back is inside the timed region
    b.record(stream)
    torch.cuda.synchronize()
    wall_ms = (time.perf_counter() - t0) * 1e3
    e2e_ms = max(a.elapsed_time(b), wall_ms)
    agg2 = aggregate(e2e_ms, float(step_bytes) * steps, dev if world > 1 else None)
    h2d, d2h = M * n * 4, n * 4
    return {"value": agg2["units"] / (agg2["ms"] * 1e-3) / 1e9, "unit": "GB/s",
            "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": steps,
            "ms_per_step": agg2["ms"] / steps,
            "h2d_GBps": h2d * steps * world / (agg2["ms"] * 1e-3) / 1e9,
            "what": "ALGORITHMIC bytes of the update, (M + 5) * 4 * P per step, over a time that is set by the "
                    "host link: M * 4 * P bytes cross it per step (h2d_GBps is that traffic over the same time), "
                    "so this figure may sit above what the bus itself carries",
            "note": f"{M} host-to-device copies per step from a pool of {len(pool)} distinct pinned buffers; "
                    + ("copy-back of the local weights on a second stream" if copy_stream is not None
                       else "copy-back on the same stream (small arena)")}


def _small_set_entry(name, dev, stream, flags, cpu_full=True, steps=4000, graph_steps=20):
    """A cache-resident set: eager launches through the bound-table call, and CUDA-graph replay."""
    import torch

    from paper_2005_06728_b200 import workloads as W
    from paper_2005_06728_b200.benchutil import algorithmic_bytes

    wl = W.workload(name)
    s = _Set(wl, wl.n_workers, dev, flags)
    ctx = s.ctx
    bound = ctx.bind_grads(s.grads)
    sh = stream.cuda_stream
    raw, slot = ctx.fused_update_bound_raw, bound.slot
    rcs = []
    eager_ms = _timed(lambda: rcs.append(raw(slot, 0, sh)), steps, stream, warm=20)
    bad = [rc for rc in rcs if rc != 0]
    if bad:
        ctx.check(bad[0])
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        for _ in range(graph_steps):
            ctx.fused_update(bound, 0)
    graph_ms = _timed(graph.replay, max(1, steps // graph_steps), stream) / graph_steps
    nb = algorithmic_bytes("fused", wl.n_params, wl.n_workers)
    entry = {"workload": workload_label(wl, wl.n_workers), "n_params": wl.n_params, "n_tensors": wl.n_tensors,
             "n_workers": wl.n_workers, "bytes_per_step": nb,
             "l2": "effective, L2-resident: the working set fits in the 126 MB L2, so these are not HBM figures",
             "fused": {"eager_us_per_step": eager_ms * 1e3, "eager_effective_GBps": nb / eager_ms / 1e6,
                       "graph_us_per_step": graph_ms * 1e3, "graph_effective_GBps": nb / graph_ms / 1e6,
                       "frac": None, "steps": steps,
                       "launch": "eager: odsgd_fused_update_bound from a Python loop, one launch per step; "
                                 f"graph: {graph_steps} steps captured once and replayed"},
             "params_per_s": wl.n_params / (eager_ms * 1e-3)}
    bound.unbind()
    rules = _all_rules(s, 200, stream, 1.0, hbm_bound=False)
    for k, r in rules.items():
        if k != "fused":
            entry[k] = {"us": r["ms"] * 1e3, "effective_GBps": r["GBps"], "frac": None}
    if cpu_full:
        entry["cpu_oracle_full"] = time_oracle_full(wl, wl.n_workers, s.w_a, s.grads, passes=5)
    ctx.close()
    return entry


def _large_set_entry(name, dev, stream, flags, peak, reps, cpu_full, e2e):
    import torch

    from paper_2005_06728_b200 import workloads as W
    from paper_2005_06728_b200.benchutil import algorithmic_bytes

    wl = W.workload(name)
    s = _Set(wl, wl.n_workers, dev, flags)
    entry = {"workload": workload_label(wl, wl.n_workers), "n_params": wl.n_params, "n_tensors": wl.n_tensors,
             "n_workers": wl.n_workers, "bytes_per_step": algorithmic_bytes("fused", wl.n_params, wl.n_workers),
             "l2": "inputs per step exceed the 126 MB L2 many times over: no flush", "reps": reps}
    entry.update(_all_rules(s, reps, stream, peak))
    entry["params_per_s"] = wl.n_params / (entry["fused"]["ms"] * 1e-3)
    entry["grad_elems_per_s"] = wl.n_workers * entry["params_per_s"]
    if e2e:
        entry["e2e"] = _end_to_end(s, entry["bytes_per_step"], 6, stream, dev)
    if cpu_full:
        entry["cpu_oracle_full"] = time_oracle_full(wl, wl.n_workers, s.w_a, s.grads)
    s.ctx.close()
    del s
    torch.cuda.empty_cache()
    return entry


def run_cuda(args):
    import torch

    from paper_2005_06728_b200 import binding
    from paper_2005_06728_b200 import workloads as W
    from paper_2005_06728_b200.benchutil import (ClockSampler, aggregate, algorithmic_bytes, barrier,
                                                 init_process_group, rank_info)

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the update pass has no CPU path")
    from paper_2005_06728_b200 import build as cuda_build

    if cuda_build.is_stale():
        cuda_build.build()  # raises if nvcc is missing or the build fails
    binding.load_library()  # fail now if the CUDA library is missing
    ri = rank_info()
    world = ri["world_size"]
    if world > 1:
        init_process_group("nccl")
    dev = torch.device("cuda", ri["local_rank"] if world > 1 else 0)
    torch.cuda.set_device(dev)
    rank0 = ri["rank"] == 0

    wl = W.workload(args.workload)
    M = args.workers or wl.n_workers
    n, P = wl.arena_len, wl.n_params
    free, total = torch.cuda.mem_get_info()
    need = (M + 5 + (3 * M if args.all_locals else 0)) * n * 4
    if need > 0.9 * free:
        raise SystemExit(f"{wl.name} with {M} workers needs {need / 2**30:.1f} GiB; {free / 2**30:.1f} GiB free")

    flags = binding.FLAG_ALLOW_FMA if args.allow_fma else 0
    n_locals = M if args.all_locals else 1
    wid = -1 if args.all_locals else 0
    head = _Set(wl, M, dev, flags, n_locals)
    ctx, local, grad_list = head.ctx, head.local, head.grads
    w_a = head.w_a
    if args.block or args.ctas_per_sm:
        ctx.set_launch_config(args.block, args.ctas_per_sm)
    stream = torch.cuda.current_stream()
    extra_streams = 0  # arenas touched per local update beyond the plain rule's single store
    if args.local_rule != "sgd":
        rule = {"dc_c": binding.LOCAL_DC_C, "dc_a": binding.LOCAL_DC_A, "momentum": binding.LOCAL_MOMENTUM}[args.local_rule]
        ms = [torch.zeros_like(w_a) for _ in range(n_locals)] + [None] * (M - n_locals) if rule != binding.LOCAL_DC_C else None
        ctx.set_local_rule(rule, 0.04 if rule != binding.LOCAL_MOMENTUM else wl.wd, 0.95, 1e-7, ms)
        # arenas touched per local update beyond the store of x: x_prev read (Eq. 4, 5), state read + write
        extra_streams = n_locals * {binding.LOCAL_DC_C: 1, binding.LOCAL_DC_A: 3, binding.LOCAL_MOMENTUM: 2}[rule]
    if args.multipliers:
        ctx.set_tensor_multipliers(None, [1.0 if t.kind == "weight" else 0.0 for t in wl.tensors])

    step_bytes = algorithmic_bytes("fused", P, M, n_locals) + extra_streams * 4 * P
    hbm_bound = step_bytes > 8 * L2_BYTES
    grads = ctx.bind_grads(grad_list)  # validated once, as a training loop would
    l2_note = ("inputs per step exceed the 126 MB L2 many times over: no flush" if hbm_bound
               else "working set fits in L2: effective GB/s, not an HBM figure")

    for _ in range(max(3, args.warmup)):
        ctx.fused_update(grads, wid, stream)
    torch.cuda.synchronize()
    graph = None
    if args.graph:
        if args.graph % 2 or args.steps % args.graph:
            raise SystemExit("--graph must be even (the weight halves swap every step) and divide --steps")
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            for _ in range(args.graph):
                ctx.fused_update(grads, wid)  # lands on the capturing stream
        for _ in range(3):
            graph.replay()
        torch.cuda.synchronize()
    barrier(dev)
    torch.cuda.synchronize()
    if graph is None:
        # an event after every step for steps of half a millisecond or more; for short steps (where
        # the event itself would cost as much as the step) one every `stride` steps
        probe_ms = _timed(lambda: ctx.fused_update(grads, wid, stream), 4, stream, warm=0)
        stride = 1 if probe_ms >= 0.5 else max(1, min(50, args.steps // 8))
        marks = list(range(0, args.steps, stride)) + [args.steps]
        ev = {k: torch.cuda.Event(enable_timing=True) for k in marks}
        launches_before = ctx.launch_count
        with ClockSampler(dev.index or 0) as clocks:
            # the bound-table entry point with the slot and the stream handle looked up once: on
            # the small sets the wrapper's own marshalling would be a third of a step
            raw, slot, sh, rcs = ctx.fused_update_bound_raw, grads.slot, stream.cuda_stream, []
            ev[0].record(stream)
            for k in range(args.steps):
                rcs.append(raw(slot, wid, sh))
                if k + 1 in ev:
                    ev[k + 1].record(stream)
            torch.cuda.synchronize()
        for rc in rcs:
            ctx.check(rc)
        gpu_launches = ctx.launch_count - launches_before
        per_step = [ev[a].elapsed_time(ev[b]) / (b - a) for a, b in zip(marks[:-1], marks[1:])]
        total_ms = ev[0].elapsed_time(ev[args.steps])
    else:
        replays = args.steps // args.graph
        evl = [torch.cuda.Event(enable_timing=True) for _ in range(replays + 1)]
        with ClockSampler(dev.index or 0) as clocks:
            evl[0].record(stream)
            for k in range(replays):
                graph.replay()
                evl[k + 1].record(stream)
            torch.cuda.synchronize()
        gpu_launches = args.steps  # one kernel node per captured step, replayed
        per_step = [evl[k].elapsed_time(evl[k + 1]) / args.graph for k in range(replays)]
        total_ms = evl[0].elapsed_time(evl[-1])
    barrier(dev)
    torch.cuda.synchronize()
    agg = aggregate(total_ms, float(step_bytes) * args.steps, dev if world > 1 else None)
    ms_per_step = agg["ms"] / args.steps
    value = agg["units"] / (agg["ms"] * 1e-3) / 1e9
    kernel_ms = total_ms / args.steps  # one launch per step, back to back on one stream
    achieved = step_bytes / (kernel_ms * 1e-3) / 1e9
    peak, peak_src = hbm_peak()

    # ---- the other rules on the same arena (context only; not part of `value`)
    extra = {}
    if not args.no_extra_kernels and rank0:
        reps = max(5, min(50, args.steps))
        for name, fn in (("global", lambda: ctx.global_update(grads, stream)),
                         ("local", lambda: ctx.local_update(0, stream)),
                         ("ssgd", lambda: ctx.ssgd_step(grads, stream)),
                         ("asgd", lambda: ctx.asgd_step(0, grad_list[0], stream))):
            if name == "local":
                ctx.global_update(grads, stream)
            extra[name] = _rate(algorithmic_bytes(name, P, M), _timed(fn, reps, stream), peak, hbm_bound)

    # ---- worker-count sweep on the same arena (fused update, first m gradient buffers)
    sweep_counts = [int(x) for x in args.sweep_workers.split(",") if x]
    if not sweep_counts and not args.no_configs and world == 1 and args.workload == "vgg16" and not args.workers:
        sweep_counts = [1, 2, 4, 8, 16, 32]
    sweep = _sweep(head, sweep_counts, max(20, min(200, args.steps)), stream, peak) if sweep_counts and rank0 else []

    # ---- end to end: gradients start in pinned host memory, local weights come back
    e2e = None
    if not args.no_e2e:
        e2e = _end_to_end(head, step_bytes, max(2, min(args.steps, 6)), stream, dev, world)

    if not rank0:
        return 0

    cpu = None
    if not args.no_cpu_baseline and world == 1:
        info = time_oracle_full(wl, M, w_a, grad_list)
        cpu = {k: info[k] for k in ("value", "unit", "cores", "kind", "sample", "ms_per_call")}
        cpu["host"] = info["host"]

    # ---- the other parameter sets (reported under `configs`; not part of `value`)
    configs = []
    if not args.no_configs and world == 1 and args.workload == "vgg16" and not args.workers:
        grads.unbind()
        ctx.close()
        del head, ctx, local, grad_list, grads, w_a
        torch.cuda.empty_cache()
        for name in ("alexnet", "resnet50"):
            configs.append(_large_set_entry(name, dev, stream, flags, peak, reps=200,
                                            cpu_full=not args.no_cpu_baseline, e2e=not args.no_e2e))
        for name in ("resnet56", "lenet5"):
            configs.append(_small_set_entry(name, dev, stream, flags, cpu_full=not args.no_cpu_baseline))

    ck = clocks.summary()
    roof_frac = achieved / peak if hbm_bound else None
    line = {
        "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps,
        "warmup": max(3, args.warmup), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": workload_label(wl, M),
                   "n_params": P, "n_tensors": wl.n_tensors, "n_workers": M,
                   "bytes_per_step": step_bytes, "l2": l2_note,
                   "flavour": "FMA contraction allowed" if args.allow_fma else "default: one rounding per operator, bit-exact against the CPU oracle",
                   "variant": {"local_rule": args.local_rule, "locals_updated": n_locals, "multipliers": args.multipliers},
                   "launch": f"CUDA graph of {args.graph} steps, replayed" if args.graph else "one launch per step from the host",
                   "parallelism": "independent replicas" if world > 1 else "single GPU"},
        "clocks": {"sm_mhz": ck.get("sm_mhz"), "sm_max_mhz": ck.get("sm_max_mhz"), "reasons": ck.get("reasons", []),
                   "power_w_max": ck.get("power_w_max"), "samples": ck.get("samples"), "source": ck.get("source")},
        "e2e": e2e, "gpu_launches": gpu_launches,
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": roof_frac,
                     "traffic": measured_traffic(step_bytes) if hbm_bound else None, "peak_source": f"of {peak_src}",
                     "kernel": "server_kernel (fused, one local)", "kernel_ms": kernel_ms,
                     "frac_of_nominal_8000": achieved / NOMINAL_HBM_GBS if hbm_bound else None,
                     "note": None if hbm_bound else "cache-resident working set: effective GB/s, no HBM fraction"},
        "cpu_baseline": cpu,
        "params_per_s": P * args.steps * world / (agg["ms"] * 1e-3),
        "grad_elems_per_s": M * P * args.steps * world / (agg["ms"] * 1e-3),
        "step_ms": {"median": statistics.median(per_step), "min": min(per_step), "max": max(per_step)},
        "other_kernels": extra,
    }
    if sweep:
        line["worker_sweep"] = sweep
    if configs:
        line["configs"] = configs
    print(json.dumps(line), flush=True)
    return 0


# ----------------------------------------------------------------------------- sharded server arm
def run_sharded(args):
    """One OD-SGD iteration per step with the server role sharded over the ranks: every rank hosts
    M / N workers, pushes the slices of their gradients to the owners, updates the slice it owns
    and gathers the new weights, while the hosted workers' local updates run on a second stream.
    Total work is fixed as N grows (strong scaling)."""
    import torch
    import torch.distributed as dist

    from paper_2005_06728_b200 import binding, shard
    from paper_2005_06728_b200 import workloads as W
    from paper_2005_06728_b200.benchutil import ClockSampler, aggregate, barrier, init_process_group, rank_info

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the update pass has no CPU path")
    binding.load_library()
    ri = rank_info()
    world, rank = ri["world_size"], ri["rank"]
    dev = torch.device("cuda", ri["local_rank"])
    torch.cuda.set_device(dev)
    if world > 1:
        init_process_group("nccl")
    elif not dist.is_initialized():
        import socket

        with socket.socket() as sock:
            sock.bind(("127.0.0.1", 0))
            port = sock.getsockname()[1]
        dist.init_process_group("nccl", init_method=f"tcp://127.0.0.1:{port}", rank=0, world_size=1)
    wl = W.workload(args.workload)
    M = args.workers or wl.n_workers
    if M % world:
        raise SystemExit(f"--sharded: {M} workers do not divide over {world} ranks")
    k = M // world
    n = wl.arena_len
    lay = shard.ShardLayout(n, world, k)
    w0 = W.make_weights(wl, dev)
    exchange = shard.PeerExchange(lay, rank, dev) if args.peer else shard.ShardExchange(lay, rank)
    sh = shard.ShardedOdsgd(lay, rank, w0, lr=wl.lr, local_lr=wl.local_lr, momentum=wl.momentum, wd=wl.wd,
                            exchange=exchange, flags=binding.FLAG_ALLOW_FMA if args.allow_fma else 0)
    sg, pads = W.sigma_arena(wl, dev), W.pad_mask(wl, dev)
    grads = []
    for j in range(k):
        # the peer exchange reads the gradients where the workers produce them: its own arenas
        g = exchange.grad_arenas[j] if args.peer else torch.zeros(lay.padded_len, dtype=torch.float32, device=dev)
        W.make_grad(wl, lay.worker_id(rank, j), 0, dev, out=g[:n], _sigma=sg, _pads=pads)
        grads.append(g)
    stream = torch.cuda.current_stream()
    for _ in range(max(3, args.warmup)):
        sh.step(grads)
    torch.cuda.synchronize()
    barrier(dev)
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with ClockSampler(dev.index or 0) as clocks:
        a.record(stream)
        for _ in range(args.steps):
            sh.step(grads)
        b.record(stream)
        torch.cuda.synchronize()
    barrier(dev)
    torch.cuda.synchronize()
    P = wl.n_params
    own = sh.end - sh.begin
    # bytes this rank's kernels move per step: server rule on its slice, local rule for its k workers
    local_bytes = (M + 4) * 4 * own + k * 3 * 4 * P
    agg = aggregate(a.elapsed_time(b), float(local_bytes) * args.steps, dev)
    if args.peer:
        exchange.quiesce()  # no rank drops its symmetric buffers while a peer may still touch them
    if rank != 0:
        return 0
    S = lay.shard_len
    ck = clocks.summary()
    value = agg["units"] / (agg["ms"] * 1e-3) / 1e9
    line = {
        "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps,
        "warmup": max(3, args.warmup), "ms_per_step": agg["ms"] / args.steps, "higher_is_better": True,
        "scaling": "strong", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": f"{wl.name}-shaped parameter set, M={M} workers, sharded server + local updates",
                   "n_params": P, "n_workers": M, "workers_per_rank": k, "shard_len": S,
                   "bytes_per_step": (M + 4) * 4 * P + M * 3 * 4 * P,
                   "exchange_bytes_per_rank_per_step": {"push_sent": k * (world - 1) * S * 4,
                                                        "pull_received": (world - 1) * S * 4},
                   "parallelism": (f"server role sharded over {world} rank(s): the kernel on the owned slice reads "
                                   "the other ranks' gradient slices and writes their replicas through symmetric "
                                   "memory, one fence either side; local updates on a second stream") if args.peer else
                                  (f"server role sharded over {world} rank(s): all-to-all of gradient slices, "
                                   "kernel on the owned slice, all-gather of the weights; local updates on a second stream"),
                   "note": "value counts the bytes the update kernels move (server rule on every slice + every worker's "
                           "local rule), not the bytes on the links"},
        "clocks": {"sm_mhz": ck.get("sm_mhz"), "sm_max_mhz": ck.get("sm_max_mhz"), "reasons": ck.get("reasons", []),
                   "samples": ck.get("samples"), "source": ck.get("source")},
        "e2e": None, "gpu_launches": args.steps * (k + (1 if own > 0 else 0)),
        "params_per_s": P * args.steps / (agg["ms"] * 1e-3),
    }
    print(json.dumps(line), flush=True)
    sh.close()
    return 0


# ----------------------------------------------------------------------------- launching N ranks
def self_launch_command(argv, n_gpus, port):
    """The torchrun command line that runs this script as `n_gpus` ranks on this node."""
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n_gpus}",
            "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.join(ROOT, "bench.py"), *argv]


def self_launch(argv, n_gpus):
    import socket

    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    return subprocess.run(self_launch_command(argv, n_gpus, port), cwd=ROOT).returncode


def main(argv=None):
    argv = list(sys.argv[1:] if argv is None else argv)
    args = parse_args(argv)
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # started plainly: become the launcher of the N ranks (each re-enters main() under torchrun)
        if args.impl == "cuda":
            import torch

            have = torch.cuda.device_count()
            if have < args.gpus:
                raise SystemExit(f"--gpus {args.gpus}: only {have} CUDA device(s) visible")
        return self_launch(argv, args.gpus)
    if args.impl == "reference":
        return run_reference(args)
    try:
        return run_sharded(args) if args.sharded else run_cuda(args)
    finally:
        try:
            import torch.distributed as dist

            if dist.is_available() and dist.is_initialized():
                dist.destroy_process_group()
        except Exception:
            pass


if __name__ == "__main__":
    sys.exit(main())
