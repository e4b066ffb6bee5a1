"""The N > 1 plumbing of the benchmark on CPU: world size 2 over gloo.

The ranks of the benchmark share no data (independent replicas); what crosses between them is
a barrier and the reduction of two scalars, which is what these tests cover.
"""
import json
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _torchrun(script_args, nproc=2, timeout=240):
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={nproc}",
           "--master-addr", "127.0.0.1", "--master-port", str(_free_port()), *script_args]
    env = dict(os.environ, CUDA_VISIBLE_DEVICES="", OMP_NUM_THREADS="1")
    return subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=timeout)


def _json_lines(text):
    out = []
    for line in text.splitlines():
        line = line.strip()
        if line.startswith("{") and line.endswith("}"):
            out.append(json.loads(line))
    return out


def test_aggregate_takes_slowest_rank_and_sums_work():
    res = _torchrun([os.path.join("tests", "_rank_worker.py")])
    assert res.returncode == 0, res.stderr[-2000:]
    lines = _json_lines(res.stdout)
    assert len(lines) == 1
    assert lines[0] == {"ms": 15.0, "units": 3000.0, "world_size": 2}


def test_reference_arm_prints_one_line_from_rank_zero():
    res = _torchrun(["bench.py", "--impl", "reference", "--gpus", "2", "--steps", "2", "--warmup", "1",
                     "--workload", "lenet5", "--cpu-sample", "100000"])
    assert res.returncode == 0, res.stderr[-2000:]
    lines = _json_lines(res.stdout)
    assert len(lines) == 1, "rank 0 alone prints; the other rank exits quietly"
    d = lines[0]
    assert d["impl"] == "reference" and d["n_gpus"] == 2 and d["unit"] == "GB/s" and d["value"] > 0
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] == 1
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["e2e"]["value"] == d["value"]
    assert d["vs_baseline"] is None and d["higher_is_better"] is True


def test_plain_start_with_gpus_launches_the_ranks_itself():
    """`python bench.py --gpus 2` without torchrun becomes the launcher of its two ranks."""
    env = dict(os.environ, CUDA_VISIBLE_DEVICES="", OMP_NUM_THREADS="1")
    for k in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT"):
        env.pop(k, None)
    res = subprocess.run([sys.executable, "bench.py", "--impl", "reference", "--gpus", "2", "--steps", "2",
                          "--warmup", "1", "--workload", "lenet5", "--cpu-sample", "100000"],
                         cwd=ROOT, env=env, capture_output=True, text=True, timeout=240)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = _json_lines(res.stdout)
    assert len(lines) == 1 and lines[0]["n_gpus"] == 2 and lines[0]["impl"] == "reference"
    # the CUDA arm refuses, in words, to start more ranks than there are devices
    res = subprocess.run([sys.executable, "bench.py", "--gpus", "2", "--steps", "2"], cwd=ROOT, env=env,
                         capture_output=True, text=True, timeout=240)
    assert res.returncode != 0 and "CUDA device" in res.stderr
    import bench

    cmd = bench.self_launch_command(["--gpus", "4", "--steps", "3"], 4, 29999)
    assert "--nproc-per-node=4" in cmd and cmd[-4:] == ["--gpus", "4", "--steps", "3"] and "127.0.0.1" in cmd


def test_single_process_aggregate_is_identity():
    from paper_2005_06728_b200 import benchutil

    assert benchutil.aggregate(3.5, 7.0) == {"ms": 3.5, "units": 7.0, "world_size": 1}


def test_algorithmic_bytes():
    from paper_2005_06728_b200.benchutil import algorithmic_bytes as ab

    P = 1000
    assert ab("global", P, 8) == 12 * 4 * P and ab("ssgd", P, 8) == 12 * 4 * P
    assert ab("local", P, 8) == 3 * 4 * P and ab("asgd", P, 8) == 5 * 4 * P
    assert ab("fused", P, 8) == 13 * 4 * P, "(M + 3) read + 2 written, times 4P"
    assert ab("fused", P, 8, n_locals=8) == 20 * 4 * P


def test_profiled_traffic_constants_match_the_committed_capture(tmp_path):
    """bench.py carries the traffic ratio and the kernel-source digest of the ncu capture as
    constants; they must be the ones the profile summary records, and the traffic is only
    reported while the kernel source still is the profiled one (comments aside)."""
    import importlib.util
    import re

    spec = importlib.util.spec_from_file_location("bench_module", os.path.join(ROOT, "bench.py"))
    bench = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(bench)
    note = open(os.path.join(ROOT, "profiles", "server_kernel_fused_m32_resnet50_arena.md")).read()
    assert float(re.search(r"^traffic_ratio:\s*([0-9.]+)", note, re.M).group(1)) == bench.PROFILED_TRAFFIC_RATIO
    assert re.search(r"^kernel_source_digest:\s*([0-9a-f]+)", note, re.M).group(1) == bench.PROFILED_KERNEL_DIGEST
    current = bench.kernel_source_digest() == bench.PROFILED_KERNEL_DIGEST
    got = bench.measured_traffic(1000)
    assert got == (bench.PROFILED_TRAFFIC_RATIO * 1000 if current else None)
    # the digest ignores comments and blank lines, and nothing else
    src = open(bench.KERNEL_SOURCE, encoding="utf-8").read()
    a = tmp_path / "a.cuh"
    a.write_text("// a new remark\n\n" + src.replace("#pragma once", "#pragma once  // reworded"))
    assert bench.kernel_source_digest(str(a)) == bench.kernel_source_digest()
    a.write_text(src.replace("#define ODSGD_BATCH 8", "#define ODSGD_BATCH 4"))
    assert bench.kernel_source_digest(str(a)) != bench.kernel_source_digest()
