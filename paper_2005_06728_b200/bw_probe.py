"""Builds and runs the bandwidth-ceiling probe (csrc/bw_probe.cu) on the current GPU.

    python -m paper_2005_06728_b200.bw_probe [GiB]

Prints the probe's table and a one-line summary of the ceilings: best pure-read rate for
128-bit loads, 256-bit loads and TMA bulk copies, and best 1:1 copy rate (read + written bytes).
"""
from __future__ import annotations

import os
import re
import subprocess
import sys
from typing import Dict

from .build import CSRC, PKG, nvcc_path

EXE = os.path.join(PKG, "bw_probe_bin")
SRC = os.path.join(CSRC, "bw_probe.cu")


def build(force: bool = False) -> str:
    if force or not os.path.exists(EXE) or os.path.getmtime(EXE) < os.path.getmtime(SRC):
        cmd = [nvcc_path(), "-O3", "-std=c++17", "-lineinfo", "-gencode", "arch=compute_100a,code=sm_100a",
               "-o", EXE, SRC]
        res = subprocess.run(cmd, capture_output=True, text=True)
        if res.returncode != 0:
            raise RuntimeError("nvcc failed:\n" + res.stdout + res.stderr)
    return EXE


def run(gib: int = 8) -> Dict[str, float]:
    out = subprocess.run([build(), str(gib)], capture_output=True, text=True, check=True).stdout
    sys.stdout.write(out)
    best: Dict[str, float] = {}
    for line in out.splitlines():
        m = re.match(r"(read128|read256|tma|copy128|cudaMemcpy)\b.*?([0-9.]+) GB/s", line)
        if m:
            key = {"copy128": "copy", "cudaMemcpy": "copy"}.get(m.group(1), m.group(1))
            best[key] = max(best.get(key, 0.0), float(m.group(2)))
    return best


if __name__ == "__main__":
    print(run(int(sys.argv[1]) if len(sys.argv) > 1 else 8))
