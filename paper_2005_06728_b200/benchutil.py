"""Measurement plumbing for the benchmark: clock sampling, rank aggregation, byte counts.

Nothing here computes an update; it only watches the GPU and adds up numbers.
"""
from __future__ import annotations

import os
import statistics
import subprocess
import threading
from typing import Dict, List, Optional

BAD_REASONS = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown")


# ----------------------------------------------------------------------------- byte counts
def algorithmic_bytes(kernel: str, n_params: int, n_workers: int, n_locals: int = 1) -> int:
    """Bytes the rule itself must move per call (every buffer touched once), fp32.

    global / ssgd : M gradients + w + v read, w + v written          -> (M + 4) * 4P
    local         : w_bak + g read, x written                        -> 3 * 4P
    fused         : M gradients + w + v read, w + v + L locals written -> (M + 4 + L) * 4P
    asgd          : g + w + v read, w + v written                    -> 5 * 4P
    """
    p4 = 4 * n_params
    if kernel in ("global", "ssgd"):
        return (n_workers + 4) * p4
    if kernel == "local":
        return 3 * p4
    if kernel == "fused":
        return (n_workers + 4 + n_locals) * p4
    if kernel == "asgd":
        return 5 * p4
    raise KeyError(kernel)


# ----------------------------------------------------------------------------- clocks
class ClockSampler:
    """Samples SM clock, power and throttle reasons of one GPU while a region runs.

    Reads only (NVML queries, or `nvidia-smi --query-gpu` as a fallback); never changes a
    setting.  Use as a context manager around the timed region.
    """

    def __init__(self, cuda_index: int = 0, period_s: float = 0.005):
        self.cuda_index = cuda_index
        self.period_s = period_s
        self.samples: List[Dict] = []
        self.sm_max_mhz: Optional[float] = None
        self._stop = threading.Event()
        self._thread: Optional[threading.Thread] = None
        self._proc: Optional[subprocess.Popen] = None
        self._nvml = None
        self._handle = None
        self.source = "none"

    def _physical_index(self) -> str:
        vis = os.environ.get("CUDA_VISIBLE_DEVICES")
        if vis:
            parts = [p.strip() for p in vis.split(",") if p.strip()]
            if self.cuda_index < len(parts):
                return parts[self.cuda_index]
        return str(self.cuda_index)

    def _open_nvml(self) -> bool:
        try:
            import pynvml

            pynvml.nvmlInit()
            ident = self._physical_index()
            if ident.isdigit():
                self._handle = pynvml.nvmlDeviceGetHandleByIndex(int(ident))
            else:
                self._handle = pynvml.nvmlDeviceGetHandleByUUID(ident.encode())
            self.sm_max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(self._handle, pynvml.NVML_CLOCK_SM))
            self._nvml = pynvml
            self.source = "nvml"
            return True
        except Exception:
            self._nvml = None
            return False

    def _reasons_nvml(self) -> List[str]:
        n = self._nvml
        try:
            mask = n.nvmlDeviceGetCurrentClocksEventReasons(self._handle)
        except Exception:
            mask = n.nvmlDeviceGetCurrentClocksThrottleReasons(self._handle)
        names = {
            "sw_power_cap": getattr(n, "nvmlClocksThrottleReasonSwPowerCap", 0x4),
            "hw_slowdown": getattr(n, "nvmlClocksThrottleReasonHwSlowdown", 0x8),
            "sync_boost": getattr(n, "nvmlClocksThrottleReasonSyncBoost", 0x10),
            "sw_thermal_slowdown": getattr(n, "nvmlClocksThrottleReasonSwThermalSlowdown", 0x20),
            "hw_thermal_slowdown": getattr(n, "nvmlClocksThrottleReasonHwThermalSlowdown", 0x40),
            "hw_power_brake": getattr(n, "nvmlClocksThrottleReasonHwPowerBrakeSlowdown", 0x80),
            "applications_clocks": getattr(n, "nvmlClocksThrottleReasonApplicationsClocksSetting", 0x2),
        }
        return [k for k, bit in names.items() if mask & bit]

    def _loop_nvml(self) -> None:
        n = self._nvml
        while not self._stop.is_set():
            try:
                s = {"sm_mhz": float(n.nvmlDeviceGetClockInfo(self._handle, n.NVML_CLOCK_SM)),
                     "power_w": n.nvmlDeviceGetPowerUsage(self._handle) / 1000.0,
                     "reasons": self._reasons_nvml()}
                self.samples.append(s)
            except Exception:
                pass
            self._stop.wait(self.period_s)

    def _loop_smi(self) -> None:
        q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")
        try:
            self._proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={q}", "--format=csv,noheader,nounits",
                 "-lms", str(max(20, int(self.period_s * 1000))), "-i", self._physical_index()],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            return
        self.source = "nvidia-smi"
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for line in self._proc.stdout:  # ends when the process is terminated
            f = [x.strip() for x in line.split(",")]
            try:
                self.sm_max_mhz = float(f[1])
                self.samples.append({"sm_mhz": float(f[0]), "power_w": float(f[2]),
                                     "reasons": [n for n, v in zip(names, f[3:7]) if v.lower().startswith("active")]})
            except (ValueError, IndexError):
                continue

    def __enter__(self) -> "ClockSampler":
        target = self._loop_nvml if self._open_nvml() else self._loop_smi
        self._thread = threading.Thread(target=target, daemon=True)
        self._thread.start()
        return self

    def __exit__(self, *exc) -> None:
        self._stop.set()
        if self._proc is not None:
            self._proc.terminate()  # our own child, by handle
        if self._thread is not None:
            self._thread.join(timeout=2.0)
        if self._nvml is not None:
            try:
                self._nvml.nvmlShutdown()
            except Exception:
                pass

    def summary(self) -> Dict:
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.sm_max_mhz, "reasons": [], "samples": 0,
                    "source": self.source}
        busy = [s for s in self.samples if s["power_w"] is not None]
        mhz = [s["sm_mhz"] for s in busy]
        reasons = sorted({r for s in busy for r in s["reasons"]})
        return {"sm_mhz": statistics.median(mhz), "sm_max_mhz": self.sm_max_mhz, "reasons": reasons,
                "power_w_max": max(s["power_w"] for s in busy), "samples": len(busy), "source": self.source,
                "rejected": any(r in BAD_REASONS for r in reasons)}


# ----------------------------------------------------------------------------- ranks
def rank_info() -> Dict[str, int]:
    return {"rank": int(os.environ.get("RANK", "0")), "local_rank": int(os.environ.get("LOCAL_RANK", "0")),
            "world_size": int(os.environ.get("WORLD_SIZE", "1"))}


def init_process_group(backend: str):
    """Joins the job torchrun started (MASTER_ADDR / MASTER_PORT / RANK / WORLD_SIZE from the env)."""
    import torch.distributed as dist

    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    os.environ.setdefault("MASTER_PORT", "29511")
    if not dist.is_initialized():
        dist.init_process_group(backend=backend, rank=rank_info()["rank"], world_size=rank_info()["world_size"])
    return dist


def aggregate(ms_local: float, units_local: float, device=None) -> Dict[str, float]:
    """Whole-job figures from per-rank ones: the slowest rank's time, the sum of the work.

    The ranks share no data (each updates its own parameter arena), so the only traffic between
    them is this reduction of two scalars after the timed region.
    """
    import torch
    import torch.distributed as dist

    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return {"ms": ms_local, "units": units_local, "world_size": 1}
    t = torch.tensor([ms_local], dtype=torch.float64, device=device)
    u = torch.tensor([units_local], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return {"ms": float(t.item()), "units": float(u.item()), "world_size": dist.get_world_size()}


def barrier(device=None) -> None:
    import torch.distributed as dist

    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        if device is not None and str(device).startswith("cuda"):
            dist.barrier(device_ids=[int(str(device).split(":")[1])] if ":" in str(device) else None)
        else:
            dist.barrier()


def host_info() -> Dict:
    model = "unknown"
    try:
        with open("/proc/cpuinfo") as fh:
            for line in fh:
                if line.lower().startswith("model name"):
                    model = line.split(":", 1)[1].strip()
                    break
    except OSError:
        pass
    return {"nproc": os.cpu_count(), "cpu": model}
