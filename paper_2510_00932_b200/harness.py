"""Host-side logic of the benchmark: byte accounting, rank aggregation, clock sampling, peaks.

Nothing here computes any of the five operations; it only counts bytes, times and ranks, so it
runs (and is tested) without a GPU.
"""
from __future__ import annotations

import json
import os
import statistics
import subprocess
import threading

from .streamops import ARRAYS_MOVED, OPS

NOMINAL_HBM_GBS = 8000.0           # the HBM3e figure the target is quoted against
FALLBACK_HBM_GBS = 6650.0          # earlier copy measurement on the same GPU pool
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def op_bytes(op: str, n: int, itemsize: int) -> int:
    """Algorithmic bytes of one launch, counted the standard STREAM way: two arrays for
    copy/scale/dot, three for add/triad; no write-allocate traffic is counted."""
    return ARRAYS_MOVED[op] * n * itemsize


def step_bytes(n: int, itemsize: int) -> int:
    """Algorithmic bytes of one pass of all five operations."""
    return sum(op_bytes(op, n, itemsize) for op in OPS)


def measured_peak():
    """(GB/s, source) of the HBM roofline denominator: the measured copy bandwidth if the
    per-pod measurement file is present, else the documented fallback."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except (OSError, KeyError, ValueError):
        return FALLBACK_HBM_GBS, "fallback"


def dist_env():
    """(rank, local_rank, world_size) from the torchrun environment; (0, 0, 1) when absent."""
    return (int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)),
            int(os.environ.get("WORLD_SIZE", 1)))


def max_over_ranks(value: float, device=None) -> float:
    """MAX of a per-rank scalar over the default process group (identity without one)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device or "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, device=None) -> float:
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device or "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def whole_job_gbs(bytes_this_rank: float, elapsed_ms_this_rank: float, device=None) -> tuple[float, float]:
    """Whole-job throughput of a weak-scaling run: the bytes ALL ranks moved divided by the
    slowest rank's time. Returns (GB/s, max elapsed ms)."""
    total_bytes = sum_over_ranks(bytes_this_rank, device)
    max_ms = max_over_ranks(elapsed_ms_this_rank, device)
    return total_bytes / (max_ms * 1e-3) / 1e9, max_ms


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while a timed region runs."""

    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int = 0, period_ms: int = 100):
        self.gpu_index, self.period_ms = gpu_index, period_ms
        self.lines: list[str] = []
        self.proc = None
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.gpu_index}", f"--query-gpu={self.QUERY}",
                 "--format=csv,noheader,nounits", "-lms", str(self.period_ms)],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return self

        def pump():
            for line in self.proc.stdout:
                self.lines.append(line.strip())
        self.thread = threading.Thread(target=pump, daemon=True)
        self.thread.start()
        return self

    def mark(self) -> int:
        return len(self.lines)

    def stop(self):
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()
            if self.thread is not None:
                self.thread.join(timeout=2)

    def summary(self, first: int = 0, last: int | None = None) -> dict:
        return summarize_clock_lines(self.lines[first:last])


def summarize_clock_lines(lines) -> dict:
    """Median SM clock under load and the set of throttle reasons seen in nvidia-smi CSV rows."""
    sm, smax, reasons = [], [], set()
    names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
    for line in lines:
        f = [x.strip() for x in line.split(",")]
        if len(f) < 9:
            continue
        try:
            sm.append(float(f[1])); smax.append(float(f[2]))
        except ValueError:
            continue
        for name, val in zip(names, f[5:9]):
            if val.lower().startswith("active"):
                reasons.add(name)
    if not sm:
        return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
    return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(smax), "reasons": sorted(reasons),
            "samples": len(sm)}


def pin_bandwidth_gbs(memory_clock_khz: float, bus_width_bits: int) -> float:
    """What the memory pins of the device can carry: double data rate x bus width, from the two
    attributes the device reports (a B200 with 7680 of 8192 bits enabled at 3996 MHz: 7672 GB/s)."""
    return 2.0 * memory_clock_khz * 1e3 * bus_width_bits / 8 / 1e9


def per_op_report(durations_ms: dict, n: int, itemsize: int, peak_gbs: float, pin_gbs: float | None = None) -> dict:
    """GB/s per operation from average launch durations, with the roofline fractions: of the measured
    copy rate, of the nominal 8 TB/s, and (when given) of the device's own pin bandwidth."""
    out = {}
    for op, ms in durations_ms.items():
        gbs = op_bytes(op, n, itemsize) / (ms * 1e-3) / 1e9
        out[op] = {"ms": round(ms, 5), "gbs": round(gbs, 1), "frac_measured_peak": round(gbs / peak_gbs, 4),
                   "frac_nominal_8tbs": round(gbs / NOMINAL_HBM_GBS, 4)}
        if pin_gbs:
            out[op]["frac_pin_bandwidth"] = round(gbs / pin_gbs, 4)
    return out


def launch_ranks(script: str, argv: list, nproc: int, extra_env: dict | None = None) -> int:
    """Starts `nproc` ranks of `script argv...` on this node with torch.distributed.run (one process
    per GPU, rendezvous on 127.0.0.1 at a free port) and returns the launcher's exit code. NCCL's
    initialisation log is switched on (to stderr) unless the caller configured NCCL_DEBUG, so that
    the communicator's size can be read off a run's output."""
    import socket
    import sys
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    env = dict(os.environ)
    if "NCCL_DEBUG" not in env:
        env.update(NCCL_DEBUG="INFO", NCCL_DEBUG_SUBSYS="INIT", NCCL_DEBUG_FILE="/dev/stderr")
    env.update(extra_env or {})
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={int(nproc)}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), script, *argv]
    return subprocess.call(cmd, env=env)


def traffic_file(workload: str) -> str:
    return os.path.join(ROOT, "profiles", f"ncu_dram_traffic_opmajor_{workload}.txt")


def read_traffic_file(path: str):
    """The JSON object stored after the '#' comment lines of a traffic summary, or None."""
    try:
        with open(path) as f:
            body = "".join(line for line in f if not line.lstrip().startswith("#"))
        return json.loads(body)
    except (OSError, ValueError):
        return None


def captured_traffic(workload: str, op: str, tuning: dict):
    """DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) of `op` from the stored
    ncu capture of this workload, or None when there is no capture or when it was taken under a
    tuning other than the one in force (the kernel has changed since)."""
    data = read_traffic_file(traffic_file(workload))
    if not data:
        return None
    entry = data.get("kernels", {}).get(op)
    if not entry or entry.get("tuning") != tuning:
        return None
    return int(entry["dram_read_bytes"] + entry["dram_write_bytes"])
