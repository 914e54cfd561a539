"""Host-side helpers of bench.py: rank bookkeeping, the cross-rank reduction of the timing, the
clock sampler and the bounded CPU sample.  No operator arithmetic lives here."""
from __future__ import annotations

import json
import os
import statistics
import subprocess
import tempfile
import time
from typing import Optional

import numpy as np


def rank_info():
    """(rank, local_rank, world_size) from the torchrun environment (1 process: 0, 0, 1)."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def rank_seed(base_seed: int, rank: int) -> int:
    """Every rank owns its own tables and batch (independent units, no exchange step)."""
    return base_seed + rank


def init_process_group(backend: str):
    import torch.distributed as dist
    if int(os.environ.get("WORLD_SIZE", "1")) > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group(backend=backend)
    return dist


def reduce_job(units_local: float, elapsed_ms_local: float, device=None):
    """Whole-job figures: units summed over ranks, time = the slowest rank's.
    Returns (total_units, max_elapsed_ms).  Works without a process group (one rank)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(units_local), float(elapsed_ms_local)
    u = torch.tensor([float(units_local)], dtype=torch.float64, device=device)
    t = torch.tensor([float(elapsed_ms_local)], dtype=torch.float64, device=device)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(u.item()), float(t.item())


def barrier():
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.barrier()


class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU with nvidia-smi while a region runs."""
    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_id, period_ms: int = 100):
        """gpu_id: anything `nvidia-smi -i` accepts (index or GPU-<uuid>)."""
        self.gpu_index = gpu_id
        self.period_ms = period_ms
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.gpu_index), f"--query-gpu={self.QUERY}",
                 "--format=csv,noheader,nounits", "-lms", str(self.period_ms)],
                stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None
        return self

    def stop(self) -> Optional[dict]:
        if self.proc is None:
            return None
        time.sleep(self.period_ms / 1000.0 * 1.5)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        try:
            lines = [l.strip() for l in open(self.path) if l.strip()]
            os.unlink(self.path)
        except OSError:
            return None
        return parse_clock_samples(lines)


def parse_clock_samples(lines):
    sm, mx, reasons = [], [], set()
    names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
    for l in lines:
        f = [x.strip() for x in l.split(",")]
        if len(f) < 7:
            continue
        try:
            sm.append(float(f[0]))
            mx.append(float(f[1]))
        except ValueError:
            continue
        for name, v in zip(names, f[3:7]):
            if v.lower().startswith("active"):
                reasons.add(name)
    if not sm:
        return None
    return {"sm_mhz": statistics.median(sm), "sm_mhz_min": min(sm), "sm_max_mhz": max(mx),
            "samples": len(sm), "reasons": sorted(reasons)}


def measured_peaks(root: str) -> dict:
    """HBM copy bandwidth measured on this machine (GB/s), else the documented fallback."""
    path = os.path.join(root, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            d = json.load(f)
        return {"hbm_gbs": float(d["hbm_gbs"]), "source": "measured"}
    except (OSError, KeyError, ValueError):
        return {"hbm_gbs": 6650.0, "source": "fallback"}


def cpu_sample(w, jag, max_lookups: int):
    """The bounded sample the CPU oracle is timed on: the leading tables of the workload with all
    their bags, as many as hold ``max_lookups`` lookups; if table 0 alone holds more, its leading
    bags only.  Returns (n_tables, indices, offsets, weights, B_sample, n_lookups)."""
    per_table = [int(jag.offsets[(t + 1) * w.B]) for t in range(w.T)]     # cumulative lookups
    k = int(np.searchsorted(per_table, max_lookups, side="right"))
    if k >= 1:
        k = min(k, w.T)
        n = per_table[k - 1]
        weights = None if jag.weights is None else jag.weights[:n]
        return k, jag.indices[:n], jag.offsets[:k * w.B + 1], weights, w.B, n
    off = jag.offsets[:w.B + 1]
    nb = int(np.searchsorted(off, max_lookups, side="right")) - 1
    nb = max(1, min(nb, w.B))
    n = int(off[nb])
    weights = None if jag.weights is None else jag.weights[:n]
    return 1, jag.indices[:n], off[:nb + 1].copy(), weights, nb, n
