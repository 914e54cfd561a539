"""Host logic of the benchmark, including the N > 1 reduction on a 2-rank gloo group (CPU)."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2512_23236_b200 import benchlib as bl
from paper_2512_23236_b200 import workloads as wl


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, q):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    assert bl.rank_info() == (rank, rank, world)
    bl.init_process_group("gloo")
    # every rank draws its own batch: independent units, no exchange
    w = wl.make_workload(1, seed=bl.rank_seed(0, rank))
    n = int(wl.gen_jagged(w).lengths.sum())
    bl.barrier()
    total, slowest = bl.reduce_job(n * 3, 10.0 * (rank + 1))
    q.put((rank, n, total, slowest))
    dist.destroy_process_group()


def test_two_rank_reduction_sums_units_and_takes_slowest_time():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (_, n0, tot0, slow0), (_, n1, tot1, slow1) = res
    assert n0 != n1                              # different seeds, different batches
    assert tot0 == tot1 == 3 * (n0 + n1)
    assert slow0 == slow1 == 20.0


def test_single_rank_reduction_is_identity():
    assert bl.reduce_job(7, 3.5) == (7.0, 3.5)
    assert bl.rank_seed(0, 3) == 3


def test_clock_sample_parsing():
    lines = ["1965, 1965, 400.1, Not Active, Not Active, Not Active, Not Active",
             "1350, 1965, 990.0, Not Active, Not Active, Not Active, Active",
             "1410, 1965, 980.0, Not Active, Not Active, Not Active, Active",
             "garbage"]
    c = bl.parse_clock_samples(lines)
    assert c["sm_mhz"] == 1410 and c["sm_max_mhz"] == 1965 and c["reasons"] == ["sw_power_cap"]
    assert bl.parse_clock_samples([]) is None


def test_cpu_sample_is_a_prefix_of_the_workload():
    w = wl.make_workload(4, scale_rows=0.001, scale_B=1 / 32, max_tables=3)
    jag = wl.gen_jagged(w)
    # smaller than table 0: leading bags of table 0
    k, idx, off, wts, nb, n = bl.cpu_sample(w, jag, 5000)
    assert k == 1 and 1 <= nb < w.B and off[0] == 0 and off[-1] == n <= 5000
    assert np.array_equal(idx, jag.indices[:n]) and np.array_equal(wts, jag.weights[:n])
    assert np.array_equal(off, jag.offsets[:nb + 1])
    # room for two whole tables
    two = int(jag.offsets[2 * w.B])
    k, idx, off, wts, nb, n = bl.cpu_sample(w, jag, two + 10)
    assert (k, nb, n) == (2, w.B, two) and off.shape[0] == 2 * w.B + 1
    # more than everything: the whole workload
    k, idx, off, wts, nb, n = bl.cpu_sample(w, jag, 10 ** 12)
    assert (k, n) == (3, jag.indices.shape[0])


def test_measured_peaks_fallback(tmp_path):
    assert bl.measured_peaks(str(tmp_path)) == {"hbm_gbs": 6650.0, "source": "fallback"}
    (tmp_path / "MEASURED_PEAKS.json").write_text('{"hbm_gbs": 6459.0}')
    assert bl.measured_peaks(str(tmp_path)) == {"hbm_gbs": 6459.0, "source": "measured"}
