#!/usr/bin/env python
"""Benchmark of the pooled embedding-bag forward on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload 1..10] [--impl reference]

One step = one pass of the whole hot path (one ebag_forward launch over all tables of the
workload).  Default workload: 3, the batched 32-table bf16 TBE (the largest batched-table
configuration the metric is quoted on).  Prints ONE JSON line:

  value     pooled lookups/s, whole job, inputs resident in HBM, CUDA-event time of K steps
  e2e       the same through ebag_forward_host: pinned host ids/offsets/weights in, pinned host
            output back, copies inside the timed region
  roofline  the forward kernel against the measured HBM copy bandwidth (algorithmic bytes)
  cpu_baseline  the CPU oracle, as it stands, on a bounded sample of the same workload

With N > 1 (launched by torchrun) every rank owns its own tables and batch (independent units,
no exchange step): weak scaling, value = lookups of all ranks / slowest rank's time.

--impl reference times the CPU oracle on the machine's host cores (rank 0 only); each step is the
bounded sample.
"""
import argparse
import json
import os
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402
import torch  # noqa: E402

from paper_2512_23236_b200 import benchlib as bl  # noqa: E402
from paper_2512_23236_b200 import workloads as wl  # noqa: E402

METRIC = "pooled_lookups_per_sec"
UNIT = "lookups/s"
L2_FLUSH_BYTES = 256 << 20

# DRAM bytes per forward launch (dram__bytes_read.sum + dram__bytes_write.sum) from the ncu
# captures summarised under profiles/.  The full-size workloads are too large to capture with
# more than one pass, so each figure is a smaller case of the same kernel scaled to a full launch
# by lookups (DRAM traffic here is compulsory misses + ids + output, all proportional to
# tables x bags); every entry says which capture it came from, and the line carries that along.
NCU_TRAFFIC = {
    3: {"small_case_bytes": 991.3e6, "small_case_lookups": 18.83e6, "small_case": "--max-tables 6",
        "summary": "profiles/ebag_fwd_bf16_cfg3.md", "captured_at_commit": "72112d9"},
    4: {"small_case_bytes": 1.7087e9, "small_case_lookups": 1.637e6, "small_case": "--max-tables 1",
        "summary": "profiles/ebag_fwd_f32_cfg4.md", "captured_at_commit": "72112d9"},
    5: {"small_case_bytes": 1.3074e9, "small_case_lookups": 20.97e6, "small_case": "--max-tables 8",
        "summary": "profiles/ebag_fwd_int8_cfg5.md", "captured_at_commit": "72112d9"},
}
# What the ncu counters of those captures show to be the limit of each workload's launch.
BOUND = {1: "launch-latency", 2: "latency", 3: "l1+issue", 4: "hbm", 5: "l1+issue"}
HBM_CASE_WORKLOAD = 4          # uniform ids over 41 GB of tables: DRAM bytes = algorithmic bytes


def ncu_traffic(number, lookups):
    """(bytes per full launch, provenance) or (None, None)."""
    c = NCU_TRAFFIC.get(number)
    if c is None:
        return None, None
    scale = lookups / c["small_case_lookups"]
    src = dict(c, scale_by_lookups=scale,
               note="extrapolated from a small-case ncu capture, not measured on the timed launch")
    return c["small_case_bytes"] * scale, src


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--e2e-steps", type=int, default=0, help="0: min(steps, 10)")
    ap.add_argument("--cpu-seconds", type=float, default=15.0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-hbm-case", action="store_true",
                    help="skip the extra leg that times the HBM-bound workload beside workload 3")
    ap.add_argument("--item-bytes", type=int, default=0)
    ap.add_argument("--split-bytes", type=int, default=-1,
                    help="bags gathering this many bytes or more are pooled in parts (0: never)")
    ap.add_argument("--ctas-per-sm", type=int, default=0)
    ap.add_argument("--bwd-sorted", type=int, default=-1,
                    help="workload 9: 1/0 = the reproducible (sorted) / the reduction backward; -1: the library's default")
    ap.add_argument("--bwd-base", type=int, default=3, choices=[3, 4, 5],
                    help="workload 9: whose jagged ids (and weights) and table shapes the backward runs on")
    ap.add_argument("--gw-base", type=int, default=3, choices=[3, 4, 5],
                    help="workload 10: whose tables and ids the weights' gradient runs on")
    # shrunk variants of a workload, for profiler captures and quick checks (not bench lines)
    ap.add_argument("--row-d", type=int, default=0, help="every table with rows of this many elements instead")
    ap.add_argument("--max-tables", type=int, default=0)
    ap.add_argument("--scale-rows", type=float, default=1.0)
    ap.add_argument("--scale-b", type=float, default=1.0)
    return ap.parse_args()


MAPID_WORKLOAD = 6     # workload 3 with 1/100 of the rows and RAW ids, MapId fused into the forward


def make_workload(args, seed):
    if args.workload == MAPID_WORKLOAD:
        w = wl.make_workload(3, scale_rows=0.01 * args.scale_rows, scale_B=args.scale_b,
                             max_tables=args.max_tables or None, seed=seed)
        w.name = "cfg3_rows_div100_raw_ids_mapid"
        return w
    w = wl.make_workload(args.workload, scale_rows=args.scale_rows, scale_B=args.scale_b,
                         max_tables=args.max_tables or None, seed=seed)
    if args.row_d:          # the same jagged structure over rows of another width (a probe, not a bench line)
        w.D = [args.row_d] * w.T
        w.name += f"_D{args.row_d}"
    return w


def workload_config(w, ab, args=None):
    shrunk = args is not None and (args.max_tables or args.scale_rows != 1.0 or args.scale_b != 1.0 or args.row_d)
    extra = {}
    if args is not None and args.workload == MAPID_WORKLOAD:
        extra = {"mapid": "per table a sorted list of rows-1 known raw ids (1 k - 100 k; the paper's "
                          "MapId sizes are 100 - 10 000); ids arrive raw and are searched in the kernel"}
    return {"workload": w.name + ("_SHRUNK" if shrunk else ""), "tables": w.T, "bags_per_table": w.B, "sum_D": w.sumD,
            "table_dtype": wl.DTYPE_NAMES[w.dtype],
            "pooling": "mean" if w.mode == wl.MEAN else ("weighted_sum" if w.weighted else "sum"),
            "lookups_per_step": ab["lookups"], "algorithmic_bytes_per_step": ab["total"],
            "index_dtype": "int64", "seed": w.seed,
            "l2": f"{L2_FLUSH_BYTES >> 20} MiB written between timed steps (L2 flush)", **extra}


def oracle_inputs(w, jag, host_table, max_lookups, mapid=None):
    """Host arrays of the bounded CPU sample.  host_table(t) returns table t as host tensors.
    mapid = (raw values, mappings) makes it a sample of the fused MapId workload."""
    k, idx, off, wts, nb, n = bl.cpu_sample(w, jag, max_lookups)
    tabs, sc, bi = [], [], []
    for t in range(k):
        tab = host_table(t)
        if w.dtype == wl.INT8_ROWWISE:
            tabs.append(wl.raw_numpy(tab[0]))
            sc.append(wl.raw_numpy(tab[1]))
            bi.append(wl.raw_numpy(tab[2]))
        else:
            tabs.append(wl.raw_numpy(tab))
    inp = dict(tables=tabs, scales=sc or None, biases=bi or None, indices=idx, offsets=off,
               weights=wts, B=nb, lookups=n, n_tables=k, rows=w.rows[:k], D=w.D[:k])
    if mapid is not None:
        inp["values"] = mapid[0][:n]
        inp["mappings"] = mapid[1][:k]
    return inp


def time_oracle(w, inp):
    from oracle import ebag_oracle as orc
    t0 = time.perf_counter()
    if "mappings" in inp:
        from oracle import mapid_oracle as mo
        mo.forward_mapid(inp["tables"], w.dtype, inp["values"], inp["offsets"], inp["B"],
                         inp["mappings"], w.mode, weights=inp["weights"], scales=inp["scales"],
                         biases=inp["biases"])
    else:
        orc.forward(inp["tables"], w.dtype, inp["indices"], inp["offsets"], inp["B"], w.mode,
                    weights=inp["weights"], scales=inp["scales"], biases=inp["biases"], want64=True)
    return time.perf_counter() - t0


def sized_cpu_sample(w, jag, host_table, seconds, mapid=None):
    """Pick the sample size from a short probe so that one oracle pass takes about `seconds`
    (the whole workload if that is less work)."""
    from oracle import ebag_oracle as orc
    probe = oracle_inputs(w, jag, host_table, 200_000, mapid)
    t = max(time_oracle(w, probe), 1e-4)
    rate = probe["lookups"] / t
    inp = oracle_inputs(w, jag, host_table, int(rate * seconds), mapid)
    whole = inp["lookups"] == int(jag.indices.shape[0])
    desc = (("the whole workload: " if whole else "") +
            f"the first {inp['n_tables']} of {w.T} tables, {inp['B']} bags each, "
            f"{inp['lookups']} of {int(jag.indices.shape[0])} lookups, "
            f"all {orc.max_threads()} host threads")
    return inp, desc, orc.max_threads()


def run_reference(args, rank):
    """The CPU oracle as the reference arm (rank 0 only)."""
    if rank != 0:
        return
    w = make_workload(args, 0)
    jag = wl.gen_jagged(w)
    ab = wl.algorithmic_bytes(w, jag.lengths)
    cache = {}

    def host_table(t):
        if t not in cache:
            cache[t] = wl.gen_table(w, t, "cpu")
        return cache[t]

    # a step must stay short enough for warmup + steps to end within a few minutes
    per_step = max(0.5, min(args.cpu_seconds, 120.0 / max(1, args.steps + args.warmup)))
    mapid = None
    if args.workload == MAPID_WORKLOAD:
        maps = wl.gen_mappings(w)
        mapid = (wl.raw_values(w, jag, maps), maps)
    inp, desc, cores = sized_cpu_sample(w, jag, host_table, per_step, mapid)
    for _ in range(args.warmup):
        time_oracle(w, inp)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        time_oracle(w, inp)
    dt = time.perf_counter() - t0
    value = inp["lookups"] * args.steps / dt
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic", "config": workload_config(w, ab, args),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                             "sample": desc},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


MBDT_WORKLOAD = 7      # MergeBucketizedDense transform (paper Sec. 5.4.2)


def run_mbdt(args, rank, local_rank, world):
    """Workload 7: MBDT on F=64 features x B=1,048,576 values with 10 borders each (the paper
    measures Batch x Features x Borders up to 2048 x 2 x 4, which is launch-bound here and is
    reported beside it).  12 algorithmic bytes per value (fp32 in, int64 out)."""
    from oracle import mbdt_oracle as mb
    F, B, K = 64, 1 << 20, 10
    rng = np.random.default_rng(bl.rank_seed(0, rank))
    borders = [np.sort(rng.standard_normal(K)).astype(np.float32) for _ in range(F)]
    values = rng.standard_normal((F, B)).astype(np.float32)
    flat, boff = mb.flatten_borders(borders)
    ooff = mb.bin_offsets(borders)
    config = {"workload": "mbdt_F64_B1048576_K10", "features": F, "batch": B, "borders": K,
              "algorithmic_bytes_per_step": 12 * F * B, "data": "N(0,1) values and borders, seed 0",
              "l2": f"{L2_FLUSH_BYTES >> 20} MiB written between timed steps (L2 flush)"}
    if args.impl == "reference":
        if rank != 0:
            return
        sample = values[:, :B // 8]
        for _ in range(args.warmup):
            mb.mbdt_fast(sample, borders, ooff)
        t0 = time.perf_counter()
        for _ in range(args.steps):
            mb.mbdt_fast(sample, borders, ooff)
        dt = time.perf_counter() - t0
        v = sample.size * args.steps / dt
        print(json.dumps({"impl": "reference", "metric": "bucketized_values_per_sec", "value": v,
                          "unit": "values/s", "n_gpus": args.gpus, "steps": args.steps,
                          "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
                          "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
                          "dtype": "f32", "data": "synthetic", "config": config,
                          "cpu_baseline": {"value": v, "unit": "values/s", "cores": 1, "kind": "oracle",
                                           "sample": "the first eighth of every feature's values"},
                          "e2e": {"value": v, "unit": "values/s", "h2d_bytes_per_step": 0,
                                  "d2h_bytes_per_step": 0}, "gpu_launches": 0}), flush=True)
        return
    import paper_2512_23236_b200 as eb
    eb.lib()
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    bl.init_process_group("nccl")
    warmup = max(3, args.warmup)
    h_val = torch.from_numpy(values).pin_memory()
    d_val = h_val.to(dev)
    d_flat, d_boff, d_ooff = (torch.from_numpy(x).to(dev) for x in (flat, boff, ooff))
    d_out = torch.empty((F, B), dtype=torch.int64, device=dev)
    h_out = torch.empty((F, B), dtype=torch.int64).pin_memory()
    d_stage = torch.empty_like(d_val)
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=dev)
    stream = torch.cuda.Stream(device=dev)
    sampler = bl.ClockSampler(f"GPU-{torch.cuda.get_device_properties(dev).uuid}").start()
    with torch.cuda.stream(stream):
        for _ in range(warmup):
            flush.fill_(1)
            eb.ebag_mbdt(d_val, d_flat, d_boff, d_ooff, out=d_out, stream=stream)
        bl.barrier()
        torch.cuda.synchronize()
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
              for _ in range(args.steps)]
        for a, b in ev:
            flush.fill_(1)
            a.record(stream)
            eb.ebag_mbdt(d_val, d_flat, d_boff, d_ooff, out=d_out, stream=stream)
            b.record(stream)
        torch.cuda.synchronize()
        bl.barrier()
        step_ms = [a.elapsed_time(b) for a, b in ev]
        elapsed_ms = float(sum(step_ms))
        e2e_steps = args.e2e_steps or min(args.steps, 10)
        ev2 = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
               for _ in range(e2e_steps)]
        for a, b in ev2:                      # host values in, host ids out, copies timed
            a.record(stream)
            d_stage.copy_(h_val, non_blocking=True)
            eb.ebag_mbdt(d_stage, d_flat, d_boff, d_ooff, out=d_out, stream=stream)
            h_out.copy_(d_out, non_blocking=True)
            b.record(stream)
        torch.cuda.synchronize()
        bl.barrier()
        e2e_ms = float(sum(a.elapsed_time(b) for a, b in ev2))
        # the paper's largest measured shape, Batch x Features x Borders = 2048 x 2 x 4
        pb = [np.sort(rng.standard_normal(4)).astype(np.float32) for _ in range(2)]
        pflat, pboff = mb.flatten_borders(pb)
        pv = torch.randn(2, 2048, device=dev)
        pargs = (pv, torch.from_numpy(pflat).to(dev), torch.from_numpy(pboff).to(dev),
                 torch.from_numpy(mb.bin_offsets(pb)).to(dev))
        pout = torch.empty((2, 2048), dtype=torch.int64, device=dev)
        eb.ebag_mbdt(*pargs, out=pout, stream=stream)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for _ in range(100):
            eb.ebag_mbdt(*pargs, out=pout, stream=stream)
        b.record(stream)
        torch.cuda.synchronize()
        paper_shape_us = a.elapsed_time(b) * 10.0
    clocks = sampler.stop()
    assert torch.equal(h_out, d_out.cpu())
    total, max_ms = bl.reduce_job(F * B * args.steps, elapsed_ms, dev)
    e2e_total, e2e_max = bl.reduce_job(F * B * e2e_steps, e2e_ms, dev)
    if rank != 0:
        return
    peaks = bl.measured_peaks(ROOT)
    ms = elapsed_ms / args.steps
    achieved = 12.0 * F * B / (ms * 1e-3) / 1e9
    t0 = time.perf_counter()
    ref = mb.mbdt_fast(values[:, :B // 8], borders, ooff)
    dt = time.perf_counter() - t0
    assert np.array_equal(ref, h_out.numpy()[:, :B // 8])
    line = {"metric": "bucketized_values_per_sec", "value": total / (max_ms * 1e-3), "unit": "values/s",
            "n_gpus": world, "steps": args.steps, "warmup": warmup, "ms_per_step": max_ms / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
            "data": "synthetic", "config": config, "clocks": clocks, "gpu_launches": args.steps,
            "e2e": {"value": e2e_total / (e2e_max * 1e-3), "unit": "values/s",
                    "h2d_bytes_per_step": 4 * F * B, "d2h_bytes_per_step": 8 * F * B,
                    "steps": e2e_steps, "ms_per_step": e2e_max / e2e_steps},
            "roofline": {"bound": "hbm", "kernel": "mbdt_kernel", "achieved": achieved,
                         "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": achieved / peaks["hbm_gbs"],
                         "peak_source": f"{peaks['source']} HBM copy bandwidth (burst)",
                         "algorithmic_bytes_per_launch": 12 * F * B, "ms_per_launch": ms,
                         "ms_per_launch_min": min(step_ms), "traffic": None},
            "cpu_baseline": {"value": ref.size / dt, "unit": "values/s", "cores": 1, "kind": "oracle",
                             "sample": "the first eighth of every feature's values (numpy searchsorted "
                                       "per feature, one thread)", "seconds": dt},
            "paper_shape": {"batch_x_features_x_borders": "2048 x 2 x 4", "us_per_call": paper_shape_us,
                            "paper_ms": "0.027-0.064 (MTIA v2i), 0.029-0.045 (MTIA v3), other hardware"}}
    print(json.dumps(line), flush=True)


BET_WORKLOAD = 8       # Batch Event Truncate (paper Sec. 5.5)


def run_bet(args, rank, local_rank, world):
    """Workload 8: Batch Event Truncate on 32,768 users x 100-200 events x 9 features (the paper's
    production shape is 9 features, 200 events, length limit 100/200; it does not print its batch
    size), 0-4 attributes per event, truncated to N = 100 events."""
    from oracle import bet_oracle as bo
    U, F, N = 32768, 9, 100
    rng = np.random.default_rng(bl.rank_seed(0, rank))
    outer = rng.integers(100, 201, size=U).astype(np.int64)
    E = int(outer.sum())
    inner = rng.integers(0, 5, size=(F, E)).astype(np.int64)
    vlen = inner.sum(axis=1)
    voff = np.zeros(F + 1, np.int64)
    np.cumsum(vlen, out=voff[1:])
    values = rng.integers(0, 1 << 40, size=int(voff[-1])).astype(np.int64)
    keep_ev = np.concatenate([np.arange(n) for n in outer]) < N
    kept_events = int(keep_ev.sum())
    kept_values = int(sum(inner[f][keep_ev].sum() for f in range(F)))
    # the method must read every inner length once, read and write the kept values and write the
    # kept inner lengths; outer lengths in and out
    alg = 8 * (F * E + 2 * kept_values + F * kept_events + 2 * U)
    config = {"workload": "bet_U32768_F9_events100-200_N100", "users": U, "features": F,
              "events": E, "values": int(voff[-1]), "truncate_to": N,
              "algorithmic_bytes_per_step": alg, "data": "synthetic, seed 0",
              "l2": f"{L2_FLUSH_BYTES >> 20} MiB written between timed steps (L2 flush)"}
    su = 256                                              # users in the CPU sample
    se = int(outer[:su].sum())

    def cpu_once():
        io = np.zeros(F + 1, np.int64)
        feats_i, feats_v = [], []
        for f in range(F):
            n = int(inner[f, :se].sum())
            feats_i.append(inner[f, :se])
            feats_v.append(values[voff[f]:voff[f] + n])
        t0 = time.perf_counter()
        bo.truncate(outer[:su], feats_i, feats_v, N)
        return time.perf_counter() - t0

    if args.impl == "reference":
        if rank != 0:
            return
        for _ in range(args.warmup):
            cpu_once()
        dt = sum(cpu_once() for _ in range(args.steps))
        v = F * se * args.steps / dt
        print(json.dumps({"impl": "reference", "metric": "feature_events_per_sec", "value": v,
                          "unit": "events/s", "n_gpus": args.gpus, "steps": args.steps,
                          "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
                          "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
                          "dtype": "int64", "data": "synthetic", "config": config,
                          "cpu_baseline": {"value": v, "unit": "events/s", "cores": 1, "kind": "oracle",
                                           "sample": f"the first {su} users, all {F} features"},
                          "e2e": {"value": v, "unit": "events/s", "h2d_bytes_per_step": 0,
                                  "d2h_bytes_per_step": 0}, "gpu_launches": 0}), flush=True)
        return
    import paper_2512_23236_b200 as eb
    eb.lib()
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    bl.init_process_group("nccl")
    warmup = max(3, args.warmup)
    h = [torch.from_numpy(x).pin_memory() for x in (outer, inner, values, voff)]
    d_outer, d_inner, d_values, d_voff = (x.to(dev) for x in h)
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=dev)
    stream = torch.cuda.Stream(device=dev)
    sampler = bl.ClockSampler(f"GPU-{torch.cuda.get_device_properties(dev).uuid}").start()
    with torch.cuda.stream(stream):
        for _ in range(warmup):
            flush.fill_(1)
            res = eb.ebag_batch_event_truncate(d_outer, d_inner, d_values, d_voff, N, stream=stream)
        bl.barrier()
        torch.cuda.synchronize()
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
              for _ in range(args.steps)]
        for a, b in ev:
            flush.fill_(1)
            a.record(stream)
            res = eb.ebag_batch_event_truncate(d_outer, d_inner, d_values, d_voff, N, stream=stream)
            b.record(stream)
        torch.cuda.synchronize()
        bl.barrier()
        step_ms = [a.elapsed_time(b) for a, b in ev]
        elapsed_ms = float(sum(step_ms))
        e2e_steps = args.e2e_steps or min(args.steps, 10)
        s_in = [torch.empty_like(x) for x in (d_outer, d_inner, d_values)]
        h_out = [torch.empty_like(x).pin_memory() for x in (h[0], h[1], h[2])]
        h_cnt = torch.empty(1 + F, dtype=torch.int64).pin_memory()
        ev2 = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
               for _ in range(e2e_steps)]
        for a, b in ev2:                      # host batch in, host batch out, copies timed
            a.record(stream)
            for dst, src in zip(s_in, h[:3]):
                dst.copy_(src, non_blocking=True)
            r = eb.ebag_batch_event_truncate(s_in[0], s_in[1], s_in[2], d_voff, N, stream=stream)
            for dst, src in zip(h_out, r[:3]):
                dst.copy_(src, non_blocking=True)
            h_cnt.copy_(r[3], non_blocking=True)
            b.record(stream)
        torch.cuda.synchronize()
        bl.barrier()
        e2e_ms = float(sum(a.elapsed_time(b) for a, b in ev2))
    clocks = sampler.stop()
    counts = res[3].cpu().numpy()
    assert counts[0] == kept_events and int(counts[1:].sum()) == kept_values
    total, max_ms = bl.reduce_job(F * E * args.steps, elapsed_ms, dev)
    e2e_total, e2e_max = bl.reduce_job(F * E * e2e_steps, e2e_ms, dev)
    if rank != 0:
        return
    # parity on the CPU sample (the first `su` users are a prefix of every output)
    feats_i = [inner[f, :se] for f in range(F)]
    feats_v = [values[voff[f]:voff[f] + int(inner[f, :se].sum())] for f in range(F)]
    t0 = time.perf_counter()
    want = bo.truncate(outer[:su], feats_i, feats_v, N)
    dt = time.perf_counter() - t0
    io, vo = res[1].cpu().numpy(), res[2].cpu().numpy()
    for f in range(F):
        assert np.array_equal(io[f, :want[1][f].shape[0]], want[1][f])
        assert np.array_equal(vo[voff[f]:voff[f] + want[2][f].shape[0]], want[2][f])
    peaks = bl.measured_peaks(ROOT)
    ms = elapsed_ms / args.steps
    achieved = alg / (ms * 1e-3) / 1e9
    line = {"metric": "feature_events_per_sec", "value": total / (max_ms * 1e-3), "unit": "events/s",
            "n_gpus": world, "steps": args.steps, "warmup": warmup, "ms_per_step": max_ms / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int64",
            "data": "synthetic", "config": config, "clocks": clocks, "gpu_launches": 4 * args.steps,
            "e2e": {"value": e2e_total / (e2e_max * 1e-3), "unit": "events/s",
                    "h2d_bytes_per_step": 8 * (U + F * E + int(voff[-1])),
                    "d2h_bytes_per_step": 8 * (U + F * E + int(voff[-1]) + 1 + F),
                    "steps": e2e_steps, "ms_per_step": e2e_max / e2e_steps},
            "roofline": {"bound": "hbm", "kernel": "bet_copy (+ bet_user_sums, two scans)",
                         "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                         "frac": achieved / peaks["hbm_gbs"],
                         "peak_source": f"{peaks['source']} HBM copy bandwidth (burst)",
                         "algorithmic_bytes_per_launch": alg, "ms_per_launch": ms,
                         "ms_per_launch_min": min(step_ms), "traffic": None},
            "cpu_baseline": {"value": F * se / dt, "unit": "events/s", "cores": 1, "kind": "oracle",
                             "sample": f"the first {su} users, all {F} features (plain Python loops)",
                             "seconds": dt},
            "paper_context": "Table 'Batch Event Truncate performance': 9 features, 200 events: "
                             "1.443 -> 0.148 ms (platform unnamed, batch size not printed)"}
    print(json.dumps(line), flush=True)


BWD_WORKLOAD = 9       # backward (gradient with respect to the tables)


def run_bwd(args, rank, local_rank, world):
    """Workload 9: ebag_backward on workload 3's jagged structure (32 tables, Zipf ids, 87.7 M
    lookups): dense fp32 gradient tables (31.9 GB), grad_out [65536, 4352] fp32.  Algorithmic
    bytes: per lookup the reduction's payload (4 D) + id (8); per bag grad_out (4 D) + offset (8).
    The reductions are resolved in L2, so the HBM copy bandwidth is a reference, not the bound."""
    from oracle import ebag_bwd_oracle as bo
    base = wl.make_workload(args.bwd_base, scale_rows=args.scale_rows, scale_B=args.scale_b,
                            max_tables=args.max_tables or None, seed=bl.rank_seed(0, rank))
    jag = wl.gen_jagged(base)
    T, B = base.T, base.B
    lookups = int(jag.lengths.sum())
    per_table = np.add.reduceat(jag.lengths, np.arange(0, T * B, B))
    wbytes = 4 if jag.weights is not None else 0
    alg = int(sum(int(per_table[t]) * (4 * base.D[t] + 8 + wbytes) for t in range(T)) + B * (4 * base.sumD + 8 * T))
    config = {"workload": "bwd_" + base.name, "tables": T, "bags_per_table": B, "lookups": lookups,
              "sum_D": base.sumD, "gradient_tables": "dense fp32", "algorithmic_bytes_per_step": alg,
              "data": f"workload {args.bwd_base}'s seeded jagged ids (and weights); grad_out N(0,1)",
              "l2": f"{L2_FLUSH_BYTES >> 20} MiB written between timed steps (L2 flush)"}
    rng = np.random.default_rng(bl.rank_seed(0, rank) + 1)
    sb = min(B, 512)                                       # CPU sample: the first bags of table 0

    def cpu_sample():
        off = jag.offsets[:sb + 1]
        idx = jag.indices[:off[-1]]
        G = rng.standard_normal((sb, base.D[0]))
        t0 = time.perf_counter()
        bo.backward([base.rows[0]], [base.D[0]], G, idx, off, sb)
        return int(off[-1]), time.perf_counter() - t0

    if args.impl == "reference":
        if rank != 0:
            return
        for _ in range(args.warmup):
            cpu_sample()
        n = dt = 0
        for _ in range(args.steps):
            a, b = cpu_sample()
            n += a
            dt += b
        v = n / dt
        print(json.dumps({"impl": "reference", "metric": "pooled_lookups_per_sec", "value": v,
                          "unit": "lookups/s", "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
                          "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
                          "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": config,
                          "cpu_baseline": {"value": v, "unit": "lookups/s", "cores": 1, "kind": "oracle",
                                           "sample": f"the first {sb} bags of table 0 (Python loops over lookups)"},
                          "e2e": {"value": v, "unit": "lookups/s", "h2d_bytes_per_step": 0,
                                  "d2h_bytes_per_step": 0}, "gpu_launches": 0}), flush=True)
        return
    import paper_2512_23236_b200 as eb
    eb.lib()
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    bl.init_process_group("nccl")
    warmup = max(3, args.warmup)
    grads = [torch.zeros(r, d, device=dev) for r, d in zip(base.rows, base.D)]
    h_idx = torch.from_numpy(jag.indices).pin_memory()
    h_off = torch.from_numpy(jag.offsets).pin_memory()
    gen = torch.Generator(device=dev)
    gen.manual_seed(bl.rank_seed(0, rank) + 7)
    d_G = torch.randn((B, base.sumD), device=dev, generator=gen)
    h_G = d_G.cpu().pin_memory()
    d_idx, d_off = h_idx.to(dev), h_off.to(dev)
    h_w = None if jag.weights is None else torch.from_numpy(jag.weights).pin_memory()
    d_w = None if h_w is None else h_w.to(dev)
    s_w = None if h_w is None else torch.empty_like(d_w)
    s_idx, s_off, s_G = torch.empty_like(d_idx), torch.empty_like(d_off), torch.empty_like(d_G)
    h_status = torch.zeros(2, dtype=torch.int64).pin_memory()
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=dev)
    tbe = eb.TBE(base.rows, base.D, wl.F32, device=local_rank)
    if args.bwd_sorted >= 0:
        tbe.set_param("bwd_sorted", args.bwd_sorted)
    stream = torch.cuda.Stream(device=dev)
    sampler = bl.ClockSampler(f"GPU-{torch.cuda.get_device_properties(dev).uuid}").start()
    with torch.cuda.stream(stream):
        for _ in range(warmup):
            flush.fill_(1)
            tbe.backward(d_G, d_idx, d_off, B, grads, base.mode, d_w, stream=stream)
        stream.synchronize()
        assert tbe.last_status(stream) == (0, 0, 0)
        bl.barrier()
        torch.cuda.synchronize()
        launches0 = tbe.launch_count()
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
              for _ in range(args.steps)]
        for a, b in ev:
            flush.fill_(1)
            a.record(stream)
            tbe.backward(d_G, d_idx, d_off, B, grads, base.mode, d_w, stream=stream)
            b.record(stream)
        torch.cuda.synchronize()
        bl.barrier()
        launches = tbe.launch_count() - launches0
        step_ms = [a.elapsed_time(b) for a, b in ev]
        elapsed_ms = float(sum(step_ms))
        # end to end: host grad_out, ids and offsets in; the gradient tables stay on the device
        # (they are the optimizer's input), the status words come back
        e2e_steps = args.e2e_steps or min(args.steps, 10)
        ev2 = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
               for _ in range(e2e_steps)]
        for a, b in ev2:
            a.record(stream)
            s_idx.copy_(h_idx, non_blocking=True)
            s_off.copy_(h_off, non_blocking=True)
            s_G.copy_(h_G, non_blocking=True)
            if s_w is not None:
                s_w.copy_(h_w, non_blocking=True)
            tbe.backward(s_G, s_idx, s_off, B, grads, base.mode, s_w, stream=stream)
            h_status.copy_(grads[0][0, :2].to(torch.int64), non_blocking=True)
            b.record(stream)
        torch.cuda.synchronize()
        bl.barrier()
        e2e_ms = float(sum(a.elapsed_time(b) for a, b in ev2))
    clocks = sampler.stop()
    n_steps = warmup + args.steps + e2e_steps           # every step added into the same tables
    total, max_ms = bl.reduce_job(lookups * args.steps, elapsed_ms, dev)
    e2e_total, e2e_max = bl.reduce_job(lookups * e2e_steps, e2e_ms, dev)
    tbe.close()
    if rank != 0:
        return
    peaks = bl.measured_peaks(ROOT)
    ms = elapsed_ms / args.steps
    achieved = alg / (ms * 1e-3) / 1e9
    n_cpu, dt = cpu_sample()
    # the kernel that takes most of the call (profiles/ebag_bwd_cfg3.md)
    bwd_kernel = "ebag_bwd_kernel" if args.bwd_sorted == 0 else "bwds_run_sums_kernel"
    line = {"metric": "pooled_lookups_per_sec", "value": total / (max_ms * 1e-3), "unit": "lookups/s",
            "n_gpus": world, "steps": args.steps, "warmup": warmup, "ms_per_step": max_ms / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
            "data": "synthetic", "config": config, "clocks": clocks, "gpu_launches": launches,
            "e2e": {"value": e2e_total / (e2e_max * 1e-3), "unit": "lookups/s",
                    "h2d_bytes_per_step": int(h_idx.numel() * 8 + h_off.numel() * 8 + h_G.numel() * 4 +
                                              (0 if h_w is None else h_w.numel() * 4)),
                    "d2h_bytes_per_step": 16, "steps": e2e_steps, "ms_per_step": e2e_max / e2e_steps},
            "roofline": {"bound": "hbm", "kernel": bwd_kernel, "achieved": achieved,
                         "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": achieved / peaks["hbm_gbs"],
                         "peak_source": f"{peaks['source']} HBM copy bandwidth (burst); the reductions are "
                                        "resolved in L2, so this is a reference, not the binding limit",
                         "algorithmic_bytes_per_launch": alg, "ms_per_launch": ms,
                         "ms_per_launch_min": min(step_ms), "traffic": None},
            "cpu_baseline": {"value": n_cpu / dt, "unit": "lookups/s", "cores": 1, "kind": "oracle",
                             "sample": f"the first {sb} bags of table 0 (Python loops over lookups)",
                             "seconds": dt},
            "steps_accumulated": n_steps}
    print(json.dumps(line), flush=True)


GW_WORKLOAD = 10       # gradient with respect to the per-sample weights


def run_gw(args, rank, local_rank, world):
    """Workload 10: ebag_backward_weights on the tables and jagged ids of workload --gw-base (3, 4
    or 5): grad_w[i] = <grad_out[b, Doff[t]:+D], value(t, indices[i], :)>.  Algorithmic bytes: per
    lookup the row + id (8) + the gradient written (4); per bag its grad_out slice (4 D) + offset
    (8)."""
    from oracle import ebag_bwd_oracle as bo
    base = wl.make_workload(args.gw_base, scale_rows=args.scale_rows, scale_B=args.scale_b,
                            max_tables=args.max_tables or None, seed=bl.rank_seed(0, rank))
    jag = wl.gen_jagged(base)
    T, B = base.T, base.B
    lookups = int(jag.lengths.sum())
    per_table = np.add.reduceat(jag.lengths, np.arange(0, T * B, B))
    elem = {wl.F32: 4, wl.F16: 2, wl.BF16: 2, wl.INT8_ROWWISE: 1, wl.UINT8_ROWWISE: 1}[base.dtype]
    row_bytes = [d * elem + (8 if elem == 1 else 0) for d in base.D]
    alg = int(sum(int(per_table[t]) * (row_bytes[t] + 12) for t in range(T)) + B * (4 * base.sumD + 8 * T))
    config = {"workload": "gradw_" + base.name, "tables": T, "bags_per_table": B, "lookups": lookups,
              "sum_D": base.sumD, "algorithmic_bytes_per_step": alg,
              "data": f"workload {args.gw_base}'s seeded tables and jagged ids; grad_out N(0,1)",
              "l2": f"{L2_FLUSH_BYTES >> 20} MiB written between timed steps (L2 flush)"}
    rng = np.random.default_rng(bl.rank_seed(0, rank) + 1)
    sb = min(B, 256)                                       # CPU sample: the first bags of table 0
    rs = min(base.rows[0], 1 << 16)                        # the CPU sample's table: ids folded into its rows
    cpu_tab = rng.standard_normal((rs, base.D[0])).astype(np.float32)

    def cpu_sample():
        off = jag.offsets[:sb + 1]
        idx = jag.indices[:off[-1]] % rs
        G = rng.standard_normal((sb, base.D[0]))
        t0 = time.perf_counter()
        bo.backward_weights([cpu_tab], G, idx, off, sb)
        return int(off[-1]), time.perf_counter() - t0

    cpu_note = f"the first {sb} bags of table 0 over a {rs}-row table of N(0,1) values (Python loops over lookups)"
    if args.impl == "reference":
        if rank != 0:
            return
        for _ in range(args.warmup):
            cpu_sample()
        n = dt = 0
        for _ in range(args.steps):
            a, b = cpu_sample()
            n += a
            dt += b
        v = n / dt
        print(json.dumps({"impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": args.gpus,
                          "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
                          "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
                          "data": "synthetic", "config": config,
                          "cpu_baseline": {"value": v, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": cpu_note},
                          "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
                          "gpu_launches": 0}), flush=True)
        return
    import paper_2512_23236_b200 as eb
    eb.lib()
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    bl.init_process_group("nccl")
    warmup = max(3, args.warmup)
    raw_tables = [wl.gen_table(base, t, dev) for t in range(T)]
    tables = ([eb.ebag_pack_int8_rowwise(q, s, b) for q, s, b in raw_tables]
              if base.dtype == wl.INT8_ROWWISE else raw_tables)
    h_idx = torch.from_numpy(jag.indices).pin_memory()
    h_off = torch.from_numpy(jag.offsets).pin_memory()
    gen = torch.Generator(device=dev)
    gen.manual_seed(bl.rank_seed(0, rank) + 7)
    d_G = torch.randn((B, base.sumD), device=dev, generator=gen)
    h_G = d_G.cpu().pin_memory()
    d_idx, d_off = h_idx.to(dev), h_off.to(dev)
    s_idx, s_off, s_G = torch.empty_like(d_idx), torch.empty_like(d_off), torch.empty_like(d_G)
    d_gw = torch.zeros(lookups, device=dev)
    h_gw = torch.empty(lookups).pin_memory()
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=dev)
    tbe = eb.TBE(base.rows, base.D, base.dtype, device=local_rank)
    stream = torch.cuda.Stream(device=dev)
    sampler = bl.ClockSampler(f"GPU-{torch.cuda.get_device_properties(dev).uuid}").start()
    with torch.cuda.stream(stream):
        for _ in range(warmup):
            flush.fill_(1)
            tbe.backward_weights(tables, d_G, d_idx, d_off, B, base.mode, out=d_gw, stream=stream)
        stream.synchronize()
        assert tbe.last_status(stream) == (0, 0, 0)
        bl.barrier()
        torch.cuda.synchronize()
        launches0 = tbe.launch_count()
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
              for _ in range(args.steps)]
        for a, b in ev:
            flush.fill_(1)
            a.record(stream)
            tbe.backward_weights(tables, d_G, d_idx, d_off, B, base.mode, out=d_gw, stream=stream)
            b.record(stream)
        torch.cuda.synchronize()
        bl.barrier()
        launches = tbe.launch_count() - launches0
        step_ms = [a.elapsed_time(b) for a, b in ev]
        elapsed_ms = float(sum(step_ms))
        # end to end: host grad_out, ids and offsets in, the weights' gradient back to the host
        e2e_steps = args.e2e_steps or min(args.steps, 10)
        ev2 = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
               for _ in range(e2e_steps)]
        for a, b in ev2:
            a.record(stream)
            s_idx.copy_(h_idx, non_blocking=True)
            s_off.copy_(h_off, non_blocking=True)
            s_G.copy_(h_G, non_blocking=True)
            tbe.backward_weights(tables, s_G, s_idx, s_off, B, base.mode, out=d_gw, stream=stream)
            h_gw.copy_(d_gw, non_blocking=True)
            b.record(stream)
        torch.cuda.synchronize()
        bl.barrier()
        e2e_ms = float(sum(a.elapsed_time(b) for a, b in ev2))
    clocks = sampler.stop()
    total, max_ms = bl.reduce_job(lookups * args.steps, elapsed_ms, dev)
    e2e_total, e2e_max = bl.reduce_job(lookups * e2e_steps, e2e_ms, dev)
    tbe.close()
    if rank != 0:
        return
    peaks = bl.measured_peaks(ROOT)
    ms = elapsed_ms / args.steps
    achieved = alg / (ms * 1e-3) / 1e9
    n_cpu, dt = cpu_sample()
    line = {"metric": METRIC, "value": total / (max_ms * 1e-3), "unit": UNIT,
            "n_gpus": world, "steps": args.steps, "warmup": warmup, "ms_per_step": max_ms / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
            "data": "synthetic", "config": config, "clocks": clocks, "gpu_launches": launches,
            "e2e": {"value": e2e_total / (e2e_max * 1e-3), "unit": UNIT,
                    "h2d_bytes_per_step": int(h_idx.numel() * 8 + h_off.numel() * 8 + h_G.numel() * 4),
                    "d2h_bytes_per_step": int(h_gw.numel() * 4), "steps": e2e_steps,
                    "ms_per_step": e2e_max / e2e_steps},
            "roofline": {"bound": "hbm", "kernel": "ebag_bwd_weights_kernel", "achieved": achieved,
                         "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": achieved / peaks["hbm_gbs"],
                         "peak_source": f"{peaks['source']} HBM copy bandwidth (burst); with skewed ids most row "
                                        "bytes are served by L1 and L2, so this is a reference, not the binding limit",
                         "algorithmic_bytes_per_launch": alg, "ms_per_launch": ms,
                         "ms_per_launch_min": min(step_ms), "traffic": None},
            "cpu_baseline": {"value": n_cpu / dt, "unit": UNIT, "cores": 1, "kind": "oracle",
                             "sample": cpu_note, "seconds": dt}}
    print(json.dumps(line), flush=True)


def hbm_case(args, dev, local_rank, peaks):
    """The HBM-bound leg beside the headline workload: workload 4 (uniform ids over 41 GB of fp32
    tables, weighted sum), whose DRAM bytes equal its algorithmic bytes, timed exactly like the
    headline (CUDA events on the launching stream, L2 flushed between steps, clocks sampled)."""
    import paper_2512_23236_b200 as eb
    w = wl.make_workload(HBM_CASE_WORKLOAD, seed=0)
    need = sum(r * eb.ebag_row_stride(w.dtype, d) for r, d in zip(w.rows, w.D))
    free, _ = torch.cuda.mem_get_info()
    if free < need + (6 << 30):
        return {"workload": w.name, "skipped": f"needs {need >> 30} GiB of device memory, {free >> 30} GiB free"}
    jag = wl.gen_jagged(w)
    ab = wl.algorithmic_bytes(w, jag.lengths)
    tables = [wl.gen_table(w, t, dev) for t in range(w.T)]
    d_idx = torch.from_numpy(jag.indices).to(dev)
    d_off = torch.from_numpy(jag.offsets).to(dev)
    d_w = None if jag.weights is None else torch.from_numpy(jag.weights).to(dev)
    d_out = torch.empty((w.B, w.sumD), dtype=torch.float32, device=dev)
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=dev)
    tbe = eb.TBE(w.rows, w.D, w.dtype, device=local_rank)
    stream = torch.cuda.Stream(device=dev)
    steps = max(20, args.steps)
    torch.cuda.synchronize()
    sampler = bl.ClockSampler(f"GPU-{torch.cuda.get_device_properties(dev).uuid}").start()
    with torch.cuda.stream(stream):
        for _ in range(max(3, args.warmup)):
            flush.fill_(1)
            tbe.forward(tables, d_idx, d_off, w.B, w.mode, d_w, out=d_out, stream=stream)
        stream.synchronize()
        assert tbe.last_status(stream) == (0, 0, 0)
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
              for _ in range(steps)]
        for a, b in ev:
            flush.fill_(1)
            a.record(stream)
            tbe.forward(tables, d_idx, d_off, w.B, w.mode, d_w, out=d_out, stream=stream)
            b.record(stream)
        torch.cuda.synchronize()
    clocks = sampler.stop()
    tbe.close()
    step_ms = sorted(a.elapsed_time(b) for a, b in ev)
    ms = sum(step_ms) / steps
    achieved = ab["total"] / (ms * 1e-3) / 1e9
    traffic, src = ncu_traffic(w.number, ab["lookups"])
    return {"workload": w.name, "bound": BOUND[w.number], "steps": steps, "lookups_per_launch": ab["lookups"],
            "ms_per_launch": ms, "min": step_ms[0], "median": step_ms[len(step_ms) // 2],
            "algorithmic_bytes": ab["total"], "achieved": achieved, "unit": "GB/s",
            "peak": peaks["hbm_gbs"], "frac": achieved / peaks["hbm_gbs"],
            "peak_source": f"{peaks['source']} HBM copy bandwidth (burst)",
            "frac_of_nominal_8TBs": achieved / 8000.0,
            "traffic": traffic, "traffic_source": src,
            "frac_dram": None if traffic is None else traffic / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
            "clocks": clocks}


def main():
    args = parse_args()
    rank, local_rank, world = bl.rank_info()
    if args.workload == BET_WORKLOAD:
        run_bet(args, rank, local_rank, world)
        return
    if args.workload == MBDT_WORKLOAD:
        run_mbdt(args, rank, local_rank, world)
        return
    if args.workload == BWD_WORKLOAD:
        run_bwd(args, rank, local_rank, world)
        return
    if args.workload == GW_WORKLOAD:
        run_gw(args, rank, local_rank, world)
        return
    if args.impl == "reference":
        run_reference(args, rank)
        return
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    import paper_2512_23236_b200 as eb
    eb.lib()                                   # fail loudly if the CUDA library is missing
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = bl.init_process_group("nccl")
    warmup = max(3, args.warmup)

    # ---------------- inputs: seeded, synthetic; every rank owns its own tables and batch
    w = make_workload(args, bl.rank_seed(0, rank))
    jag = wl.gen_jagged(w)
    ab = wl.algorithmic_bytes(w, jag.lengths)
    raw_tables = [wl.gen_table(w, t, dev) for t in range(w.T)]
    if w.dtype == wl.INT8_ROWWISE:
        tables = [eb.ebag_pack_int8_rowwise(q, s, b) for q, s, b in raw_tables]
    else:
        tables = raw_tables

    def host_table(t):
        x = raw_tables[t]
        return tuple(y.cpu() for y in x) if isinstance(x, tuple) else x.cpu()

    mapid = args.workload == MAPID_WORKLOAD
    d_maps = None
    if mapid:
        maps = wl.gen_mappings(w)
        raw = wl.raw_values(w, jag, maps)
        d_maps = [torch.from_numpy(m).to(dev) for m in maps]
        d_raw = torch.from_numpy(raw).to(dev)
    h_idx = torch.from_numpy(jag.indices).pin_memory()
    h_off = torch.from_numpy(jag.offsets).pin_memory()
    h_w = None if jag.weights is None else torch.from_numpy(jag.weights).pin_memory()
    d_idx, d_off = h_idx.to(dev), h_off.to(dev)
    d_w = None if h_w is None else h_w.to(dev)
    d_out = torch.empty((w.B, w.sumD), dtype=torch.float32, device=dev)
    h_out = torch.empty((w.B, w.sumD), dtype=torch.float32).pin_memory()
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=dev)

    tbe = eb.TBE(w.rows, w.D, w.dtype, device=local_rank)
    if args.item_bytes:
        tbe.set_param("item_bytes", args.item_bytes)
    if args.split_bytes >= 0:
        tbe.set_param("split_bytes", args.split_bytes)
    if args.ctas_per_sm:
        tbe.set_param("ctas_per_sm", args.ctas_per_sm)
    stream = torch.cuda.Stream(device=dev)

    def step():
        if mapid:
            tbe.forward_mapid(tables, d_raw, d_off, d_maps, w.B, w.mode, d_w, out=d_out, stream=stream)
        else:
            tbe.forward(tables, d_idx, d_off, w.B, w.mode, d_w, out=d_out, stream=stream)

    def step_host():
        tbe.forward_host(tables, h_idx, h_off, w.B, w.mode, h_w, out=h_out, stream=stream)

    torch.cuda.synchronize()
    sampler = bl.ClockSampler(f"GPU-{torch.cuda.get_device_properties(dev).uuid}").start()
    with torch.cuda.stream(stream):
        for _ in range(warmup):
            flush.fill_(1)
            step()
        stream.synchronize()
        assert tbe.last_status(stream) == (0, 0, 0)

        # ---------------- device-resident timing: K steps, CUDA events on the launching stream
        bl.barrier()
        torch.cuda.synchronize()
        launches0 = tbe.launch_count()
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
              for _ in range(args.steps)]
        for a, b in ev:
            flush.fill_(1)                     # outside the event pair
            a.record(stream)
            step()
            b.record(stream)
        torch.cuda.synchronize()
        bl.barrier()
        launches = tbe.launch_count() - launches0
        step_ms = [a.elapsed_time(b) for a, b in ev]
        elapsed_ms = float(sum(step_ms))

        # ---------------- the same inputs back to back, no flush in between (the warm regime,
        # reported beside the cold one; at these sizes little of a step's data survives in L2)
        warm_n = min(args.steps, 10)
        wa, wb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        step()
        wa.record(stream)
        for _ in range(warm_n):
            step()
        wb.record(stream)
        torch.cuda.synchronize()
        warm_ms = wa.elapsed_time(wb) / warm_n

        # ---------------- end to end: host buffers in, host result out, copies timed
        e2e_steps = args.e2e_steps or min(args.steps, 10)
        for _ in range(2):
            step_host()
        stream.synchronize()
        bl.barrier()
        torch.cuda.synchronize()
        ev2 = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
               for _ in range(e2e_steps)]
        for a, b in ev2:
            a.record(stream)
            step_host()
            b.record(stream)
        torch.cuda.synchronize()
        bl.barrier()
        e2e_ms = float(sum(a.elapsed_time(b) for a, b in ev2))
        # ---------------- beside it: the same call with 32-bit ids and bf16 output (fewer bytes on
        # both legs); an extra figure, the headline keeps the int64 ids and fp32 output of the config
        e2e_narrow = None
        if not mapid and max(w.rows) < 2 ** 31:
            import paper_2512_23236_b200 as ebm
            h_idx32 = torch.from_numpy(jag.indices.astype(np.int32)).pin_memory()
            h_out16 = torch.empty((w.B, w.sumD), dtype=torch.bfloat16).pin_memory()
            tbe.set_param("out_dtype", ebm.EBAG_BF16)
            for _ in range(2):
                tbe.forward_host(tables, h_idx32, h_off, w.B, w.mode, h_w, out=h_out16, stream=stream)
            stream.synchronize()
            na, nb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            na.record(stream)
            for _ in range(e2e_steps):
                tbe.forward_host(tables, h_idx32, h_off, w.B, w.mode, h_w, out=h_out16, stream=stream)
            nb.record(stream)
            torch.cuda.synchronize()
            tbe.set_param("out_dtype", ebm.EBAG_F32)
            narrow_ms = na.elapsed_time(nb) / e2e_steps
            e2e_narrow = {"ids": "int32", "out": "bf16", "ms_per_step": narrow_ms,
                          "value": ab["lookups"] / (narrow_ms * 1e-3), "unit": UNIT,
                          "h2d_bytes_per_step": ab["indices"] // 2 + ab["offsets"] + ab["weights"],
                          "d2h_bytes_per_step": ab["out"] // 2}
    mapid_extra = None
    if mapid:
        # the timed call runs the transform in a launch of its own and then the plain forward (the
        # library's default); beside it: the search fused into the forward kernel, and the parts
        ids = torch.empty_like(d_raw)

        def fused():
            tbe.set_param("mapid_fused", 1)
            tbe.forward_mapid(tables, d_raw, d_off, d_maps, w.B, w.mode, d_w, out=d_out, stream=stream)
            tbe.set_param("mapid_fused", 0)

        def fused_binary_search():
            tbe.set_param("mapid_hash", 0)
            fused()
            tbe.set_param("mapid_hash", 1)

        def mapid_only():
            tbe.mapid(d_raw, d_off, d_maps, w.B, out=ids, stream=stream)

        def plain():
            tbe.forward(tables, d_idx, d_off, w.B, w.mode, d_w, out=d_out, stream=stream)

        def timed(fn, reps=10):
            with torch.cuda.stream(stream):
                fn()
                total = 0.0
                for _ in range(reps):
                    flush.fill_(1)
                    a = torch.cuda.Event(enable_timing=True)
                    b = torch.cuda.Event(enable_timing=True)
                    a.record(stream)
                    fn()
                    b.record(stream)
                    stream.synchronize()
                    total += a.elapsed_time(b)
            return total / reps

        default_out = d_out.clone()
        mapid_extra = {"mapid_then_forward_ms": elapsed_ms / args.steps, "fused_ms": timed(fused)}
        assert torch.equal(default_out, d_out), "fused MapId forward and the two-launch path disagree"
        mapid_extra["fused_binary_search_ms"] = timed(fused_binary_search)
        assert torch.equal(default_out, d_out), "fused MapId forward and the two-launch path disagree"
        mapid_extra["mapid_alone_ms"] = timed(mapid_only)              # hash tables of the mappings
        assert torch.equal(ids, d_idx)
        tbe.set_param("mapid_hash", 0)
        mapid_extra["mapid_alone_binary_search_ms"] = timed(mapid_only)
        tbe.set_param("mapid_hash", 1)
        mapid_extra["plain_forward_ms"] = timed(plain)
        assert torch.equal(default_out, d_out), "MapId forward and plain forward disagree"
        assert torch.equal(ids, d_idx)
    clocks = sampler.stop()
    assert tbe.last_status(stream) == (0, 0, 0)
    assert torch.equal(h_out, d_out.cpu()), "host-buffer path and device path disagree"

    total_lookups, max_ms = bl.reduce_job(ab["lookups"] * args.steps, elapsed_ms, dev)
    e2e_lookups, e2e_max_ms = bl.reduce_job(ab["lookups"] * e2e_steps, e2e_ms, dev)
    if rank != 0:
        tbe.close()
        return

    peaks = bl.measured_peaks(ROOT)
    # one forward kernel per step (the short parts kernel that may follow it is inside the same
    # event pair and counted in gpu_launches)
    ms_per_launch = elapsed_ms / max(1, args.steps)
    achieved = ab["total"] / (ms_per_launch * 1e-3) / 1e9
    full_size = not (args.max_tables or args.scale_rows != 1.0 or args.scale_b != 1.0)
    traffic, traffic_src = ncu_traffic(w.number, ab["lookups"]) if (full_size and not mapid) else (None, None)
    dram_gbs = None if traffic is None else traffic / (ms_per_launch * 1e-3) / 1e9
    line = {
        "metric": METRIC, "value": total_lookups / (max_ms * 1e-3), "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": warmup, "ms_per_step": max_ms / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic", "config": workload_config(w, ab, args),
        "clocks": clocks, "gpu_launches": launches,
        "e2e": {"value": e2e_lookups / (e2e_max_ms * 1e-3), "unit": UNIT,
                "h2d_bytes_per_step": ab["indices"] + ab["offsets"] + ab["weights"],
                "d2h_bytes_per_step": ab["out"], "steps": e2e_steps,
                "ms_per_step": e2e_max_ms / e2e_steps,
                "narrow": e2e_narrow if world == 1 else None},
        # `bound` names what the ncu counters show to be the limit of this launch.  `achieved` and
        # `frac` are ALGORITHMIC bytes over the launch time against the measured copy bandwidth:
        # on the skewed workloads L1 and L2 serve most of those bytes, so that ratio passes 1 and is
        # not a fraction of a binding ceiling; `frac_dram` is the same launch seen from DRAM.  The
        # workload whose DRAM bytes equal its algorithmic bytes is timed beside it (`hbm_case`).
        "roofline": {"bound": BOUND.get(w.number, "hbm"), "kernel": "ebag_fwd_kernel", "achieved": achieved,
                     "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": achieved / peaks["hbm_gbs"],
                     "peak_source": f"{peaks['source']} HBM copy bandwidth (burst)",
                     "frac_of_nominal_8TBs": achieved / 8000.0,
                     "algorithmic_bytes_per_launch": ab["total"],
                     "ms_per_launch": ms_per_launch, "ms_per_launch_min": min(step_ms),
                     "ms_per_launch_median": sorted(step_ms)[len(step_ms) // 2],
                     "ms_per_launch_warm_l2": warm_ms,
                     "traffic": traffic, "traffic_source": traffic_src,
                     "dram_gbs": dram_gbs,
                     "frac_dram": None if dram_gbs is None else dram_gbs / peaks["hbm_gbs"],
                     "l1_l2_served_bytes": None if traffic is None else ab["total"] - traffic},
        "bags_per_sec": w.T * w.B * world * args.steps / (max_ms * 1e-3),
    }
    if mapid_extra:
        line["mapid"] = mapid_extra
    if world == 1 and not args.no_cpu_baseline:
        inp, desc, cores = sized_cpu_sample(w, jag, host_table, args.cpu_seconds,
                                            (raw, maps) if mapid else None)
        dt = time_oracle(w, inp)
        line["cpu_baseline"] = {"value": inp["lookups"] / dt, "unit": UNIT, "cores": cores,
                                "kind": "oracle", "sample": desc, "seconds": dt}
    else:
        line["cpu_baseline"] = None
    tbe.close()
    if world == 1 and full_size and w.number == 3 and not mapid and not args.no_hbm_case:
        # free the headline workload's device memory first: the HBM-bound one needs 41 GB
        del tables, raw_tables, d_idx, d_off, d_w, d_out, flush
        torch.cuda.empty_cache()
        line["roofline"]["hbm_case"] = hbm_case(args, dev, local_rank, peaks)
    print(json.dumps(line), flush=True)


if __name__ == "__main__":
    main()
