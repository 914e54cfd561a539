"""Seeded synthetic inputs for the pooled embedding-bag forward.

This module only draws inputs (table values, jagged id lists, per-sample weights).  It holds
none of the operator's arithmetic and imports neither the CUDA binding nor the CPU oracle, so
both sides can be fed the very same arrays.

The five workloads stand in for production DLRM sparse features (jagged int64 id lists and
(id, float32 score) pairs, Sec. 2.2 "Feature Types and Memory Layout"; embedding tables that
stress memory bandwidth, Sec. 2.1 "DLRM Architecture").  The paper itself evaluates on synthetic
data matched to production statistics (Appendix "1D Convolution", input generation), which is
the precedent for doing the same here.

Recipe (identical for every workload; seed 0, one numpy PCG64 stream per workload keyed by
SeedSequence([seed, workload number, 0]) for the table shapes (rows, D, per-table mean length)
and one per table keyed by [seed, workload number, 1, table] for its bag lengths, Zipf ranks /
uniform ids, row permutation and weights, in that order; table values come from a torch
generator keyed by (seed, workload number, table)):

  1  1 table 10,000 x 64 fp32 N(0,1); B=512; lengths integer-uniform on 0..20; uniform ids; sum
  2  1 table 1,000,000 x 128 fp16 N(0,1); B=16,384; Poisson(30); Zipf(1.05) ranks through a
     random row permutation; mean
  3  32 tables, rows floor(10^U(5,7)), D drawn from {64,128,256}, bf16 N(0,0.02); B=65,536 per
     table; per-table mean length U(1,80), lengths Poisson; Zipf(1.1) + permutation; sum
  4  8 tables 5,000,000 x 256 fp32 N(0,1); B=32,768; lengths geometric(p=1/50) on {1,2,..}
     capped at 1024; uniform ids; weights U(0,1) fp32; weighted sum
  5  64 tables 2,000,000 x 128 rowwise int8 (codes U{-128..127}, scale U(0.01,0.03),
     bias N(0,0.1)); B=131,072; Poisson(20); Zipf(1.2) + permutation; sum

Bounded Zipf: rank k in 1..rows with P(k) proportional to k^-alpha, drawn by inverting the
cumulative table; the id is perm[k-1] for a per-table uniform random permutation.
"""
from __future__ import annotations

import dataclasses
from typing import List, Optional

import numpy as np
import torch

F32, F16, BF16, INT8_ROWWISE, UINT8_ROWWISE = 0, 1, 2, 3, 4
SUM, MEAN, MAX = 0, 1, 2

DTYPE_NAMES = {F32: "f32", F16: "f16", BF16: "bf16", INT8_ROWWISE: "int8_rowwise",
               UINT8_ROWWISE: "uint8_rowwise"}
_TORCH_DT = {F32: torch.float32, F16: torch.float16, BF16: torch.bfloat16,
             INT8_ROWWISE: torch.int8, UINT8_ROWWISE: torch.uint8}


@dataclasses.dataclass
class Workload:
    number: int                    # 1..5 (the five published workloads); 0 for ad-hoc ones
    name: str
    dtype: int
    rows: List[int]
    D: List[int]
    B: int
    mode: int
    weighted: bool
    length_kind: str               # "uniform_int" | "poisson" | "geometric_capped"
    length_params: List[float]     # per table: mean (poisson), hi (uniform_int), mean (geometric)
    length_cap: int
    index_kind: str                # "uniform" | "zipf"
    zipf_alpha: float
    value_std: float
    seed: int = 0

    @property
    def T(self) -> int:
        return len(self.rows)

    @property
    def sumD(self) -> int:
        return int(sum(self.D))


def make_workload(number: int, scale_rows: float = 1.0, scale_B: float = 1.0,
                  max_tables: Optional[int] = None, seed: int = 0) -> Workload:
    """Workload ``number`` (1..5).  ``scale_rows``/``scale_B``/``max_tables`` shrink it for
    cases the CPU oracle must finish in seconds; the draws for the structure stay in the same
    order, so a shrunk workload has the same D mix and mean lengths as the full one."""
    rng = np.random.default_rng(np.random.SeedSequence([seed, number, 0]))

    def srows(r):
        return max(16, int(r * scale_rows))

    def sB(b):
        return max(1, int(b * scale_B))

    if number == 1:
        w = Workload(1, "cfg1_single_f32_sum", F32, [srows(10_000)], [64], sB(512), SUM, False,
                     "uniform_int", [20], 0, "uniform", 0.0, 1.0, seed)
    elif number == 2:
        w = Workload(2, "cfg2_single_f16_mean_zipf", F16, [srows(1_000_000)], [128], sB(16_384),
                     MEAN, False, "poisson", [30.0], 0, "zipf", 1.05, 1.0, seed)
    elif number == 3:
        T = 32
        rows = [srows(int(np.floor(10.0 ** u))) for u in rng.uniform(5.0, 7.0, size=T)]
        D = [int(d) for d in rng.choice([64, 128, 256], size=T)]
        lam = [float(x) for x in rng.uniform(1.0, 80.0, size=T)]
        w = Workload(3, "cfg3_tbe32_bf16_sum_zipf", BF16, rows, D, sB(65_536), SUM, False,
                     "poisson", lam, 0, "zipf", 1.1, 0.02, seed)
    elif number == 4:
        T = 8
        w = Workload(4, "cfg4_tbe8_f32_weighted_uniform", F32, [srows(5_000_000)] * T, [256] * T,
                     sB(32_768), SUM, True, "geometric_capped", [50.0] * T, 1024, "uniform", 0.0,
                     1.0, seed)
    elif number == 5:
        T = 64
        w = Workload(5, "cfg5_tbe64_int8_sum_zipf", INT8_ROWWISE, [srows(2_000_000)] * T,
                     [128] * T, sB(131_072), SUM, False, "poisson", [20.0] * T, 0, "zipf", 1.2,
                     1.0, seed)
    else:
        raise ValueError("workload number must be 1..5")
    if max_tables is not None and max_tables < w.T:
        w.rows, w.D = w.rows[:max_tables], w.D[:max_tables]
        w.length_params = w.length_params[:max_tables]
    return w


@dataclasses.dataclass
class Jagged:
    indices: np.ndarray            # int64 [N]
    offsets: np.ndarray            # int64 [T*B+1], bag id = t*B + b
    weights: Optional[np.ndarray]  # float32 [N] or None
    lengths: np.ndarray            # int64 [T*B]


def _draw_lengths(rng, w: Workload, t: int) -> np.ndarray:
    p = w.length_params[t]
    if w.length_kind == "uniform_int":
        return rng.integers(0, int(p) + 1, size=w.B, dtype=np.int64)
    if w.length_kind == "poisson":
        return rng.poisson(p, size=w.B).astype(np.int64)
    if w.length_kind == "geometric_capped":
        return np.minimum(rng.geometric(1.0 / p, size=w.B).astype(np.int64), w.length_cap)
    raise ValueError(w.length_kind)


def _draw_ids(rng, w: Workload, t: int, n: int) -> np.ndarray:
    rows = w.rows[t]
    if w.index_kind == "uniform":
        return rng.integers(0, rows, size=n, dtype=np.int64)
    pmf = np.arange(1, rows + 1, dtype=np.float64) ** (-w.zipf_alpha)
    cdf = np.cumsum(pmf)
    cdf /= cdf[-1]
    ranks = np.searchsorted(cdf, rng.random(n), side="right")
    np.minimum(ranks, rows - 1, out=ranks)
    perm = rng.permutation(rows)
    return perm[ranks].astype(np.int64, copy=False)


def _gen_table_jagged(w: Workload, t: int):
    rng = np.random.default_rng(np.random.SeedSequence([w.seed, w.number, 1, t]))
    lengths = _draw_lengths(rng, w, t)
    n = int(lengths.sum())
    ids = _draw_ids(rng, w, t, n)
    weights = rng.random(n, dtype=np.float32) if w.weighted else None
    return lengths, ids, weights


def gen_jagged(w: Workload) -> Jagged:
    """Bag lengths, offsets, ids and weights for all T tables (host, numpy, seeded; one
    independent stream per table, drawn on a thread pool)."""
    import concurrent.futures
    import os
    with concurrent.futures.ThreadPoolExecutor(max_workers=min(w.T, os.cpu_count() or 1)) as ex:
        parts = list(ex.map(lambda t: _gen_table_jagged(w, t), range(w.T)))
    lengths = np.concatenate([p[0] for p in parts])
    offsets = np.zeros(w.T * w.B + 1, dtype=np.int64)
    np.cumsum(lengths, out=offsets[1:])
    indices = np.concatenate([p[1] for p in parts])
    weights = np.concatenate([p[2] for p in parts]) if w.weighted else None
    return Jagged(indices, offsets, weights, lengths)


def gen_table(w: Workload, t: int, device="cpu"):
    """Values of table ``t`` as torch tensors on ``device``.

    F32/F16/BF16: one tensor [rows, D] of that dtype.  INT8_ROWWISE / UINT8_ROWWISE: (codes int8 /
    uint8 [rows, D], scale float32 [rows], bias float32 [rows])."""
    dev = torch.device(device)
    g = torch.Generator(device=dev)
    g.manual_seed((w.seed * 1_000_003 + w.number) * 4099 + t)
    rows, D = w.rows[t], w.D[t]
    if w.dtype in (INT8_ROWWISE, UINT8_ROWWISE):
        if w.dtype == INT8_ROWWISE:
            q = torch.randint(-128, 128, (rows, D), dtype=torch.int8, device=dev, generator=g)
        else:
            q = torch.randint(0, 256, (rows, D), dtype=torch.uint8, device=dev, generator=g)
        scale = torch.empty(rows, dtype=torch.float32, device=dev).uniform_(0.01, 0.03,
                                                                            generator=g)
        bias = torch.empty(rows, dtype=torch.float32, device=dev).normal_(0.0, 0.1, generator=g)
        return q, scale, bias
    x = torch.empty((rows, D), dtype=_TORCH_DT[w.dtype], device=dev)
    x.normal_(0.0, w.value_std, generator=g)
    return x


def gen_tables(w: Workload, device="cpu"):
    return [gen_table(w, t, device) for t in range(w.T)]


def gen_mappings(w: Workload) -> List[np.ndarray]:
    """MapId inputs for workload ``w``: per table a strictly increasing int64 list of
    rows[t] - 1 known raw ids (row 0 of the table is the "unknown" embedding), gaps of 1..3."""
    out = []
    for t in range(w.T):
        rng = np.random.default_rng(np.random.SeedSequence([w.seed, w.number, 2, t]))
        out.append(np.cumsum(rng.integers(1, 4, size=max(w.rows[t] - 1, 0), dtype=np.int64)))
    return out


def raw_values(w: Workload, jag: Jagged, mappings: List[np.ndarray]) -> np.ndarray:
    """Raw ids whose MapId image is ``jag.indices``: row k >= 1 comes from the k-th known id,
    row 0 from -1, which no mapping contains."""
    vals = np.empty_like(jag.indices)
    for t in range(w.T):
        lo, hi = int(jag.offsets[t * w.B]), int(jag.offsets[(t + 1) * w.B])
        idx = jag.indices[lo:hi]
        m = mappings[t]
        vals[lo:hi] = np.where(idx == 0, -1, m[np.maximum(idx, 1) - 1]) if m.size else -1
    return vals


def raw_numpy(x: torch.Tensor) -> np.ndarray:
    """Host numpy view of a table for the oracle: float32 / int8 as is, fp16 and bf16 as their
    uint16 bit patterns."""
    x = x.detach().cpu().contiguous()
    if x.dtype in (torch.float16, torch.bfloat16):
        return x.view(torch.int16).numpy().view(np.uint16)
    return x.numpy()


def algorithmic_bytes(w: Workload, lengths: np.ndarray) -> dict:
    """Bytes the operator itself must move for this input: per lookup the stored row
    (D*elem, plus 8 for rowwise int8 scale+bias), the int64 id and, if weighted, the fp32
    weight; per bag one int64 offset and the fp32 output row."""
    elem = {F32: 4, F16: 2, BF16: 2, INT8_ROWWISE: 1, UINT8_ROWWISE: 1}[w.dtype]
    extra = 8 if w.dtype in (INT8_ROWWISE, UINT8_ROWWISE) else 0
    gathered = 0
    n = 0
    for t in range(w.T):
        nt = int(lengths[t * w.B:(t + 1) * w.B].sum())
        n += nt
        gathered += nt * (w.D[t] * elem + extra)
    idx = 8 * n
    wts = 4 * n if w.weighted else 0
    off = 8 * (w.T * w.B + 1)
    out = 4 * w.B * w.sumD
    return dict(lookups=n, gathered=gathered, indices=idx, weights=wts, offsets=off, out=out,
                total=gathered + idx + wts + off + out)
