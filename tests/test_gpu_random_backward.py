"""Randomized shapes through both backward entry points: table count (empty tables included),
gradient row widths from one vector to three column tiles, row counts that
need one to three sorting passes, bag lengths from all-empty to thousands, skipped ids, weights,
mean, both id widths.  ebag_backward against the backward oracle (and bit for bit against a second
run when the reproducible path applies), ebag_backward_weights against its oracle.

The bar per gradient element is the one of tests/test_gpu_backward.py, (8 * sqrt(n) + 4) * u * S,
plus n / 16 * u * S: the generator can send thousands of lookups of ONE bag to one row of a tiny
table, i.e. add the same fp32 value n times, and then the roundings all go one way (the error grows
like n, not like sqrt(n); a longer run of these seeds measured up to 1.05 of the plain bar in four
of 364 cases, for the reduction kernel and the sorted path alike).  The worst case of a sequential
sum is (n - 1) * u * S, sixteen times above what is added here."""
import numpy as np
import pytest
import torch

import paper_2512_23236_b200 as eb
from oracle import ebag_bwd_oracle as bo
from paper_2512_23236_b200 import workloads as wl

pytestmark = pytest.mark.gpu
U = 2.0 ** -24


def _case(seed):
    rng = np.random.default_rng(1000 + seed)
    T = int(rng.integers(1, 6))
    wide = seed % 6 == 5
    Ds = [int(rng.integers(1, 90 if wide else 65)) * 4 for _ in range(T)]
    B = int(rng.integers(1, 200))
    rows = [int(rng.choice([1, 7, 200, 300, 70_000, 1 << 17])) for _ in Ds]
    maxlen = int(rng.choice([0, 2, 30, 300]))
    lengths = rng.integers(0, maxlen + 1, size=T * B)
    if seed % 5 == 0:
        lengths[int(rng.integers(0, T * B))] = int(rng.integers(3000, 9000))     # a run of many units
    if T > 1 and seed % 4 == 1:
        t0 = int(rng.integers(0, T))
        lengths[t0 * B:(t0 + 1) * B] = 0                                         # a table without lookups
    off = np.zeros(T * B + 1, np.int64)
    np.cumsum(lengths, out=off[1:])
    parts = []
    for t in range(T):
        n = int(lengths[t * B:(t + 1) * B].sum())
        hot = np.minimum((rows[t] * rng.random(n) ** 5).astype(np.int64), rows[t] - 1)
        parts.append(hot if seed % 2 else rng.integers(0, rows[t], size=n))
    idx = np.concatenate(parts).astype(np.int64) if parts else np.zeros(0, np.int64)
    if idx.size and seed % 3 == 0:
        idx[rng.choice(idx.size, size=max(1, idx.size // 50), replace=False)] = -3
    w = rng.uniform(-1.5, 1.5, size=idx.size).astype(np.float32) if seed % 3 == 1 else None
    mode = [wl.SUM, wl.MEAN][(seed // 2) % 2]
    G = rng.standard_normal((B, sum(Ds))).astype(np.float32)
    return rows, Ds, B, lengths, off, idx, w, mode, G


@pytest.mark.parametrize("seed", range(36))
def test_random_backward(seed):
    rows, Ds, B, lengths, off, idx, w, mode, G = _case(seed)
    ids = idx.astype(np.int32) if seed % 4 == 2 else idx
    ref = bo.backward(rows, Ds, G, idx, off, B, mode, weights=w)
    outs = []
    tbe = eb.TBE(rows, Ds, wl.F32, device=torch.cuda.current_device())
    try:
        for _ in range(2):
            grads = [torch.zeros(r, d, device="cuda") for r, d in zip(rows, Ds)]
            tbe.backward(torch.from_numpy(G).cuda(), torch.from_numpy(ids).cuda(), torch.from_numpy(off).cuda(),
                         B, grads, mode, None if w is None else torch.from_numpy(w).cuda())
            status = tbe.last_status()
            assert status[1:] == (ref["n_oob"], 0)
            outs.append([g.cpu().numpy() for g in grads])
    finally:
        tbe.close()
    for t, g in enumerate(outs[0]):
        err = np.abs(g.astype(np.float64) - ref["grads"][t])
        n = ref["counts"][t][:, None].astype(np.float64)
        assert np.all(err <= (8.0 * np.sqrt(n) + n / 16.0 + 4.0) * U * ref["S"][t]), (seed, t)
        assert not g[ref["counts"][t] == 0].any()
        if idx.size:                                         # the reproducible path ran
            assert np.array_equal(g.view(np.uint32), outs[1][t].view(np.uint32)), (seed, t)


@pytest.mark.parametrize("seed", range(24))
def test_random_backward_weights(seed):
    rows, Ds, B, lengths, off, idx, w, mode, G = _case(seed)
    rng = np.random.default_rng(seed)
    vals = [rng.standard_normal((r, d)).astype(np.float32) for r, d in zip(rows, Ds)]
    ref = bo.backward_weights(vals, G, idx, off, B, mode)
    tbe = eb.TBE(rows, Ds, wl.F32, device=torch.cuda.current_device())
    try:
        got = tbe.backward_weights([torch.from_numpy(v).cuda() for v in vals], torch.from_numpy(G).cuda(),
                                   torch.from_numpy(idx).cuda(), torch.from_numpy(off).cuda(), B, mode)
        status = tbe.last_status()
    finally:
        tbe.close()
    assert status[1:] == (ref["n_oob"], 0)
    g = got.cpu().numpy().astype(np.float64)
    width = np.zeros(idx.size)
    for t in range(len(rows)):
        width[off[t * B]:off[(t + 1) * B]] = Ds[t]
    assert np.all(np.abs(g - ref["grad_w"]) <= (width + 4) * U * ref["S"] + 1e-30)
