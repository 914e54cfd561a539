"""GPU parity of ebag_backward with the backward oracle, element by element.

Tolerance per gradient element: the GPU adds n fp32 terms in an order that is not fixed, the
oracle adds them in fp64.  With u = 2^-24, each product w*g is rounded once (error <= u*|term|)
and a sum of n terms picks up at most (n-1)*u*S in the worst case, about sqrt(n)*u*S for
rounding errors of random sign (S = sum of |terms|, from the oracle).  The bar used is
    |gpu - oracle| <= (8 * sqrt(n) + 4) * u * S
which is far below the weight of a single dropped or doubled term (about S / n) for every n
that occurs here.  Rows no lookup touches must keep their previous contents bit for bit."""
import numpy as np
import pytest
import torch

import paper_2512_23236_b200 as eb
from oracle import ebag_bwd_oracle as bo
from paper_2512_23236_b200 import workloads as wl

pytestmark = pytest.mark.gpu
U = 2.0 ** -24


def _problem(rng, rows, D, B, max_len, weighted, zipf=False):
    T = len(rows)
    lengths = rng.integers(0, max_len + 1, size=T * B)
    lengths[rng.random(T * B) < 0.1] = 0
    off = np.zeros(T * B + 1, np.int64)
    np.cumsum(lengths, out=off[1:])
    parts = []
    for t in range(T):
        n = int(lengths[t * B:(t + 1) * B].sum())
        if zipf:
            parts.append(np.minimum((rows[t] * rng.random(n) ** 6).astype(np.int64), rows[t] - 1))
        else:
            parts.append(rng.integers(0, rows[t], size=n))
    idx = np.concatenate(parts).astype(np.int64)
    w = rng.uniform(-1.5, 1.5, size=idx.size).astype(np.float32) if weighted else None
    G = rng.standard_normal((B, sum(D))).astype(np.float32)
    return lengths, off, idx, w, G


def _run(dtype, rows, D, B, off, idx, w, G, mode, start=None, params=None):
    tbe = eb.TBE(rows, D, dtype, device=torch.cuda.current_device())
    try:
        for k, v in (params or {}).items():
            tbe.set_param(k, v)
        grads = [torch.zeros(r, d, device="cuda") if start is None else torch.from_numpy(start[t]).cuda()
                 for t, (r, d) in enumerate(zip(rows, D))]
        tbe.backward(torch.from_numpy(G).cuda(), torch.from_numpy(idx).cuda(), torch.from_numpy(off).cuda(),
                     B, grads, mode, None if w is None else torch.from_numpy(w).cuda())
        status = tbe.last_status()
        return [g.cpu().numpy() for g in grads], status
    finally:
        tbe.close()


def _compare(got, ref, start=None):
    worst = 0.0
    for t, g in enumerate(got):
        base = 0.0 if start is None else start[t].astype(np.float64)
        err = np.abs(g.astype(np.float64) - (base + ref["grads"][t]))
        n = ref["counts"][t][:, None].astype(np.float64)
        S = ref["S"][t] + (0.0 if start is None else np.abs(base))
        tol = (8.0 * np.sqrt(n) + 4.0) * U * S
        bad = err > tol
        assert not bad.any(), f"table {t}: {bad.sum()} elements beyond the bar, first {np.argwhere(bad)[0]}"
        untouched = ref["counts"][t] == 0
        want = np.zeros_like(g[untouched]) if start is None else start[t][untouched]
        assert np.array_equal(g[untouched].view(np.uint32), want.view(np.uint32))
        pos = S > 0
        if pos.any():
            worst = max(worst, float((err[pos] / S[pos]).max()))
    return worst


@pytest.mark.parametrize("dtype,Ds", [(wl.F32, [4, 8, 12, 64, 100, 256, 260, 1028]),
                                      (wl.BF16, [8, 16, 72, 128, 512, 2056]),
                                      (wl.INT8_ROWWISE, [16, 48, 128, 528])])
@pytest.mark.parametrize("mode,weighted", [(wl.SUM, False), (wl.MEAN, False), (wl.SUM, True), (wl.MEAN, True)])
def test_all_row_widths(dtype, Ds, mode, weighted):
    rng = np.random.default_rng(3 + dtype)
    rows = [int(rng.integers(5, 300)) for _ in Ds]
    B = 61
    lengths, off, idx, w, G = _problem(rng, rows, Ds, B, 30, weighted)
    ref = bo.backward(rows, Ds, G, idx, off, B, mode, weights=w)
    got, status = _run(dtype, rows, Ds, B, off, idx, w, G, mode)
    assert status == (0, 0, 0)
    _compare(got, ref)


def test_hot_rows_int32_ids_and_accumulation():
    # skewed ids: a few rows collect thousands of terms; 32-bit ids; gradients added to what is there
    rng = np.random.default_rng(11)
    rows, D, B = [2000, 50], [64, 128], 400
    lengths, off, idx, w, G = _problem(rng, rows, D, B, 60, True, zipf=True)
    ref = bo.backward(rows, D, G, idx, off, B, wl.SUM, weights=w)
    assert max(int(c.max()) for c in ref["counts"]) > 1000
    start = [rng.standard_normal((r, d)).astype(np.float32) for r, d in zip(rows, D)]
    got64, st64 = _run(wl.F32, rows, D, B, off, idx, w, G, wl.SUM, start)
    got32, st32 = _run(wl.F32, rows, D, B, off, idx.astype(np.int32), w, G, wl.SUM, start)
    assert st64 == st32 == (0, 0, 0)
    _compare(got64, ref, start)
    _compare(got32, ref, start)


def test_rejected_ids_and_malformed_bags():
    rng = np.random.default_rng(5)
    rows, D, B = [100, 40], [32, 8], 50
    lengths, off, idx, w, G = _problem(rng, rows, D, B, 12, True)
    bad = rng.choice(idx.size, size=12, replace=False)
    idx[bad[:6]] = -5
    idx[bad[6:]] = 10 ** 12
    off[9] = off[8] - 2
    off[70] = idx.size + 5
    ref = bo.backward(rows, D, G, idx, off, B, wl.MEAN, weights=w)
    got, status = _run(wl.F32, rows, D, B, off, idx, w, G, wl.MEAN)
    assert ref["n_oob"] > 0 and ref["n_bad_offsets"] > 0
    assert status[1:] == (ref["n_oob"], ref["n_bad_offsets"]) and status[0] != eb.EBAG_OK
    _compare(got, ref)


def test_many_warps_and_tables_against_an_index_add_in_fp64():
    """A size at which every warp of the grid has work in every table and the hot-row sums are
    flushed many times: 0.6 M skewed lookups over four tables.  The oracle's Python loops are too
    slow here; the check is the operator's definition through a library routine (torch index_add_
    in fp64 on the CPU), with the same bar as the oracle-sized cases."""
    rng = np.random.default_rng(17)
    rows, D, B = [50_000, 3_000, 200_000, 64], [32, 64, 8, 128], 6000
    lengths, off, idx, w, G = _problem(rng, rows, D, B, 50, True, zipf=True)
    got, status = _run(wl.F32, rows, D, B, off, idx, w, G, wl.SUM)
    assert status == (0, 0, 0)
    col = 0
    for t, (r, d) in enumerate(zip(rows, D)):
        lo, hi = int(off[t * B]), int(off[(t + 1) * B])
        bag = np.repeat(np.arange(B), lengths[t * B:(t + 1) * B])
        terms = torch.from_numpy(G[bag, col:col + d].astype(np.float64) * w[lo:hi, None].astype(np.float64))
        ids = torch.from_numpy(idx[lo:hi])
        ref = torch.zeros(r, d, dtype=torch.float64).index_add_(0, ids, terms).numpy()
        S = torch.zeros(r, d, dtype=torch.float64).index_add_(0, ids, terms.abs()).numpy()
        n = np.bincount(idx[lo:hi], minlength=r)[:, None].astype(np.float64)
        err = np.abs(got[t].astype(np.float64) - ref)
        assert np.all(err <= (8.0 * np.sqrt(n) + 4.0) * U * S), t
        assert not got[t][n[:, 0] == 0].any()
        col += d


@pytest.mark.parametrize("mode,weighted,idx32", [(wl.SUM, False, False), (wl.MEAN, True, False), (wl.SUM, True, True)])
def test_sorted_path_is_reproducible_and_agrees_with_the_reductions(mode, weighted, idx32):
    """0.9 M skewed lookups over five tables (several sorting tiles per table, hot rows whose runs
    span many sub-chunks, row ids that need one, two and three sorting passes, an empty table
    segment): the default path (lookups sorted by row) gives the same bits on every run, and both
    it and the reduction kernel meet the bar against an fp64 index_add."""
    rng = np.random.default_rng(23 + mode)
    rows, D, B = [40_000, 200, 70_000, 9, 300_000], [64, 256, 32, 128, 8], 5000
    lengths, off, idx, w, G = _problem(rng, rows, D, B, 70, weighted, zipf=True)
    # table 3 gets no lookups at all
    lo3, hi3 = int(off[3 * B]), int(off[4 * B])
    idx = np.concatenate([idx[:lo3], idx[hi3:]])
    if w is not None:
        w = np.concatenate([w[:lo3], w[hi3:]])
    lengths[3 * B:4 * B] = 0
    off = np.zeros_like(off)
    np.cumsum(lengths, out=off[1:])
    idx[::1013] = -1                                       # skipped ids
    ids = idx.astype(np.int32) if idx32 else idx
    a, st_a = _run(wl.F32, rows, D, B, off, ids, w, G, mode)
    b, st_b = _run(wl.F32, rows, D, B, off, ids, w, G, mode)
    c, st_c = _run(wl.F32, rows, D, B, off, ids, w, G, mode, params=dict(bwd_sorted=0))
    n_skipped = int((idx < 0).sum())
    assert st_a == st_b == st_c == (eb.EBAG_ERR_INDEX_OOB, n_skipped, 0)
    for x, y in zip(a, b):
        assert np.array_equal(x.view(np.uint32), y.view(np.uint32)), "two runs differ"
    col = 0
    for t, (r, d) in enumerate(zip(rows, D)):
        lo, hi = int(off[t * B]), int(off[(t + 1) * B])
        bag = np.repeat(np.arange(B), lengths[t * B:(t + 1) * B])
        scale = np.ones(hi - lo) if w is None else w[lo:hi].astype(np.float64)
        if mode == wl.MEAN:
            scale = scale / np.repeat(lengths[t * B:(t + 1) * B], lengths[t * B:(t + 1) * B])
        keep = idx[lo:hi] >= 0
        terms = torch.from_numpy(G[bag, col:col + d].astype(np.float64) * scale[:, None])[keep]
        tid = torch.from_numpy(idx[lo:hi][keep])
        ref = torch.zeros(r, d, dtype=torch.float64).index_add_(0, tid, terms).numpy()
        S = torch.zeros(r, d, dtype=torch.float64).index_add_(0, tid, terms.abs()).numpy()
        n = np.bincount(idx[lo:hi][keep], minlength=r)[:, None].astype(np.float64)
        for got in (a[t], c[t]):
            err = np.abs(got.astype(np.float64) - ref)
            assert np.all(err <= (8.0 * np.sqrt(n) + 4.0) * U * S), t
            assert not got[n[:, 0] == 0].any()
        col += d


def test_offsets_that_reach_past_an_empty_id_list_are_counted():
    """No ids at all, but a bag that claims five: a malformed bag, counted as the oracle counts it
    (the call must not take "no ids" for "nothing to do")."""
    rows, D, B = [7], [8], 1
    off = np.array([0, 5], np.int64)
    idx = np.zeros(0, np.int64)
    G = np.ones((B, 8), np.float32)
    ref = bo.backward(rows, D, G, idx, off, B, wl.SUM)
    assert (ref["n_oob"], ref["n_bad_offsets"]) == (0, 1)
    got, status = _run(wl.F32, rows, D, B, off, idx, None, G, wl.SUM)
    assert status == (eb.EBAG_ERR_BAD_OFFSETS, 0, 1)
    assert not got[0].any()


def test_adjoint_of_the_gpu_forward():
    """<forward(T), G> = <T, backward(G)> with both sides computed on the GPU."""
    rng = np.random.default_rng(8)
    rows, D, B = [300, 80, 1000], [64, 16, 256], 200
    lengths, off, idx, w, G = _problem(rng, rows, D, B, 25, True)
    tabs = [torch.randn(r, d, device="cuda") for r, d in zip(rows, D)]
    tbe = eb.TBE(rows, D, wl.F32, device=torch.cuda.current_device())
    try:
        didx, doff, dw = (torch.from_numpy(x).cuda() for x in (idx, off, w))
        out = tbe.forward(tabs, didx, doff, B, wl.MEAN, dw)
        grads = [torch.zeros_like(t) for t in tabs]
        dG = torch.from_numpy(G).cuda()
        tbe.backward(dG, didx, doff, B, grads, wl.MEAN, dw)
        lhs = float((out.double() * dG.double()).sum())
        rhs = float(sum((t.double() * g.double()).sum() for t, g in zip(tabs, grads)))
        scale = float((out.abs().double() * dG.abs().double()).sum())
    finally:
        tbe.close()
    assert abs(lhs - rhs) <= 1e-5 * scale


def test_empty_and_argument_checks():
    tbe = eb.TBE([10], [16], wl.F32)
    try:
        g = torch.zeros(10, 16, device="cuda")
        off = torch.zeros(4, dtype=torch.int64, device="cuda")
        idx = torch.zeros(0, dtype=torch.int64, device="cuda")
        tbe.backward(torch.zeros(3, 16, device="cuda"), idx, off, 3, [g])
        assert tbe.last_status() == (0, 0, 0) and float(g.abs().sum()) == 0.0
        with pytest.raises(TypeError):
            tbe.backward(torch.zeros(3, 16, device="cuda"), idx, off, 3, [g.half()])
    finally:
        tbe.close()
