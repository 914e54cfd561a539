"""GPU parity of ebag_backward_weights (gradient of the per-sample weights) with its oracle,
lookup by lookup, for every storage type, both id widths, sum and mean, with planted bad ids and
a malformed bag.

Tolerance per lookup: a dot product of D fp32 products added in some fixed order; with
u = 2^-24 the worst case is (D + 4) * u * S, S = sum_d |grad_out * value| from the oracle (the
value itself is exact on both sides: 16-bit storage widens exactly, and a rowwise 8-bit value is
scale * code + bias with product and sum rounded separately, which is how the test prepares the
oracle's input).  Two runs must give the same bits."""
import numpy as np
import pytest
import torch

import paper_2512_23236_b200 as eb
from oracle import ebag_bwd_oracle as bo
from paper_2512_23236_b200 import workloads as wl

import parity_util as pu

pytestmark = pytest.mark.gpu
U = 2.0 ** -24
_TORCH = {wl.F32: torch.float32, wl.F16: torch.float16, wl.BF16: torch.bfloat16}


def _tables(rng, dtype, rows, D):
    """(tables as the library takes them on the CPU, the values they hold as float32 arrays)"""
    tabs, vals = [], []
    for r, d in zip(rows, D):
        if dtype in pu.ROWWISE8:
            if dtype == wl.INT8_ROWWISE:
                q = rng.integers(-128, 128, size=(r, d)).astype(np.int8)
            else:
                q = rng.integers(0, 256, size=(r, d)).astype(np.uint8)
            s = rng.uniform(0.01, 0.03, r).astype(np.float32)
            b = rng.normal(0, 0.1, r).astype(np.float32)
            tabs.append((torch.from_numpy(q), torch.from_numpy(s), torch.from_numpy(b)))
            vals.append((s[:, None] * q.astype(np.float32)).astype(np.float32) + b[:, None])   # two roundings
        else:
            x = torch.from_numpy(rng.standard_normal((r, d)).astype(np.float32)).to(_TORCH[dtype])
            tabs.append(x)
            vals.append(x.float().numpy())
    return tabs, vals


def _device_tables(dtype, tabs):
    out = []
    for t in tabs:
        if dtype in pu.ROWWISE8:
            q, s, b = (x.cuda() for x in t)
            out.append(eb.ebag_pack_int8_rowwise(q, s, b) if dtype == wl.INT8_ROWWISE
                       else eb.ebag_pack_uint8_rowwise(q, s, b))
        else:
            out.append(t.cuda().contiguous())
    return out


def _jagged(rng, rows, B, max_len):
    T = len(rows)
    lengths = rng.integers(0, max_len + 1, size=T * B)
    lengths[rng.random(T * B) < 0.1] = 0
    off = np.zeros(T * B + 1, np.int64)
    np.cumsum(lengths, out=off[1:])
    idx = np.concatenate([rng.integers(0, rows[t], size=int(lengths[t * B:(t + 1) * B].sum()))
                          for t in range(T)]).astype(np.int64)
    return lengths, off, idx


@pytest.mark.parametrize("dtype", [wl.F32, wl.F16, wl.BF16, wl.INT8_ROWWISE, wl.UINT8_ROWWISE])
@pytest.mark.parametrize("mode", [wl.SUM, wl.MEAN])
@pytest.mark.parametrize("idx32", [False, True])
def test_weights_gradient_matches_the_oracle(dtype, mode, idx32):
    rng = np.random.default_rng(11 * dtype + 3 * mode + idx32)
    # row widths of 1, 16 and 64 vectors (two column tiles of 32 lanes), a ragged 5, and 2 and 4 (groups
    # of fewer lanes than the eight rows of a batch)
    D = {wl.F32: [4, 64, 256, 20, 8, 16], wl.F16: [8, 128, 512, 40, 16, 32],
         wl.BF16: [8, 128, 512, 40, 16, 32]}.get(dtype, [16, 128, 1024, 48, 32, 64])
    rows = [37, 1000, 211, 64, 150, 90]
    B = 97
    lengths, off, idx = _jagged(rng, rows, B, 23)
    idx[::41] = -2                                           # skipped, counted, gradient 0
    idx[5::53] = 10 ** 6
    off[-1] += 5                                             # the last bag reaches past the id list: malformed
    tabs, vals = _tables(rng, dtype, rows, D)
    G = rng.standard_normal((B, sum(D))).astype(np.float32)
    ref = bo.backward_weights(vals, G, idx, off, B, mode)
    tbe = eb.TBE(rows, D, dtype, device=torch.cuda.current_device())
    try:
        dev = _device_tables(dtype, tabs)
        d_idx = torch.from_numpy(idx.astype(np.int32) if idx32 else idx).cuda()
        d_off, d_G = torch.from_numpy(off).cuda(), torch.from_numpy(G).cuda()
        got = tbe.backward_weights(dev, d_G, d_idx, d_off, B, mode)
        status = tbe.last_status()
        again = tbe.backward_weights(dev, d_G, d_idx, d_off, B, mode)
        tbe.last_status()
    finally:
        tbe.close()
    if idx32:       # 10**6 fits in 32 bits and is still outside every table
        assert (idx.astype(np.int32) == idx).all()
    assert status[1:] == (ref["n_oob"], ref["n_bad_offsets"]) and ref["n_oob"] > 0 and ref["n_bad_offsets"] >= 1
    assert torch.equal(got, again), "two runs differ"
    g = got.cpu().numpy().astype(np.float64)
    # the bar per lookup, by the width of its table
    width = np.zeros(idx.size)
    for t in range(len(rows)):
        width[off[t * B]:max(off[t * B], off[(t + 1) * B])] = D[t]
    err = np.abs(g - ref["grad_w"])
    assert np.all(err <= (width + 4) * U * ref["S"] + 1e-30)
    assert np.all(g[ref["S"] == 0] == 0.0)


@pytest.mark.parametrize("dtype", [wl.F32, wl.INT8_ROWWISE])
def test_weights_gradient_with_a_table_without_rows(dtype):
    # every id that names the empty table is skipped and counted and gets the gradient 0
    rng = np.random.default_rng(77 + dtype)
    rows, D, B = [40, 0, 9], [32, 64, 16], 31
    lengths = rng.integers(0, 14, size=3 * B)
    off = np.zeros(3 * B + 1, np.int64)
    np.cumsum(lengths, out=off[1:])
    idx = np.concatenate([rng.integers(0, max(rows[t], 3), size=int(lengths[t * B:(t + 1) * B].sum()))
                          for t in range(3)]).astype(np.int64)
    tabs, vals = _tables(rng, dtype, rows, D)
    G = rng.standard_normal((B, sum(D))).astype(np.float32)
    ref = bo.backward_weights(vals, G, idx, off, B, wl.SUM)
    tbe = eb.TBE(rows, D, dtype, device=torch.cuda.current_device())
    try:
        got = tbe.backward_weights(_device_tables(dtype, tabs), torch.from_numpy(G).cuda(),
                                   torch.from_numpy(idx).cuda(), torch.from_numpy(off).cuda(), B, wl.SUM)
        status = tbe.last_status()
    finally:
        tbe.close()
    n1 = int(off[2 * B] - off[B])
    assert n1 > 0 and ref["n_oob"] == n1 and status[1:] == (n1, 0)
    g = got.cpu().numpy().astype(np.float64)
    assert np.all(g[off[B]:off[2 * B]] == 0.0)
    width = np.concatenate([np.full(int(off[(t + 1) * B] - off[t * B]), D[t]) for t in range(3)])
    assert np.all(np.abs(g - ref["grad_w"]) <= (width + 4) * U * ref["S"] + 1e-30)


def test_weights_gradient_at_a_workload_shape():
    # workload 4's shape scaled down (fp32, 1 KB rows: two column tiles), checked against the oracle
    w = wl.make_workload(4, scale_rows=0.002, scale_B=1 / 256, max_tables=3)
    jag = wl.gen_jagged(w)
    tables = wl.gen_tables(w, "cpu")
    rng = np.random.default_rng(5)
    G = rng.standard_normal((w.B, w.sumD)).astype(np.float32)
    ref = bo.backward_weights([t.numpy() for t in tables], G, jag.indices, jag.offsets, w.B, w.mode)
    tbe = eb.TBE(w.rows, w.D, w.dtype, device=torch.cuda.current_device())
    try:
        got = tbe.backward_weights([t.cuda() for t in tables], torch.from_numpy(G).cuda(),
                                   torch.from_numpy(jag.indices).cuda(), torch.from_numpy(jag.offsets).cuda(),
                                   w.B, w.mode)
        assert tbe.last_status() == (0, 0, 0)
    finally:
        tbe.close()
    err = np.abs(got.cpu().numpy().astype(np.float64) - ref["grad_w"])
    assert np.all(err <= (w.D[0] + 4) * U * ref["S"])
