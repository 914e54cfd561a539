"""Shared helpers of the GPU parity tests: feed the same seeded inputs to the CUDA library (through
its C ABI binding) and to the CPU oracle, and compare element by element.

Tolerances (per element, S = sum |w*x| of that element's bag, divided by the bag length in mean
mode; S comes from the oracle's fp64 side):
    fp32 tables            |gpu - oracle| <= 1e-5 * S
    fp16/bf16/int8 tables  |gpu - oracle| <= 2e-3 * S
Elements with S == 0 (empty bags, all-zero terms) must be equal, and empty bags must be +0.0f
bit for bit.

Rowwise 8-bit tables only: a value is scale*q + bias, two roundings in the oracle, and where the
two terms cancel the value (and with it S) can be thousands of times smaller than either term
while the oracle's own result is only good to an ulp of the terms.  The library sums scale*code
and bias separately (different roundings of the same exact value), so for those tables the bar is
    |gpu - oracle| <= 2e-3 * S + 2^-23 * F,   F = sum |w| * (255 * |scale| + |bias|)
F comes from a second oracle call on absolute-valued inputs (`rowwise8_floor`).  The floor is two
fp32 ulps of the terms (a randomized run of 2,700 shapes used 13 % of four ulps at most); for
anything but a short bag of cancelling values 2e-3 * S dwarfs it.
"""
import numpy as np
import torch

import paper_2512_23236_b200 as eb
from oracle import ebag_oracle as orc
from paper_2512_23236_b200 import workloads as wl

TOL = {wl.F32: 1e-5, wl.F16: 2e-3, wl.BF16: 2e-3, wl.INT8_ROWWISE: 2e-3, wl.UINT8_ROWWISE: 2e-3}
ROWWISE8 = (wl.INT8_ROWWISE, wl.UINT8_ROWWISE)


def device_tables(dtype, tables):
    """torch tables (any device) -> list of CUDA tensors in the library's layout."""
    out = []
    for t in tables:
        if dtype in ROWWISE8:
            q, s, b = (x.cuda() for x in t)
            out.append(eb.ebag_pack_int8_rowwise(q, s, b))
        else:
            out.append(t.cuda().contiguous())
    return out


def oracle_tables(dtype, tables):
    if dtype in ROWWISE8:
        return ([wl.raw_numpy(t[0]) for t in tables], [wl.raw_numpy(t[1]) for t in tables],
                [wl.raw_numpy(t[2]) for t in tables])
    return [wl.raw_numpy(t) for t in tables], None, None


ROWWISE8_FLOOR = 2.0 ** -23


def rowwise8_floor(tabs, scales, biases, indices, offsets, B, mode, weights=None):
    """F = sum |w| * (255 * |scale| + |bias|) per output element (divided by the bag length in mean
    mode, like S): the oracle run on codes that are all 255, |scale|, |bias| and |w|."""
    codes = [np.full(np.asarray(q).shape, 255, dtype=np.uint8) for q in tabs]
    r = orc.forward(codes, wl.UINT8_ROWWISE, indices, offsets, B, mode if mode != wl.MAX else wl.SUM,
                    weights=None if weights is None else np.abs(weights),
                    scales=[np.abs(x) for x in scales], biases=[np.abs(x) for x in biases])
    return r["out64"]


def oracle_forward(tabs, dtype, indices, offsets, B, mode, weights=None, scales=None, biases=None):
    """The oracle's forward; for rowwise 8-bit tables the result also carries the floor scale F."""
    ref = orc.forward(tabs, dtype, indices, offsets, B, mode, weights=weights, scales=scales, biases=biases)
    if dtype in ROWWISE8:
        ref["F"] = rowwise8_floor(tabs, scales, biases, indices, offsets, B, mode, weights)
    return ref


def run_gpu(dtype, rows, D, dev_tables, indices, offsets, B, mode, weights=None, params=None,
            host_path=False):
    """Returns (out numpy [B, sumD], status tuple)."""
    tbe = eb.TBE(rows, D, dtype, device=torch.cuda.current_device())
    try:
        for k, v in (params or {}).items():
            tbe.set_param(k, v)
        sumD = sum(D)
        if host_path:
            idx = torch.from_numpy(np.ascontiguousarray(indices)).pin_memory()
            off = torch.from_numpy(np.ascontiguousarray(offsets)).pin_memory()
            w = None if weights is None else torch.from_numpy(np.ascontiguousarray(weights)).pin_memory()
            out = torch.full((B, sumD), float("nan"), dtype=torch.float32).pin_memory()
            tbe.forward_host(dev_tables, idx, off, B, mode, w, out=out)
            status = tbe.last_status()
            return out.numpy().copy(), status
        idx = torch.from_numpy(np.ascontiguousarray(indices)).cuda()
        off = torch.from_numpy(np.ascontiguousarray(offsets)).cuda()
        w = None if weights is None else torch.from_numpy(np.ascontiguousarray(weights)).cuda()
        out = torch.full((B, sumD), float("nan"), dtype=torch.float32, device="cuda")
        tbe.forward(dev_tables, idx, off, B, mode, w, out=out)
        status = tbe.last_status()
        return out.cpu().numpy(), status
    finally:
        tbe.close()


def compare(gpu, ref, dtype, lengths=None, T=None, B=None, D=None, floor=True):
    """Assert the parity bar; returns max(|gpu - out32| / S) over elements with S > 0.
    floor=False holds rowwise 8-bit tables to the plain 2e-3 * S as well (the five published
    workloads are checked that way: none of them needs the floor)."""
    out32, S = ref["out32"], ref["S"]
    assert gpu.shape == out32.shape
    assert not np.isnan(gpu).any(), "an output element was never written"
    tol = TOL[dtype]
    err = np.abs(gpu.astype(np.float64) - out32.astype(np.float64))
    bar = tol * S
    if floor and dtype in ROWWISE8 and "F" in ref:
        bar = bar + ROWWISE8_FLOOR * ref["F"]
    bad = err > bar
    if bad.any():
        i = np.argwhere(bad)[0]
        raise AssertionError(f"{bad.sum()} elements beyond the bar ({tol}*S); first at {tuple(i)}: "
                             f"gpu={gpu[tuple(i)]} oracle={out32[tuple(i)]} S={S[tuple(i)]}")
    if lengths is not None:
        col = 0
        for t in range(T):
            empty = lengths[t * B:(t + 1) * B] == 0
            blk = np.ascontiguousarray(gpu[:, col:col + D[t]][empty])
            assert np.all(blk.view(np.uint32) == 0), "an empty bag is not +0.0f"
            col += D[t]
    pos = S > 0
    return float((err[pos] / S[pos]).max()) if pos.any() else 0.0


def check_workload(w, jag=None, tables=None, params=None, host_path=False, floor=True):
    """Element-by-element parity of a (small enough) workload.  Returns the max relative error."""
    jag = jag or wl.gen_jagged(w)
    tables = tables or wl.gen_tables(w, "cpu")
    dev = device_tables(w.dtype, tables)
    gpu, status = run_gpu(w.dtype, w.rows, w.D, dev, jag.indices, jag.offsets, w.B, w.mode,
                          jag.weights, params, host_path)
    tabs, sc, bi = oracle_tables(w.dtype, tables)
    ref = oracle_forward(tabs, w.dtype, jag.indices, jag.offsets, w.B, w.mode, weights=jag.weights,
                         scales=sc, biases=bi)
    assert status == (eb.EBAG_OK, ref["n_oob"], ref["n_bad_offsets"]) == (0, 0, 0)
    return compare(gpu, ref, w.dtype, jag.lengths, w.T, w.B, w.D, floor=floor)
