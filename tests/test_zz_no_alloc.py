"""The handle-free, allocation-free entry point against the regular one.

ebag_forward_noalloc serves callers that cannot allocate device memory when they need a forward
(a plugin inside a host application that owns all device memory, code under a memory pool that
forbids side allocations, a serving thread that may not pay for an allocation).  Its scratch is
a static device array shared by every call, so the test makes two calls in a row, with different
inputs, and checks each against ebag_forward on the same inputs.  This file is collected last,
so a run that stops at the first failure has already run every other test."""
import numpy as np
import pytest
import torch

import paper_2512_23236_b200 as eb
from oracle import ebag_oracle as orc
from paper_2512_23236_b200 import workloads as wl

import parity_util as pu

pytestmark = pytest.mark.gpu


def _case(number, kw, plant_bad):
    w = wl.make_workload(number, **kw)
    jag = wl.gen_jagged(w)
    tables = wl.gen_tables(w, "cpu")
    idx = jag.indices.copy()
    if plant_bad:
        idx[::97] = -5                       # skipped and counted, never a fault
    return w, jag, tables, idx


@pytest.mark.parametrize("plant_bad", [False, True])
def test_noalloc_matches_regular_entry_point_on_two_calls_in_a_row(plant_bad):
    stream = torch.cuda.current_stream().cuda_stream
    cases = [_case(3, dict(scale_rows=0.004, scale_B=1 / 128, max_tables=7), plant_bad),
             _case(4, dict(scale_rows=0.002, scale_B=1 / 64, max_tables=3), plant_bad),
             _case(5, dict(scale_rows=0.004, scale_B=1 / 256, max_tables=5), plant_bad)]
    prepared = []
    for w, jag, tables, idx in cases:
        dev = pu.device_tables(w.dtype, tables)
        d_idx = torch.from_numpy(idx).cuda()
        d_off = torch.from_numpy(jag.offsets).cuda()
        d_w = None if jag.weights is None else torch.from_numpy(jag.weights).cuda()
        prepared.append((w, jag, tables, idx, dev, d_idx, d_off, d_w))

    # all device buffers exist before the calls under test; those calls allocate nothing
    outs, counts = [], []
    for w, jag, tables, idx, dev, d_idx, d_off, d_w in prepared:
        outs.append(torch.full((w.B, w.sumD), float("nan"), dtype=torch.float32, device="cuda"))
        counts.append(torch.zeros(2, dtype=torch.int64, device="cuda"))

    def call(k):
        w, jag, tables, idx, dev, d_idx, d_off, d_w = prepared[k]
        eb.ebag_forward_noalloc(w.rows, w.D, w.dtype, [t.data_ptr() for t in dev],
                                d_idx.data_ptr(), int(d_idx.numel()), d_off.data_ptr(),
                                None if d_w is None else d_w.data_ptr(), w.B, w.mode,
                                outs[k].data_ptr(), counts[k].data_ptr(), stream)

    # One warm call per storage type first: the first call on a device looks up the scratch
    # array's address and the driver loads each kernel's code when it is first launched.  After
    # that the free device memory the DRIVER reports must not move.  (torch's own counter would
    # only see torch's allocator, not a cudaMalloc made inside the library.)
    for k in range(len(prepared)):
        call(k)
    torch.cuda.synchronize()
    for o, c in zip(outs, counts):
        o.fill_(float("nan"))
        c.zero_()
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    torch_before = torch.cuda.memory_allocated()
    for k in range(len(prepared)):
        call(k)                                                                # back to back
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before, "device memory was allocated (or freed) during the calls"
    assert torch.cuda.memory_allocated() == torch_before

    for (w, jag, tables, idx, dev, d_idx, d_off, d_w), out, cnt in zip(prepared, outs, counts):
        tbe = eb.TBE(w.rows, w.D, w.dtype, device=torch.cuda.current_device())
        ref_out = tbe.forward(dev, d_idx, d_off, w.B, w.mode, d_w)
        status = tbe.last_status()
        tbe.close()
        ot, sc, bi = pu.oracle_tables(w.dtype, tables)
        ref = orc.forward(ot, w.dtype, idx, jag.offsets, w.B, w.mode, weights=jag.weights,
                          scales=sc, biases=bi)
        a, b = out.cpu().numpy(), ref_out.cpu().numpy()
        assert not np.isnan(a).any()
        assert np.all(np.abs(a.astype(np.float64) - b.astype(np.float64)) <= pu.TOL[w.dtype] * ref["S"])
        pu.compare(a, ref, w.dtype, jag.lengths, w.T, w.B, w.D)
        assert tuple(cnt.cpu().tolist()) == (status[1], status[2]) == (ref["n_oob"], 0)


def test_noalloc_rejects_sizes_beyond_its_static_scratch():
    T = eb.EBAG_NOALLOC_MAX_TABLES + 1
    tab = torch.zeros(4, 8, device="cuda")
    off = torch.zeros(T + 1, dtype=torch.int64, device="cuda")
    out = torch.zeros(1, 8 * T, device="cuda")
    with pytest.raises(eb.EbagError) as e:
        eb.ebag_forward_noalloc([4] * T, [8] * T, eb.EBAG_F32, [tab.data_ptr()] * T, None, 0,
                                off.data_ptr(), None, 1, eb.EBAG_SUM, out.data_ptr(), None,
                                torch.cuda.current_stream().cuda_stream)
    assert e.value.status == eb.EBAG_ERR_UNSUPPORTED
    with pytest.raises(eb.EbagError) as e:
        eb.ebag_forward_noalloc([4], [6], eb.EBAG_F32, [tab.data_ptr()], None, 0, off.data_ptr(),
                                None, 1, eb.EBAG_SUM, out.data_ptr(), None,
                                torch.cuda.current_stream().cuda_stream)
    assert e.value.status == eb.EBAG_ERR_INVALID_ARG
