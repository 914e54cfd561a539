"""GPU parity at the published sizes of workloads 3, 4 and 5, in the launch configuration that
bench.py times (default handle parameters, one ebag_forward call over all tables).  The oracle
cannot hold these tables on every host, so it checks sampled bags: per table the longest bag, an
empty one, the first, the last and random ones, against the rows they reference (copied from
the device, renumbered).  Plus properties that hold at any size: nothing was skipped, every
output element was written, empty bags are +0.0f."""
import numpy as np
import pytest
import torch

import paper_2512_23236_b200 as eb
from paper_2512_23236_b200 import workloads as wl

import parity_util as pu

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("number,bags_per_table", [(3, 24), (4, 12), (5, 12)])
def test_full_size_sampled(number, bags_per_table):
    w = wl.make_workload(number)
    need = sum(r * eb.ebag_row_stride(w.dtype, d) for r, d in zip(w.rows, w.D))
    free, _ = torch.cuda.mem_get_info()
    if free < 2.4 * need + (8 << 30):
        pytest.skip("not enough free device memory for the full-size tables")
    jag = wl.gen_jagged(w)
    raw = [wl.gen_table(w, t, "cuda") for t in range(w.T)]
    if w.dtype == wl.INT8_ROWWISE:
        tables = [eb.ebag_pack_int8_rowwise(q, s, b) for q, s, b in raw]
    else:
        tables = raw
    tbe = eb.TBE(w.rows, w.D, w.dtype, device=torch.cuda.current_device())
    idx = torch.from_numpy(jag.indices).cuda()
    off = torch.from_numpy(jag.offsets).cuda()
    wts = None if jag.weights is None else torch.from_numpy(jag.weights).cuda()
    out = torch.full((w.B, w.sumD), float("nan"), dtype=torch.float32, device="cuda")
    tbe.forward(tables, idx, off, w.B, w.mode, wts, out=out)
    assert tbe.last_status() == (0, 0, 0) and tbe.launch_count() == 2     # forward + parts
    tbe.close()
    assert not bool(torch.isnan(out).any()), "an output element was never written"
    # every empty bag is +0.0f, bit for bit, at full size
    col = 0
    lengths = torch.from_numpy(jag.lengths).cuda()
    for t in range(w.T):
        empty = (lengths[t * w.B:(t + 1) * w.B] == 0).nonzero().flatten()
        if empty.numel():
            blk = out.index_select(0, empty)[:, col:col + w.D[t]].contiguous()
            assert int(blk.view(torch.int32).abs().max()) == 0
        col += w.D[t]
    worst = pu.sampled_check(w, jag, raw, out, bags_per_table, seed=number)
    assert worst <= pu.TOL[w.dtype]
