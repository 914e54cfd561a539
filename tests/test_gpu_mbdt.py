"""GPU parity of the MBDT transform (paper Sec. 5.4.2) against the CPU oracle: integer output,
bit-exact.  Covers the paper's worked example and its measured shapes (Batch x Features x Borders
from 64 x 2 x 2 to 2048 x 2 x 4), ties, special values, empty and long border lists."""
import numpy as np
import pytest
import torch

import paper_2512_23236_b200 as eb
from golden_io import read_fixture
from oracle import mbdt_oracle as mb

pytestmark = pytest.mark.gpu


def _gpu(values, borders):
    flat, boff = mb.flatten_borders(borders)
    ooff = mb.bin_offsets(borders)
    out = eb.ebag_mbdt(torch.from_numpy(np.ascontiguousarray(values, dtype=np.float32)).cuda(),
                       torch.from_numpy(flat).cuda() if flat.size else torch.zeros(1, device="cuda"),
                       torch.from_numpy(boff).cuda(), torch.from_numpy(ooff).cuda())
    return out.cpu().numpy(), ooff


def test_paper_worked_example_on_gpu():
    fx = read_fixture("mbdt_example.txt")
    values = np.stack([fx["values0"], fx["values1"]]).astype(np.float32)
    borders = [fx["borders0"].astype(np.float32), fx["borders1"].astype(np.float32)]
    got, _ = _gpu(values, borders)
    assert np.array_equal(got, np.stack([fx["output0"], fx["output1"]]).astype(np.int64))


@pytest.mark.parametrize("B,F,K", [(64, 2, 2), (256, 2, 3), (2048, 2, 4), (1000, 7, 10), (5000, 3, 64),
                                   (5000, 3, 65), (33333, 5, 1000), (10, 4, 0),
                                   (1 << 20, 3, 10), ((1 << 20) + 2, 2, 10)])   # the benchmark's batch; the same, not a multiple of 4
def test_matches_oracle_bit_for_bit(B, F, K):
    rng = np.random.default_rng(B + F + K)
    borders = [np.sort(rng.standard_normal(K + (f % 2 if K else 0))).astype(np.float32) for f in range(F)]
    values = rng.standard_normal((F, B)).astype(np.float32)
    for f in range(F):                                   # ties, infinities, NaN
        if borders[f].size:
            values[f, ::5] = borders[f][rng.integers(0, borders[f].size, size=values[f, ::5].shape[0])]
        values[f, :3] = [np.inf, -np.inf, np.nan]
    got, ooff = _gpu(values, borders)
    assert np.array_equal(got, mb.mbdt_fast(values, borders, ooff))
    if B * F <= 20000:
        assert np.array_equal(got, mb.mbdt(values, borders, ooff))


def test_degenerate_sizes_and_arguments():
    off = torch.zeros(2, dtype=torch.int64, device="cuda")
    v = torch.zeros((1, 0), device="cuda")
    assert eb.ebag_mbdt(v, torch.zeros(1, device="cuda"), off, off[:1]).shape == (1, 0)
    assert eb.lib().ebag_mbdt(None, 1, 5, None, None, None, None, None) == eb.EBAG_ERR_INVALID_ARG
    assert eb.lib().ebag_mbdt(None, -1, 5, None, None, None, None, None) == eb.EBAG_ERR_INVALID_ARG
