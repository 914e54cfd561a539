"""GPU parity of Batch Event Truncate (paper Sec. 5.5) against the CPU oracle: integer and index
work, bit-exact.  Covers the paper's worked example, its measured shapes (1-32 features, 200
events, lengths up to 100/200), no-op truncation, N = 0, empty users and ragged sizes."""
import numpy as np
import pytest
import torch

import paper_2512_23236_b200 as eb
from golden_io import read_fixture
from oracle import bet_oracle as bo

pytestmark = pytest.mark.gpu


def _gpu(outer, inner_list, values_list, N):
    F = len(inner_list)
    E = int(np.sum(outer))
    inner = np.stack(inner_list).astype(np.int64) if E or F else np.zeros((F, 0), np.int64)
    voff = np.zeros(F + 1, np.int64)
    np.cumsum([v.shape[0] for v in values_list], out=voff[1:])
    values = np.concatenate(values_list + [np.zeros(0, np.int64)]).astype(np.int64)
    t = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
    oo, io, vo, counts = eb.ebag_batch_event_truncate(t(np.asarray(outer, np.int64)), t(inner.reshape(F, E)),
                                                      t(values) if values.size else torch.zeros(1, dtype=torch.int64, device="cuda"),
                                                      t(voff), N)
    counts = counts.cpu().numpy()
    io, vo = io.cpu().numpy(), vo.cpu().numpy()
    inner_out = [io[f, :counts[0]] for f in range(F)]
    values_out = [vo[voff[f]:voff[f] + counts[1 + f]] for f in range(F)]
    return oo.cpu().numpy(), inner_out, values_out


def _check(outer, inner, values, N):
    got = _gpu(outer, inner, values, N)
    want = bo.truncate(outer, inner, values, N)
    assert np.array_equal(got[0], want[0])
    for f in range(len(inner)):
        assert np.array_equal(got[1][f], want[1][f]), f
        assert np.array_equal(got[2][f], want[2][f]), f


def test_paper_worked_example_on_gpu():
    fx = read_fixture("bet_example.txt")
    i64 = lambda k: fx[k].astype(np.int64)
    got = _gpu(i64("outer"), [i64("inner0"), i64("inner1")], [i64("values0"), i64("values1")], 2)
    assert np.array_equal(got[0], i64("outer_out"))
    assert np.array_equal(got[1][0], i64("inner0_out")) and np.array_equal(got[2][0], i64("values0_out"))
    assert np.array_equal(got[1][1], i64("inner1_out")) and np.array_equal(got[2][1], i64("values1_out"))


@pytest.mark.parametrize("U,F,max_events,max_attr,N", [
    (3, 1, 5, 3, 2), (64, 1, 200, 12, 100), (64, 5, 200, 12, 100), (40, 9, 200, 6, 200),
    (33, 32, 50, 5, 20), (1500, 3, 9, 4, 3), (2049, 2, 3, 2, 1), (10, 2, 4, 3, 0), (7, 3, 6, 0, 2),
    # more users than one scan tile of 4096 holds: the tiles' prefixes come from separate CTAs
    (4097, 2, 4, 3, 2), (9000, 3, 6, 3, 2), (20001, 1, 3, 2, 1), (40000, 2, 60, 2, 25),
    (32768, 2, 200, 4, 100)])                      # the benchmark's users, events and N (two of its nine features)
def test_matches_oracle_bit_for_bit(U, F, max_events, max_attr, N):
    rng = np.random.default_rng(U * 31 + F)
    outer = rng.integers(0, max_events + 1, size=U)
    outer[rng.random(U) < 0.1] = 0                       # users without events
    E = int(outer.sum())
    inner = [rng.integers(0, max_attr + 1, size=E) for _ in range(F)]
    values = [rng.integers(-10 ** 12, 10 ** 12, size=int(i.sum())).astype(np.int64) for i in inner]
    _check(outer, inner, values, N)


def test_degenerate_inputs_and_arguments():
    _check(np.zeros(5, np.int64), [np.zeros(0, np.int64)], [np.zeros(0, np.int64)], 3)   # no events at all
    assert eb.lib().ebag_bet_workspace_bytes(2, 3) == 8 * (2 * 4 + 2 * 6 + 2 * 8)
    assert eb.lib().ebag_bet_workspace_bytes(-1, 3) == -1
    st = eb.lib().ebag_batch_event_truncate(None, 4, None, 0, None, None, 1, 2, None, None, None, None, None, 0, None)
    assert st == eb.EBAG_ERR_INVALID_ARG
