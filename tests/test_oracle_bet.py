"""Pins for the Batch Event Truncate oracle.  CPU only."""
import numpy as np
import pytest

from golden_io import read_fixture
from oracle import bet_oracle as bo


def _random_batch(rng, U, F, max_events, max_attr):
    outer = rng.integers(0, max_events + 1, size=U)
    E = int(outer.sum())
    inner = [rng.integers(0, max_attr + 1, size=E) for _ in range(F)]
    values = [rng.integers(-1000, 1000, size=int(i.sum())).astype(np.int64) for i in inner]
    return outer, inner, values


def test_paper_worked_example():
    fx = read_fixture("bet_example.txt")
    i64 = lambda k: fx[k].astype(np.int64)
    oo, io, vo = bo.truncate(i64("outer"), [i64("inner0"), i64("inner1")],
                             [i64("values0"), i64("values1")], int(fx["N"][0]))
    assert np.array_equal(oo, i64("outer_out"))
    assert np.array_equal(io[0], i64("inner0_out")) and np.array_equal(vo[0], i64("values0_out"))
    assert np.array_equal(io[1], i64("inner1_out")) and np.array_equal(vo[1], i64("values1_out"))


@pytest.mark.parametrize("seed", range(4))
def test_against_label_formulation_and_invariants(seed):
    rng = np.random.default_rng(seed)
    U, F = 23, 3
    outer, inner, values = _random_batch(rng, U, F, 7, 4)
    N = int(rng.integers(0, 6))
    oo, io, vo = bo.truncate(outer, inner, values, N)
    assert np.array_equal(oo, np.minimum(outer, N))
    # second formulation: label every event with (user, position in user) and every value with its event
    ev_user = np.repeat(np.arange(U), outer)
    ev_pos = np.concatenate([np.arange(n) for n in outer]) if outer.sum() else np.zeros(0, np.int64)
    keep_ev = ev_pos < N
    for f in range(F):
        assert np.array_equal(io[f], inner[f][keep_ev])
        val_event = np.repeat(np.arange(inner[f].shape[0]), inner[f])
        assert np.array_equal(vo[f], values[f][keep_ev[val_event]])
        assert io[f].sum() == vo[f].shape[0] and io[f].shape[0] == oo.sum()
    # N >= every length: identity; N = 0: everything empty
    big = bo.truncate(outer, inner, values, 100)
    assert np.array_equal(big[0], outer) and all(np.array_equal(a, b) for a, b in zip(big[1], inner))
    assert all(np.array_equal(a, b) for a, b in zip(big[2], values))
    zero = bo.truncate(outer, inner, values, 0)
    assert zero[0].sum() == 0 and all(a.size == 0 for a in zero[1]) and all(a.size == 0 for a in zero[2])


def test_rejects_inconsistent_lengths():
    with pytest.raises(ValueError):
        bo.truncate([2], [np.array([1])], [np.array([5])], 1)
    with pytest.raises(ValueError):
        bo.truncate([1], [np.array([2])], [np.array([5])], 1)
