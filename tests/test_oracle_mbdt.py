"""Pins for the MBDT oracle: the paper's printed example, brute force, ties, special values."""
import numpy as np
import pytest

from golden_io import read_fixture
from oracle import mbdt_oracle as mb


def test_paper_worked_example():
    fx = read_fixture("mbdt_example.txt")
    values = np.stack([fx["values0"], fx["values1"]]).astype(np.float32)
    borders = [fx["borders0"].astype(np.float32), fx["borders1"].astype(np.float32)]
    got = mb.mbdt(values, borders, fx["offsets"].astype(np.int64))
    assert np.array_equal(got, np.stack([fx["output0"], fx["output1"]]).astype(np.int64))
    assert np.array_equal(mb.bin_offsets(borders), fx["offsets"].astype(np.int64))
    flat, off = mb.flatten_borders(borders)
    assert np.array_equal(off, [0, 2, 4]) and flat.shape == (4,)


@pytest.mark.parametrize("seed", range(4))
def test_brute_force_count_of_borders_below(seed):
    rng = np.random.default_rng(seed)
    F, B = 5, 200
    borders = [np.sort(rng.standard_normal(int(rng.integers(0, 12)))).astype(np.float32) for _ in range(F)]
    values = rng.standard_normal((F, B)).astype(np.float32)
    values[:, ::7] = np.array([b[0] if b.size else 0.0 for b in borders], np.float32)[:, None]   # ties
    offs = mb.bin_offsets(borders)
    want = np.array([[sum(1 for x in borders[f] if x < values[f, i]) + offs[f] for i in range(B)]
                     for f in range(F)], dtype=np.int64)
    assert np.array_equal(mb.mbdt(values, borders, offs), want)
    assert np.array_equal(mb.mbdt_fast(values, borders, offs), want)


def test_ties_go_left_and_special_values():
    b = [np.array([0.3, 0.6], np.float32)]
    v = np.array([[0.3, 0.6, np.nextafter(np.float32(0.3), np.float32(1)), -np.inf, np.inf, np.nan]], np.float32)
    got = mb.mbdt(v, b, np.array([10]))
    assert np.array_equal(got, [[10, 11, 11, 10, 12, 12]])      # tie -> left bin; NaN -> last bin
    # no borders: one bin
    assert np.array_equal(mb.mbdt(np.array([[1.0, -2.0]], np.float32), [np.zeros(0, np.float32)], np.array([7])), [[7, 7]])
    with pytest.raises(ValueError):
        mb.mbdt(np.zeros((1, 1), np.float32), [np.array([2.0, 1.0], np.float32)], np.array([0]))
