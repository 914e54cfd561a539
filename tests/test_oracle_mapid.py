"""Pins for the MapId oracle: the paper's printed example, brute force, closed forms.  CPU only."""
import numpy as np
import pytest

from golden_io import read_fixture
from oracle import ebag_oracle as orc
from oracle import mapid_oracle as mo


def test_paper_worked_example():
    fx = read_fixture("mapid_example.txt")
    got = mo.mapid(fx["values"].astype(np.int64), fx["mapping"].astype(np.int64))
    assert np.array_equal(got, fx["output"].astype(np.int64))


@pytest.mark.parametrize("seed", range(5))
def test_brute_force_dictionary(seed):
    rng = np.random.default_rng(seed)
    m = int(rng.integers(1, 200))
    mapping = np.sort(rng.choice(np.arange(-500, 500), size=m, replace=False)).astype(np.int64)
    values = rng.integers(-600, 600, size=1000).astype(np.int64)
    rank = {int(v): i + 1 for i, v in enumerate(mapping)}
    want = np.array([rank.get(int(v), 0) for v in values], dtype=np.int64)
    assert np.array_equal(mo.mapid(values, mapping), want)


def test_closed_forms_and_edges():
    mapping = np.array([-7, 0, 3, 2 ** 40, 2 ** 62], dtype=np.int64)
    assert np.array_equal(mo.mapid(mapping, mapping), np.arange(1, 6))          # members -> rank
    outside = np.array([-8, -6, 1, 4, 2 ** 40 - 1, 2 ** 40 + 1, 2 ** 62 + 5, -2 ** 63], np.int64)
    assert np.all(mo.mapid(outside, mapping) == 0)                              # non-members -> 0
    assert np.array_equal(mo.mapid(np.array([5, 5, 4, 6]), np.array([5])), [1, 1, 0, 0])
    assert mo.mapid(np.zeros(0, np.int64), mapping).shape == (0,)
    with pytest.raises(ValueError):
        mo.mapid(np.array([1]), np.zeros(0, np.int64))
    with pytest.raises(ValueError):
        mo.mapid(np.array([1]), np.array([3, 3]))


def test_fused_forward_is_mapid_then_pooling():
    rng = np.random.default_rng(9)
    T, B = 2, 6
    mappings = [np.array([10, 20, 30, 40], np.int64), np.array([7, 8, 100], np.int64)]
    tables = [rng.standard_normal((len(m) + 1, 4)).astype(np.float32) for m in mappings]
    lengths = rng.integers(0, 5, size=T * B)
    offsets = np.zeros(T * B + 1, np.int64)
    np.cumsum(lengths, out=offsets[1:])
    values = np.concatenate([rng.choice([10, 20, 25, 30, 40, 99], size=int(offsets[B])),
                             rng.choice([7, 8, 9, 100], size=int(offsets[-1] - offsets[B]))])
    r = mo.forward_mapid(tables, orc.F32, values, offsets, B, mappings)
    # by hand for one bag: unknown ids pool row 0, known ids their rank
    for t in range(T):
        for b in range(B):
            seg = values[offsets[t * B + b]:offsets[t * B + b + 1]]
            want = np.zeros(4)
            for v in seg:
                hit = np.nonzero(mappings[t] == v)[0]
                want += tables[t][hit[0] + 1 if hit.size else 0].astype(np.float64)
            assert np.allclose(r["out64"][b, 4 * t:4 * t + 4], want, rtol=1e-12, atol=1e-12)
    assert r["n_oob"] == 0
