"""Host checks of the seeded input generators (CPU only)."""
import numpy as np
import torch

from paper_2512_23236_b200 import workloads as wl


def test_generators_are_deterministic_and_well_formed():
    for n in range(1, 6):
        w = wl.make_workload(n, scale_rows=0.01, scale_B=0.01, max_tables=4)
        a, b = wl.gen_jagged(w), wl.gen_jagged(w)
        assert np.array_equal(a.indices, b.indices) and np.array_equal(a.offsets, b.offsets)
        assert a.offsets[0] == 0 and a.offsets[-1] == a.indices.shape[0]
        assert np.all(np.diff(a.offsets) >= 0) and a.offsets.shape[0] == w.T * w.B + 1
        for t in range(w.T):
            seg = a.indices[a.offsets[t * w.B]:a.offsets[(t + 1) * w.B]]
            assert seg.size == 0 or (seg.min() >= 0 and seg.max() < w.rows[t])
        assert (a.weights is not None) == w.weighted
        if w.weighted:
            assert a.weights.dtype == np.float32 and a.weights.min() >= 0 and a.weights.max() < 1
        t0 = wl.gen_table(w, 0)
        t1 = wl.gen_table(w, 0)
        x0 = t0[0] if isinstance(t0, tuple) else t0
        x1 = t1[0] if isinstance(t1, tuple) else t1
        assert torch.equal(x0, x1) and tuple(x0.shape) == (w.rows[0], w.D[0])


def test_published_shapes():
    w1, w2, w3, w4, w5 = [wl.make_workload(n) for n in range(1, 6)]
    assert (w1.rows, w1.D, w1.B, w1.dtype, w1.mode) == ([10_000], [64], 512, wl.F32, wl.SUM)
    assert (w2.rows, w2.D, w2.B, w2.dtype, w2.mode) == ([1_000_000], [128], 16_384, wl.F16, wl.MEAN)
    assert w3.T == 32 and w3.B == 65_536 and set(w3.D) <= {64, 128, 256} and w3.dtype == wl.BF16
    assert min(w3.rows) >= 100_000 and max(w3.rows) <= 10_000_000
    assert all(1.0 <= m <= 80.0 for m in w3.length_params)
    assert w4.T == 8 and w4.rows[0] == 5_000_000 and w4.D[0] == 256 and w4.weighted
    assert w5.T == 64 and w5.rows[0] == 2_000_000 and w5.dtype == wl.INT8_ROWWISE and w5.B == 131_072


def test_length_and_id_distributions():
    w = wl.make_workload(1)
    j = wl.gen_jagged(w)
    assert j.lengths.min() == 0 and j.lengths.max() == 20
    w = wl.make_workload(4, scale_rows=0.001, max_tables=1)
    j = wl.gen_jagged(w)
    assert j.lengths.min() >= 1 and j.lengths.max() <= 1024 and abs(j.lengths.mean() - 50) < 2
    w = wl.make_workload(2, scale_rows=0.1)
    j = wl.gen_jagged(w)
    assert abs(j.lengths.mean() - 30) < 0.5
    # bounded Zipf(1.05) over 1e5 rows: the hottest id takes 1/H(1e5, 1.05) ~ 11 % of the draws
    top = np.bincount(j.indices).max() / j.indices.shape[0]
    H = (np.arange(1, w.rows[0] + 1, dtype=np.float64) ** -1.05).sum()
    assert abs(top - 1.0 / H) < 0.01


def test_algorithmic_bytes_cfg1():
    w = wl.make_workload(1)
    j = wl.gen_jagged(w)
    ab = wl.algorithmic_bytes(w, j.lengths)
    n = int(j.lengths.sum())
    assert ab["lookups"] == n and ab["gathered"] == n * 256 and ab["indices"] == 8 * n
    assert ab["out"] == 512 * 64 * 4 and ab["offsets"] == 8 * 513 and ab["weights"] == 0


def test_mapid_inputs_round_trip():
    """raw_values() produces raw ids whose 1-based rank in the mapping is the row index."""
    w = wl.make_workload(3, scale_rows=0.001, scale_B=1 / 256, max_tables=3)
    j = wl.gen_jagged(w)
    maps = wl.gen_mappings(w)
    vals = wl.raw_values(w, j, maps)
    for t in range(w.T):
        assert maps[t].shape[0] == w.rows[t] - 1 and np.all(np.diff(maps[t]) > 0)
        lo, hi = j.offsets[t * w.B], j.offsets[(t + 1) * w.B]
        pos = np.searchsorted(maps[t], vals[lo:hi])
        rank = np.where((pos < maps[t].shape[0]) & (maps[t][np.minimum(pos, maps[t].shape[0] - 1)] == vals[lo:hi]), pos + 1, 0)
        assert np.array_equal(rank, j.indices[lo:hi])
