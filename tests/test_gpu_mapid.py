"""GPU parity of the MapId transform (paper Sec. 5.4.1) and of the pooled forward with MapId
fused into the id fetch, against the CPU oracle.  Integer work: bit-exact."""
import numpy as np
import pytest
import torch

import paper_2512_23236_b200 as eb
from golden_io import read_fixture
from oracle import ebag_oracle as orc
from oracle import mapid_oracle as mo
from paper_2512_23236_b200 import workloads as wl

import parity_util as pu

pytestmark = pytest.mark.gpu


def _gpu_mapid(values, mapping):
    v = torch.from_numpy(np.ascontiguousarray(values, dtype=np.int64)).cuda()
    m = torch.from_numpy(np.ascontiguousarray(mapping, dtype=np.int64)).cuda()
    return eb.ebag_mapid(v, m).cpu().numpy()


def test_paper_worked_example_on_gpu():
    fx = read_fixture("mapid_example.txt")
    got = _gpu_mapid(fx["values"].astype(np.int64), fx["mapping"].astype(np.int64))
    assert np.array_equal(got, fx["output"].astype(np.int64))


@pytest.mark.parametrize("m,n", [(1, 1000), (2, 1000), (5, 77), (100, 10_000), (10_000, 50_000),
                                 (1_048_576, 300_000), (1_000_003, 300_001)])
def test_mapid_matches_oracle_bit_for_bit(m, n):
    """Includes the paper's shapes (unique ids x batch = 100 x 10000 ... 10000 x 50000), a full
    2^20-entry mapping, odd sizes, members, non-members, below-range and above-range values."""
    rng = np.random.default_rng(m + n)
    mapping = np.sort(rng.choice(np.arange(-2 * m, 4 * m + 10, dtype=np.int64), size=m, replace=False))
    values = rng.integers(-3 * m - 5, 5 * m + 20, size=n).astype(np.int64)
    values[::3] = mapping[rng.integers(0, m, size=values[::3].shape[0])]      # plenty of members
    values[:2] = [np.iinfo(np.int64).min, np.iinfo(np.int64).max]
    assert np.array_equal(_gpu_mapid(values, mapping), mo.mapid(values, mapping))


def test_mapid_degenerate_sizes():
    assert _gpu_mapid(np.zeros(0, np.int64), np.array([1, 2, 3])).shape == (0,)
    v = torch.tensor([5, 6, 7], dtype=torch.int64, device="cuda")
    empty = torch.zeros(0, dtype=torch.int64, device="cuda")
    assert torch.equal(eb.ebag_mapid(v, empty).cpu(), torch.zeros(3, dtype=torch.int64))


@pytest.mark.parametrize("dtype", [wl.F32, wl.BF16, wl.INT8_ROWWISE])
@pytest.mark.parametrize("mode,weighted", [(wl.SUM, False), (wl.MEAN, False), (wl.SUM, True)])
@pytest.mark.parametrize("path", ["fused", "fused_hash", "hash", "search"])
def test_fused_mapid_forward(dtype, mode, weighted, path):
    rng = np.random.default_rng(31 + dtype)
    T, B = 5, 300
    Ds = {wl.F32: [64, 8, 256, 132, 32], wl.BF16: [64, 128, 256, 8, 1032],
          wl.INT8_ROWWISE: [128, 16, 512, 48, 1040]}[dtype]
    mlens = [1000, 1, 37, 5000, 64]
    mappings = [np.sort(rng.choice(np.arange(0, 20 * m + 50, dtype=np.int64), size=m, replace=False))
                for m in mlens]
    rows = [m + 1 for m in mlens]
    lengths = np.concatenate([rng.integers(0, 80, size=B) for _ in range(T)])
    offsets = np.zeros(T * B + 1, np.int64)
    np.cumsum(lengths, out=offsets[1:])
    vals = []
    for t in range(T):
        n = int(offsets[(t + 1) * B] - offsets[t * B])
        v = rng.integers(-10, 20 * mlens[t] + 100, size=n).astype(np.int64)          # mostly unknown
        hit = rng.random(n) < 0.7
        v[hit] = mappings[t][rng.integers(0, mlens[t], size=int(hit.sum()))]         # mostly known
        vals.append(v)
    values = np.concatenate(vals)
    w = rng.random(values.shape[0]).astype(np.float32) if weighted else None
    tabs = []
    for r, d in zip(rows, Ds):
        if dtype == wl.INT8_ROWWISE:
            tabs.append((torch.from_numpy(rng.integers(-128, 128, size=(r, d)).astype(np.int8)),
                         torch.from_numpy(rng.uniform(0.01, 0.03, r).astype(np.float32)),
                         torch.from_numpy(rng.normal(0, 0.1, r).astype(np.float32))))
        else:
            x = torch.from_numpy(rng.standard_normal((r, d)).astype(np.float32))
            tabs.append(x.to(torch.bfloat16) if dtype == wl.BF16 else x)
    dev = pu.device_tables(dtype, tabs)
    dmaps = [torch.from_numpy(m).cuda() for m in mappings]
    tbe = eb.TBE(rows, Ds, dtype, device=torch.cuda.current_device())
    # fused: search inside the forward kernel; else the transform runs first, through hash tables
    # of the mappings (this call has more values than those tables have slots) or by binary search
    tbe.set_param("mapid_fused", int(path.startswith("fused")))
    tbe.set_param("mapid_hash", int(path.endswith("hash")))
    before = tbe.launch_count()
    out = torch.full((B, sum(Ds)), float("nan"), dtype=torch.float32, device="cuda")
    tbe.forward_mapid(dev, torch.from_numpy(values).cuda(), torch.from_numpy(offsets).cuda(), dmaps, B,
                      mode, None if w is None else torch.from_numpy(w).cuda(), out=out)
    assert tbe.last_status() == (0, 0, 0)
    assert tbe.launch_count() - before == {"fused": 2, "fused_hash": 3, "hash": 4, "search": 3}[path]   # the forward itself is two launches
    # the fused call equals MapId followed by the plain forward, bit for bit
    ids = torch.cat([eb.ebag_mapid(torch.from_numpy(vals[t]).cuda(), dmaps[t]) for t in range(T)])
    out2 = tbe.forward(dev, ids, torch.from_numpy(offsets).cuda(), B, mode,
                       None if w is None else torch.from_numpy(w).cuda())
    assert torch.equal(out, out2)
    # ... and so does MapId for all tables in one launch
    ids3 = tbe.mapid(torch.from_numpy(values).cuda(), torch.from_numpy(offsets).cuda(), dmaps, B)
    assert torch.equal(ids3, ids)
    tbe.close()
    ot, sc, bi = pu.oracle_tables(dtype, tabs)
    ref = mo.forward_mapid(ot, dtype, values, offsets, B, mappings, mode, weights=w, scales=sc, biases=bi)
    if dtype in pu.ROWWISE8:            # the floor of the bar for rowwise 8-bit tables, on the mapped ids
        ref["F"] = pu.rowwise8_floor(ot, sc, bi, ids.cpu().numpy(), offsets, B, mode, w)
    pu.compare(out.cpu().numpy(), ref, dtype, lengths, T, B, Ds)


def test_fused_mapid_rejects_bad_arguments_and_counts_rows_beyond_the_table():
    tab = torch.randn(4, 8, device="cuda")                 # 4 rows: room for 3 known ids
    mapping = torch.tensor([10, 20, 30, 40, 50], dtype=torch.int64, device="cuda")   # 5 known ids
    vals = torch.tensor([10, 50, 99, 40], dtype=torch.int64, device="cuda")
    off = torch.tensor([0, 4], dtype=torch.int64, device="cuda")
    tbe = eb.TBE([4], [8], eb.EBAG_F32, device=torch.cuda.current_device())
    out = tbe.forward_mapid([tab], vals, off, [mapping], 1)
    # 10 -> row 1, 99 -> row 0; 50 -> row 5 and 40 -> row 4 do not exist: skipped and counted
    assert tbe.last_status() == (eb.EBAG_ERR_INDEX_OOB, 2, 0)
    assert torch.allclose(out[0], tab[1] + tab[0])
    with pytest.raises(eb.EbagError):
        eb.ebag_forward_mapid(tbe._h, [tab.data_ptr()], [8], vals.data_ptr(), 4, off.data_ptr(), None,
                              [mapping.data_ptr()], [-1], 1, 0, out.data_ptr(), 0)
    tbe.close()


@pytest.mark.parametrize("use_hash", [0, 1])
def test_mapid_for_all_tables_with_duplicates_empty_mappings_and_extreme_values(use_hash):
    """Equal keys in a mapping map to the first of their run on both paths; a table without a
    mapping maps everything to 0; the extreme int64 values and 0 are ordinary keys."""
    rng = np.random.default_rng(5 + use_hash)
    B = 64
    lo64, hi64 = np.iinfo(np.int64).min, np.iinfo(np.int64).max
    mappings = [np.array([lo64, -7, -7, -7, 0, 0, 5, 9, 9, hi64], np.int64),
                np.zeros(0, np.int64),
                np.sort(rng.integers(-50_000, 50_000, size=30_000).astype(np.int64)),     # many duplicates
                np.arange(0, 3 * 70_001, 3, dtype=np.int64),
                np.array([42], np.int64)]
    T = len(mappings)
    lengths = rng.integers(0, 6000, size=T * B)     # more values than hash slots: the hash path is taken
    offsets = np.zeros(T * B + 1, np.int64)
    np.cumsum(lengths, out=offsets[1:])
    vals = []
    for t, m in enumerate(mappings):
        n = int(offsets[(t + 1) * B] - offsets[t * B])
        v = rng.integers(-60_000, 220_000, size=n).astype(np.int64)
        if m.size:
            hit = rng.random(n) < 0.5
            v[hit] = m[rng.integers(0, m.size, size=int(hit.sum()))]
        v[:3] = [lo64, hi64, 0]
        vals.append(v)
    values = np.concatenate(vals)
    tbe = eb.TBE([8] * T, [8] * T, eb.EBAG_F32, device=torch.cuda.current_device())
    tbe.set_param("mapid_hash", use_hash)
    before = tbe.launch_count()
    got = tbe.mapid(torch.from_numpy(values).cuda(), torch.from_numpy(offsets).cuda(),
                    [torch.from_numpy(m).cuda() for m in mappings], B).cpu().numpy()
    assert tbe.launch_count() - before == (2 if use_hash else 1)
    tbe.close()
    want = []
    for t, m in enumerate(mappings):
        if m.size and np.all(m[1:] > m[:-1]):
            want.append(mo.mapid(vals[t], m))                 # the oracle's domain: strictly increasing
        else:                                                 # outside it: position of the first equal entry
            first = {}
            for i, key in enumerate(m.tolist()):
                first.setdefault(key, i + 1)
            want.append(np.array([first.get(v, 0) for v in vals[t].tolist()], np.int64))
    assert np.array_equal(got, np.concatenate(want))


@pytest.mark.parametrize("use_hash", [0, 1])
def test_mapid_for_many_small_tables(use_hash):
    """More tables than threads in a CTA (the per-table chunk and hash-table offsets are prefix
    sums taken by the whole CTA), mapping sizes from 0 to a few hundred, some tables without values."""
    rng = np.random.default_rng(77)
    T, B = 700, 24
    mappings = []
    for t in range(T):
        m = int(rng.integers(0, 300)) if t % 7 else 0
        mappings.append(np.sort(rng.choice(np.arange(-1000, 5000, dtype=np.int64), size=m, replace=False)))
    lengths = rng.integers(0, 120, size=T * B)
    lengths[5 * B:9 * B] = 0                                # four tables in a row without values
    offsets = np.zeros(T * B + 1, np.int64)
    np.cumsum(lengths, out=offsets[1:])
    values = rng.integers(-1200, 5200, size=int(offsets[-1])).astype(np.int64)
    tbe = eb.TBE([8] * T, [8] * T, eb.EBAG_F32, device=torch.cuda.current_device())
    tbe.set_param("mapid_hash", use_hash)
    before = tbe.launch_count()
    got = tbe.mapid(torch.from_numpy(values).cuda(), torch.from_numpy(offsets).cuda(),
                    [torch.from_numpy(m).cuda() for m in mappings], B).cpu().numpy()
    assert tbe.launch_count() - before == (2 if use_hash else 1)
    tbe.close()
    for t in range(T):
        lo, hi = int(offsets[t * B]), int(offsets[(t + 1) * B])
        want = mo.mapid(values[lo:hi], mappings[t]) if mappings[t].size else np.zeros(hi - lo, np.int64)
        assert np.array_equal(got[lo:hi], want), t


def test_mapid_with_a_mapping_too_large_for_the_hash_scratch_uses_the_binary_search():
    """Hash tables are capped at 2^24 slots per handle; a mapping of 5 M ids would need 2^25, so
    the call keeps to the binary search (one launch) and still maps every value."""
    rng = np.random.default_rng(123)
    m = 5_000_000
    mapping = np.cumsum(rng.integers(1, 4, size=m)).astype(np.int64)        # strictly increasing
    B = 256
    lengths = rng.integers(0, 400, size=B)
    offsets = np.zeros(B + 1, np.int64)
    np.cumsum(lengths, out=offsets[1:])
    n = int(offsets[-1])
    values = rng.integers(0, int(mapping[-1]) + 10, size=n).astype(np.int64)
    values[::2] = mapping[rng.integers(0, m, size=values[::2].shape[0])]
    tbe = eb.TBE([8], [8], eb.EBAG_F32, device=torch.cuda.current_device())
    before = tbe.launch_count()
    got = tbe.mapid(torch.from_numpy(values).cuda(), torch.from_numpy(offsets).cuda(),
                    [torch.from_numpy(mapping).cuda()], B).cpu().numpy()
    assert tbe.launch_count() - before == 1
    tbe.close()
    assert np.array_equal(got, mo.mapid(values, mapping))
