"""GPU parity: the CUDA library (through its C ABI) against the CPU oracle on the same seeded
inputs.  All tests here need a B200."""
import numpy as np
import pytest
import torch

import paper_2512_23236_b200 as eb
from oracle import ebag_oracle as orc
from paper_2512_23236_b200 import workloads as wl

import parity_util as pu

pytestmark = pytest.mark.gpu


def _jagged_from_lengths(rng, lengths_per_table, rows):
    T = len(lengths_per_table)
    B = len(lengths_per_table[0])
    lengths = np.concatenate([np.asarray(l, dtype=np.int64) for l in lengths_per_table])
    offsets = np.zeros(T * B + 1, dtype=np.int64)
    np.cumsum(lengths, out=offsets[1:])
    idx = np.concatenate([rng.integers(0, rows[t], size=int(np.sum(lengths_per_table[t])))
                          for t in range(T)]).astype(np.int64)
    return idx, offsets, lengths


def _rand_tables(rng, dtype, rows, D, small_ints=False):
    tabs = []
    for r, d in zip(rows, D):
        if dtype in (wl.INT8_ROWWISE, wl.UINT8_ROWWISE):
            if dtype == wl.INT8_ROWWISE:
                q = torch.from_numpy(rng.integers(-128, 128, size=(r, d)).astype(np.int8))
            else:
                q = torch.from_numpy(rng.integers(0, 256, size=(r, d)).astype(np.uint8))
            if small_ints:
                s, b = torch.ones(r), torch.zeros(r)
            else:
                s = torch.from_numpy(rng.uniform(0.01, 0.03, r).astype(np.float32))
                b = torch.from_numpy(rng.normal(0, 0.1, r).astype(np.float32))
            tabs.append((q, s, b))
        else:
            x = rng.integers(-8, 9, size=(r, d)).astype(np.float32) if small_ints \
                else rng.standard_normal((r, d)).astype(np.float32)
            tabs.append(torch.from_numpy(x).to({wl.F32: torch.float32, wl.F16: torch.float16,
                                                wl.BF16: torch.bfloat16}[dtype]))
    return tabs


def _both(dtype, rows, D, tabs, idx, off, B, mode, w=None, params=None, host_path=False):
    dev = pu.device_tables(dtype, tabs)
    gpu, status = pu.run_gpu(dtype, rows, D, dev, idx, off, B, mode, w, params, host_path)
    ot, sc, bi = pu.oracle_tables(dtype, tabs)
    ref = pu.oracle_forward(ot, dtype, idx, off, B, mode, weights=w, scales=sc, biases=bi)
    return gpu, status, ref


# ------------------------------------------------------------------ the five published workloads
def test_cfg1_full_size():
    pu.check_workload(wl.make_workload(1), floor=False)


def test_cfg2_full_size():
    pu.check_workload(wl.make_workload(2), floor=False)


@pytest.mark.parametrize("number,kw", [
    (3, dict(scale_rows=0.01, scale_B=1 / 64)),
    (4, dict(scale_rows=0.01, scale_B=1 / 32)),
    (5, dict(scale_rows=0.01, scale_B=1 / 64)),
])
def test_cfg345_scaled_down_elementwise(number, kw):
    pu.check_workload(wl.make_workload(number, **kw), floor=False)      # the bar exactly as stated


@pytest.mark.parametrize("item_bytes,ctas", [(256, 1), (4096, 0), (1 << 20, 2)])
def test_work_partition_settings_do_not_change_results(item_bytes, ctas):
    w = wl.make_workload(3, scale_rows=0.005, scale_B=1 / 128, max_tables=8)
    pu.check_workload(w, params=dict(item_bytes=item_bytes, ctas_per_sm=ctas))


@pytest.mark.parametrize("chunks", [0, 1, 3, 16])
def test_host_buffer_entry_point(chunks):
    """Host buffers in and out, in one piece and pipelined over ragged ranges of bags."""
    params = dict(host_chunks=chunks) if chunks else None
    pu.check_workload(wl.make_workload(4, scale_rows=0.002, scale_B=1 / 64, max_tables=3),
                      host_path=True, params=params)
    pu.check_workload(wl.make_workload(2, scale_rows=0.05, scale_B=1 / 8), host_path=True,
                      params=params)
    pu.check_workload(wl.make_workload(3, scale_rows=0.004, scale_B=1 / 97, max_tables=5),
                      host_path=True, params=params)


@pytest.mark.parametrize("chunks", [1, 3])
@pytest.mark.parametrize("idx32", [False, True])
@pytest.mark.parametrize("out_dtype", [wl.F32, wl.F16, wl.BF16])
def test_host_buffer_entry_point_with_narrow_ids_and_output(chunks, idx32, out_dtype):
    """Host buffers with 32-bit ids and / or 16-bit output: bit for bit what the device entry point
    gives for the same settings (which the tests above and below hold to the oracle)."""
    w = wl.make_workload(3, scale_rows=0.004, scale_B=1 / 97, max_tables=5)
    jag = wl.gen_jagged(w)
    dev = pu.device_tables(w.dtype, wl.gen_tables(w, "cpu"))
    idx = torch.from_numpy(jag.indices.astype(np.int32) if idx32 else jag.indices)
    off = torch.from_numpy(jag.offsets)
    tbe = eb.TBE(w.rows, w.D, w.dtype, device=torch.cuda.current_device())
    try:
        tbe.set_param("out_dtype", out_dtype)
        tbe.set_param("host_chunks", chunks)
        want = tbe.forward(dev, idx.cuda(), off.cuda(), w.B, w.mode)
        got = tbe.forward_host(dev, idx.pin_memory(), off.pin_memory(), w.B, w.mode)
        assert tbe.last_status() == (0, 0, 0)
    finally:
        tbe.close()
    assert got.dtype == want.dtype and got.dtype == {wl.F32: torch.float32, wl.F16: torch.float16,
                                                     wl.BF16: torch.bfloat16}[out_dtype]
    assert torch.equal(got, want.cpu())


def test_host_buffer_entry_point_with_malformed_offsets_falls_back():
    rng = np.random.default_rng(12)
    rows, D, B = [100, 50], [16, 8], 40
    lens = [rng.integers(1, 10, size=B) for _ in rows]
    idx, off, lengths = _jagged_from_lengths(rng, lens, rows)
    bad = off.copy()
    bad[10] = bad[9] - 1 if bad[9] > 0 else 0
    tabs = _rand_tables(rng, wl.F32, rows, D)
    gpu, status, ref = _both(wl.F32, rows, D, tabs, idx, bad, B, wl.SUM, params=dict(host_chunks=4),
                             host_path=True)
    assert status == (eb.EBAG_ERR_BAD_OFFSETS, ref["n_oob"], ref["n_bad_offsets"])
    pu.compare(gpu, ref, wl.F32)


# ------------------------------------------------------------------ shapes: every row-group path
@pytest.mark.parametrize("dtype,Ds", [
    (wl.F32, [4, 8, 12, 36, 64, 100, 132, 256, 260, 520, 1028]),
    (wl.F16, [8, 24, 64, 128, 264, 520, 1032]),
    (wl.BF16, [8, 16, 72, 256, 512, 1032, 2056]),
    (wl.INT8_ROWWISE, [16, 48, 128, 512, 528, 1040, 2064]),
    (wl.UINT8_ROWWISE, [16, 64, 128, 528, 2064]),
])
@pytest.mark.parametrize("mode,weighted", [(wl.SUM, False), (wl.MEAN, False), (wl.SUM, True),
                                           (wl.MEAN, True)])
def test_all_row_widths(dtype, Ds, mode, weighted):
    rng = np.random.default_rng(42 + dtype)
    T, B = len(Ds), 77                      # ragged tail: 77 is not a multiple of any item size
    rows = [int(rng.integers(5, 400)) for _ in Ds]
    lens = [rng.integers(0, 40, size=B) for _ in Ds]
    for l in lens:
        l[rng.random(B) < 0.15] = 0
    idx, off, lengths = _jagged_from_lengths(rng, lens, rows)
    w = (rng.random(idx.shape[0]).astype(np.float32) - 0.25) if weighted else None
    tabs = _rand_tables(rng, dtype, rows, Ds)
    gpu, status, ref = _both(dtype, rows, Ds, tabs, idx, off, B, mode, w)
    assert status == (0, 0, 0)
    pu.compare(gpu, ref, dtype, lengths, T, B, Ds)


# ------------------------------------------------------------------ 32-bit ids
@pytest.mark.parametrize("dtype,Ds", [(wl.F32, [8, 64, 260]), (wl.BF16, [16, 128, 1032]),
                                      (wl.INT8_ROWWISE, [16, 128, 528])])
@pytest.mark.parametrize("mode,weighted", [(wl.SUM, False), (wl.MEAN, True)])
def test_int32_ids(dtype, Ds, mode, weighted):
    """ebag_forward_i32: parity with the oracle, the same bits as the 64-bit entry point on the
    same ids, and ids outside the table (negative ones too) skipped and counted."""
    rng = np.random.default_rng(77 + dtype)
    T, B = len(Ds), 130
    rows = [int(rng.integers(20, 500)) for _ in Ds]
    lens = [rng.integers(0, 50, size=B) for _ in Ds]
    idx, off, lengths = _jagged_from_lengths(rng, lens, rows)
    bad = rng.choice(idx.shape[0], size=25, replace=False)
    idx[bad[:10]] = -1 - rng.integers(0, 1000, size=10)
    idx[bad[10:]] = 2**31 - 1 - rng.integers(0, 1000, size=15)
    w = (rng.random(idx.shape[0]).astype(np.float32) - 0.25) if weighted else None
    tabs = _rand_tables(rng, dtype, rows, Ds)
    gpu64, st64, ref = _both(dtype, rows, Ds, tabs, idx, off, B, mode, w)
    gpu32, st32, _ = _both(dtype, rows, Ds, tabs, idx.astype(np.int32), off, B, mode, w)
    assert ref["n_oob"] == 25
    assert st32 == st64 == (eb.EBAG_ERR_INDEX_OOB, 25, 0)
    pu.compare(gpu32, ref, dtype)
    assert np.array_equal(gpu32.view(np.uint32), gpu64.view(np.uint32))


# ------------------------------------------------------------------ max pooling
@pytest.mark.parametrize("dtype,Ds", [
    (wl.F32, [4, 12, 64, 260, 1028]),
    (wl.F16, [8, 128, 520]),
    (wl.BF16, [16, 72, 256, 2056]),
    (wl.INT8_ROWWISE, [16, 128, 528, 2064]),
    (wl.UINT8_ROWWISE, [16, 128]),
])
def test_max_pooling_is_bit_exact(dtype, Ds):
    """A maximum involves no rounding, so the GPU must equal the oracle bit for bit, whatever the
    order (rowwise 8-bit: scale*q and +bias are rounded separately on both sides).  Skipped ids
    take no part, bags with no valid lookup are +0, a very long bag is pooled by one warp."""
    rng = np.random.default_rng(61 + dtype)
    T, B = len(Ds), 90
    rows = [int(rng.integers(5, 400)) for _ in Ds]
    lens = [rng.integers(0, 40, size=B) for _ in Ds]
    for l in lens:
        l[rng.random(B) < 0.15] = 0
    lens[0][7] = 3000
    idx, off, lengths = _jagged_from_lengths(rng, lens, rows)
    bad = rng.choice(idx.shape[0], size=40, replace=False)
    idx[bad] = -3
    lens_last = lengths[(T - 1) * B + 4]
    g = (T - 1) * B + 4                                     # one bag made of skipped ids only
    idx[off[g]:off[g + 1]] = 10 ** 9
    tabs = _rand_tables(rng, dtype, rows, Ds)
    for ids in (idx, idx.astype(np.int32)):
        gpu, status, ref = _both(dtype, rows, Ds, tabs, ids, off, B, wl.MAX)
        assert status == (eb.EBAG_ERR_INDEX_OOB, ref["n_oob"], 0) and ref["n_oob"] >= 40
        assert np.array_equal(gpu.view(np.uint32), ref["out32"].view(np.uint32))
    col = sum(Ds[:T - 1])
    assert np.all(gpu[4, col:col + Ds[T - 1]] == 0.0) and lens_last >= 0


def test_max_pooling_argument_rules():
    tbe = eb.TBE([10], [16], eb.EBAG_F32, device=torch.cuda.current_device())
    try:
        tab = torch.zeros(10, 16, device="cuda")
        idx = torch.zeros(4, dtype=torch.int64, device="cuda")
        off = torch.tensor([0, 4], dtype=torch.int64, device="cuda")
        with pytest.raises(eb.EbagError) as e:
            tbe.forward([tab], idx, off, 1, eb.EBAG_MAX, torch.ones(4, device="cuda"))
        assert e.value.status == eb.EBAG_ERR_UNSUPPORTED
        out = tbe.forward([tab - 2.0], idx, off, 1, eb.EBAG_MAX)
        assert tbe.launch_count() == 1 and float(out.max()) == -2.0
    finally:
        tbe.close()


# ------------------------------------------------------------------ 16-bit output
def _round_bf16(x32):
    """fp32 array rounded to nearest-even bf16, returned as fp32."""
    b = x32.astype(np.float32).view(np.uint32).astype(np.uint64)
    b = (b + 0x7FFF + ((b >> 16) & 1)) & 0xFFFF0000
    return b.astype(np.uint32).view(np.float32)


@pytest.mark.parametrize("dtype,Ds", [(wl.F32, [4, 64, 260]), (wl.BF16, [8, 128, 1032]),
                                      (wl.INT8_ROWWISE, [16, 128, 528])])
@pytest.mark.parametrize("out_dtype", [eb.EBAG_F16, eb.EBAG_BF16])
@pytest.mark.parametrize("mode,weighted", [(wl.SUM, False), (wl.MEAN, True)])
def test_sixteen_bit_output(dtype, Ds, out_dtype, mode, weighted):
    """out_dtype fp16 / bf16: fp32 sums rounded once at the store.  The value must lie within the
    usual bar of the oracle plus one rounding of the output type (2^-11 relative for fp16, 2^-8
    for bf16), it must be EXACTLY the rounding of some fp32 value within the bar (checked on the
    integer-valued case below), empty bags are +0, and a long bag takes the parts path."""
    rng = np.random.default_rng(91 + dtype)
    T, B = len(Ds), 70
    rows = [int(rng.integers(20, 400)) for _ in Ds]
    lens = [rng.integers(0, 40, size=B) for _ in Ds]
    lens[0][5] = 2000                                     # pooled in parts
    idx, off, lengths = _jagged_from_lengths(rng, lens, rows)
    w = (rng.random(idx.shape[0]).astype(np.float32) - 0.25) if weighted else None
    tabs = _rand_tables(rng, dtype, rows, Ds)
    dev = pu.device_tables(dtype, tabs)
    ot, sc, bi = pu.oracle_tables(dtype, tabs)
    ref = pu.oracle_forward(ot, dtype, idx, off, B, mode, weights=w, scales=sc, biases=bi)
    tbe = eb.TBE(rows, Ds, dtype, device=torch.cuda.current_device())
    try:
        tbe.set_param("out_dtype", out_dtype)
        out = tbe.forward(dev, torch.from_numpy(idx).cuda(), torch.from_numpy(off).cuda(), B, mode,
                          None if w is None else torch.from_numpy(w).cuda())
        assert out.dtype == (torch.float16 if out_dtype == eb.EBAG_F16 else torch.bfloat16)
        assert tbe.last_status() == (0, 0, 0)
        got = out.float().cpu().numpy().astype(np.float64)
    finally:
        tbe.close()
    rel = 2.0 ** -11 if out_dtype == eb.EBAG_F16 else 2.0 ** -8
    err = np.abs(got - ref["out64"])
    bar = pu.TOL[dtype] * ref["S"] + rel * np.abs(ref["out64"]) + 2.0 ** -24
    assert np.all(err <= bar), f"{(err > bar).sum()} elements beyond the bar"
    col = 0
    for t in range(T):
        empty = lengths[t * B:(t + 1) * B] == 0
        assert np.all(got[:, col:col + Ds[t]][empty] == 0.0)
        col += Ds[t]


@pytest.mark.parametrize("out_dtype", [eb.EBAG_F16, eb.EBAG_BF16])
def test_sixteen_bit_output_rounds_to_nearest_even(out_dtype):
    # integer-valued sums are exact in fp32, so the 16-bit result must be exactly their rounding
    rng = np.random.default_rng(17)
    rows, D, B = [500], [64], 300
    lens = [rng.integers(0, 80, size=B)]
    idx, off, lengths = _jagged_from_lengths(rng, lens, rows)
    tabs = _rand_tables(rng, wl.F32, rows, D, small_ints=True)
    w = np.full(idx.shape[0], 37.0, np.float32)            # sums in the thousands: they need rounding
    ref = orc.forward([wl.raw_numpy(tabs[0])], wl.F32, idx, off, B, wl.SUM, weights=w)
    tbe = eb.TBE(rows, D, wl.F32, device=torch.cuda.current_device())
    try:
        tbe.set_param("out_dtype", out_dtype)
        out = tbe.forward(pu.device_tables(wl.F32, tabs), torch.from_numpy(idx).cuda(),
                          torch.from_numpy(off).cuda(), B, wl.SUM, torch.from_numpy(w).cuda())
        got = out.float().cpu().numpy()
    finally:
        tbe.close()
    want = ref["out32"].astype(np.float16).astype(np.float32) if out_dtype == eb.EBAG_F16 \
        else _round_bf16(ref["out32"])
    assert np.abs(ref["out32"]).max() > 2048               # values that do need rounding occur
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))


# ------------------------------------------------------------------ degenerate and extreme bags
@pytest.mark.parametrize("dtype,D", [(wl.F32, 256), (wl.BF16, 64), (wl.INT8_ROWWISE, 128)])
def test_planted_bag_lengths(dtype, D):
    rng = np.random.default_rng(5)
    lens = [[0, 1, 1023, 1024, 0, 0, 7, 5000, 31, 32, 33, 255, 256, 257, 1, 0, 8, 9, 15, 16, 17]]
    rows = [3000]
    idx, off, lengths = _jagged_from_lengths(rng, lens, rows)
    B = len(lens[0])
    w = rng.random(idx.shape[0]).astype(np.float32)
    tabs = _rand_tables(rng, dtype, rows, [D])
    for mode, ww in ((wl.SUM, None), (wl.MEAN, None), (wl.SUM, w)):
        gpu, status, ref = _both(dtype, rows, [D], tabs, idx, off, B, mode, ww)
        assert status == (0, 0, 0)
        pu.compare(gpu, ref, dtype, lengths, 1, B, [D])


def test_empty_inputs():
    rng = np.random.default_rng(6)
    rows, D = [50, 60], [16, 32]
    tabs = _rand_tables(rng, wl.F32, rows, D)
    dev = pu.device_tables(wl.F32, tabs)
    # B == 0: nothing to do, nothing launched
    gpu, status = pu.run_gpu(wl.F32, rows, D, dev, np.zeros(0, np.int64), np.zeros(1, np.int64), 0, wl.SUM)
    assert gpu.shape == (0, 48) and status == (0, 0, 0)
    # all bags empty, no lookups at all
    B = 100
    gpu, status = pu.run_gpu(wl.F32, rows, D, dev, np.zeros(0, np.int64),
                             np.zeros(2 * B + 1, np.int64), B, wl.MEAN)
    assert status == (0, 0, 0) and np.all(gpu.view(np.uint32) == 0)
    # a table with zero lookups next to one with some
    lens = [np.zeros(B, np.int64), rng.integers(0, 5, size=B)]
    idx, off, lengths = _jagged_from_lengths(rng, lens, rows)
    gpu, status, ref = _both(wl.F32, rows, D, tabs, idx, off, B, wl.SUM)
    pu.compare(gpu, ref, wl.F32, lengths, 2, B, D)


def test_single_bag_single_lookup():
    tabs = [torch.arange(32, dtype=torch.float32).reshape(4, 8)]
    gpu, status, ref = _both(wl.F32, [4], [8], tabs, np.array([2], np.int64),
                             np.array([0, 1], np.int64), 1, wl.SUM)
    assert np.array_equal(gpu, np.arange(16, 24, dtype=np.float32)[None, :])


# ------------------------------------------------------------------ integer-exact cases, bit for bit
@pytest.mark.parametrize("dtype", [wl.F32, wl.F16, wl.BF16, wl.INT8_ROWWISE, wl.UINT8_ROWWISE])
def test_integer_valued_tables_match_bit_for_bit(dtype):
    """Products and partial sums are integers below 2^24, so every summation order gives the same
    fp32 result: the GPU must equal the oracle exactly."""
    rng = np.random.default_rng(7)
    rows, D = [300, 40, 1000], [16, 64, 128]
    B = 200
    lens = [rng.integers(0, 60, size=B) for _ in rows]
    idx, off, lengths = _jagged_from_lengths(rng, lens, rows)
    tabs = _rand_tables(rng, dtype, rows, D, small_ints=True)
    w = rng.integers(-3, 4, size=idx.shape[0]).astype(np.float32)
    for ww in (None, w):
        gpu, status, ref = _both(dtype, rows, D, tabs, idx, off, B, wl.SUM, ww)
        assert status == (0, 0, 0)
        assert np.array_equal(gpu.view(np.uint32), ref["out32"].view(np.uint32))


def test_one_hot_table_counts():
    rng = np.random.default_rng(8)
    rows, B = 64, 300
    lens = [rng.integers(0, 50, size=B)]
    idx, off, lengths = _jagged_from_lengths(rng, lens, [rows])
    tabs = [torch.eye(rows, dtype=torch.float32)]
    gpu, status, ref = _both(wl.F32, [rows], [rows], tabs, idx, off, B, wl.SUM)
    want = np.zeros((B, rows), np.float32)
    for b in range(B):
        np.add.at(want[b], idx[off[b]:off[b + 1]], 1.0)
    assert np.array_equal(gpu, want) and np.array_equal(ref["out32"], want)


# ------------------------------------------------------------------ malformed inputs never fault
def test_out_of_range_ids_skipped_and_counted():
    rng = np.random.default_rng(9)
    rows, D, B = [100, 30], [32, 8], 64
    lens = [rng.integers(1, 20, size=B) for _ in rows]
    idx, off, lengths = _jagged_from_lengths(rng, lens, rows)
    bad = idx.copy()
    planted = rng.choice(idx.shape[0], size=25, replace=False)
    bad[planted[:8]] = -1
    bad[planted[8:16]] = 2 ** 40
    bad[planted[16:]] = 100          # == rows[0]; in range for nothing, out of range for both tables
    tabs = _rand_tables(rng, wl.F32, rows, D)
    for mode in (wl.SUM, wl.MEAN):
        gpu, status, ref = _both(wl.F32, rows, D, tabs, bad, off, B, mode)
        assert ref["n_oob"] == 25
        assert status == (eb.EBAG_ERR_INDEX_OOB, 25, 0)
        pu.compare(gpu, ref, wl.F32, lengths, 2, B, D)


@pytest.mark.parametrize("dtype", [wl.F32, wl.BF16, wl.INT8_ROWWISE])
def test_table_without_rows(dtype):
    """A table of zero rows (it may come without memory): every id that names it is skipped and
    counted, its output columns read +0, and the other tables are pooled as ever."""
    rng = np.random.default_rng(21 + dtype)
    rows, D, B = [50, 0, 20], [32, 64, 16], 37
    lens = [rng.integers(0, 12, size=B) for _ in rows]
    lengths = np.concatenate(lens).astype(np.int64)
    off = np.zeros(3 * B + 1, np.int64)
    np.cumsum(lengths, out=off[1:])
    idx = np.concatenate([rng.integers(0, max(r, 5), size=int(l.sum())) for r, l in zip(rows, lens)]).astype(np.int64)
    tabs = _rand_tables(rng, dtype, rows, D)
    for mode in (wl.SUM, wl.MEAN):
        gpu, status, ref = _both(dtype, rows, D, tabs, idx, off, B, mode)
        n1 = int(lens[1].sum())
        assert n1 > 0 and ref["n_oob"] == n1
        assert status == (eb.EBAG_ERR_INDEX_OOB, n1, 0)
        pu.compare(gpu, ref, dtype, lengths, 3, B, D)
        assert float(np.abs(gpu[:, 32:96]).max()) == 0.0


def test_bad_offsets_treated_as_empty_and_counted():
    rng = np.random.default_rng(10)
    rows, D, B = [100], [16], 40
    lens = [rng.integers(1, 10, size=B)]
    idx, off, lengths = _jagged_from_lengths(rng, lens, rows)
    bad = off.copy()
    bad[10] = bad[9] - 1 if bad[9] > 0 else 0       # bag 9 runs backwards, bag 10 grows
    bad[-1] = idx.shape[0] + 5                      # last bag reaches past the id list
    tabs = _rand_tables(rng, wl.F32, rows, D)
    gpu, status, ref = _both(wl.F32, rows, D, tabs, idx, bad, B, wl.SUM)
    assert ref["n_bad_offsets"] >= 2
    assert status == (eb.EBAG_ERR_BAD_OFFSETS, ref["n_oob"], ref["n_bad_offsets"])
    pu.compare(gpu, ref, wl.F32)


@pytest.mark.parametrize("dtype,D", [(wl.F32, [16, 260]), (wl.BF16, [64, 8]), (wl.INT8_ROWWISE, [128, 16])])
def test_offsets_that_jump_forward_and_come_back(dtype, D):
    """An offset far ahead of its neighbours makes the bag before it reach over later bags (still
    a well-formed bag: it is pooled, overlap and all) and the bag after it run backwards (empty,
    counted).  The bags that follow start BEFORE that offset and are well-formed themselves: they
    must be pooled too, wherever the work items happen to be cut."""
    rng = np.random.default_rng(12 + dtype)
    T, B = len(D), 70
    rows = [150] * T
    lens = [rng.integers(0, 12, size=B) for _ in D]
    idx, off, lengths = _jagged_from_lengths(rng, lens, rows)
    tabs = _rand_tables(rng, dtype, rows, D)
    for g in (1, 7, 32, 33, 64, B + 3, B + 31, 2 * B - 2):          # first bags of items, middles, table ends
        bad = off.copy()
        bad[g] = min(bad[g + 1] + 5, idx.shape[0])
        for params in (None, dict(item_bytes=256)):                   # small items: other cut points
            gpu, status, ref = _both(dtype, rows, D, tabs, idx, bad, B, wl.SUM, params=params)
            assert ref["n_bad_offsets"] == (1 if bad[g] > bad[g + 1] else 0)
            assert status[1:] == (ref["n_oob"], ref["n_bad_offsets"]), (g, params)
            pu.compare(gpu, ref, dtype)


def test_maximum_number_of_tables():
    """EBAG_MAX_TABLES tables in one launch (the item table of the kernel lives in shared memory
    and grows with T); one more table is refused at create time."""
    rng = np.random.default_rng(31)
    T, B = 2048, 5
    Ds = [int(4 * rng.integers(1, 9)) for _ in range(T)]
    rows = [int(rng.integers(1, 30)) for _ in range(T)]
    lens = [rng.integers(0, 6, size=B) for _ in range(T)]
    idx, off, lengths = _jagged_from_lengths(rng, lens, rows)
    tabs = _rand_tables(rng, wl.F32, rows, Ds)
    gpu, status, ref = _both(wl.F32, rows, Ds, tabs, idx, off, B, wl.MEAN)
    assert status == (0, 0, 0)
    pu.compare(gpu, ref, wl.F32, lengths, T, B, Ds)
    with pytest.raises(eb.EbagError) as e:
        eb.TBE([4] * 2049, [4] * 2049, eb.EBAG_F32)
    assert e.value.status == eb.EBAG_ERR_UNSUPPORTED
    tbe = eb.TBE([4] * 2048, [4] * 2048, eb.EBAG_F32)
    try:
        z = torch.zeros(4, 4, device="cuda")
        off = torch.zeros(1, dtype=torch.int64, device="cuda")
        with pytest.raises(eb.EbagError) as e:                 # T * B must stay below 2^31
            eb.ebag_forward(tbe._h, [z.data_ptr()] * 2048, [4] * 2048, None, 0, off.data_ptr(), None,
                            1 << 20, 0, z.data_ptr(), 0)
        assert e.value.status == eb.EBAG_ERR_UNSUPPORTED
    finally:
        tbe.close()


def test_host_side_argument_errors():
    tbe = eb.TBE([10], [16], eb.EBAG_F32, device=torch.cuda.current_device())
    tab = torch.zeros(10, 16, device="cuda")
    idx = torch.zeros(4, dtype=torch.int64, device="cuda")
    off = torch.tensor([0, 4], dtype=torch.int64, device="cuda")
    with pytest.raises(eb.EbagError) as e:
        eb.ebag_forward(tbe._h, [tab.data_ptr()], [32], idx.data_ptr(), 4, off.data_ptr(), None, 1, 0,
                        tab.data_ptr(), 0)
    assert e.value.status == eb.EBAG_ERR_INVALID_ARG          # D differs from create time
    with pytest.raises(eb.EbagError):
        eb.ebag_forward(tbe._h, [tab.data_ptr() + 4], [16], idx.data_ptr(), 4, off.data_ptr(), None,
                        1, 0, tab.data_ptr(), 0)              # misaligned table
    assert tbe.launch_count() == 0
    out = tbe.forward([tab], idx, off, 1)
    assert tbe.launch_count() == 1 and tbe.last_status() == (0, 0, 0)
    tbe.close()
    with pytest.raises(eb.EbagError):
        eb.TBE([10], [6], eb.EBAG_F32)                        # 24-byte rows


def test_repeated_calls_and_changing_table_pointers():
    """The work queue re-arms itself after every launch, and a new table-pointer array is picked
    up even when many different arrays are in flight."""
    rng = np.random.default_rng(11)
    rows, D, B = [200, 300], [64, 32], 128
    lens = [rng.integers(0, 30, size=B) for _ in rows]
    idx, off, lengths = _jagged_from_lengths(rng, lens, rows)
    tbe = eb.TBE(rows, D, eb.EBAG_F32, device=torch.cuda.current_device())
    didx, doff = torch.from_numpy(idx).cuda(), torch.from_numpy(off).cuda()
    outs, refs = [], []
    for k in range(10):
        tabs = _rand_tables(rng, wl.F32, rows, D)
        dev = pu.device_tables(wl.F32, tabs)
        outs.append((tbe.forward(dev, didx, doff, B), dev))
        ot, _, _ = pu.oracle_tables(wl.F32, tabs)
        refs.append(orc.forward(ot, wl.F32, idx, off, B, wl.SUM))
    assert tbe.last_status() == (0, 0, 0) and tbe.launch_count() == 20    # forward + parts kernel each
    for (o, _), r in zip(outs, refs):
        pu.compare(o.cpu().numpy(), r, wl.F32, lengths, 2, B, D)
    tbe.close()


# ------------------------------------------------------------------ output alignment
@pytest.mark.parametrize("dtype,Ds", [(wl.BF16, [8, 64, 136]), (wl.INT8_ROWWISE, [16, 128, 48]),
                                      (wl.F32, [4, 64])])
def test_output_that_is_only_16_byte_aligned(dtype, Ds):
    """16- and 8-bit tables write whole 32-byte sectors with one store where the output allows it;
    an output buffer that starts 16 bytes into a sector must give the same bits through the
    16-byte stores."""
    rng = np.random.default_rng(9 + dtype)
    T, B = len(Ds), 50
    rows = [int(rng.integers(5, 200)) for _ in Ds]
    lens = [rng.integers(0, 30, size=B) for _ in Ds]
    idx, off, lengths = _jagged_from_lengths(rng, lens, rows)
    tabs = _rand_tables(rng, dtype, rows, Ds)
    dev = pu.device_tables(dtype, tabs)
    sumD = sum(Ds)
    d_idx, d_off = torch.from_numpy(idx).cuda(), torch.from_numpy(off).cuda()
    tbe = eb.TBE(rows, Ds, dtype, device=torch.cuda.current_device())
    aligned = torch.full((B, sumD), float("nan"), dtype=torch.float32, device="cuda")
    assert aligned.data_ptr() % 32 == 0
    tbe.forward(dev, d_idx, d_off, B, wl.SUM, None, out=aligned)
    store = torch.full((B * sumD + 8,), float("nan"), dtype=torch.float32, device="cuda")
    shifted = store[4:4 + B * sumD].view(B, sumD)
    assert shifted.data_ptr() % 32 == 16
    tbe.forward(dev, d_idx, d_off, B, wl.SUM, None, out=shifted)
    assert tbe.last_status() == (0, 0, 0)
    tbe.close()
    assert torch.equal(aligned, shifted)
    assert torch.isnan(store[:4]).all() and torch.isnan(store[4 + B * sumD:]).all()   # nothing written outside
    ot, sc, bi = pu.oracle_tables(dtype, tabs)
    ref = pu.oracle_forward(ot, dtype, idx, off, B, wl.SUM, scales=sc, biases=bi)
    pu.compare(aligned.cpu().numpy(), ref, dtype, lengths, T, B, Ds)
