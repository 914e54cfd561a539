"""Pins for the CPU oracle: values fixed by hand, by a library routine, by brute force and by
algebra, so that a dropped term, a wrong sign or index, or a transposed operand fails here.
CPU only."""
import numpy as np
import pytest
import torch

from golden_io import read_fixture
from oracle import ebag_oracle as orc


def _bits(x):
    return np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)


def _f16_bits(a):
    return np.asarray(a, dtype=np.float16).view(np.uint16)


def _bf16_bits(a):
    return torch.tensor(np.asarray(a, dtype=np.float32)).to(torch.bfloat16).view(torch.int16) \
        .numpy().view(np.uint16)


def _random_jagged(rng, T, B, rows, max_len, empty_frac=0.2):
    lengths = rng.integers(0, max_len + 1, size=T * B)
    lengths[rng.random(T * B) < empty_frac] = 0
    offsets = np.zeros(T * B + 1, dtype=np.int64)
    np.cumsum(lengths, out=offsets[1:])
    idx = np.concatenate([rng.integers(0, rows[t], size=int(offsets[(t + 1) * B] - offsets[t * B]))
                          for t in range(T)]).astype(np.int64)
    return idx, offsets, lengths


# ---------------------------------------------------------------- hand-worked examples
def test_worked_example_sum_mean_weighted():
    fx = read_fixture("worked_example.txt")
    table = fx["table"].astype(np.float32)
    idx = fx["indices"].astype(np.int64)
    off = fx["offsets"].astype(np.int64)
    B = off.shape[0] - 1
    r = orc.forward([table], orc.F32, idx, off, B, orc.SUM)
    assert np.array_equal(r["out32"].ravel(), fx["sum"].astype(np.float32))
    assert np.array_equal(r["out64"].ravel(), fx["sum"])
    r = orc.forward([table], orc.F32, idx, off, B, orc.MEAN)
    assert np.array_equal(_bits(r["out32"].ravel()), _bits(fx["mean"].astype(np.float32)))
    r = orc.forward([table], orc.F32, idx, off, B, orc.SUM, weights=fx["weights"])
    assert np.array_equal(r["out32"].ravel(), fx["weighted"].astype(np.float32))
    # S for bag 0, column 0: |1*1| + |0.5*3| + |0.25*3| = 3.25 ; column 1: |1*-2| = 2
    assert r["S"][0, 0] == 3.25 and r["S"][0, 1] == 2.0
    # the same values stored as fp16 / bf16 (all exactly representable) give the same answers
    for dt, conv in ((orc.F16, _f16_bits), (orc.BF16, _bf16_bits)):
        r = orc.forward([conv(table)], dt, idx, off, B, orc.SUM, weights=fx["weights"])
        assert np.array_equal(r["out32"].ravel(), fx["weighted"].astype(np.float32))


def test_int8_rowwise_example():
    fx = read_fixture("int8_rowwise_example.txt")
    q = fx["table"].astype(np.int8)
    idx = fx["indices"].astype(np.int64)
    off = fx["offsets"].astype(np.int64)
    kw = dict(scales=[fx["scale"].astype(np.float32)], biases=[fx["bias"].astype(np.float32)])
    r = orc.forward([q], orc.INT8_ROWWISE, idx, off, 2, orc.SUM, **kw)
    assert np.array_equal(r["out32"].ravel(), fx["sum"].astype(np.float32))
    r = orc.forward([q], orc.INT8_ROWWISE, idx, off, 2, orc.MEAN, **kw)
    assert np.array_equal(r["out32"].ravel(), fx["mean"].astype(np.float32))


# ---------------------------------------------------------------- storage formats
def test_fp16_widening_all_bit_patterns():
    bits = np.arange(65536, dtype=np.uint32).astype(np.uint16).reshape(-1, 1)
    idx = np.arange(65536, dtype=np.int64)
    off = np.arange(65537, dtype=np.int64)
    got = orc.forward([bits], orc.F16, idx, off, 65536, orc.SUM)["out32"].ravel()
    want = bits.ravel().view(np.float16).astype(np.float32)
    nan = np.isnan(want)
    assert np.array_equal(np.isnan(got), nan)
    # 0.0f + 1.0f*x keeps every non-NaN value; -0 becomes +0 through the initial +0.0f
    w = want[~nan].copy()
    w[w == 0] = 0.0
    assert np.array_equal(_bits(got[~nan]), _bits(w))


def test_bf16_widening_all_bit_patterns():
    bits = np.arange(65536, dtype=np.uint32).astype(np.uint16).reshape(-1, 1)
    idx = np.arange(65536, dtype=np.int64)
    off = np.arange(65537, dtype=np.int64)
    got = orc.forward([bits], orc.BF16, idx, off, 65536, orc.SUM)["out32"].ravel()
    want = torch.from_numpy(bits.ravel().view(np.int16).copy()).view(torch.bfloat16).float().numpy()
    nan = np.isnan(want)
    assert np.array_equal(np.isnan(got), nan)
    w = want[~nan].copy()
    w[w == 0] = 0.0
    assert np.array_equal(_bits(got[~nan]), _bits(w))


# ---------------------------------------------------------------- library routine
@pytest.mark.parametrize("dtype", [orc.F32, orc.F16, orc.BF16, orc.INT8_ROWWISE])
@pytest.mark.parametrize("mode,weighted", [(orc.SUM, False), (orc.MEAN, False), (orc.SUM, True)])
def test_against_torch_embedding_bag(dtype, mode, weighted):
    rng = np.random.default_rng(100 + dtype * 10 + mode * 3 + weighted)
    T, B = 3, 37
    rows = [53, 17, 200]
    D = [8, 20, 12]
    idx, off, lengths = _random_jagged(rng, T, B, rows, 9)
    w = rng.random(idx.shape[0]).astype(np.float32) - 0.3 if weighted else None
    tabs, f32, sc, bi = [], [], [], []
    for t in range(T):
        x = rng.standard_normal((rows[t], D[t])).astype(np.float32)
        if dtype == orc.F32:
            tabs.append(x); f32.append(torch.from_numpy(x))
        elif dtype == orc.F16:
            h = x.astype(np.float16)
            tabs.append(h.view(np.uint16)); f32.append(torch.from_numpy(h.astype(np.float32)))
        elif dtype == orc.BF16:
            bt = torch.from_numpy(x).to(torch.bfloat16)
            tabs.append(bt.view(torch.int16).numpy().view(np.uint16)); f32.append(bt.float())
        else:
            q = rng.integers(-128, 128, size=(rows[t], D[t])).astype(np.int8)
            s = rng.uniform(0.01, 0.03, rows[t]).astype(np.float32)
            b = rng.normal(0, 0.1, rows[t]).astype(np.float32)
            tabs.append(q); sc.append(s); bi.append(b)
            deq = torch.from_numpy(s)[:, None] * torch.from_numpy(q).float()
            deq = deq + torch.from_numpy(b)[:, None]
            f32.append(deq)
    r = orc.forward(tabs, dtype, idx, off, B, mode, weights=w, scales=sc or None,
                    biases=bi or None)
    col = 0
    for t in range(T):
        lo, hi = off[t * B], off[(t + 1) * B]
        ref = torch.nn.functional.embedding_bag(
            torch.from_numpy(idx[lo:hi]), f32[t], torch.from_numpy(off[t * B:(t + 1) * B + 1] - lo),
            mode="sum" if mode == orc.SUM else "mean",
            per_sample_weights=None if w is None else torch.from_numpy(w[lo:hi]),
            include_last_offset=True).numpy()
        got = r["out32"][:, col:col + D[t]]
        S = r["S"][:, col:col + D[t]]
        assert np.all(np.abs(got - ref) <= 1e-6 * S + 1e-30), (t, np.abs(got - ref).max())
        # empty bags are zeros in the library routine too
        empty = lengths[t * B:(t + 1) * B] == 0
        assert np.all(ref[empty] == 0) and np.all(_bits(got[empty]) == 0)
        col += D[t]


# ---------------------------------------------------------------- brute force, other formulation
@pytest.mark.parametrize("seed", range(6))
def test_brute_force_dense_one_hot_product(seed):
    rng = np.random.default_rng(seed)
    T = int(rng.integers(1, 4))
    B = int(rng.integers(1, 6))
    rows = [int(rng.integers(1, 8)) for _ in range(T)]
    D = [int(rng.choice([4, 8])) for _ in range(T)]
    idx, off, lengths = _random_jagged(rng, T, B, rows, 4)
    w = rng.standard_normal(idx.shape[0]).astype(np.float32)
    tabs = [rng.standard_normal((rows[t], D[t])).astype(np.float32) for t in range(T)]
    for weights, mode in ((None, orc.SUM), (None, orc.MEAN), (w, orc.SUM)):
        r = orc.forward(tabs, orc.F32, idx, off, B, mode, weights=weights)
        col = 0
        for t in range(T):
            P = np.zeros((B, rows[t]))
            for b in range(B):
                for i in range(off[t * B + b], off[t * B + b + 1]):
                    P[b, idx[i]] += 1.0 if weights is None else float(weights[i])
                if mode == orc.MEAN and lengths[t * B + b] > 0:
                    P[b] /= lengths[t * B + b]
            ref = P @ tabs[t].astype(np.float64)
            got64 = r["out64"][:, col:col + D[t]]
            assert np.allclose(got64, ref, rtol=1e-12, atol=1e-12)
            L = lengths[t * B:(t + 1) * B][:, None]
            assert np.all(np.abs(r["out32"][:, col:col + D[t]] - ref)
                          <= (L + 2) * 2.0 ** -24 * r["S"][:, col:col + D[t]] + 1e-30)
            col += D[t]


# ---------------------------------------------------------------- closed forms (bit-exact)
def test_one_hot_table_gives_multiplicities():
    rng = np.random.default_rng(7)
    rows, B = 33, 40
    idx, off, lengths = _random_jagged(rng, 1, B, [rows], 25)
    eye = np.eye(rows, dtype=np.float32)
    want = np.zeros((B, rows), dtype=np.float32)
    for b in range(B):
        for i in range(off[b], off[b + 1]):
            want[b, idx[i]] += 1
    for dt, tab in ((orc.F32, eye), (orc.F16, _f16_bits(eye)), (orc.BF16, _bf16_bits(eye))):
        got = orc.forward([tab], dt, idx, off, B, orc.SUM)["out32"]
        assert np.array_equal(_bits(got), _bits(want))
    q = np.eye(rows, dtype=np.int8)
    got = orc.forward([q], orc.INT8_ROWWISE, idx, off, B, orc.SUM,
                      scales=[np.ones(rows, np.float32)], biases=[np.zeros(rows, np.float32)])
    assert np.array_equal(_bits(got["out32"]), _bits(want))


def test_row_id_table_gives_sum_of_ids_and_all_ones_gives_weight_sum():
    rng = np.random.default_rng(8)
    rows, B, D = 1000, 64, 5
    idx, off, lengths = _random_jagged(rng, 1, B, [rows], 30)
    tab = np.repeat(np.arange(rows, dtype=np.float32)[:, None], D, axis=1)
    got = orc.forward([tab], orc.F32, idx, off, B, orc.SUM)["out32"]
    want = np.array([idx[off[b]:off[b + 1]].sum() for b in range(B)], dtype=np.float32)
    assert np.array_equal(got, np.repeat(want[:, None], D, axis=1))
    assert np.array_equal(_bits(got[lengths == 0]), np.zeros((int((lengths == 0).sum()), D), np.uint32))
    # all-ones table with dyadic weights: the sum of weights, exactly
    w = (rng.integers(-8, 9, size=idx.shape[0]) / 4.0).astype(np.float32)
    got = orc.forward([np.ones((rows, D), np.float32)], orc.F32, idx, off, B, orc.SUM, weights=w)
    want = np.array([w[off[b]:off[b + 1]].astype(np.float64).sum() for b in range(B)])
    assert np.array_equal(got["out32"].astype(np.float64), np.repeat(want[:, None], D, axis=1))


def test_offsets_end_is_lookup_count_and_mean_times_len_is_sum():
    rng = np.random.default_rng(9)
    T, B = 2, 50
    rows, D = [70, 90], [12, 4]
    idx, off, lengths = _random_jagged(rng, T, B, rows, 40)
    assert off[-1] == idx.shape[0]
    tabs = [rng.standard_normal((rows[t], D[t])).astype(np.float32) for t in range(T)]
    s = orc.forward(tabs, orc.F32, idx, off, B, orc.SUM)
    m = orc.forward(tabs, orc.F32, idx, off, B, orc.MEAN)
    col = 0
    for t in range(T):
        L = lengths[t * B:(t + 1) * B][:, None].astype(np.float64)
        Ls = np.maximum(L, 1)
        a = m["out32"][:, col:col + D[t]].astype(np.float64) * Ls
        b = s["out32"][:, col:col + D[t]].astype(np.float64)
        assert np.all(np.abs(a - b) <= 2.0 ** -23 * np.abs(b))       # one division rounding
        assert np.allclose(m["out64"][:, col:col + D[t]] * Ls, s["out64"][:, col:col + D[t]],
                           rtol=1e-14, atol=0)
        assert np.allclose(m["S"][:, col:col + D[t]] * Ls, s["S"][:, col:col + D[t]], rtol=1e-14)
        col += D[t]


# ---------------------------------------------------------------- structure invariants
def test_linearity_columns_bag_permutation_batching_threads():
    rng = np.random.default_rng(10)
    T, B = 3, 45
    rows, D = [64, 30, 11], [8, 16, 4]
    idx, off, lengths = _random_jagged(rng, T, B, rows, 20)
    w = rng.random(idx.shape[0]).astype(np.float32)
    A = [rng.standard_normal((rows[t], D[t])).astype(np.float32) for t in range(T)]
    Bm = [rng.standard_normal((rows[t], D[t])).astype(np.float32) for t in range(T)]
    fa = orc.forward(A, orc.F32, idx, off, B, orc.SUM, weights=w)
    fb = orc.forward(Bm, orc.F32, idx, off, B, orc.SUM, weights=w)
    C = [(2.0 * a.astype(np.float64) - 0.5 * b.astype(np.float64)).astype(np.float32)
         for a, b in zip(A, Bm)]
    fc = orc.forward(C, orc.F32, idx, off, B, orc.SUM, weights=w)
    lin = 2.0 * fa["out64"] - 0.5 * fb["out64"]
    tolS = 2.0 * fa["S"] + 0.5 * fb["S"]
    assert np.all(np.abs(fc["out64"] - lin) <= 2.0 ** -23 * tolS + 1e-30)

    # 1 thread == all threads, bit for bit
    f1 = orc.forward(A, orc.F32, idx, off, B, orc.SUM, weights=w, nthreads=1)
    assert np.array_equal(_bits(f1["out32"]), _bits(fa["out32"]))
    assert np.array_equal(f1["out64"], fa["out64"])

    # T tables batched == T single-table calls, bit for bit; columns of a table are independent
    col = 0
    for t in range(T):
        lo, hi = off[t * B], off[(t + 1) * B]
        single = orc.forward([A[t]], orc.F32, idx[lo:hi], off[t * B:(t + 1) * B + 1] - lo, B,
                             orc.SUM, weights=w[lo:hi])
        assert np.array_equal(_bits(single["out32"]), _bits(fa["out32"][:, col:col + D[t]]))
        half = orc.forward([np.ascontiguousarray(A[t][:, 1:3])], orc.F32, idx[lo:hi],
                           off[t * B:(t + 1) * B + 1] - lo, B, orc.SUM, weights=w[lo:hi])
        assert np.array_equal(_bits(half["out32"]), _bits(single["out32"][:, 1:3]))
        col += D[t]

    # permuting the bags of a table permutes its output rows, bit for bit
    t = 0
    lo = off[0]
    perm = rng.permutation(B)
    lens = lengths[:B][perm]
    off2 = np.zeros(B + 1, dtype=np.int64)
    np.cumsum(lens, out=off2[1:])
    idx2 = np.concatenate([idx[off[p]:off[p + 1]] for p in perm] + [np.zeros(0, np.int64)])
    w2 = np.concatenate([w[off[p]:off[p + 1]] for p in perm] + [np.zeros(0, np.float32)])
    fp = orc.forward([A[0]], orc.F32, idx2, off2, B, orc.SUM, weights=w2)
    assert np.array_equal(_bits(fp["out32"]), _bits(fa["out32"][perm, :D[0]]))


def test_fp32_path_obeys_sequential_sum_error_bound():
    rng = np.random.default_rng(11)
    B = 16
    rows, D = 5000, 16
    lengths = np.array([0, 1, 2, 3, 17, 64, 255, 256, 257, 1000, 1023, 1024, 5, 9, 33, 700])
    off = np.zeros(B + 1, dtype=np.int64)
    np.cumsum(lengths, out=off[1:])
    idx = rng.integers(0, rows, size=int(off[-1])).astype(np.int64)
    w = rng.random(idx.shape[0]).astype(np.float32)
    tab = rng.standard_normal((rows, D)).astype(np.float32)
    for mode, ww in ((orc.SUM, None), (orc.SUM, w), (orc.MEAN, None)):
        r = orc.forward([tab], orc.F32, idx, off, B, mode, weights=ww)
        bound = (lengths[:, None] + 2) * 2.0 ** -24 * r["S"]
        err = np.abs(r["out32"].astype(np.float64) - r["out64"])
        assert np.all(err <= bound + 1e-300)
        # and it is a genuine fp32 accumulation, not fp64 rounded at the end
        assert err[lengths >= 255].max() > 0


# ---------------------------------------------------------------- malformed inputs
def test_out_of_range_ids_are_skipped_and_counted():
    rng = np.random.default_rng(12)
    rows, B, D = 20, 10, 4
    idx, off, lengths = _random_jagged(rng, 1, B, [rows], 6, empty_frac=0.0)
    tab = rng.standard_normal((rows, D)).astype(np.float32)
    bad = idx.copy()
    planted = [0, 3, idx.shape[0] - 1]
    bad[planted[0]] = -1
    bad[planted[1]] = rows
    bad[planted[2]] = 2 ** 40
    r = orc.forward([tab], orc.F32, bad, off, B, orc.MEAN)
    assert r["n_oob"] == 3 and r["n_bad_offsets"] == 0
    # reference: drop the planted lookups but keep the divisor L
    keep = np.ones(idx.shape[0], bool)
    keep[planted] = False
    w = keep.astype(np.float32)
    ref = orc.forward([tab], orc.F32, idx, off, B, orc.SUM, weights=w)
    L = np.maximum(lengths, 1)[:, None].astype(np.float32)
    assert np.array_equal(_bits(r["out32"]), _bits(ref["out32"] / L))


def test_bad_offsets_make_empty_bags_and_are_counted():
    tab = np.arange(12, dtype=np.float32).reshape(6, 2)
    idx = np.array([0, 1, 2, 3], dtype=np.int64)
    off = np.array([0, 3, 2, 4], dtype=np.int64)        # bag 1 runs backwards
    r = orc.forward([tab], orc.F32, idx, off, 3, orc.SUM)
    assert r["n_bad_offsets"] == 1
    assert np.array_equal(r["out32"], np.array([[6, 9], [0, 0], [10, 12]], np.float32))
    off = np.array([0, 2, 9], dtype=np.int64)           # bag 1 runs past the id list
    r = orc.forward([tab], orc.F32, idx, off, 2, orc.SUM)
    assert r["n_bad_offsets"] == 1 and np.all(r["out32"][1] == 0)


def test_uint8_rowwise_is_scale_times_unsigned_code_plus_bias():
    """UINT8_ROWWISE: value = scale * u + bias with u the unsigned byte.  Pinned against the F32
    path (pinned above) on the dequantised table, where the two must agree bit for bit: scale a
    power of two and bias a small integer make scale*u + bias exact in fp32."""
    rng = np.random.default_rng(33)
    rows, D, B = 40, 16, 25
    u = rng.integers(0, 256, size=(rows, D)).astype(np.uint8)
    scale = (2.0 ** rng.integers(-3, 3, size=rows)).astype(np.float32)
    bias = rng.integers(-5, 6, size=rows).astype(np.float32)
    lengths = rng.integers(0, 7, size=B)
    off = np.zeros(B + 1, np.int64)
    np.cumsum(lengths, out=off[1:])
    idx = rng.integers(0, rows, size=int(off[-1])).astype(np.int64)
    w = rng.integers(-2, 3, size=idx.size).astype(np.float32)
    deq = (scale[:, None] * u.astype(np.float32) + bias[:, None]).astype(np.float32)
    for mode, ww in ((orc.SUM, None), (orc.SUM, w), (orc.MEAN, None)):
        a = orc.forward([u], orc.UINT8_ROWWISE, idx, off, B, mode, weights=ww, scales=[scale], biases=[bias])
        b = orc.forward([deq], orc.F32, idx, off, B, mode, weights=ww)
        assert np.array_equal(a["out32"].view(np.uint32), b["out32"].view(np.uint32))
    # and it differs from reading the same bytes as signed codes
    u_sum = orc.forward([u], orc.UINT8_ROWWISE, idx, off, B, orc.SUM, scales=[scale], biases=[bias])
    s8 = orc.forward([u.view(np.int8)], orc.INT8_ROWWISE, idx, off, B, orc.SUM, scales=[scale], biases=[bias])
    assert not np.array_equal(s8["out32"], u_sum["out32"])


@pytest.mark.parametrize("dtype", [orc.F32, orc.BF16, orc.INT8_ROWWISE])
def test_max_pooling_against_numpy(dtype):
    """MAX: element-wise maximum over the looked-up rows, by brute force with numpy; skipped ids
    take no part, a bag with no valid lookup is +0, weights are refused."""
    rng = np.random.default_rng(55 + dtype)
    rows, D, B = 60, 12, 50
    kw = {}
    if dtype == orc.F32:
        tab = rng.standard_normal((rows, D)).astype(np.float32)
        val = tab
    elif dtype == orc.BF16:
        f = rng.standard_normal((rows, D)).astype(np.float32)
        tab = (f.view(np.uint32) >> 16).astype(np.uint16)
        val = (tab.astype(np.uint32) << 16).view(np.float32)
    else:
        tab = rng.integers(-128, 128, size=(rows, D)).astype(np.int8)
        sc = rng.uniform(0.5, 2.0, rows).astype(np.float32)
        bi = rng.normal(0, 1, rows).astype(np.float32)
        kw = dict(scales=[sc], biases=[bi])
        val = (sc[:, None] * tab.astype(np.float32)).astype(np.float32) + bi[:, None]
    lengths = rng.integers(0, 9, size=B)
    off = np.zeros(B + 1, np.int64)
    np.cumsum(lengths, out=off[1:])
    idx = rng.integers(0, rows, size=int(off[-1])).astype(np.int64)
    idx[rng.random(idx.size) < 0.1] = -1                  # skipped
    r = orc.forward([tab], dtype, idx, off, B, orc.MAX, **kw)
    for b in range(B):
        ids = [i for i in idx[off[b]:off[b + 1]] if 0 <= i < rows]
        want = np.max(val[ids], axis=0) if ids else np.zeros(D, np.float32)
        assert np.array_equal(r["out32"][b], want.astype(np.float32)), b
    with pytest.raises(ValueError):
        orc.forward([tab], dtype, idx, off, B, orc.MAX, weights=np.ones(idx.size, np.float32), **kw)


def test_weighted_mean_divides_the_weighted_sum_by_the_lookup_count():
    """mean with per-sample weights = (sum of w*x) / L, L the number of lookups of the bag (the
    divisor is not the sum of the weights).  Pinned against the weighted sum, which has its own
    pins above, and against a brute-force evaluation in fp64."""
    rng = np.random.default_rng(21)
    rows, D, B = 50, 8, 40
    tab = rng.standard_normal((rows, D)).astype(np.float32)
    lengths = rng.integers(0, 9, size=B)
    off = np.zeros(B + 1, np.int64)
    np.cumsum(lengths, out=off[1:])
    idx = rng.integers(0, rows, size=int(off[-1])).astype(np.int64)
    w = rng.uniform(-2, 2, size=idx.size).astype(np.float32)
    s = orc.forward([tab], orc.F32, idx, off, B, orc.SUM, weights=w)
    m = orc.forward([tab], orc.F32, idx, off, B, orc.MEAN, weights=w)
    for b in range(B):
        L = lengths[b]
        if L == 0:
            assert np.all(m["out32"][b].view(np.uint32) == 0)
            continue
        assert np.array_equal(m["out32"][b], s["out32"][b] / np.float32(L))
        brute = sum(np.float64(w[i]) * tab[idx[i]].astype(np.float64) for i in range(off[b], off[b + 1])) / L
        assert np.allclose(m["out64"][b], brute, rtol=1e-12, atol=1e-12)
        assert np.allclose(m["S"][b], s["S"][b] / L, rtol=1e-12)


def test_rejects_bad_shapes():
    tab = np.zeros((4, 4), np.float32)
    with pytest.raises(ValueError):
        orc.forward([tab], orc.F32, np.zeros(1, np.int64), np.array([0, 1, 1]), 1, orc.SUM)
