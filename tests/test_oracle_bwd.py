"""Pins for the backward oracle.  CPU only.  The main pin is the adjoint identity against the
forward oracle (which has its own pins): a wrong index, sign, weight or mean divisor in the
backward breaks <forward(T), G> = <T, backward(G)> for random T and G."""
import numpy as np
import pytest

from oracle import ebag_bwd_oracle as bo
from oracle import ebag_oracle as orc


def _problem(rng, T=3, B=17, max_len=9, weighted=True):
    rows = [int(rng.integers(3, 40)) for _ in range(T)]
    D = [int(4 * rng.integers(1, 6)) for _ in range(T)]
    lengths = rng.integers(0, max_len, size=T * B)
    off = np.zeros(T * B + 1, np.int64)
    np.cumsum(lengths, out=off[1:])
    idx = np.concatenate([rng.integers(0, rows[t], size=int(lengths[t * B:(t + 1) * B].sum()))
                          for t in range(T)]).astype(np.int64)
    w = rng.uniform(-2, 2, size=idx.size).astype(np.float32) if weighted else None
    return rows, D, lengths, off, idx, w


@pytest.mark.parametrize("mode", [orc.SUM, orc.MEAN])
@pytest.mark.parametrize("weighted", [False, True])
@pytest.mark.parametrize("seed", range(3))
def test_adjoint_of_the_forward(mode, weighted, seed):
    rng = np.random.default_rng(seed)
    rows, D, lengths, off, idx, w = _problem(rng, weighted=weighted)
    B = 17
    tabs = [rng.standard_normal((r, d)).astype(np.float32) for r, d in zip(rows, D)]
    G = rng.standard_normal((B, sum(D)))
    fwd = orc.forward(tabs, orc.F32, idx, off, B, mode, weights=w)
    bwd = bo.backward(rows, D, G, idx, off, B, mode, weights=w)
    lhs = float((fwd["out64"] * G).sum())
    rhs = float(sum((tab.astype(np.float64) * g).sum() for tab, g in zip(tabs, bwd["grads"])))
    scale = float(sum((np.abs(tab.astype(np.float64)) * s).sum() for tab, s in zip(tabs, bwd["S"])))
    assert abs(lhs - rhs) <= 1e-12 * scale


def test_hand_worked_example():
    # one table of 3 rows x 4, two bags: bag 0 = rows [2, 0, 2] with weights [1, 2, 3],
    # bag 1 = row [1] with weight 5.  grad_out rows g0, g1.
    g0 = np.array([1.0, -1.0, 0.5, 2.0])
    g1 = np.array([4.0, 0.0, -2.0, 1.0])
    idx = np.array([2, 0, 2, 1])
    off = np.array([0, 3, 4])
    w = np.array([1.0, 2.0, 3.0, 5.0], np.float32)
    r = bo.backward([3], [4], np.stack([g0, g1]), idx, off, 2, bo.SUM, weights=w)
    want = np.stack([2 * g0, 5 * g1, (1 + 3) * g0])
    assert np.array_equal(r["grads"][0], want)
    assert np.array_equal(r["counts"][0], [1, 1, 2])
    m = bo.backward([3], [4], np.stack([g0, g1]), idx, off, 2, bo.MEAN, weights=w)
    want_mean = np.stack([2 * g0 / 3, 5 * g1 / 1, (1 + 3) * g0 / 3])
    assert np.allclose(m["grads"][0], want_mean, rtol=1e-15)


def test_closed_forms():
    rows, D, B = [5], [8], 6
    # every lookup on row 3, weight 1, grad_out all ones: the row collects the lookup count
    lengths = np.array([4, 0, 1, 7, 2, 3])
    off = np.zeros(B + 1, np.int64)
    np.cumsum(lengths, out=off[1:])
    idx = np.full(int(off[-1]), 3)
    r = bo.backward(rows, D, np.ones((B, 8)), idx, off, B)
    assert np.all(r["grads"][0][3] == lengths.sum()) and r["grads"][0][[0, 1, 2, 4]].sum() == 0
    # mean mode: every non-empty bag contributes exactly 1
    m = bo.backward(rows, D, np.ones((B, 8)), idx, off, B, bo.MEAN)
    assert np.allclose(m["grads"][0][3], (lengths > 0).sum())
    # one-hot grad_out (bag 3, column 5): only column 5 of the rows bag 3 looks up is touched
    G = np.zeros((B, 8))
    G[3, 5] = 1.0
    idx2 = np.arange(int(off[-1])) % 5
    h = bo.backward(rows, D, G, idx2, off, B)
    want = np.zeros((5, 8))
    for i in range(off[3], off[4]):
        want[idx2[i], 5] += 1
    assert np.array_equal(h["grads"][0], want)


def test_linearity_and_counts():
    rng = np.random.default_rng(9)
    rows, D, lengths, off, idx, w = _problem(rng)
    B = 17
    G1, G2 = rng.standard_normal((2, B, sum(D)))
    a = bo.backward(rows, D, G1, idx, off, B, weights=w)
    b = bo.backward(rows, D, G2, idx, off, B, weights=w)
    c = bo.backward(rows, D, 2 * G1 - 3 * G2, idx, off, B, weights=w)
    for x, y, z in zip(a["grads"], b["grads"], c["grads"]):
        assert np.allclose(z, 2 * x - 3 * y, rtol=1e-12, atol=1e-12)
    assert sum(int(c_.sum()) for c_ in a["counts"]) == idx.size


def test_rejected_ids_and_malformed_bags_match_the_forward():
    rng = np.random.default_rng(4)
    rows, D, lengths, off, idx, w = _problem(rng, weighted=False)
    B = 17
    idx[[1, 5, 9]] = [-3, 10 ** 9, rows[0]]
    off[7] = off[6] - 1                                # bags 6 and 7 of table 0 become malformed
    tabs = [np.zeros((r, d), np.float32) for r, d in zip(rows, D)]
    f = orc.forward(tabs, orc.F32, idx, off, B, orc.SUM)
    r = bo.backward(rows, D, np.ones((B, sum(D))), idx, off, B)
    assert (r["n_oob"], r["n_bad_offsets"]) == (f["n_oob"], f["n_bad_offsets"])


# ------------------------------------------------------------------ gradient of the per-sample weights
@pytest.mark.parametrize("mode", [orc.SUM, orc.MEAN])
@pytest.mark.parametrize("seed", range(4))
def test_weights_gradient_is_the_adjoint_in_the_weights(mode, seed):
    # the forward is linear in w: <forward(w), G> = sum_i w_i * grad_w[i], for any w
    rng = np.random.default_rng(100 + seed)
    rows, D, lengths, off, idx, w = _problem(rng, weighted=True)
    B = 17
    tabs = [rng.standard_normal((r, d)).astype(np.float32) for r, d in zip(rows, D)]
    G = rng.standard_normal((B, sum(D)))
    fwd = orc.forward(tabs, orc.F32, idx, off, B, mode, weights=w)
    gw = bo.backward_weights(tabs, G, idx, off, B, mode)
    lhs = float((fwd["out64"] * G).sum())
    rhs = float((w.astype(np.float64) * gw["grad_w"]).sum())
    scale = float((np.abs(w.astype(np.float64)) * gw["S"]).sum())
    assert abs(lhs - rhs) <= 1e-12 * scale
    # and it does not depend on w at all (linearity): a second w gives the same identity
    w2 = rng.uniform(-3, 3, size=idx.size).astype(np.float32)
    fwd2 = orc.forward(tabs, orc.F32, idx, off, B, mode, weights=w2)
    assert abs(float((fwd2["out64"] * G).sum()) - float((w2.astype(np.float64) * gw["grad_w"]).sum())) <= \
        1e-12 * float((np.abs(w2.astype(np.float64)) * gw["S"]).sum())


def test_weights_gradient_hand_worked_example():
    # table rows r0=[1,-2], r1=[0.5,4], r2=[3,0]; bag 0 = rows [2, 0, 2], bag 1 = row [1];
    # grad_out g0=[1,2], g1=[-1,0.5]
    tab = np.array([[1.0, -2.0], [0.5, 4.0], [3.0, 0.0]])
    G = np.array([[1.0, 2.0], [-1.0, 0.5]])
    idx = np.array([2, 0, 2, 1])
    off = np.array([0, 3, 4])
    r = bo.backward_weights([tab], G, idx, off, 2, bo.SUM)
    assert np.array_equal(r["grad_w"], [3.0, 1.0 - 4.0, 3.0, -0.5 + 2.0])
    assert np.array_equal(r["S"], [3.0, 5.0, 3.0, 2.5])
    m = bo.backward_weights([tab], G, idx, off, 2, bo.MEAN)
    assert np.allclose(m["grad_w"], [1.0, -1.0, 1.0, 1.5], rtol=1e-15)


def test_weights_gradient_closed_forms_and_skips():
    rng = np.random.default_rng(7)
    B, D = 5, [4, 8]
    lengths = rng.integers(0, 6, size=2 * B)
    off = np.zeros(2 * B + 1, np.int64)
    np.cumsum(lengths, out=off[1:])
    idx = rng.integers(0, 6, size=int(off[-1]))
    G = rng.standard_normal((B, 12))
    # all-ones tables: every lookup collects the row sum of its bag's grad_out slice
    r = bo.backward_weights([np.ones((6, 4)), np.ones((6, 8))], G, idx, off, B, bo.SUM)
    for t, (c0, c1) in enumerate([(0, 4), (4, 12)]):
        for b in range(B):
            lo, hi = off[t * B + b], off[t * B + b + 1]
            assert np.allclose(r["grad_w"][lo:hi], G[b, c0:c1].sum(), rtol=1e-14)
    # planted bad ids and a malformed bag: zeros there, counted
    idx2 = idx.copy()
    bad_at = [1, int(off[-1]) - 1]
    idx2[bad_at] = [-3, 6]
    off2 = off.copy()
    off2[3] = off2[2] - 1 if off2[2] > 0 else off2[3]           # bag 2 of table 0 runs backwards (if it can)
    tabs = [rng.standard_normal((6, 4)), rng.standard_normal((6, 8))]
    r2 = bo.backward_weights(tabs, G, idx2, off2, B, bo.SUM)
    assert r2["n_oob"] >= 1 and np.all(r2["grad_w"][bad_at] == 0.0)
    # agreement with the tables' gradient: sum_i w_i grad_w[i] = <T, backward(G)>
    w = rng.uniform(-2, 2, size=idx.size)
    gw = bo.backward_weights(tabs, G, idx, off, B, bo.MEAN)
    gt = bo.backward([6, 6], D, G, idx, off, B, bo.MEAN, weights=w)
    lhs = float((w * gw["grad_w"]).sum())
    rhs = float(sum((tab * g).sum() for tab, g in zip(tabs, gt["grads"])))
    assert abs(lhs - rhs) <= 1e-12 * float((np.abs(w) * gw["S"]).sum())
