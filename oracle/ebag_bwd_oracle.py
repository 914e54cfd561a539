"""CPU oracle for the backward of the pooled embedding-bag forward (the training half the
paper's abstract refers to: "training and inference workloads").

TEST INFRASTRUCTURE ONLY (tests, smoke check, benchmark CPU-baseline leg); the CUDA library
never imports it.

The forward is linear in the tables:
    out[b, Doff[t] + d] = (1/L_g or 1) * sum_{i in bag g = t*B + b} w_i * table_t[indices[i], d]
so the gradient of a scalar loss with respect to table t is the transpose of that map applied
to grad_out = d loss / d out, the definition written out below:
    grad_t[r, d] = sum over bags g of table t, over lookups i of g with indices[i] == r, of
                   w_i * grad_out[b, Doff[t] + d] * (1/L_g in mean mode, else 1)
Ids outside [0, rows_t) contribute nothing and are counted (they still count in L, as in the
forward); malformed bags (end before start, or outside the id list) contribute nothing and are
counted.  Everything is fp64; alongside the gradient the oracle returns
    S_t[r, d]  = the same sum over absolute values (the scale tolerances are relative to)
    n_t[r]     = how many lookups hit row r (the number of terms of each sum)
Plain loops over bags; numpy only for the per-lookup vector arithmetic.

Pins (tests/test_oracle_bwd.py): the adjoint identity <forward(T), G> = <T, backward(G)> against
the separately pinned forward oracle, a hand-worked example, closed forms (all lookups on one
row; one-hot grad_out), linearity in grad_out and the mean/sum relation.

The forward is linear in the per-sample weights as well (the scores of Sec. 2.2's weighted
sparse features), so their gradient is the other transpose, `backward_weights`:
    grad_w[i] = (1/L_g in mean mode, else 1) * sum_d grad_out[b, Doff[t] + d] * value(t, indices[i], d)
for lookup i of bag g = t*B + b; 0 for a skipped id or a malformed bag.  Pins: the adjoint
identity in the weights, <forward(w), G> = <w, backward_weights(G)>, against the forward oracle; a
hand-worked example; the all-ones table (every lookup of a bag collects the bag's grad_out row
sum); agreement with `backward` through sum_i w_i grad_w[i] = <T, backward(G)>.
"""
from __future__ import annotations

import numpy as np

SUM, MEAN = 0, 1


def backward(rows, D, grad_out, indices, offsets, B, mode=SUM, weights=None):
    """rows, D: per-table sizes.  grad_out: [B, sum(D)].  Returns dict(grads=[T arrays f64
    [rows_t, D_t]], S=[...], counts=[T arrays int64 [rows_t]], n_oob, n_bad_offsets)."""
    T = len(rows)
    grad_out = np.asarray(grad_out, dtype=np.float64)
    indices = np.asarray(indices, dtype=np.int64)
    offsets = np.asarray(offsets, dtype=np.int64)
    if offsets.shape[0] != T * B + 1:
        raise ValueError("offsets must hold T*B+1 entries")
    if grad_out.shape != (B, int(sum(D))):
        raise ValueError("grad_out must be [B, sum(D)]")
    if mode not in (SUM, MEAN):
        raise ValueError("mode")
    w = None if weights is None else np.asarray(weights, dtype=np.float64)
    if w is not None and w.shape[0] != indices.shape[0]:
        raise ValueError("weights must pair with indices")
    n = indices.shape[0]
    grads = [np.zeros((rows[t], D[t]), dtype=np.float64) for t in range(T)]
    S = [np.zeros((rows[t], D[t]), dtype=np.float64) for t in range(T)]
    counts = [np.zeros(rows[t], dtype=np.int64) for t in range(T)]
    n_oob = n_bad = 0
    col = 0
    for t in range(T):
        for b in range(B):
            g = t * B + b
            lo, hi = int(offsets[g]), int(offsets[g + 1])
            if lo < 0 or hi < lo or hi > n:
                n_bad += 1
                continue
            L = hi - lo
            if L == 0:
                continue
            go = grad_out[b, col:col + D[t]]
            if mode == MEAN:
                go = go / L
            for i in range(lo, hi):
                r = int(indices[i])
                if r < 0 or r >= rows[t]:
                    n_oob += 1
                    continue
                wi = 1.0 if w is None else w[i]
                grads[t][r] += wi * go
                S[t][r] += np.abs(wi * go)
                counts[t][r] += 1
        col += D[t]
    return dict(grads=grads, S=S, counts=counts, n_oob=n_oob, n_bad_offsets=n_bad)


def backward_weights(tables, grad_out, indices, offsets, B, mode=SUM):
    """tables: T float arrays [rows_t, D_t] holding the VALUES the forward pools (16-bit storage
    widened, rowwise 8-bit codes dequantised as scale * code + bias in fp32, by the caller).
    grad_out: [B, sum(D)].  Returns dict(grad_w f64 [n], S f64 [n] = the same sums over absolute
    values, n_oob, n_bad_offsets)."""
    T = len(tables)
    D = [int(t.shape[1]) for t in tables]
    grad_out = np.asarray(grad_out, dtype=np.float64)
    indices = np.asarray(indices, dtype=np.int64)
    offsets = np.asarray(offsets, dtype=np.int64)
    if offsets.shape[0] != T * B + 1:
        raise ValueError("offsets must hold T*B+1 entries")
    if grad_out.shape != (B, int(sum(D))):
        raise ValueError("grad_out must be [B, sum(D)]")
    if mode not in (SUM, MEAN):
        raise ValueError("mode")
    n = indices.shape[0]
    gw = np.zeros(n, dtype=np.float64)
    S = np.zeros(n, dtype=np.float64)
    n_oob = n_bad = 0
    col = 0
    for t in range(T):
        tab = np.asarray(tables[t], dtype=np.float64)
        for b in range(B):
            g = t * B + b
            lo, hi = int(offsets[g]), int(offsets[g + 1])
            if lo < 0 or hi < lo or hi > n:
                n_bad += 1
                continue
            L = hi - lo
            if L == 0:
                continue
            go = grad_out[b, col:col + D[t]]
            if mode == MEAN:
                go = go / L
            for i in range(lo, hi):
                r = int(indices[i])
                if r < 0 or r >= tab.shape[0]:
                    n_oob += 1
                    continue
                gw[i] += float((go * tab[r]).sum())
                S[i] += float(np.abs(go * tab[r]).sum())
        col += D[t]
    return dict(grad_w=gw, S=S, n_oob=n_oob, n_bad_offsets=n_bad)
