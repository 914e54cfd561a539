"""CPU oracle for Batch Event Truncate on nested jagged event features.

TEST INFRASTRUCTURE ONLY; the CUDA library never imports it.

Paper Sec. 5.5 "Sequence Learning: Batch Event Truncate": a batch holds, per user, a number of
events (outer_lengths, shared by all features) and, per feature, the number of attributes of
every event (inner_lengths) and the flattened attribute values.  Truncating to N keeps the
first N events of every user, in every feature at once: outer lengths become min(len, N), the
inner lengths and the values of the dropped events disappear, everything stays in order.

The oracle is that definition written as plain Python loops over users and events (slow on
purpose).  Pins (tests/test_oracle_bet.py): the paper's worked example (Fig. "Batch Event
Truncate with multiple features"), N >= every length (identity), N = 0 (everything empty),
conservation (kept + dropped = input), and a second formulation through per-value user/event
labels.
"""
from __future__ import annotations

import numpy as np


def truncate(outer_lengths, inner_lengths_per_feature, values_per_feature, N):
    """Returns (outer_out [U], [inner_out_f], [values_out_f])."""
    outer = np.asarray(outer_lengths, dtype=np.int64)
    if N < 0 or np.any(outer < 0):
        raise ValueError("lengths and N must be non-negative")
    outer_out = np.minimum(outer, N)
    inner_out, values_out = [], []
    for inner, values in zip(inner_lengths_per_feature, values_per_feature):
        inner = np.asarray(inner, dtype=np.int64)
        values = np.asarray(values)
        if inner.shape[0] != int(outer.sum()) or int(inner.sum()) != values.shape[0] or np.any(inner < 0):
            raise ValueError("inconsistent nested lengths")
        keep_inner, keep_vals = [], []
        e = 0          # running event index
        v = 0          # running value index
        for u in range(outer.shape[0]):
            for j in range(int(outer[u])):
                n = int(inner[e])
                if j < N:
                    keep_inner.append(n)
                    keep_vals.extend(values[v:v + n].tolist())
                e += 1
                v += n
        inner_out.append(np.array(keep_inner, dtype=np.int64))
        values_out.append(np.array(keep_vals, dtype=values.dtype))
    return outer_out, inner_out, values_out
