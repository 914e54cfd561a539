"""CPU oracle for the MergeBucketizedDense transform (MBDT).

TEST INFRASTRUCTURE ONLY; the CUDA library never imports it.

Paper Sec. 5.4.2 "MergeBucketizedDense Transform": for values X [F, B] (F features, B batch) and
per-feature sorted border lists B_f, the output is the bin of every value plus a per-feature
offset that makes the bins of different features distinct embedding ids:

    Y[f, i] = bucketize(X[f, i], B_f) + offsets[f]

This follows the sequential pseudocode the paper prints (two loops, torch.bucketize with its
default side, then the offset).  Reading of a point where the paper is at odds with itself: its
Eq. for Y says min{k : X < B_f[k]} (a value equal to a border goes right), while its worked
example labels the bins (-inf, 0.3], (0.3, 0.6], ... and its pseudocode calls torch.bucketize,
whose default puts a value equal to a border LEFT (bin = number of borders strictly below the
value).  The example and the pseudocode win; the example contains no ties, so it pins
everything but this choice.  NaN goes to the last bin, as in the library routine.

numpy's searchsorted(side="left") is the library primitive for the per-value search.  Pins
(tests/test_oracle_mbdt.py): the paper's worked example (Fig. "MBDT execution example"), a
brute-force count of borders below the value, ties, infinities, NaN, empty border lists.
"""
from __future__ import annotations

import numpy as np


def flatten_borders(borders_list):
    """Per-feature border lists -> (flat float32 array, int64 offsets [F+1])."""
    off = np.zeros(len(borders_list) + 1, dtype=np.int64)
    for f, b in enumerate(borders_list):
        off[f + 1] = off[f] + len(b)
    flat = np.concatenate([np.asarray(b, dtype=np.float32) for b in borders_list]) \
        if off[-1] else np.zeros(0, np.float32)
    return flat, off


def bin_offsets(borders_list):
    """The paper's `offsets`: first global bin id of every feature (K_f + 1 bins each)."""
    out = np.zeros(len(borders_list), dtype=np.int64)
    for f in range(1, len(borders_list)):
        out[f] = out[f - 1] + len(borders_list[f - 1]) + 1
    return out


def mbdt(values: np.ndarray, borders_list, offsets: np.ndarray) -> np.ndarray:
    values = np.ascontiguousarray(values, dtype=np.float32)
    F, B = values.shape
    if len(borders_list) != F or len(offsets) != F:
        raise ValueError("one border list and one offset per feature")
    out = np.empty((F, B), dtype=np.int64)
    for f in range(F):
        b = np.asarray(borders_list[f], dtype=np.float32)
        if b.size > 1 and np.any(b[1:] < b[:-1]):
            raise ValueError("borders must be sorted")
        for i in range(B):                                   # the paper's two loops
            out[f, i] = int(np.searchsorted(b, values[f, i], side="left")) + int(offsets[f])
    return out


def mbdt_fast(values: np.ndarray, borders_list, offsets: np.ndarray) -> np.ndarray:
    """The same result with the inner loop handed to numpy (used only to time large cases; a test
    checks it against mbdt())."""
    values = np.ascontiguousarray(values, dtype=np.float32)
    out = np.empty(values.shape, dtype=np.int64)
    for f in range(values.shape[0]):
        out[f] = np.searchsorted(np.asarray(borders_list[f], dtype=np.float32), values[f],
                                 side="left") + int(offsets[f])
    return out
