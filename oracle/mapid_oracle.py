"""CPU oracle for the MapId transform and for the pooled forward fed by it.

TEST INFRASTRUCTURE ONLY (tests, smoke check, benchmark CPU-baseline leg); the CUDA library
never imports it.

MapId (paper Sec. 5.4.1 "MapId Transform"): a sorted mapping tensor M of known ids turns every
input value v into its 1-based position in M, 0 meaning "unknown".  The three steps of the
paper's algorithm, in its order:
  1. insertion index by binary search:  idx = bucketize(v, M)   (first i with M[i] >= v)
  2. clamp:                              idx = min(idx, |M| - 1)
  3. validate:                           out = idx + 1 if M[idx] == v else 0
numpy's searchsorted(side="left") is the library primitive for step 1.  Pins
(tests/test_oracle_mapid.py): the paper's worked example (Table "MapIdTransform example"), a
dictionary brute force, and the closed forms (every member of M maps to its rank, every
non-member to 0).

The fused operator is the composition: ids = MapId_t(values) per table, then the pooled
embedding-bag forward over tables with |M_t| + 1 rows (row 0 holds the "unknown" embedding).
"""
from __future__ import annotations

import numpy as np

from oracle import ebag_oracle


def mapid(values: np.ndarray, mapping: np.ndarray) -> np.ndarray:
    values = np.ascontiguousarray(values, dtype=np.int64)
    mapping = np.ascontiguousarray(mapping, dtype=np.int64)
    if mapping.ndim != 1 or mapping.shape[0] == 0:
        raise ValueError("mapping must be a non-empty 1-D array")
    if np.any(mapping[1:] <= mapping[:-1]):
        raise ValueError("mapping must be strictly increasing")
    idx = np.searchsorted(mapping, values, side="left")            # step 1
    idx = np.minimum(idx, mapping.shape[0] - 1)                    # step 2
    return np.where(mapping[idx] == values, idx + 1, 0).astype(np.int64)   # step 3


def forward_mapid(tables, dtype, values, offsets, B, mappings, mode=ebag_oracle.SUM, weights=None,
                  scales=None, biases=None):
    """MapId per table, then the pooled forward.  tables[t] has len(mappings[t]) + 1 rows."""
    T = len(tables)
    values = np.ascontiguousarray(values, dtype=np.int64)
    offsets = np.ascontiguousarray(offsets, dtype=np.int64)
    ids = np.empty_like(values)
    for t in range(T):
        lo, hi = int(offsets[t * B]), int(offsets[(t + 1) * B])
        ids[lo:hi] = mapid(values[lo:hi], mappings[t])
    return ebag_oracle.forward(tables, dtype, ids, offsets, B, mode, weights=weights,
                               scales=scales, biases=biases)
