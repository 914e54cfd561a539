"""ctypes wrapper around the CPU oracle (``ebag_oracle.cpp``).

TEST INFRASTRUCTURE ONLY: the tests, the smoke check and the benchmark's CPU-baseline leg use
it; the CUDA library and its binding never import it.  Inputs and outputs are numpy arrays.
The operator it defines is the pooled embedding-bag forward over jagged id lists
(motivated in Sec. 1.1, paragraph "Model Diversity Across Ranking Stages"; input types from
Sec. 2.2, paragraph "Feature Types and Memory Layout").
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ebag_oracle.cpp")
_LIB = os.path.join(_HERE, "libebag_oracle.so")

F32, F16, BF16, INT8_ROWWISE, UINT8_ROWWISE = 0, 1, 2, 3, 4
SUM, MEAN, MAX = 0, 1, 2

_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle into its own shared library (g++, OpenMP, no FMA contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["g++", "-O2", "-std=c++17", "-fopenmp", "-ffp-contract=off", "-fPIC", "-shared",
               _SRC, "-o", _LIB]
        subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        vp = ctypes.c_void_p
        lib.ebag_oracle_forward.restype = ctypes.c_int
        lib.ebag_oracle_forward.argtypes = [
            ctypes.c_int32, vp, vp, ctypes.c_int32, vp, vp, vp, vp, ctypes.c_int64, vp, vp,
            ctypes.c_int64, ctypes.c_int32, vp, vp, vp, vp, vp, ctypes.c_int32]
        lib.ebag_oracle_max_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


def max_threads() -> int:
    return int(_load().ebag_oracle_max_threads())


_TABLE_NP = {F32: np.float32, F16: np.uint16, BF16: np.uint16, INT8_ROWWISE: np.int8,
             UINT8_ROWWISE: np.uint8}


def _ptr_array(arrs):
    return (ctypes.c_void_p * len(arrs))(*[a.ctypes.data for a in arrs])


def forward(tables, dtype, indices, offsets, B, mode=SUM, weights=None, scales=None, biases=None,
            nthreads=0, want64=True):
    """Run the oracle.

    tables : list of T numpy arrays [rows_t, D_t]; float32 (F32), uint16 bit patterns (F16/BF16)
             or int8 / uint8 codes (INT8_ROWWISE / UINT8_ROWWISE, with ``scales``/``biases`` lists of
             float32 [rows_t]: value = scale * code + bias).
    Returns dict(out32 [B, sumD] f32, out64, S (f64 or None), n_oob, n_bad_offsets).
    """
    lib = _load()
    T = len(tables)
    want = _TABLE_NP[dtype]
    tabs = []
    for a in tables:
        if a.dtype != want or a.ndim != 2:
            raise TypeError(f"table must be 2-D {want}, got {a.dtype} ndim {a.ndim}")
        tabs.append(np.ascontiguousarray(a))
    rows = np.array([a.shape[0] for a in tabs], dtype=np.int64)
    D = np.array([a.shape[1] for a in tabs], dtype=np.int32)
    indices = np.ascontiguousarray(indices, dtype=np.int64)
    offsets = np.ascontiguousarray(offsets, dtype=np.int64)
    if offsets.shape[0] != T * B + 1:
        raise ValueError("offsets must hold T*B+1 entries")
    w = None if weights is None else np.ascontiguousarray(weights, dtype=np.float32)
    if w is not None and w.shape[0] != indices.shape[0]:
        raise ValueError("weights must pair with indices")
    sc = bi = None
    if dtype in (INT8_ROWWISE, UINT8_ROWWISE):
        sc = [np.ascontiguousarray(s, dtype=np.float32) for s in scales]
        bi = [np.ascontiguousarray(s, dtype=np.float32) for s in biases]
    sumD = int(D.sum())
    out32 = np.empty((B, sumD), dtype=np.float32)
    out64 = np.empty((B, sumD), dtype=np.float64) if want64 else None
    S = np.empty((B, sumD), dtype=np.float64) if want64 else None
    n_oob = ctypes.c_int64(0)
    n_bad = ctypes.c_int64(0)
    tp = _ptr_array(tabs)
    sp = _ptr_array(sc) if sc is not None else None
    bp = _ptr_array(bi) if bi is not None else None
    rc = lib.ebag_oracle_forward(
        T, rows.ctypes.data, D.ctypes.data, dtype, ctypes.cast(tp, ctypes.c_void_p),
        None if sp is None else ctypes.cast(sp, ctypes.c_void_p),
        None if bp is None else ctypes.cast(bp, ctypes.c_void_p),
        indices.ctypes.data, indices.shape[0], offsets.ctypes.data,
        None if w is None else w.ctypes.data, B, mode, out32.ctypes.data,
        None if out64 is None else out64.ctypes.data, None if S is None else S.ctypes.data,
        ctypes.addressof(n_oob), ctypes.addressof(n_bad), nthreads)
    if rc != 0:
        raise ValueError("ebag_oracle_forward rejected its arguments")
    return dict(out32=out32, out64=out64, S=S, n_oob=int(n_oob.value),
                n_bad_offsets=int(n_bad.value))
