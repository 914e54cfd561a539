"""Python binding of libebag.so: the pooled embedding-bag forward on one B200.

Argument marshalling only.  Every step of the operator runs in the library's CUDA kernels;
torch is used to hold device memory and to name the stream.  The functions carry the names of
the C entry points declared in ``include/ebag.h``; ``TBE`` is a small convenience wrapper around
a handle.  There is no CPU fallback: if ``libebag.so`` has not been built (``python -m
paper_2512_23236_b200.build``) or no CUDA device is usable, calls raise.
"""
from __future__ import annotations

import ctypes
import os
from typing import List, Optional, Sequence

EBAG_F32, EBAG_F16, EBAG_BF16, EBAG_INT8_ROWWISE, EBAG_UINT8_ROWWISE = 0, 1, 2, 3, 4
EBAG_SUM, EBAG_MEAN, EBAG_MAX = 0, 1, 2
EBAG_OK, EBAG_ERR_INVALID_ARG, EBAG_ERR_UNSUPPORTED, EBAG_ERR_CUDA = 0, 1, 2, 3
EBAG_ERR_INDEX_OOB, EBAG_ERR_BAD_OFFSETS = 4, 5
EBAG_NOALLOC_MAX_TABLES = 64

_PKG = os.path.dirname(os.path.abspath(__file__))
# EBAG_LIB points the binding at another build of the same library (kernel-tuning experiments)
LIB_PATH = os.environ.get("EBAG_LIB") or os.path.join(_PKG, "libebag.so")

# name -> (restype, argtypes); kept in step with include/ebag.h (a test parses the header)
_vp, _i32, _i64, _int = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_int
SIGNATURES = {
    "ebag_row_stride": (_i64, [_int, _i32]),
    "ebag_create_tbe": (_int, [_i32, _vp, _vp, _int, _int, _vp]),
    "ebag_forward": (_int, [_vp, _vp, _vp, _vp, _i64, _vp, _vp, _i64, _int, _vp, _vp]),
    "ebag_forward_i32": (_int, [_vp, _vp, _vp, _vp, _i64, _vp, _vp, _i64, _int, _vp, _vp]),
    "ebag_backward": (_int, [_vp, _vp, _vp, _i32, _i64, _vp, _vp, _i64, _int, _vp, _vp]),
    "ebag_backward_weights": (_int, [_vp, _vp, _vp, _vp, _vp, _i32, _i64, _vp, _i64, _int, _vp, _vp]),
    "ebag_forward_host": (_int, [_vp, _vp, _vp, _vp, _i64, _vp, _vp, _i64, _int, _vp, _vp]),
    "ebag_forward_host_i32": (_int, [_vp, _vp, _vp, _vp, _i64, _vp, _vp, _i64, _int, _vp, _vp]),
    "ebag_forward_noalloc": (_int, [_i32, _vp, _vp, _int, _vp, _vp, _i64, _vp, _vp, _i64, _int, _vp,
                                    _vp, _vp]),
    "ebag_mapid": (_int, [_vp, _i64, _vp, _i64, _vp, _vp]),
    "ebag_bet_workspace_bytes": (_i64, [_i32, _i64]),
    "ebag_batch_event_truncate": (_int, [_vp, _i64, _vp, _i64, _vp, _vp, _i32, _i64, _vp, _vp, _vp, _vp,
                                         _vp, _i64, _vp]),
    "ebag_mbdt": (_int, [_vp, _i32, _i64, _vp, _vp, _vp, _vp, _vp]),
    "ebag_mapid_tbe": (_int, [_vp, _vp, _i64, _vp, _vp, _vp, _i64, _vp, _vp]),
    "ebag_forward_mapid": (_int, [_vp, _vp, _vp, _vp, _i64, _vp, _vp, _vp, _vp, _i64, _int, _vp,
                                  _vp]),
    "ebag_last_status": (_int, [_vp, _vp, _vp, _vp]),
    "ebag_pack_int8_rowwise": (_int, [_vp, _vp, _vp, _i64, _i32, _vp, _vp]),
    "ebag_pack_uint8_rowwise": (_int, [_vp, _vp, _vp, _i64, _i32, _vp, _vp]),
    "ebag_set_param": (_int, [_vp, ctypes.c_char_p, _i64]),
    "ebag_launch_count": (_i64, [_vp]),
    "ebag_last_cuda_error": (ctypes.c_char_p, [_vp]),
    "ebag_destroy": (None, [_vp]),
    "ebag_status_string": (ctypes.c_char_p, [_int]),
}

_lib = None


class EbagError(RuntimeError):
    def __init__(self, status: int, what: str = ""):
        self.status = status
        msg = lib().ebag_status_string(status).decode()
        super().__init__(f"{what}: {msg}" if what else msg)


def lib():
    """The loaded library (loads it on first use; raises if it is missing)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} not found: build it with "
                              "`python -m paper_2512_23236_b200.build` (there is no fallback path)")
        L = ctypes.CDLL(LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(L, name)
            fn.restype = res
            fn.argtypes = args
        _lib = L
    return _lib


def _check(status: int, what: str):
    if status != EBAG_OK:
        raise EbagError(status, what)


def _stream_ptr(stream) -> int:
    import torch
    if stream is None:
        stream = torch.cuda.current_stream()
    return int(stream.cuda_stream) if hasattr(stream, "cuda_stream") else int(stream)


def _ptr(t) -> Optional[int]:
    return None if t is None else int(t.data_ptr())


# ---------------------------------------------------------------- functions named as the C ABI
def ebag_row_stride(dtype: int, D: int) -> int:
    return int(lib().ebag_row_stride(dtype, D))


def ebag_create_tbe(rows: Sequence[int], D: Sequence[int], dtype: int, device: int = 0) -> int:
    """Returns the handle as an integer address."""
    T = len(rows)
    r = (ctypes.c_int64 * T)(*[int(x) for x in rows])
    d = (ctypes.c_int32 * T)(*[int(x) for x in D])
    h = ctypes.c_void_p(0)
    st = lib().ebag_create_tbe(T, ctypes.cast(r, _vp), ctypes.cast(d, _vp), dtype, device,
                               ctypes.addressof(h))
    _check(st, "ebag_create_tbe")
    return int(h.value)


def ebag_forward(h: int, table_ptrs: Sequence[int], D: Sequence[int], indices_ptr, n_indices: int,
                 offsets_ptr, weights_ptr, B: int, mode: int, out_ptr, stream_ptr,
                 host: bool = False, idx32: bool = False) -> None:
    T = len(table_ptrs)
    tp = (ctypes.c_void_p * T)(*[int(p) if p else None for p in table_ptrs])
    d = (ctypes.c_int32 * T)(*[int(x) for x in D])
    name = ("ebag_forward_host" if host else "ebag_forward") + ("_i32" if idx32 else "")
    st = getattr(lib(), name)(h, ctypes.cast(tp, _vp), ctypes.cast(d, _vp), indices_ptr, n_indices, offsets_ptr,
                              weights_ptr, B, mode, out_ptr, stream_ptr)
    _check(st, name)


def ebag_forward_noalloc(rows: Sequence[int], D: Sequence[int], dtype: int,
                         table_ptrs: Sequence[int], indices_ptr, n_indices: int, offsets_ptr,
                         weights_ptr, B: int, mode: int, out_ptr, status_counts_ptr,
                         stream_ptr) -> None:
    """Handle-free forward for callers that must not allocate device memory (a plugin inside a
    host that owns all of it, code under a strict memory pool, a latency-critical thread): the
    kernel's scratch is a static device array inside the library.  Runs on the current device.
    Calls that overlap on the GPU race on that array; issue them one after another."""
    T = len(rows)
    r = (ctypes.c_int64 * T)(*[int(x) for x in rows])
    d = (ctypes.c_int32 * T)(*[int(x) for x in D])
    tp = (ctypes.c_void_p * T)(*[int(p) if p else None for p in table_ptrs])
    st = lib().ebag_forward_noalloc(T, ctypes.cast(r, _vp), ctypes.cast(d, _vp), dtype,
                                    ctypes.cast(tp, _vp), indices_ptr, n_indices, offsets_ptr,
                                    weights_ptr, B, mode, out_ptr, status_counts_ptr, stream_ptr)
    _check(st, "ebag_forward_noalloc")


def ebag_mapid(values, mapping, out=None, stream=None):
    """MapId transform of a device int64 tensor against a sorted device int64 mapping."""
    import torch
    if out is None:
        out = torch.empty_like(values)
    with torch.cuda.device(values.device):
        st = lib().ebag_mapid(_ptr(values), int(values.numel()), _ptr(mapping), int(mapping.numel()),
                              _ptr(out), _stream_ptr(stream))
    _check(st, "ebag_mapid")
    return out


def ebag_mbdt(values, borders, border_offsets, out_offsets, out=None, stream=None):
    """MergeBucketizedDense: device fp32 [F, B] values -> device int64 [F, B] bin ids."""
    import torch
    F, B = values.shape
    if out is None:
        out = torch.empty((F, B), dtype=torch.int64, device=values.device)
    with torch.cuda.device(values.device):
        st = lib().ebag_mbdt(_ptr(values), F, B, _ptr(borders), _ptr(border_offsets),
                             _ptr(out_offsets), _ptr(out), _stream_ptr(stream))
    _check(st, "ebag_mbdt")
    return out


def ebag_batch_event_truncate(outer, inner, values, value_offsets, N: int, stream=None):
    """Batch Event Truncate on device int64 tensors: outer [U], inner [F, E], values (features back
    to back), value_offsets [F+1].  Returns (outer_out [U], inner_out [F, E], values_out, counts
    [1+F]); only the leading counts[0] entries of every inner_out row and counts[1+f] values of
    feature f (from value_offsets[f] on) are meaningful."""
    import torch
    F, E = inner.shape
    U = int(outer.numel())
    outer_out = torch.empty_like(outer)
    inner_out = torch.empty_like(inner)
    values_out = torch.empty_like(values)
    counts = torch.empty(1 + F, dtype=torch.int64, device=outer.device)
    nbytes = int(lib().ebag_bet_workspace_bytes(F, U))
    ws = torch.empty(max(nbytes, 8) // 8, dtype=torch.int64, device=outer.device)
    with torch.cuda.device(outer.device):
        st = lib().ebag_batch_event_truncate(_ptr(outer), U, _ptr(inner), E, _ptr(values),
                                             _ptr(value_offsets), F, int(N), _ptr(outer_out),
                                             _ptr(inner_out), _ptr(values_out), _ptr(counts), _ptr(ws),
                                             nbytes, _stream_ptr(stream))
    _check(st, "ebag_batch_event_truncate")
    return outer_out, inner_out, values_out, counts


def ebag_forward_mapid(h: int, table_ptrs: Sequence[int], D: Sequence[int], values_ptr,
                       n_values: int, offsets_ptr, weights_ptr, mapping_ptrs: Sequence[int],
                       mapping_len: Sequence[int], B: int, mode: int, out_ptr, stream_ptr) -> None:
    T = len(table_ptrs)
    tp = (ctypes.c_void_p * T)(*[int(p) if p else None for p in table_ptrs])
    d = (ctypes.c_int32 * T)(*[int(x) for x in D])
    mp = (ctypes.c_void_p * T)(*[int(p) if p else None for p in mapping_ptrs])
    ml = (ctypes.c_int64 * T)(*[int(x) for x in mapping_len])
    st = lib().ebag_forward_mapid(h, ctypes.cast(tp, _vp), ctypes.cast(d, _vp), values_ptr,
                                  n_values, offsets_ptr, weights_ptr, ctypes.cast(mp, _vp),
                                  ctypes.cast(ml, _vp), B, mode, out_ptr, stream_ptr)
    _check(st, "ebag_forward_mapid")


def ebag_last_status(h: int, stream_ptr) -> tuple:
    """(status, n_oob, n_bad_offsets); synchronises the stream."""
    a, b = ctypes.c_int64(0), ctypes.c_int64(0)
    st = lib().ebag_last_status(h, stream_ptr, ctypes.addressof(a), ctypes.addressof(b))
    if st == EBAG_ERR_CUDA or st == EBAG_ERR_INVALID_ARG:
        raise EbagError(st, "ebag_last_status")
    return int(st), int(a.value), int(b.value)


def ebag_destroy(h: int) -> None:
    lib().ebag_destroy(h)


def ebag_pack_int8_rowwise(q, scale, bias, stream=None):
    """torch int8 (or uint8, for EBAG_UINT8_ROWWISE tables) [rows, D], fp32 [rows], fp32 [rows]
    (device) -> packed uint8 [rows, D+16]."""
    import torch
    if q.dtype not in (torch.int8, torch.uint8):
        raise TypeError("codes must be int8 or uint8")
    rows, D = q.shape
    stride = ebag_row_stride(EBAG_INT8_ROWWISE, D)
    if stride < 0:
        raise EbagError(EBAG_ERR_INVALID_ARG, "ebag_pack_int8_rowwise")
    q = q.contiguous()
    scale = scale.contiguous().float()
    bias = bias.contiguous().float()
    dst = torch.empty((rows, stride), dtype=torch.uint8, device=q.device)
    with torch.cuda.device(q.device):
        fn = lib().ebag_pack_uint8_rowwise if q.dtype == torch.uint8 else lib().ebag_pack_int8_rowwise
        st = fn(_ptr(q), _ptr(scale), _ptr(bias), rows, D, _ptr(dst), _stream_ptr(stream))
    _check(st, "ebag_pack_int8_rowwise")
    return dst


ebag_pack_uint8_rowwise = ebag_pack_int8_rowwise     # the code type of `q` selects the entry point


# ---------------------------------------------------------------- convenience wrapper
class TBE:
    """A handle for T tables.  ``tables`` passed to forward() are torch device tensors laid out
    as the library expects: [rows, D] of float32 / float16 / bfloat16, or for rowwise int8 the
    packed uint8 [rows, D+16] tensor from ebag_pack_int8_rowwise()."""

    def __init__(self, rows: Sequence[int], D: Sequence[int], dtype: int, device: int = 0):
        self.rows = [int(r) for r in rows]
        self.D = [int(d) for d in D]
        self.dtype = dtype
        self.device = device
        self.sumD = sum(self.D)
        self._h = ebag_create_tbe(self.rows, self.D, dtype, device)

    @property
    def T(self) -> int:
        return len(self.rows)

    def close(self):
        if self._h:
            ebag_destroy(self._h)
            self._h = 0

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def set_param(self, name: str, value: int):
        _check(lib().ebag_set_param(self._h, name.encode(), int(value)), "ebag_set_param")
        if name == "out_dtype":
            self._out_dtype = int(value)

    def _out_torch_dtype(self):
        import torch
        return {EBAG_F32: torch.float32, EBAG_F16: torch.float16,
                EBAG_BF16: torch.bfloat16}[getattr(self, "_out_dtype", EBAG_F32)]

    def launch_count(self) -> int:
        return int(lib().ebag_launch_count(self._h))

    def last_cuda_error(self) -> str:
        return lib().ebag_last_cuda_error(self._h).decode()

    def _table_array(self, tables):
        """ctypes array of the tables' device pointers, rebuilt only when they change."""
        ptrs = tuple(t.data_ptr() for t in tables)
        cached = getattr(self, "_tp_cache", None)
        if cached is None or cached[0] != ptrs:
            arr = (ctypes.c_void_p * len(ptrs))(*[p if p else None for p in ptrs])
            cached = (ptrs, arr, ctypes.cast(arr, _vp))
            self._tp_cache = cached
        return cached[2]

    def forward(self, tables: List, indices, offsets, B: int, mode: int = EBAG_SUM,
                per_sample_weights=None, out=None, stream=None):
        """Device tensors in, device tensor out ([B, sum D] float32).  Enqueues only.
        ``indices`` may be int64 or int32 (the matching entry point is called)."""
        import torch
        if out is None:
            out = torch.empty((B, self.sumD), dtype=self._out_torch_dtype(), device=indices.device)
        elif out.dtype != self._out_torch_dtype():
            raise TypeError("out must have the handle's out_dtype")
        if not hasattr(self, "_d_arr"):
            self._d_arr = (ctypes.c_int32 * self.T)(*self.D)
            self._d_ptr = ctypes.cast(self._d_arr, _vp)
        if indices.dtype == torch.int32:
            fn, name = lib().ebag_forward_i32, "ebag_forward_i32"
        elif indices.dtype == torch.int64:
            fn, name = lib().ebag_forward, "ebag_forward"
        else:
            raise TypeError("indices must be int64 or int32")
        st = fn(self._h, self._table_array(tables), self._d_ptr, _ptr(indices), int(indices.numel()),
                _ptr(offsets), _ptr(per_sample_weights), B, mode, _ptr(out), _stream_ptr(stream))
        _check(st, name)
        return out

    def backward(self, grad_out, indices, offsets, B: int, grad_tables: List, mode: int = EBAG_SUM,
                 per_sample_weights=None, stream=None):
        """Adds the gradient of the forward with respect to the tables into ``grad_tables`` (a
        list of T dense float32 CUDA tensors [rows_t, D_t]).  Enqueues only."""
        import torch
        bits = 32 if indices.dtype == torch.int32 else 64
        if indices.dtype not in (torch.int32, torch.int64):
            raise TypeError("indices must be int64 or int32")
        for g in grad_tables:
            if g.dtype != torch.float32 or not g.is_contiguous():
                raise TypeError("gradient tables must be contiguous float32")
        arr = (ctypes.c_void_p * self.T)(*[g.data_ptr() if g.numel() else None for g in grad_tables])
        st = lib().ebag_backward(self._h, _ptr(grad_out), _ptr(indices), bits, int(indices.numel()),
                                 _ptr(offsets), _ptr(per_sample_weights), B, mode,
                                 ctypes.cast(arr, _vp), _stream_ptr(stream))
        _check(st, "ebag_backward")

    def backward_weights(self, tables: List, grad_out, indices, offsets, B: int, mode: int = EBAG_SUM,
                         out=None, stream=None):
        """Gradient of the forward with respect to the per-sample weights: float32 [n_indices],
        one dot product of the bag's grad_out slice with the looked-up row per lookup.  Enqueues only."""
        import torch
        bits = 32 if indices.dtype == torch.int32 else 64
        if indices.dtype not in (torch.int32, torch.int64):
            raise TypeError("indices must be int64 or int32")
        if out is None:
            out = torch.zeros(int(indices.numel()), dtype=torch.float32, device=indices.device)
        if not hasattr(self, "_d_arr"):
            self._d_arr = (ctypes.c_int32 * self.T)(*self.D)
            self._d_ptr = ctypes.cast(self._d_arr, _vp)
        st = lib().ebag_backward_weights(self._h, self._table_array(tables), self._d_ptr, _ptr(grad_out),
                                         _ptr(indices), bits, int(indices.numel()), _ptr(offsets), B, mode,
                                         _ptr(out), _stream_ptr(stream))
        _check(st, "ebag_backward_weights")
        return out

    def forward_mapid(self, tables: List, values, offsets, mappings: List, B: int,
                      mode: int = EBAG_SUM, per_sample_weights=None, out=None, stream=None):
        """Raw ids in: table t maps them through the sorted device tensor mappings[t] first."""
        import torch
        if out is None:
            out = torch.empty((B, self.sumD), dtype=self._out_torch_dtype(), device=values.device)
        ebag_forward_mapid(self._h, [t.data_ptr() for t in tables], self.D, _ptr(values),
                           int(values.numel()), _ptr(offsets), _ptr(per_sample_weights),
                           [m.data_ptr() for m in mappings], [int(m.numel()) for m in mappings], B,
                           mode, _ptr(out), _stream_ptr(stream))
        return out

    def mapid(self, values, offsets, mappings: List, B: int, out=None, stream=None):
        """MapId of all tables in one launch: raw ids -> row ids (device int64 tensors)."""
        import torch
        if out is None:
            out = torch.empty_like(values)
        T = self.T
        mp = (ctypes.c_void_p * T)(*[int(m.data_ptr()) if m.numel() else None for m in mappings])
        ml = (ctypes.c_int64 * T)(*[int(m.numel()) for m in mappings])
        st = lib().ebag_mapid_tbe(self._h, _ptr(values), int(values.numel()), _ptr(offsets),
                                  ctypes.cast(mp, _vp), ctypes.cast(ml, _vp), B, _ptr(out),
                                  _stream_ptr(stream))
        _check(st, "ebag_mapid_tbe")
        return out

    def forward_host(self, tables: List, indices, offsets, B: int, mode: int = EBAG_SUM,
                     per_sample_weights=None, out=None, stream=None):
        """Host (ideally pinned) tensors for indices/offsets/weights/out, device tables.
        The caller synchronises the stream before reading ``out``."""
        import torch
        if out is None:
            out = torch.empty((B, self.sumD), dtype=self._out_torch_dtype()).pin_memory()
        elif out.dtype != self._out_torch_dtype():
            raise TypeError("out must have the handle's out_dtype")
        if indices.dtype not in (torch.int32, torch.int64):
            raise TypeError("indices must be int64 or int32")
        ebag_forward(self._h, [t.data_ptr() for t in tables], self.D, _ptr(indices),
                     int(indices.numel()), _ptr(offsets), _ptr(per_sample_weights), B, mode,
                     _ptr(out), _stream_ptr(stream), host=True, idx32=indices.dtype == torch.int32)
        return out

    def last_status(self, stream=None) -> tuple:
        return ebag_last_status(self._h, _stream_ptr(stream))
