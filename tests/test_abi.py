"""The C-ABI library loads and exports every symbol that include/ebag.h declares, and the Python
binding lists the same names.  No compute calls: runs without a GPU."""
import ctypes
import os
import re

import paper_2512_23236_b200 as eb

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    src = open(os.path.join(ROOT, "include", "ebag.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return set(re.findall(r"\b(ebag_[a-z0-9_]+)\s*\(", src))


def test_header_symbols_are_exported_and_bound():
    names = _declared()
    assert {"ebag_create_tbe", "ebag_forward", "ebag_destroy"} <= names
    lib = ctypes.CDLL(eb.LIB_PATH)
    for n in names:
        assert hasattr(lib, n), f"{n} declared in ebag.h but not exported"
    assert names == set(eb.SIGNATURES), names ^ set(eb.SIGNATURES)


def test_calls_that_need_no_device():
    assert eb.ebag_row_stride(eb.EBAG_F32, 64) == 256
    assert eb.ebag_row_stride(eb.EBAG_F16, 128) == 256
    assert eb.ebag_row_stride(eb.EBAG_BF16, 8) == 16
    assert eb.ebag_row_stride(eb.EBAG_INT8_ROWWISE, 128) == 144
    assert eb.ebag_row_stride(eb.EBAG_F32, 6) == -1          # 24 bytes: not 128-bit loadable
    assert eb.ebag_row_stride(eb.EBAG_INT8_ROWWISE, 24) == -1
    assert eb.ebag_row_stride(eb.EBAG_F32, 0) == -1
    assert eb.lib().ebag_status_string(0) == b"ok"
    assert b"unsupported" in eb.lib().ebag_status_string(eb.EBAG_ERR_UNSUPPORTED)
    eb.ebag_destroy(None)                                     # NULL is allowed


def test_invalid_create_arguments_fail_before_touching_the_device():
    import pytest
    with pytest.raises(eb.EbagError) as e:
        eb.ebag_create_tbe([], [], eb.EBAG_F32)
    assert e.value.status == eb.EBAG_ERR_INVALID_ARG
    with pytest.raises(eb.EbagError) as e:
        eb.ebag_create_tbe([10], [6], eb.EBAG_F32)
    assert e.value.status == eb.EBAG_ERR_INVALID_ARG
    with pytest.raises(eb.EbagError) as e:
        eb.ebag_create_tbe([2 ** 31], [8], eb.EBAG_F32)
    assert e.value.status == eb.EBAG_ERR_UNSUPPORTED
    with pytest.raises(eb.EbagError) as e:
        eb.ebag_create_tbe([1] * 3000, [8] * 3000, eb.EBAG_F32)
    assert e.value.status == eb.EBAG_ERR_UNSUPPORTED


def test_no_fallback_without_a_device():
    """With no usable CUDA device, create fails loudly; nothing is computed on the CPU."""
    import pytest
    import torch
    if torch.cuda.is_available():
        pytest.skip("a CUDA device is present")
    with pytest.raises(eb.EbagError) as e:
        eb.ebag_create_tbe([10], [8], eb.EBAG_F32)
    assert e.value.status == eb.EBAG_ERR_CUDA
