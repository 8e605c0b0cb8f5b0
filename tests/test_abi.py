"""The C-ABI library loads, exports every symbol include/qllm.h declares, and rejects bad
arguments with status codes before anything is launched (no GPU needed)."""
import ctypes
import os
import re

import numpy as np

from paper_2310_08041_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    src = open(os.path.join(ROOT, "include", "qllm.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(qllm_[a-z_0-9]+)\s*\(", src)))


def test_every_declared_symbol_is_exported():
    names = _declared()
    assert sorted(B.EXPORTS) == names
    lib = ctypes.CDLL(B.LIB_PATH)
    for n in names:
        assert hasattr(lib, n), n


def test_status_strings():
    assert B.qllm_status_string(0) == "ok"
    for s in range(-11, 0):
        assert B.qllm_status_string(s) not in ("ok", "unknown status")
    assert B.qllm_status_string(-99) == "unknown status"


def test_argument_checks_return_codes_without_a_device():
    L = B._lib
    one = ctypes.c_void_p(16)   # non-null, 16-byte aligned dummy; never dereferenced on these paths
    # bits / dtype / shape checks come before any CUDA call
    assert L.qllm_reassemble_quant(one, 0, 4, 8, one, None, 1e-5, one, one, one, 5, one, one, one, None, None) == B.QLLM_ERR_BITS
    assert L.qllm_reassemble_quant(one, 7, 4, 8, one, None, 1e-5, one, one, one, 4, one, one, one, None, None) == B.QLLM_ERR_DTYPE
    assert L.qllm_reassemble_quant(one, 0, -1, 8, one, None, 1e-5, one, one, one, 4, one, one, one, None, None) == B.QLLM_ERR_SHAPE
    assert L.qllm_reassemble_quant(one, 0, 4, 7, one, None, 1e-5, one, one, one, 4, one, one, one, None, None) == B.QLLM_ERR_SHAPE
    assert L.qllm_reassemble_quant(one, 0, 0, 8, one, None, 1e-5, one, one, one, 4, one, one, one, None, None) == B.QLLM_OK
    assert L.qllm_reassemble_quant(None, 0, 4, 8, one, None, 1e-5, one, one, one, 4, one, one, one, None, None) == B.QLLM_ERR_NULL
    assert L.qllm_reassemble_quant(ctypes.c_void_p(8), 0, 4, 8, one, None, 1e-5, one, one, one, 4, one, one, one, None, None) == B.QLLM_ERR_ALIGN
    assert L.qllm_qgemm(one, one, one, one, one, one, one, None, one, 4, 8, 8, 3, 4, 0, one, None) == B.QLLM_ERR_BITS
    assert L.qllm_qgemm(one, one, one, one, one, one, one, None, one, 4, 8, 7, 4, 4, 0, one, None) == B.QLLM_ERR_SHAPE
    assert L.qllm_qgemm(one, one, one, one, one, one, one, None, one, 4, 0, 8, 4, 4, 0, one, None) == B.QLLM_ERR_SHAPE
    assert L.qllm_qgemm(one, one, one, one, one, one, one, None, one, 4, 8, 8, 4, 4, 3, one, None) == B.QLLM_ERR_DTYPE
    assert L.qllm_qgemm(one, one, one, None, one, one, one, None, one, 4, 8, 8, 4, 4, 0, one, None) == B.QLLM_ERR_NULL
    assert L.qllm_qgemm(one, one, one, one, one, one, one, None, one, 0, 8, 8, 4, 4, 0, one, None) == B.QLLM_OK
    assert L.qllm_qgemm_acc(one, one, None, 4, 8, 8, 4, 4, None) == B.QLLM_ERR_NULL
    assert L.qllm_calib_absmax(one, 0, 4, 0, one, None, 1e-5, one, None) == B.QLLM_ERR_SHAPE


def test_builder_argument_checks():
    a = np.ones(8, np.float32)
    W = np.ones((4, 8), np.float32)
    h = ctypes.c_void_p()
    L = B._lib
    hp = lambda x: x.ctypes.data_as(ctypes.c_void_p)
    assert L.qllm_build_reassembly(None, 8, 1.0, hp(W), 4, None, None, 0, 4, ctypes.byref(h)) == B.QLLM_ERR_NULL
    assert L.qllm_build_reassembly(hp(a), 8, 0.0, hp(W), 4, None, None, 0, 4, ctypes.byref(h)) == B.QLLM_ERR_SHAPE
    assert L.qllm_build_reassembly(hp(a), 8, 1.0, hp(W), 4, None, None, 0, 5, ctypes.byref(h)) == B.QLLM_ERR_BITS
    assert L.qllm_build_reassembly(hp(a), 7, 1.0, hp(W), 4, None, None, 0, 4, ctypes.byref(h)) == B.QLLM_ERR_SHAPE
    assert L.qllm_build_reassembly(hp(a), 8, 1.0, hp(W), 4, hp(a), None, 1, 4, ctypes.byref(h)) == B.QLLM_ERR_NULL
    bad = a.copy(); bad[3] = np.nan
    assert L.qllm_build_reassembly(hp(bad), 8, 1.0, hp(W), 4, None, None, 0, 4, ctypes.byref(h)) == B.QLLM_ERR_SHAPE
    # map validator
    ptr = np.array([0, 1, 2, 4], np.int32); src = np.array([0, 1, 2, 0], np.int32)
    assert B.qllm_validate_map(ptr, src, 3) == B.QLLM_OK
    assert B.qllm_validate_map(np.array([0, 1, 1, 4], np.int32), src, 3) == B.QLLM_ERR_MAP
    assert B.qllm_validate_map(ptr, np.array([0, 1, 3, 0], np.int32), 3) == B.QLLM_ERR_MAP
    assert B.qllm_validate_map(np.array([1, 2, 3, 4], np.int32), src, 3) == B.QLLM_ERR_MAP
