"""The C-ABI library loads on a machine without a GPU, exports every symbol that
include/sasq.h declares, and rejects bad arguments on the host without a launch."""
import ctypes
import os
import re

import pytest

import paper_2512_14481_b200 as P
from paper_2512_14481_b200 import build as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    src = open(os.path.join(ROOT, "include", "sasq.h")).read()
    return re.findall(r"^SASQ_API\s+[\w\s\*]+?\b(sasq_\w+)\s*\(", src, flags=re.M)


def test_library_builds_and_exports_every_declared_symbol():
    B.build()
    lib = P.load_library()
    names = _declared()
    assert len(names) >= 10 and "sasq_fakequant_fwd" in names and "sasq_static_w8a8_linear" in names
    for n in names:
        assert hasattr(lib, n), n
    for n in names:
        assert n in P.__all__ or n == "sasq_status_string" or hasattr(P, n), f"binding lacks {n}"


def test_status_strings():
    assert P.sasq_status_string(0) == "SASQ_OK"
    for code in range(1, 7):
        assert P.sasq_status_string(code).startswith("SASQ_ERR_")


def test_workspace_queries_need_no_gpu():
    assert P.sasq_fakequant_bwd_workspace(1 << 20) >= 8
    assert P.sasq_fakequant_multi_workspace(7) == 7 * P.sasq_fakequant_multi_workspace(1)
    assert P.sasq_static_w8a8_linear_workspace(128, 4096, 4096) >= 0


def test_host_side_argument_errors_launch_nothing():
    lib = P.load_library()
    INVALID, WORKSPACE = 1, 3
    buf = (ctypes.c_char * 256)()
    base = ctypes.addressof(buf)
    a = (base + 15) & ~15          # a 16-byte aligned host address: never dereferenced, the call must fail first
    # NULL tensors
    assert lib.sasq_fakequant_fwd(None, None, 8, 1, a, 8, None) == INVALID
    # misaligned pointer
    assert lib.sasq_fakequant_fwd(a + 2, a, 8, 1, a, 8, None) == INVALID
    # bits out of range, bad dtype, negative size, NULL scale
    assert lib.sasq_fakequant_fwd(a, a, 8, 1, a, 9, None) == INVALID
    assert lib.sasq_fakequant_fwd(a, a, 8, 1, a, 1, None) == INVALID
    assert lib.sasq_fakequant_fwd(a, a, 8, 7, a, 8, None) == INVALID
    assert lib.sasq_fakequant_fwd(a, a, -1, 1, a, 8, None) == INVALID
    assert lib.sasq_fakequant_fwd(a, a, 8, 1, None, 8, None) == INVALID
    # backward: workspace missing / too small
    assert lib.sasq_fakequant_bwd(a, a, a, a, 0, 8, 1, a, 8, None, 0, None) == WORKSPACE
    assert lib.sasq_fakequant_bwd(a, a, a, a, 0, 8, 1, a, 8, a, 16, None) == WORKSPACE
    assert lib.sasq_fakequant_bwd(a, a, a, None, 0, 8, 1, a, 8, a, 1 << 20, None) == INVALID
    # multi: scale index out of range, mixed parts
    d = (P.QDesc * 2)()
    d[0] = P.QDesc(a, a, a, a, 8, 3, 0)
    assert lib.sasq_fakequant_fwd_bwd_multi(d, 1, a, a, 2, 0, 1, 8, a, 1 << 20, None) == INVALID
    d[0] = P.QDesc(a, a, a, a, 8, 0, 0)
    d[1] = P.QDesc(a, None, a, None, 8, 0, 0)
    assert lib.sasq_fakequant_fwd_bwd_multi(d, 2, a, a, 2, 0, 1, 8, a, 1 << 20, None) == INVALID
    # an empty first tensor (numel 0, no pointers) does not decide which passes run: the list is valid and the call
    # gets as far as the workspace check
    d[0] = P.QDesc(None, None, None, None, 0, 0, 0)
    d[1] = P.QDesc(a, a, a, a, 8, 1, 0)
    assert lib.sasq_fakequant_fwd_bwd_multi(d, 2, a, a, 2, 0, 1, 8, None, 0, None) == WORKSPACE
    d[0] = P.QDesc(a, a, a, a, 8, 0, 0)
    d[1] = P.QDesc(a, a, a, a, 8, 0, 1)     # reserved must be 0
    assert lib.sasq_fakequant_fwd_bwd_multi(d, 2, a, a, 2, 0, 1, 8, a, 1 << 20, None) == INVALID


def test_issue_rate_probe_rejects_bad_arguments_before_touching_a_device():
    lib = P.load_library()
    lib.sasq_debug_int8_issue_rate.restype = ctypes.c_int
    lib.sasq_debug_int8_issue_rate.argtypes = [ctypes.c_int, ctypes.c_int, ctypes.POINTER(ctypes.c_double),
                                               ctypes.POINTER(ctypes.c_double), ctypes.c_void_p]
    a, b = ctypes.c_double(0), ctypes.c_double(0)
    assert lib.sasq_debug_int8_issue_rate(8, 256, ctypes.byref(a), ctypes.byref(b), None) == 1       # too few
    assert lib.sasq_debug_int8_issue_rate(64, 260, ctypes.byref(a), ctypes.byref(b), None) == 1      # width
    assert lib.sasq_debug_int8_issue_rate(64, 256, None, ctypes.byref(b), None) == 1                 # NULL output


def test_binding_rejects_cpu_tensors():
    import torch
    x = torch.zeros(8, dtype=torch.bfloat16)
    with pytest.raises(TypeError):
        P.sasq_fakequant_fwd(x, x, torch.ones(1), 8)
