"""The C-ABI library builds, loads and exports every symbol include/adadim.h declares (no GPU
work), and the host-side argument checks answer with the documented status codes."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2309_15531_b200 import build
    path = build.build()
    return ctypes.CDLL(path)


def test_every_declared_symbol_is_exported(lib):
    header = open(os.path.join(ROOT, "include", "adadim.h")).read()
    names = re.findall(r"ADADIM_API\s+[\w\s\*]+?\b(adadim_\w+)\s*\(", header)
    assert len(names) >= 9 and {"adadim_hessian_accumulate", "adadim_quantize_rtn", "adadim_quantize_gptq",
                                "adadim_score_select"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n


def test_strerror_and_version(lib):
    lib.adadim_strerror.restype = ctypes.c_char_p
    assert lib.adadim_strerror(0) == b"ok"
    assert b"workspace" in lib.adadim_strerror(6)
    assert lib.adadim_version() >= 100


def test_workspace_sizes_grow_with_the_problem(lib):
    f = lib.adadim_workspace_bytes
    f.restype = ctypes.c_size_t
    f.argtypes = [ctypes.c_int, ctypes.c_int64, ctypes.c_int64, ctypes.c_int, ctypes.c_int]
    assert f(0, 0, 4096, 3, 128) == 0                              # bf16 activations need no Hessian workspace
    assert f(0, 256, 512, 0, 0) >= 256 * 3 * 512 * 2 + 9 * 512 * 512 * 4     # an fp32 chunk of 256 tokens: three bf16 pieces + the widened product
    g1, g2 = f(1, 256, 512, 3, 128), f(1, 4096, 4096, 3, 128)
    s1, s2 = f(2, 256, 512, 3, 128), f(2, 4096, 4096, 3, 128)
    assert 0 < g1 < g2 and 0 < s1 < s2
    assert s2 >= 2 * 4096 * 4096 * 2                                # W - Q in bf16 for two dimensions
    assert f(3, 0, 4096, 0, 0) >= 4096 * 4096 * 8


def test_host_side_argument_checks_need_no_gpu(lib):
    from paper_2309_15531_b200 import binding as B
    L = B.lib()
    q = B.QTensorC(16, 16, 16)
    # NULL weight
    assert L.adadim_quantize_rtn(None, B.F16, 128, 128, 128, 3, 128, B.DIM_OC, ctypes.byref(q), None, None) == 1
    # bad bits / group / dim
    assert L.adadim_quantize_rtn(16, B.F16, 128, 128, 128, 5, 128, B.DIM_OC, ctypes.byref(q), None, None) == 4
    assert L.adadim_quantize_rtn(16, B.F16, 128, 128, 128, 3, 100, B.DIM_OC, ctypes.byref(q), None, None) == 4
    assert L.adadim_quantize_rtn(16, B.F16, 128, 128, 128, 3, 128, 7, ctypes.byref(q), None, None) == 4
    # shape and alignment
    assert L.adadim_quantize_rtn(16, B.F16, 128, 100, 128, 3, 128, B.DIM_OC, ctypes.byref(q), None, None) == 2
    assert L.adadim_quantize_rtn(18, B.F16, 128, 128, 128, 3, 128, B.DIM_OC, ctypes.byref(q), None, None) == 5
    assert L.adadim_quantize_rtn(16, B.BF16, 128, 128, 128, 3, 128, B.DIM_OC, ctypes.byref(q), None, None) == 3
    # missing output tensor for a requested dimension
    assert L.adadim_quantize_rtn(16, B.F16, 128, 128, 128, 3, 128, B.DIM_BOTH, ctypes.byref(q), None, None) == 1
    # empty problem: accepted
    assert L.adadim_quantize_rtn(None, B.F16, 0, 128, 128, 3, 128, B.DIM_OC, None, None, None) == 0
    # hessian
    assert L.adadim_hessian_accumulate(16, B.F16, 64, 64, 64, 16, None, None, None, 0, None) == 3
    assert L.adadim_hessian_accumulate(16, B.BF16, 64, 60, 64, 16, None, None, None, 0, None) == 2
    # gptq: block size, workspace
    assert L.adadim_quantize_gptq(16, B.F16, 128, 128, 128, 16, None, 3, 128, B.DIM_OC, 0.01, 64,
                                  ctypes.byref(q), None, None, None, 256, 1 << 40, None) == 4
    assert L.adadim_quantize_gptq(16, B.F16, 128, 128, 128, 16, None, 3, 128, B.DIM_OC, 0.01, 128,
                                  ctypes.byref(q), None, None, None, 256, 1024, None) == 6
    # score: needs at least one quantized tensor
    assert L.adadim_score_select(16, B.F16, 128, 128, 128, 16, 3, 128, None, None, 16, 16, None, 256, 1 << 40, None) == 1
    # factor
    assert L.adadim_cholesky_inverse_factor(16, 100, 0.01, 16, None, 256, 1 << 40, None) == 2
