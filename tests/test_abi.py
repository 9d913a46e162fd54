"""The C-ABI library builds, loads and exports every symbol include/psa.h declares; host-side
argument validation returns the documented codes.  No GPU, no compute calls."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def B():
    from paper_2609_37001_b200 import build
    build.build()
    from paper_2609_37001_b200 import binding
    binding.lib()
    return binding


def _declared_functions():
    src = open(os.path.join(ROOT, "include", "psa.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(psa_[a-z_]+)\s*\(", src)))


def test_exports_every_declared_symbol(B):
    names = _declared_functions()
    assert {"psa_mask_build", "psa_attn_fwd", "psa_mask_sizes", "psa_status_string"} <= set(names)
    lib = ctypes.CDLL(B.LIB_PATH)
    for n in names:
        assert hasattr(lib, n), n


def test_status_strings(B):
    assert B.status_string(0) == "ok"
    for code in (-1, -2, -3, -4, -5, -6):
        assert B.status_string(code) not in ("ok", "unknown status")
    assert B.status_string(-99) == "unknown status"


def test_mask_sizes_host_arithmetic(B):
    # identity head: NB pairs; all-covering head: NB^2 pairs
    nb, nnz = B.psa_mask_sizes([(1, 0, 0, 1, 0, 0), (21, 0, 0, 15, 0, 0)], (21, 45, 80), (1, 16, 16))
    assert (nb, nnz) == (315, 315 + 315 * 315)
    nb, nnz = B.psa_mask_sizes([(5, 0, 6, 1, 0, 1)], (30, 1, 1), (1, 1, 1))
    assert (nb, nnz) == (30, 770)   # closed-form count C(30; 5, 0, 6) = 770


def test_invalid_arguments_are_rejected_on_the_host(B):
    lib = B.lib()
    hp = B._params_array([(1, 0, 0, 1, 0, 0)])
    prob = B.make_problem(1, (1, 16, 16), 0.1, 128 * 256, 128)
    nb = ctypes.c_int64()
    assert lib.psa_mask_sizes(hp, ctypes.byref(prob), 0, 4, 4, ctypes.byref(nb), None) == B.PSA_ERR_INVALID_ARG
    bad = B._params_array([(0, 0, 0, 1, 0, 0)])   # width 0
    assert lib.psa_mask_sizes(bad, ctypes.byref(prob), 4, 16, 16, ctypes.byref(nb), ctypes.byref(nb)) == B.PSA_ERR_INVALID_ARG
    # attention: null pointers, misalignment, wrong head_dim, unsupported tile, bad scale
    f = lib.psa_attn_fwd
    assert f(None, None, None, None, None, hp, ctypes.byref(prob), 1, 16, 16, None) == B.PSA_ERR_INVALID_ARG
    assert f(17, 32, 48, 64, 80, hp, ctypes.byref(prob), 1, 16, 16, None) == B.PSA_ERR_INVALID_ARG
    p64 = B.make_problem(1, (1, 16, 16), 0.1, 64 * 256, 64, head_dim=64)
    assert f(16, 32, 48, 64, 80, hp, ctypes.byref(p64), 1, 16, 16, None) == B.PSA_ERR_UNSUPPORTED
    ptile = B.make_problem(1, (1, 10, 10), 0.1, 128 * 100, 128)
    assert f(16, 32, 48, 64, 80, hp, ctypes.byref(ptile), 1, 16, 16, None) == B.PSA_ERR_UNSUPPORTED
    pscale = B.make_problem(1, (1, 16, 16), -1.0, 128 * 256, 128)
    assert f(16, 32, 48, 64, 80, hp, ctypes.byref(pscale), 1, 16, 16, None) == B.PSA_ERR_INVALID_ARG
    assert f(16, 32, 48, 16, 80, hp, ctypes.byref(prob), 1, 16, 16, None) == B.PSA_ERR_INVALID_ARG  # out aliases q
    # mask build: col_idx without row_ptr
    assert lib.psa_mask_build(hp, ctypes.byref(prob), 1, 16, 16, None, None, 64, 10, None) == B.PSA_ERR_INVALID_ARG
    assert lib.psa_mask_build(hp, ctypes.byref(prob), 1, 16, 16, None, 64, 128, 0, None) == B.PSA_ERR_CAPACITY
