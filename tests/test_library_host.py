"""Host-side checks of the C-ABI library that need no GPU: it loads, exports what the header declares,
cfi_pack agrees bit for bit with the oracle's pack, and argument errors come back as status codes."""
import ctypes
import os
import re

import numpy as np
import pytest

import oracle
from paper_2305_02299_b200 import binding as cfi, inputs

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "cfi.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(cfi_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib = ctypes.CDLL(cfi.library_path())
    names = declared_functions()
    assert "cfi_pack" in names and "cfi_create" in names and "cfi_forward" in names
    for n in names:
        assert hasattr(lib, n), f"{n} declared in cfi.h but not exported"
    assert set(names) == set(cfi.EXPORTS), "binding and header disagree on the entry points"


def test_oracle_and_library_share_no_code():
    """Neither side imports or includes the other."""
    for fn in os.listdir(os.path.join(ROOT, "oracle")):
        if fn.endswith((".py", ".c", ".h")):
            src = open(os.path.join(ROOT, "oracle", fn)).read()
            assert "paper_2305_02299_b200" not in src and "cfi.h" not in src and "csrc" not in src
    pkg = os.path.join(ROOT, "paper_2305_02299_b200")
    for base, _, files in os.walk(pkg):
        for fn in files:
            if fn.endswith((".py", ".cu", ".cpp", ".h", ".cuh")):
                src = open(os.path.join(base, fn)).read()
                assert not re.search(r"^\s*(import|from)\s+oracle\b", src, flags=re.M), fn
                assert "cfi_oracle" not in src, fn


@pytest.mark.parametrize("in_f,out_f,k,nabl", [(16, 8, 3, 2), (768, 96, 77, 9), (33, 17, 33, 0), (7, 5, 1, 4),
                                                (3072, 40, 307, 4), (5, 3, 2, 3), (1, 1, 1, 0)])
def test_pack_bit_exact_against_oracle(in_f, out_f, k, nabl):
    L = inputs.make_layer(in_f, out_f, k, n_ablated=nabl, seed=5)
    v, ix, rows = cfi.cfi_pack(L.w_dense, L.mask)
    ov, oix, orows = oracle.pack(L.w_dense, L.mask)
    assert np.array_equal(ix, oix) and np.array_equal(rows, orows)
    assert np.array_equal(v.view(np.uint32), ov.view(np.uint32))
    v2, ix2, rows2 = cfi.cfi_pack(L.w_dense, None)           # structure from w != 0 (no kept zero here)
    assert np.array_equal(ix2, oix) and np.array_equal(rows2, orows)


def test_pack_mask_semantics_and_errors():
    W = np.array([[0.0, 1.0, -0.0, 2.0], [0.0, 0.0, 3.0, 4.0]], dtype=np.float32)
    _, ix, _ = cfi.cfi_pack(W, None)
    assert np.array_equal(ix, oracle.pack(W, None)[1]) and np.array_equal(ix, [[1, 3], [2, 3]])
    M = np.array([[1, 1, 0, 0], [0, 0, 1, 1]], dtype=np.uint8)
    v, ix, _ = cfi.cfi_pack(W, M)
    assert np.array_equal(ix, [[0, 1], [2, 3]]) and np.array_equal(v, [[0, 1], [3, 4]])
    M[1, 0] = 1
    with pytest.raises(cfi.CfiError) as e:
        cfi.cfi_pack(W, M)
    assert e.value.status == 3
    with pytest.raises(oracle.NotConstantFanIn):
        oracle.pack(W, M)
    v, ix, rows = cfi.cfi_pack(np.zeros((3, 4), np.float32), None)   # every row ablated
    assert v.shape == (0, 0) and rows.shape == (0,)
    v, ix, rows = cfi.cfi_pack(np.zeros((0, 4), np.float32), None)
    assert rows.shape == (0,)


def test_pack_null_and_shape_errors():
    lib = ctypes.CDLL(cfi.library_path())
    lib.cfi_pack.restype = ctypes.c_int
    k, na = ctypes.c_int32(), ctypes.c_int32()
    w = (ctypes.c_float * 4)(1, 0, 0, 1)
    assert lib.cfi_pack(None, None, 2, 2, ctypes.byref(k), ctypes.byref(na), None, None, None) == 1
    assert lib.cfi_pack(w, None, -1, 2, ctypes.byref(k), ctypes.byref(na), None, None, None) == 2
    vals = (ctypes.c_float * 2)()
    assert lib.cfi_pack(w, None, 2, 2, ctypes.byref(k), ctypes.byref(na), vals, None, None) == 1  # partial buffers


def test_create_rejects_bad_arguments_before_touching_cuda():
    v = np.ones((2, 2), np.float32)
    rows = np.array([0, 1], np.int32)
    bad = lambda **kw: pytest.raises(cfi.CfiError, **kw)
    with bad() as e:
        cfi.cfi_create(v, np.array([[0, 5], [1, 2]], np.int32), rows, None, 4, 3)      # column out of range
    assert e.value.status == 4
    with bad() as e:
        cfi.cfi_create(v, np.array([[0, -1], [1, 2]], np.int32), rows, None, 4, 3)
    assert e.value.status == 4
    with bad() as e:
        cfi.cfi_create(v, np.zeros((2, 2), np.int32), np.array([0, 0], np.int32), None, 4, 3)  # repeated row
    assert e.value.status == 4
    with bad() as e:
        cfi.cfi_create(v, np.zeros((2, 2), np.int32), np.array([0, 3], np.int32), None, 4, 3)  # row out of range
    assert e.value.status == 4
    with bad() as e:
        cfi.cfi_create(v, np.zeros((2, 2), np.int32), rows, None, 1, 3)                 # k > in
    assert e.value.status == 2
    with bad() as e:
        cfi.cfi_create(v, np.zeros((2, 2), np.int32), rows, None, 4, 1)                 # n_active > out
    assert e.value.status == 2
    lib = ctypes.CDLL(cfi.library_path())
    h = ctypes.c_void_p()
    assert lib.cfi_create(None, None, None, None, 0, 0, 4, 3, 7, 0, ctypes.byref(h)) == 6   # unknown dtype
    assert lib.cfi_create(None, None, None, None, 2, 2, 4, 3, 0, 0, ctypes.byref(h)) == 1   # NULL arrays
    assert lib.cfi_forward(None, None, None, 1, None) == 1
    assert lib.cfi_destroy(None) == 0 and lib.cfi_stack_destroy(None) == 0
    for layouts in (0, 8, -1):                                                          # empty or unknown layout set
        with bad() as e:
            cfi.cfi_create(v, np.zeros((2, 2), np.int32), rows, None, 4, 3, layouts=layouts)
        assert e.value.status == 6
    assert lib.cfi_layer_add_layouts(None, 1) == 1 and lib.cfi_forward_dense(None, None, None, 1, None, 0, 0) == 1
    assert lib.cfi_probe_floor_launch(2, None, 0, None, None) == 6 and lib.cfi_probe_floor_launch(0, None, 0, None, None) == 1


def test_no_cpu_fallback():
    """Without a CUDA device, creating a layer must fail with a CUDA error rather than run elsewhere."""
    import torch
    if torch.cuda.is_available():
        pytest.skip("a CUDA device is present")
    L = inputs.make_layer(8, 4, 2, seed=0)
    v, ix, rows = cfi.cfi_pack(L.w_dense, L.mask)
    with pytest.raises(cfi.CfiError) as e:
        cfi.cfi_create(v, ix, rows, L.bias, 8, 4)
    assert e.value.status in (7, 8)


def test_status_strings():
    assert cfi.cfi_status_string(0) == "CFI_OK"
    for s in range(1, 11):
        assert cfi.cfi_status_string(s).startswith("CFI_ERR_")
