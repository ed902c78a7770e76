"""Python access to the CPU oracle (oracle/cfi_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by tests/, by the smoke check and by the
benchmark's CPU-baseline leg.  The CUDA library and its binding never import
this package, and this package never imports them.

The wrappers below only marshal numpy arrays into the C functions; all of the
arithmetic is in the C file, which cites the passages of the paper it follows.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "cfi_oracle.c")
_LIB = os.path.join(_HERE, "libcfi_oracle.so")

ACT_NONE, ACT_GELU = 0, 1
_ACT = {"none": ACT_NONE, "gelu": ACT_GELU, ACT_NONE: ACT_NONE, ACT_GELU: ACT_GELU, None: ACT_NONE}


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP) if the shared object is stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.run(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-o", tmp, _SRC, "-lm"],
                       check=True)
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _c():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        f32p, i32p, u8p, f64p = (ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ctypes.c_int32),
                                 ctypes.POINTER(ctypes.c_uint8), ctypes.POINTER(ctypes.c_double))
        ci = ctypes.c_int
        lib.oracle_max_threads.restype = ci
        lib.oracle_set_threads.argtypes = [ci]
        lib.oracle_gelu.restype = ctypes.c_double
        lib.oracle_gelu.argtypes = [ctypes.c_double]
        lib.oracle_round_bf16.argtypes = [f32p, f32p, ctypes.c_int64]
        lib.oracle_pack.restype = ci
        lib.oracle_pack.argtypes = [f32p, u8p, ci, ci, ctypes.POINTER(ci), ctypes.POINTER(ci), f32p, i32p, i32p]
        lib.oracle_forward.argtypes = [f32p, i32p, i32p, f32p, ci, ci, ci, ci, ci, f32p, ci, f64p, f64p]
        lib.oracle_forward_recombination.argtypes = [f32p, i32p, i32p, f32p, ci, ci, ci, ci, ci, f32p, ci, f64p]
        lib.oracle_dense_forward.argtypes = [f32p, u8p, f32p, ci, ci, ci, f32p, ci, f64p]
        _lib = lib
    return _lib


def _p(a: Optional[np.ndarray], ct):
    return None if a is None else a.ctypes.data_as(ctypes.POINTER(ct))


def _f32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float32)


def _i32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.int32)


def max_threads() -> int:
    return int(_c().oracle_max_threads())


def set_threads(n: int) -> None:
    _c().oracle_set_threads(int(n))


def gelu(v: float) -> float:
    return float(_c().oracle_gelu(float(v)))


def round_bf16(a) -> np.ndarray:
    """fp32 -> nearest bf16 (ties to even), returned as fp32."""
    src = _f32(a)
    dst = np.empty_like(src)
    _c().oracle_round_bf16(_p(src, ctypes.c_float), _p(dst, ctypes.c_float), src.size)
    return dst


class NotConstantFanIn(ValueError):
    pass


def pack(w_dense, mask=None) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """Dense masked weight -> (values [n_act,k] f32, indices [n_act,k] i32, active_rows [n_act] i32)."""
    w = _f32(w_dense)
    out_f, in_f = w.shape
    m = None if mask is None else np.ascontiguousarray(mask, dtype=np.uint8)
    k, na = ctypes.c_int(0), ctypes.c_int(0)
    rc = _c().oracle_pack(_p(w, ctypes.c_float), _p(m, ctypes.c_uint8), out_f, in_f,
                          ctypes.byref(k), ctypes.byref(na), None, None, None)
    if rc:
        raise NotConstantFanIn("kept entries per non-ablated row are not constant")
    values = np.empty((na.value, k.value), dtype=np.float32)
    indices = np.empty((na.value, k.value), dtype=np.int32)
    rows = np.empty((na.value,), dtype=np.int32)
    _c().oracle_pack(_p(w, ctypes.c_float), _p(m, ctypes.c_uint8), out_f, in_f, ctypes.byref(k), ctypes.byref(na),
                     _p(values, ctypes.c_float), _p(indices, ctypes.c_int32), _p(rows, ctypes.c_int32))
    return values, indices, rows


def forward(values, indices, active_rows, bias, in_features: int, out_features: int, x, act="none",
            want_scale: bool = False):
    """Algorithm 1 + bias + ablated rows, double accumulation.  Returns y [B,out] f64 (and S if asked)."""
    v, ix, ar, xx = _f32(values), _i32(indices), _i32(active_rows), _f32(x)
    b = None if bias is None else _f32(bias)
    na, k = (v.shape if v.ndim == 2 else (0, 0))
    assert ix.shape == v.shape and ar.shape == (na,)
    assert xx.ndim == 2 and xx.shape[1] == in_features
    if ix.size:
        assert ix.min() >= 0 and ix.max() < in_features
    if ar.size:
        assert ar.min() >= 0 and ar.max() < out_features
    B = xx.shape[0]
    y = np.empty((B, out_features), dtype=np.float64)
    S = np.empty((B, out_features), dtype=np.float64) if want_scale else None
    _c().oracle_forward(_p(v, ctypes.c_float), _p(ix, ctypes.c_int32), _p(ar, ctypes.c_int32),
                        _p(b, ctypes.c_float), na, k, in_features, out_features, _ACT[act],
                        _p(xx, ctypes.c_float), B, _p(y, ctypes.c_double), _p(S, ctypes.c_double))
    return (y, S) if want_scale else y


def forward_recombination(values, indices, active_rows, bias, in_features: int, out_features: int, x, act="none"):
    """Eq. 3 (sum over the k columns of W^c of column (.) recombination of v)."""
    v, ix, ar, xx = _f32(values), _i32(indices), _i32(active_rows), _f32(x)
    b = None if bias is None else _f32(bias)
    na, k = (v.shape if v.ndim == 2 else (0, 0))
    B = xx.shape[0]
    y = np.empty((B, out_features), dtype=np.float64)
    _c().oracle_forward_recombination(_p(v, ctypes.c_float), _p(ix, ctypes.c_int32), _p(ar, ctypes.c_int32),
                                      _p(b, ctypes.c_float), na, k, in_features, out_features, _ACT[act],
                                      _p(xx, ctypes.c_float), B, _p(y, ctypes.c_double))
    return y


def dense_forward(w_dense, mask, bias, x, act="none"):
    """Eq. 1: brute-force dense product with the masked weight."""
    w, xx = _f32(w_dense), _f32(x)
    out_f, in_f = w.shape
    m = None if mask is None else np.ascontiguousarray(mask, dtype=np.uint8)
    b = None if bias is None else _f32(bias)
    B = xx.shape[0]
    y = np.empty((B, out_f), dtype=np.float64)
    _c().oracle_dense_forward(_p(w, ctypes.c_float), _p(m, ctypes.c_uint8), _p(b, ctypes.c_float), in_f, out_f,
                              _ACT[act], _p(xx, ctypes.c_float), B, _p(y, ctypes.c_double))
    return y


def stack_forward(layers, x, dtype: str = "f32"):
    """Chain of layers, each (values, indices, active_rows, bias, in, out, act).

    With dtype == "bf16" the numbers stored in bf16 (values, x) and every
    layer's output are rounded to bf16 where a bf16 layer stores them; the bias
    stays fp32 and sums stay in double.  Returns the list of every layer's (rounded) output as float64,
    and the list of un-rounded outputs and scales for per-layer comparison.
    """
    bf = dtype == "bf16"
    cur = round_bf16(x) if bf else _f32(x)
    outs, exact, scales = [], [], []
    for (v, ix, ar, b, in_f, out_f, act) in layers:
        vv = round_bf16(v) if bf else v
        y, S = forward(vv, ix, ar, b, in_f, out_f, cur, act=act, want_scale=True)
        exact.append(y)
        scales.append(S)
        cur = round_bf16(y.astype(np.float32)) if bf else y.astype(np.float32)
        outs.append(cur.astype(np.float64))
    return outs, exact, scales
