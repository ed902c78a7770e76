"""ctypes binding of the C-ABI library declared in include/cfi.h.

Same names as the C entry points; this module only marshals arguments (numpy
arrays for host data, torch tensors or raw integer addresses for device data)
and turns a non-zero status into CfiError.  Every step of the forward runs in
the library's CUDA kernels; there is no Python or CPU implementation behind
these calls, and loading fails loudly if the shared library cannot be built or
found.
"""
from __future__ import annotations

import ctypes
import os
from typing import List, Optional, Sequence, Tuple

import numpy as np

from . import build as _build

F32, BF16 = 0, 1
ACT_NONE, ACT_GELU = 0, 1
VARIANT_AUTO, VARIANT_SIMPLE, VARIANT_SPLITK, VARIANT_BATCH, VARIANT_DENSE_TC, VARIANT_SLAB = 0, 1, 2, 3, 4, 5
_DTYPES = {"f32": F32, "fp32": F32, "float32": F32, "bf16": BF16, "bfloat16": BF16, F32: F32, BF16: BF16}
_ACTS = {"none": ACT_NONE, None: ACT_NONE, "gelu": ACT_GELU, ACT_NONE: ACT_NONE, ACT_GELU: ACT_GELU}
_VARIANTS = {"auto": 0, "simple": 1, "splitk": 2, "batch": 3, "dense_tc": 4, "slab": 5, 0: 0, 1: 1, 2: 2, 3: 3, 4: 4, 5: 5}

EXPORTS = ("cfi_status_string", "cfi_pack", "cfi_compact_producer", "cfi_compact_consumer", "cfi_srigl_workspace_bytes",
           "cfi_srigl_update", "cfi_pack_device", "cfi_create", "cfi_create_layouts", "cfi_layer_add_layouts", "cfi_forward", "cfi_forward_variant", "cfi_forward_dense",
           "cfi_forward_host",
           "cfi_layer_info", "cfi_choose_variant", "cfi_dense_tile_shape", "cfi_device_status", "cfi_destroy",
           "cfi_stack_create", "cfi_stack_forward", "cfi_stack_destroy", "cfi_stack_forward_static",
           "cfi_probe_device", "cfi_probe_floor_launch")


class CfiError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = int(status)
        super().__init__(f"{where}: {_lib.cfi_status_string(status).decode()}")


class LayerInfo(ctypes.Structure):
    _fields_ = [("in_features", ctypes.c_int32), ("out_features", ctypes.c_int32), ("n_active", ctypes.c_int32),
                ("k", ctypes.c_int32), ("dtype", ctypes.c_int32), ("act", ctypes.c_int32),
                ("k_padded", ctypes.c_int32), ("batch_slab_columns", ctypes.c_int32),
                ("batch_row_stride", ctypes.c_int32), ("reserved", ctypes.c_int32),
                ("weight_bytes_splitk", ctypes.c_int64), ("weight_bytes_batch", ctypes.c_int64),
                ("device_bytes", ctypes.c_int64), ("bytes_small_batch", ctypes.c_int64), ("bytes_gather", ctypes.c_int64),
                ("bytes_dense", ctypes.c_int64), ("layouts", ctypes.c_int32), ("reserved2", ctypes.c_int32)]


class DeviceProbe(ctypes.Structure):
    _fields_ = [("sm_count", ctypes.c_int32), ("reserved", ctypes.c_int32), ("l2_bytes", ctypes.c_int64),
                ("smem_per_block_optin", ctypes.c_int64), ("sm_clock_mhz_nominal", ctypes.c_double),
                ("fma_tflops", ctypes.c_double), ("smem_load_gbs", ctypes.c_double), ("l2_read_gbs", ctypes.c_double),
                ("l2_read_same_lines_gbs", ctypes.c_double), ("empty_launch_us", ctypes.c_double)]

    def as_dict(self):
        return {n: getattr(self, n) for n, _ in self._fields_ if n != "reserved"}


def library_path() -> str:
    return _build.LIB


def _load() -> ctypes.CDLL:
    path = _build.LIB
    if not os.path.exists(path) or os.environ.get("CFI_REBUILD"):
        path = _build.build()
    lib = ctypes.CDLL(path)
    vp, ci = ctypes.c_void_p, ctypes.c_int32
    f32p, i32p, u8p = ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ctypes.c_int32), ctypes.POINTER(ctypes.c_uint8)
    lib.cfi_status_string.restype = ctypes.c_char_p
    lib.cfi_status_string.argtypes = [ctypes.c_int]
    lib.cfi_pack.argtypes = [f32p, u8p, ci, ci, i32p, i32p, f32p, i32p, i32p]
    lib.cfi_compact_producer.argtypes = [f32p, i32p, ci, ci, f32p, i32p]
    lib.cfi_compact_consumer.argtypes = [i32p, ci, ci, f32p, f32p, i32p, i32p, ci, ci, f32p, ci]
    lib.cfi_srigl_workspace_bytes.argtypes = [ci, ci, ctypes.POINTER(ctypes.c_size_t)]
    lib.cfi_srigl_update.argtypes = [vp, vp, vp, ci, ci, ctypes.c_int64, ctypes.c_float, vp, ctypes.c_size_t, i32p, i32p, vp]
    lib.cfi_pack_device.argtypes = [vp, vp, ci, ci, vp, ctypes.c_size_t, i32p, i32p, vp, vp, vp, vp]
    lib.cfi_create.argtypes = [f32p, i32p, i32p, f32p, ci, ci, ci, ci, ctypes.c_int, ctypes.c_int, ctypes.POINTER(vp)]
    lib.cfi_create_layouts.argtypes = [f32p, i32p, i32p, f32p, ci, ci, ci, ci, ctypes.c_int, ctypes.c_int, ci, ctypes.POINTER(vp)]
    lib.cfi_layer_add_layouts.argtypes = [vp, ci]
    lib.cfi_forward.argtypes = [vp, vp, vp, ci, vp]
    lib.cfi_forward_variant.argtypes = [vp, vp, vp, ci, vp, ctypes.c_int]
    lib.cfi_forward_dense.argtypes = [vp, vp, vp, ci, vp, ci, ci]
    lib.cfi_forward_host.argtypes = [vp, vp, vp, ci, vp]
    lib.cfi_layer_info.argtypes = [vp, ctypes.POINTER(LayerInfo)]
    lib.cfi_choose_variant.argtypes = [vp, ci, i32p]
    lib.cfi_dense_tile_shape.argtypes = [vp, ci, i32p, i32p]
    lib.cfi_device_status.argtypes = [vp, vp, i32p]
    lib.cfi_destroy.argtypes = [vp]
    lib.cfi_stack_create.argtypes = [ctypes.POINTER(vp), ci, ci, ctypes.POINTER(vp)]
    lib.cfi_stack_forward.argtypes = [vp, vp, vp, ci, vp]
    lib.cfi_stack_destroy.argtypes = [vp]
    lib.cfi_stack_forward_static.argtypes = [ctypes.POINTER(vp), ci, vp, vp, ci, vp]
    lib.cfi_probe_device.argtypes = [ctypes.POINTER(DeviceProbe)]
    lib.cfi_probe_floor_launch.argtypes = [ci, vp, ctypes.c_size_t, vp, vp]
    for name in EXPORTS:
        if name != "cfi_status_string":
            getattr(lib, name).restype = ctypes.c_int
    return lib


_lib = _load()


def _check(status: int, where: str) -> None:
    if status != 0:
        raise CfiError(status, where)


def _hp(a: Optional[np.ndarray], ct):
    return None if a is None else a.ctypes.data_as(ctypes.POINTER(ct))


def _dev_ptr(t) -> int:
    """Address of a device buffer: a torch CUDA tensor (contiguous) or an int."""
    if isinstance(t, int):
        return t
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError("expected a contiguous CUDA tensor")
    return t.data_ptr()


def _stream_handle(stream) -> int:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


def cfi_status_string(status: int) -> str:
    return _lib.cfi_status_string(int(status)).decode()


def cfi_pack(w_dense: np.ndarray, mask: Optional[np.ndarray] = None) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """Dense masked weight -> (values [n_act,k] f32, indices [n_act,k] i32, active_rows [n_act] i32)."""
    w = np.ascontiguousarray(w_dense, dtype=np.float32)
    if w.ndim != 2:
        raise ValueError("w_dense must be 2-D")
    m = None if mask is None else np.ascontiguousarray(mask, dtype=np.uint8)
    if m is not None and m.shape != w.shape:
        raise ValueError("mask shape differs from w_dense")
    out_f, in_f = w.shape
    k, na = ctypes.c_int32(0), ctypes.c_int32(0)
    _check(_lib.cfi_pack(_hp(w, ctypes.c_float), _hp(m, ctypes.c_uint8), out_f, in_f, ctypes.byref(k),
                         ctypes.byref(na), None, None, None), "cfi_pack")
    values = np.empty((na.value, k.value), dtype=np.float32)
    indices = np.empty((na.value, k.value), dtype=np.int32)
    rows = np.empty((na.value,), dtype=np.int32)
    _check(_lib.cfi_pack(_hp(w, ctypes.c_float), _hp(m, ctypes.c_uint8), out_f, in_f, ctypes.byref(k),
                         ctypes.byref(na), _hp(values, ctypes.c_float), _hp(indices, ctypes.c_int32),
                         _hp(rows, ctypes.c_int32)), "cfi_pack")
    return values, indices, rows


class Layer:
    """Owner of one cfi_layer_t handle."""

    def __init__(self, handle: int, in_features: int, out_features: int, dtype: int):
        self.handle, self.in_features, self.out_features, self.dtype = handle, in_features, out_features, dtype

    def close(self) -> None:
        if self.handle:
            _lib.cfi_destroy(self.handle)
            self.handle = 0

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


LAYOUT_SMALL_BATCH, LAYOUT_GATHER, LAYOUT_DENSE, LAYOUT_ALL = 1, 2, 4, 7


def cfi_create(values, indices, active_rows, bias, in_features: int, out_features: int, dtype="f32",
               act="none", layouts: int = LAYOUT_ALL) -> Layer:
    """cfi_create, or cfi_create_layouts when `layouts` (a bit set of LAYOUT_*) is not LAYOUT_ALL."""
    v = np.ascontiguousarray(values, dtype=np.float32)
    ix = np.ascontiguousarray(indices, dtype=np.int32)
    ar = np.ascontiguousarray(active_rows, dtype=np.int32)
    b = None if bias is None else np.ascontiguousarray(bias, dtype=np.float32)
    if v.shape != ix.shape or (v.ndim != 2 and v.size) or ar.ndim != 1:
        raise ValueError("values/indices must be [n_active, k] and active_rows [n_active]")
    n_active = ar.shape[0]
    k = v.shape[1] if v.ndim == 2 else 0
    if v.ndim == 2 and v.shape[0] != n_active:
        raise ValueError("values has a different number of rows than active_rows")
    if b is not None and b.shape != (out_features,):
        raise ValueError("bias must be [out_features]")
    h = ctypes.c_void_p()
    if layouts == LAYOUT_ALL:
        _check(_lib.cfi_create(_hp(v, ctypes.c_float), _hp(ix, ctypes.c_int32), _hp(ar, ctypes.c_int32),
                               _hp(b, ctypes.c_float), n_active, k, in_features, out_features, _DTYPES[dtype],
                               _ACTS[act], ctypes.byref(h)), "cfi_create")
    else:
        _check(_lib.cfi_create_layouts(_hp(v, ctypes.c_float), _hp(ix, ctypes.c_int32), _hp(ar, ctypes.c_int32),
                                       _hp(b, ctypes.c_float), n_active, k, in_features, out_features, _DTYPES[dtype],
                                       _ACTS[act], int(layouts), ctypes.byref(h)), "cfi_create_layouts")
    return Layer(h.value, in_features, out_features, _DTYPES[dtype])


def cfi_layer_add_layouts(layer: Layer, layouts: int) -> None:
    _check(_lib.cfi_layer_add_layouts(layer.handle, int(layouts)), "cfi_layer_add_layouts")


def cfi_compact_producer(bias, active_rows, out_features: int):
    """(bias_compact, rows_compact) of the layer in the paper's compact output form (ablated columns removed)."""
    rows = np.ascontiguousarray(active_rows, dtype=np.int32)
    b = None if bias is None else np.ascontiguousarray(bias, dtype=np.float32)
    bc, rc = np.empty(rows.shape[0], np.float32), np.empty(rows.shape[0], np.int32)
    _check(_lib.cfi_compact_producer(_hp(b, ctypes.c_float), _hp(rows, ctypes.c_int32), rows.shape[0], out_features,
                                     _hp(bc, ctypes.c_float), _hp(rc, ctypes.c_int32)), "cfi_compact_producer")
    return bc, rc


def cfi_compact_consumer(prod_active_rows, prod_out: int, prod_const, values, indices, active_rows, bias):
    """Returns (values, indices, bias) of the layer that reads a compact output; inputs are not modified."""
    pr = np.ascontiguousarray(prod_active_rows, dtype=np.int32)
    pc = None if prod_const is None else np.ascontiguousarray(prod_const, dtype=np.float32)
    v = np.array(values, dtype=np.float32, order="C", copy=True)
    ix = np.array(indices, dtype=np.int32, order="C", copy=True)
    rows = np.ascontiguousarray(active_rows, dtype=np.int32)
    b = np.array(bias, dtype=np.float32, order="C", copy=True)
    n_active, k = v.shape
    _check(_lib.cfi_compact_consumer(_hp(pr, ctypes.c_int32), pr.shape[0], prod_out, _hp(pc, ctypes.c_float),
                                     _hp(v, ctypes.c_float), _hp(ix, ctypes.c_int32), _hp(rows, ctypes.c_int32), n_active, k,
                                     _hp(b, ctypes.c_float), b.shape[0]), "cfi_compact_consumer")
    return v, ix, b


def cfi_srigl_update(w, mask, grad, K: int, gamma_sal: float, stream=None):
    """One SRigL mask update in place on device tensors w (float32), mask (uint8), grad (float32), all [out, in] and
    contiguous.  Returns (k_new, n_active_new).  The workspace is a torch allocation made here."""
    import torch
    out_f, in_f = w.shape
    nbytes = ctypes.c_size_t(0)
    _check(_lib.cfi_srigl_workspace_bytes(out_f, in_f, ctypes.byref(nbytes)), "cfi_srigl_workspace_bytes")
    ws = torch.empty(nbytes.value + 256, dtype=torch.uint8, device=w.device)
    base = (ws.data_ptr() + 255) & ~255
    k_new, n_act = ctypes.c_int32(0), ctypes.c_int32(0)
    _check(_lib.cfi_srigl_update(_dev_ptr(w), _dev_ptr(mask), _dev_ptr(grad), out_f, in_f, int(K), float(gamma_sal), base,
                                 nbytes.value, ctypes.byref(k_new), ctypes.byref(n_act), _stream_handle(stream)),
           "cfi_srigl_update")
    return k_new.value, n_act.value


def cfi_pack_device(w, mask, stream=None):
    """cfi_pack on device tensors w (float32) and mask (uint8), both [out, in] and contiguous.  Returns device tensors
    (values [n_active, k] float32, indices [n_active, k] int32, active_rows [n_active] int32)."""
    import torch
    out_f, in_f = w.shape
    ws = torch.empty(8 * out_f + 512, dtype=torch.uint8, device=w.device)
    base = (ws.data_ptr() + 255) & ~255
    k, na = ctypes.c_int32(0), ctypes.c_int32(0)
    st = _stream_handle(stream)
    _check(_lib.cfi_pack_device(_dev_ptr(w), _dev_ptr(mask), out_f, in_f, base, 8 * out_f + 256, ctypes.byref(k),
                                ctypes.byref(na), None, None, None, st), "cfi_pack_device")
    values = torch.empty((na.value, k.value), dtype=torch.float32, device=w.device)
    indices = torch.empty((na.value, k.value), dtype=torch.int32, device=w.device)
    rows = torch.empty((na.value,), dtype=torch.int32, device=w.device)
    if na.value:
        _check(_lib.cfi_pack_device(_dev_ptr(w), _dev_ptr(mask), out_f, in_f, base, 8 * out_f + 256, ctypes.byref(k),
                                    ctypes.byref(na), _dev_ptr(values), _dev_ptr(indices), _dev_ptr(rows), st), "cfi_pack_device")
    return values, indices, rows


def cfi_forward(layer: Layer, x, y, batch: int, stream=None) -> None:
    _check(_lib.cfi_forward(layer.handle, _dev_ptr(x), _dev_ptr(y), batch, _stream_handle(stream)), "cfi_forward")


def cfi_forward_variant(layer: Layer, x, y, batch: int, stream=None, variant="auto") -> None:
    _check(_lib.cfi_forward_variant(layer.handle, _dev_ptr(x), _dev_ptr(y), batch, _stream_handle(stream),
                                    _VARIANTS[variant]), "cfi_forward_variant")


def cfi_forward_dense(layer: Layer, x, y, batch: int, stream=None, tile: int = 0, cluster: int = 0) -> None:
    """The tensor-core variant with its launch shape given (0 = chosen by the library); see include/cfi.h."""
    _check(_lib.cfi_forward_dense(layer.handle, _dev_ptr(x), _dev_ptr(y), batch, _stream_handle(stream), tile, cluster),
           "cfi_forward_dense")


def cfi_forward_host(layer: Layer, x_host, y_host, batch: int, stream=None) -> None:
    """x_host / y_host: CPU torch tensors (pinned for asynchronous copies) or numpy arrays."""
    xp = x_host.data_ptr() if hasattr(x_host, "data_ptr") else x_host.ctypes.data
    yp = y_host.data_ptr() if hasattr(y_host, "data_ptr") else y_host.ctypes.data
    _check(_lib.cfi_forward_host(layer.handle, xp, yp, batch, _stream_handle(stream)), "cfi_forward_host")


def cfi_layer_info(layer: Layer) -> LayerInfo:
    info = LayerInfo()
    _check(_lib.cfi_layer_info(layer.handle, ctypes.byref(info)), "cfi_layer_info")
    return info


def cfi_choose_variant(layer: Layer, batch: int) -> int:
    v = ctypes.c_int32(0)
    _check(_lib.cfi_choose_variant(layer.handle, batch, ctypes.byref(v)), "cfi_choose_variant")
    return v.value


def cfi_dense_tile_shape(layer: Layer, batch: int):
    """(outputs per tile, CTAs sharing a tile through a cluster) of the tensor-core variant at this batch size."""
    tn, cl = ctypes.c_int32(0), ctypes.c_int32(0)
    _check(_lib.cfi_dense_tile_shape(layer.handle, batch, ctypes.byref(tn), ctypes.byref(cl)), "cfi_dense_tile_shape")
    return tn.value, cl.value


def cfi_device_status(layer: Layer, stream=None) -> int:
    flag = ctypes.c_int32(0)
    st = _lib.cfi_device_status(layer.handle, _stream_handle(stream), ctypes.byref(flag))
    if st not in (0, 9):
        raise CfiError(st, "cfi_device_status")
    return flag.value


def cfi_destroy(layer: Layer) -> None:
    layer.close()


class Stack:
    def __init__(self, handle: int, layers: Sequence[Layer], max_batch: int):
        self.handle, self.layers, self.max_batch = handle, list(layers), max_batch

    def close(self) -> None:
        if self.handle:
            _lib.cfi_stack_destroy(self.handle)
            self.handle = 0

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def cfi_stack_create(layers: Sequence[Layer], max_batch: int) -> Stack:
    arr = (ctypes.c_void_p * len(layers))(*[l.handle for l in layers])
    h = ctypes.c_void_p()
    _check(_lib.cfi_stack_create(arr, len(layers), max_batch, ctypes.byref(h)), "cfi_stack_create")
    return Stack(h.value, layers, max_batch)


def cfi_stack_forward(stack: Stack, x, y, batch: int, stream=None) -> None:
    _check(_lib.cfi_stack_forward(stack.handle, _dev_ptr(x), _dev_ptr(y), batch, _stream_handle(stream)),
           "cfi_stack_forward")


def cfi_stack_destroy(stack: Stack) -> None:
    stack.close()


def cfi_stack_forward_static(layers: Sequence[Layer], x, y, batch: int, stream=None) -> None:
    """Chain of layers with the intermediates in the library's fixed 8 MiB device array: no allocation.

    For callers that may not call cudaMalloc (see include/cfi.h).  batch * widest intermediate * element size
    must not exceed 4 MiB; calls that can overlap on the GPU race on the shared array.
    """
    arr = (ctypes.c_void_p * len(layers))(*[l.handle for l in layers])
    _check(_lib.cfi_stack_forward_static(arr, len(layers), _dev_ptr(x), _dev_ptr(y), batch, _stream_handle(stream)),
           "cfi_stack_forward_static")


def cfi_probe_device() -> DeviceProbe:
    p = DeviceProbe()
    _check(_lib.cfi_probe_device(ctypes.byref(p)), "cfi_probe_device")
    return p


def cfi_probe_floor_launch(kind: int, buf, scratch, stream=None) -> None:
    """One launch of the no-work kernel (kind 0: empty, kind 1: one DRAM round trip per CTA); see include/cfi.h."""
    nbytes = 0 if buf is None else buf.numel() * buf.element_size()
    _check(_lib.cfi_probe_floor_launch(kind, 0 if buf is None else _dev_ptr(buf), nbytes, _dev_ptr(scratch), _stream_handle(stream)),
           "cfi_probe_floor_launch")
