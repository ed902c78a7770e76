"""Condensed constant-fan-in sparse linear forward for B200 (sm_100a).

`paper_2305_02299_b200.binding` is the thin ctypes layer over the C-ABI library
declared in include/cfi.h; `paper_2305_02299_b200.inputs` draws the seeded
synthetic layers and activations used by tests and benchmarks.  The binding is
loaded on first use so that the input generators stay importable on their own.
"""
import importlib

_BINDING_NAMES = ("cfi_pack", "cfi_compact_producer", "cfi_compact_consumer", "cfi_srigl_update", "cfi_pack_device", "cfi_create", "cfi_forward", "cfi_forward_variant", "cfi_forward_host",
                  "cfi_destroy", "cfi_device_status", "cfi_status_string", "cfi_layer_info",
                  "cfi_stack_create", "cfi_stack_forward", "cfi_stack_destroy", "cfi_stack_forward_static", "cfi_probe_device", "cfi_choose_variant",
                  "cfi_dense_tile_shape",
                  "CfiError", "Layer", "Stack", "library_path")


def __getattr__(name):
    if name in _BINDING_NAMES or name == "binding":
        mod = importlib.import_module(".binding", __name__)
        return mod if name == "binding" else getattr(mod, name)
    raise AttributeError(name)
