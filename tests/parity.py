"""Shared helpers for the GPU parity tests: run one layer through the C-ABI library and through the oracle."""
import numpy as np

import oracle
from paper_2305_02299_b200 import inputs

TOL = {"f32": 1e-5, "bf16": 2e-2}   # max |y - y_oracle| / S with S = |bias| + sum_j |w x|  (error relative to the sum's scale)


def torch_dtype(dtype):
    import torch
    return torch.float32 if dtype == "f32" else torch.bfloat16


def to_device(x_np, dtype):
    import torch
    return torch.from_numpy(np.ascontiguousarray(x_np)).to(device="cuda", dtype=torch_dtype(dtype)).contiguous()


def oracle_layer(layer, x_np, dtype="f32", act="none", packed=None):
    """Oracle result for a DenseMaskedLayer in the storage precision `dtype`: (y f64, S f64)."""
    v, ix, rows = packed if packed is not None else oracle.pack(layer.w_dense, layer.mask)
    if dtype == "bf16":
        v, x_np = oracle.round_bf16(v), oracle.round_bf16(x_np)
    return oracle.forward(v, ix, rows, layer.bias, layer.in_features, layer.out_features, x_np, act=act,
                          want_scale=True)


def device_layer(layer, dtype="f32", act="none"):
    from paper_2305_02299_b200 import binding as cfi
    v, ix, rows = cfi.cfi_pack(layer.w_dense, layer.mask)
    return cfi.cfi_create(v, ix, rows, layer.bias, layer.in_features, layer.out_features, dtype=dtype, act=act)


def run_device(dl, x_np, dtype="f32", variant="auto", canary=True, dense_shape=None):
    """Forward through the library; y is allocated inside guard bands that must come back untouched.
    dense_shape = (tile, cluster) runs the tensor-core variant with that launch shape (cfi_forward_dense)."""
    import torch
    from paper_2305_02299_b200 import binding as cfi
    B = x_np.shape[0]
    x_d = to_device(x_np, dtype)
    guard = 64
    n = B * dl.out_features
    buf = torch.full((n + 2 * guard,), 12345.0, device="cuda", dtype=torch_dtype(dtype))
    y_d = buf[guard:guard + n]
    assert y_d.data_ptr() % 16 == 0
    if dense_shape is not None:
        cfi.cfi_forward_dense(dl, x_d, y_d, B, tile=dense_shape[0], cluster=dense_shape[1])
    else:
        cfi.cfi_forward_variant(dl, x_d, y_d, B, variant=variant)
    torch.cuda.synchronize()
    if canary:
        assert torch.all(buf[:guard] == 12345.0) and torch.all(buf[guard + n:] == 12345.0), "wrote outside y"
    return y_d.to(torch.float64).cpu().numpy().reshape(B, dl.out_features)


def scaled_error(y, y_ref, S):
    if y.size == 0:
        return 0.0
    return float(np.max(np.abs(y - y_ref) / np.maximum(S, 1e-300)))


def assert_parity(y, y_ref, S, dtype, what=""):
    """The stated bound (error against the scale of the sum) and, for bf16 storage, the bound the arithmetic itself
    allows: exact products of the rounded inputs, fp32 accumulation (a few 2^-24 of S for these fan-ins, 1e-5 of S
    with room for the activation) and ONE rounding to nearest at the store (2^-9 of |y|, allowed 2^-8).  The second
    bound is what catches inputs rounded the wrong way, which the first, at 2e-2 of S, would let through."""
    err = scaled_error(y, y_ref, S)
    assert err <= TOL[dtype], f"{what}: scaled error {err:.3e}"
    if dtype == "bf16" and y.size:
        excess = np.abs(y - y_ref) - (2.0 ** -8 * np.abs(y_ref) + 1e-5 * S)
        i = np.unravel_index(np.argmax(excess), excess.shape)
        assert excess[i] <= 0.0, f"{what}: bf16 result off by more than its store rounding at {i}: {y[i]} vs {y_ref[i]} (S {S[i]})"
    return err


def check_layer(layer, x_np, dtype="f32", act="none", variants=("auto",), tol=None):
    y_ref, S = oracle_layer(layer, x_np, dtype, act)
    dl = device_layer(layer, dtype, act)
    errs = {}
    try:
        for v in variants:
            y = run_device(dl, x_np, dtype, v)
            assert np.all(np.isfinite(y)), f"variant {v}: non-finite output"
            errs[v] = assert_parity(y, y_ref, S, dtype, f"variant {v}")
            assert errs[v] <= (TOL[dtype] if tol is None else tol), f"variant {v}: scaled error {errs[v]:.3e}"
    finally:
        dl.close()
    return errs
