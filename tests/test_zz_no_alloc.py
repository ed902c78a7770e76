"""cfi_stack_forward_static: the layer chain for callers that may not allocate device memory.

Some users of this library run where cudaMalloc is not allowed once the process is set up (a serving loop
with hard latency bounds, a fixed memory budget, a host application that forbids allocations after start).
For them the chain's intermediate activations sit in a fixed array inside the library instead of buffers
created by cfi_stack_create.  This test calls that entry point through the C ABI twice in a row, with
different inputs, and checks each result against cfi_stack_forward on the same layers and against the CPU
oracle's chain; the second call also shows that what the first one left in the shared array does not leak
into the result.  A further test reads the device's free memory around a call: it must not move.

Collected last on purpose (file name), so a run that stops at the first failure has run everything else.
"""
import numpy as np
import pytest

import oracle
from paper_2305_02299_b200 import inputs

pytestmark = pytest.mark.gpu


def _layers(dtype):
    from paper_2305_02299_b200 import binding as cfi
    s = inputs.StackWorkload(blocks=2, d_model=96, d_hidden=384, k_up=10, k_down=38, batch=70)
    out = []
    for L, sp in zip(s.layers(seed=3), s.layer_specs()):
        v, ix, rows = cfi.cfi_pack(L.w_dense, L.mask)
        out.append(cfi.cfi_create(v, ix, rows, L.bias, sp[0], sp[1], dtype=dtype, act=sp[4]))
    return s, out


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_static_chain_matches_allocating_chain_twice(dtype):
    import torch
    from paper_2305_02299_b200 import binding as cfi
    tdt = torch.float32 if dtype == "f32" else torch.bfloat16
    s, layers = _layers(dtype)
    o_layers = []
    for L, sp in zip(s.layers(seed=3), s.layer_specs()):
        v, ix, rows = oracle.pack(L.w_dense, L.mask)
        o_layers.append((v, ix, rows, L.bias, sp[0], sp[1], sp[4]))
    stack = cfi.cfi_stack_create(layers, 70)
    for call, batch in enumerate((70, 33)):          # two calls in a row, different inputs and batch sizes
        x_np = s.x(seed=10 + call, batch=batch)
        x = torch.from_numpy(x_np).to("cuda", tdt)
        y_ref = torch.empty((batch, 96), device="cuda", dtype=tdt)
        y_new = torch.full((batch, 96), 777.0, device="cuda", dtype=tdt)
        cfi.cfi_stack_forward(stack, x, y_ref, batch)
        cfi.cfi_stack_forward_static(layers, x, y_new, batch)
        torch.cuda.synchronize()
        a, b = y_new.double().cpu().numpy(), y_ref.double().cpu().numpy()
        assert np.all(np.isfinite(a))
        # Same kernels on the same numbers: the tolerance of the parity tests (1e-5 fp32, 2e-2 bf16, relative
        # to the output's scale) is far more than needed; in practice the two agree exactly.
        tol = 1e-5 if dtype == "f32" else 2e-2
        assert np.max(np.abs(a - b)) <= tol * max(1.0, float(np.max(np.abs(b))))
        # And against the oracle's chain of the same layers (norm-wise: in bf16 the store roundings compound).
        outs, _, _ = oracle.stack_forward(o_layers, x_np, dtype=dtype)
        rel = np.linalg.norm(a - outs[-1]) / np.linalg.norm(outs[-1])
        assert rel <= (1e-5 if dtype == "f32" else 3e-2), rel
    stack.close()
    for l in layers:
        l.close()


def test_static_chain_leaves_free_device_memory_unchanged():
    """The point of the entry point: a call, once the kernels it launches have been loaded by an earlier call,
    takes no device memory and gives none back."""
    import torch
    from paper_2305_02299_b200 import binding as cfi
    s, layers = _layers("f32")
    x = torch.from_numpy(s.x(seed=1, batch=64)).to("cuda")
    y = torch.empty((64, 96), device="cuda")
    cfi.cfi_stack_forward_static(layers, x, y, 64)          # first call: symbol look-up, kernel images
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    for _ in range(3):
        cfi.cfi_stack_forward_static(layers, x, y, 64)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before
    for l in layers:
        l.close()


def test_static_chain_rejects_what_does_not_fit():
    import torch
    from paper_2305_02299_b200 import binding as cfi
    s, layers = _layers("f32")
    too_many = (4 << 20) // (384 * 4) + 1              # one row more than a 4 MiB half holds for width 384
    x = torch.zeros((too_many, 96), device="cuda")
    y = torch.zeros((too_many, 96), device="cuda")
    with pytest.raises(cfi.CfiError) as e:
        cfi.cfi_stack_forward_static(layers, x, y, too_many)
    assert e.value.status == 5
    cfi.cfi_stack_forward_static(layers[:1], x, torch.empty((too_many, 384), device="cuda"), too_many)  # one layer: no intermediate
    torch.cuda.synchronize()
    for l in layers:
        l.close()
