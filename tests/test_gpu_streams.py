"""cfi_forward only reads the layer, so calls on different streams may overlap, and a call can be captured in a
CUDA graph (the launches carry programmatic-dependent-launch and, for the tensor-core variant, cluster attributes)."""
import numpy as np
import pytest

from paper_2305_02299_b200 import inputs
from parity import device_layer, to_device, torch_dtype

pytestmark = pytest.mark.gpu

CASES = [("f32", 1, "auto"), ("f32", 16, "auto"), ("f32", 64, "batch"), ("f32", 256, "dense_tc"), ("bf16", 300, "dense_tc")]


@pytest.mark.parametrize("dtype,B,variant", CASES)
def test_concurrent_streams_share_one_layer(dtype, B, variant):
    import torch
    from paper_2305_02299_b200 import binding as cfi
    L = inputs.make_layer(3072, 768, 307, n_ablated=40, seed=5)     # few tiles, long K: the fp32 tensor-core variant splits K over clusters
    dl = device_layer(L, dtype, "gelu")
    n_streams, rounds = 4, 6
    xs = [to_device(inputs.make_x(B, L.in_features, seed=100 + s), dtype) for s in range(n_streams)]
    serial = []
    for x in xs:
        y = torch.empty((B, L.out_features), device="cuda", dtype=torch_dtype(dtype))
        cfi.cfi_forward_variant(dl, x, y, B, variant=variant)
        serial.append(y)
    torch.cuda.synchronize()
    streams = [torch.cuda.Stream() for _ in range(n_streams)]
    outs = [[torch.zeros((B, L.out_features), device="cuda", dtype=torch_dtype(dtype)) for _ in range(rounds)] for _ in range(n_streams)]
    torch.cuda.synchronize()
    for r in range(rounds):
        for s, st in enumerate(streams):
            cfi.cfi_forward_variant(dl, xs[s], outs[s][r], B, stream=st, variant=variant)
    torch.cuda.synchronize()
    assert cfi.cfi_device_status(dl) == 0
    for s in range(n_streams):
        for r in range(rounds):
            assert torch.equal(outs[s][r], serial[s]), (s, r)
    dl.close()


@pytest.mark.parametrize("dtype,B", [("f32", 1), ("f32", 256), ("bf16", 256)])
def test_forward_replays_from_a_cuda_graph(dtype, B):
    import torch
    from paper_2305_02299_b200 import binding as cfi
    L = inputs.make_layer(768, 3072, 77, n_ablated=30, seed=6)
    dl = device_layer(L, dtype)
    x = to_device(inputs.make_x(B, L.in_features, seed=1), dtype)
    y_ref = torch.empty((B, L.out_features), device="cuda", dtype=torch_dtype(dtype))
    cfi.cfi_forward(dl, x, y_ref, B)
    torch.cuda.synchronize()
    y = torch.zeros_like(y_ref)
    stream = torch.cuda.Stream()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(stream):
        with torch.cuda.graph(g, stream=stream):
            for _ in range(3):                 # back-to-back launches: each may start before the one before it ends
                cfi.cfi_forward(dl, x, y, B, stream=stream)
        for _ in range(2):
            y.zero_()
            g.replay()
            stream.synchronize()
            assert torch.equal(y, y_ref)
    dl.close()
