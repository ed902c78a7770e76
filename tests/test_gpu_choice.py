"""The automatic kernel choice (cfi_forward) against every explicit variant that can run the shape, on the named
workloads: the kernel it picks must be within 15 % (plus 0.3 us of timing noise) of the fastest one.  Times are CUDA
events around replays of a CUDA graph of 50 launches on one layer, 200 launches per figure."""
import numpy as np
import pytest

from paper_2305_02299_b200 import inputs

pytestmark = pytest.mark.gpu
W = inputs.workloads()
SHAPES = [("c1", ["c1", "c2"]), ("c3_b1", ["c3_b1", "c3_b64", "c3_b256"])] + \
         [(f"c4_s{sp}_b1", [f"c4_s{sp}_b{b}" for b in (1, 16, 256)]) for sp in (80, 90, 95, 99)]


def _time(cfi, torch, layer, x, y, batch, variant):
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        for _ in range(3):
            cfi.cfi_forward_variant(layer, x, y, batch, variant=variant)
        s.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=s):
            for _ in range(50):
                cfi.cfi_forward_variant(layer, x, y, batch, variant=variant)
        g.replay()
        s.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(s)
        for _ in range(4):
            g.replay()
        b.record(s)
        b.synchronize()
    return a.elapsed_time(b) * 1e3 / 200


@pytest.mark.parametrize("base,names", SHAPES, ids=[b for b, _ in SHAPES])
def test_auto_is_close_to_the_best_variant(base, names):
    import torch
    from paper_2305_02299_b200 import binding as cfi
    L = W[base].layer()
    v, ix, rows = cfi.cfi_pack(L.w_dense, L.mask)
    layer = cfi.cfi_create(v, ix, rows, L.bias, W[base].in_features, W[base].out_features)
    report = {}
    for name in names:
        w = W[name]
        x = torch.from_numpy(w.x()).cuda()
        y = torch.empty((w.batch, w.out_features), device="cuda")
        times = {}
        for variant in ("splitk", "batch", "slab", "dense_tc"):
            if variant == "splitk" and w.batch > 64:          # hundreds of microseconds: never a candidate there
                continue
            try:
                times[variant] = _time(cfi, torch, layer, x, y, w.batch, variant)
            except cfi.CfiError as e:
                assert e.status == 2                            # the variant cannot run this shape
        t_auto = _time(cfi, torch, layer, x, y, w.batch, "auto")
        best = min(times.values())
        report[name] = (t_auto, times)
        assert t_auto <= 1.15 * best + 0.3, (name, t_auto, times)
    layer.close()
