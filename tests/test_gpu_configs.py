"""The named workloads (ViT-B/16 MLP layer shapes, 80-99 % sparsity, batch 1-256) at full size, in the
launch configuration the benchmark times (variant auto), against the oracle."""
import numpy as np
import pytest

import oracle
from paper_2305_02299_b200 import inputs
from parity import TOL, assert_parity, check_layer, device_layer, oracle_layer, run_device, scaled_error

pytestmark = pytest.mark.gpu
W = inputs.workloads()


@pytest.mark.parametrize("name", ["c1", "c2", "c3_b1", "c3_b64", "c3_b256"])
def test_vit_layer_configs(name):
    w = W[name]
    errs = check_layer(w.layer(), w.x(), "f32", variants=("auto", "splitk" if w.batch <= 64 else "batch"))
    assert max(errs.values()) <= 1e-5


@pytest.mark.parametrize("sp", [80, 90, 95, 99])
def test_sparsity_sweep_4096(sp):
    w = W[f"c4_s{sp}_b1"]
    L = w.layer()
    dl = device_layer(L)
    packed = oracle.pack(L.w_dense, L.mask)
    for B in (1, 16, 256):
        x = w.x(batch=B)
        y_ref, S = oracle_layer(L, x, packed=packed)
        assert scaled_error(run_device(dl, x, "f32", "auto"), y_ref, S) <= 1e-5
    dl.close()


def test_vit_mlp_block_bf16_slice():
    """One block of the bf16 MLP stack on a 788-row slice of its 50,432-row batch (per-layer, oracle inputs)."""
    s = inputs.StackWorkload(blocks=1)
    Ls, specs = s.layers(seed=0), s.layer_specs()
    x = s.x(seed=0, batch=788)
    cur = oracle.round_bf16(x)
    for L, sp in zip(Ls, specs):
        y_ref, S = oracle_layer(L, cur, "bf16", sp[4])
        dl = device_layer(L, "bf16", sp[4])
        y = run_device(dl, cur, "bf16")
        assert_parity(y, y_ref, S, "bf16")
        dl.close()
        cur = oracle.round_bf16(y_ref.astype(np.float32))


def test_vit_mlp_stack_bf16_full_size_sampled():
    """All 12 blocks (24 layers) of the bf16 MLP stack at the full 50,432 rows, in the launch configuration the
    benchmark times (variant auto, i.e. the tensor-core kernels).  Per layer: every output of 48 sampled batch rows
    against the oracle fed with the device's own input rows (so each layer is judged on its own arithmetic); the
    device's output feeds the next layer.  End to end: the same 48 rows through the oracle's own chain from x,
    compared norm-wise, because the store roundings of 24 layers compound."""
    import torch
    from paper_2305_02299_b200 import binding as cfi
    s = inputs.StackWorkload(blocks=12)
    Ls, specs = s.layers(seed=0), s.layer_specs()
    rng = np.random.default_rng(0)
    rows = np.sort(rng.choice(s.batch, size=48, replace=False))
    rows[0], rows[-1] = 0, s.batch - 1                      # first row, and the last row of the ragged last tile
    rows_d = torch.from_numpy(rows).cuda()
    x = s.x(seed=0)
    packed = [oracle.pack(L.w_dense, L.mask) for L in Ls]
    chain, _, _ = oracle.stack_forward([(p[0], p[1], p[2], L.bias, sp[0], sp[1], sp[4]) for p, L, sp in zip(packed, Ls, specs)],
                                       x[rows], dtype="bf16")
    x_d = torch.from_numpy(x).to("cuda", torch.bfloat16)
    worst = 0.0
    for li, (L, sp, pk) in enumerate(zip(Ls, specs, packed)):
        dl = device_layer(L, "bf16", sp[4])
        assert cfi.cfi_choose_variant(dl, s.batch) == 4
        y_d = torch.empty((s.batch, sp[1]), device="cuda", dtype=torch.bfloat16)
        cfi.cfi_forward(dl, x_d, y_d, s.batch)
        torch.cuda.synchronize()
        assert cfi.cfi_device_status(dl) == 0
        x_rows = x_d[rows_d].float().cpu().numpy()           # bf16 numbers: the rounding inside oracle_layer is a no-op
        y_ref, S = oracle_layer(L, x_rows, "bf16", sp[4], packed=pk)
        y = y_d[rows_d].double().cpu().numpy()
        worst = max(worst, assert_parity(y, y_ref, S, "bf16", f"layer {li}"))
        dl.close()
        x_d = y_d
    y_end = x_d[rows_d].double().cpu().numpy()
    rel = np.linalg.norm(y_end - chain[-1]) / np.linalg.norm(chain[-1])
    assert rel <= 3e-2, rel


def test_headline_workload_full_size_in_bench_configuration():
    """c2 exactly as bench.py runs it (variant auto through cfi_forward), every output against the oracle, and
    the gather and tensor-core variants against each other."""
    w = W["c2"]
    L, x = w.layer(), w.x()
    y_ref, S = oracle_layer(L, x)
    dl = device_layer(L)
    ys = {v: run_device(dl, x, "f32", v) for v in ("auto", "batch", "dense_tc")}
    dl.close()
    for v, y in ys.items():
        assert scaled_error(y, y_ref, S) <= 1e-5, v
    assert np.max(np.abs(ys["batch"] - ys["dense_tc"]) / S) <= 1e-5   # two summation orders, each within tolerance
