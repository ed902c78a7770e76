"""Parity of the CUDA forward (through the C-ABI) with the CPU oracle, element by element.

Tolerance: max |y - y_oracle| / S <= 1e-5 (fp32) or 2e-2 (bf16 storage, fp32 accumulate), where
S = |bias| + sum_j |w x| is the scale of the sum (a plain ratio to |y| is unbounded when terms cancel).
Integer-valued cases must agree bit for bit whatever the summation order.
"""
import numpy as np
import pytest

import oracle
from paper_2305_02299_b200 import inputs
from parity import TOL, assert_parity, check_layer, device_layer, oracle_layer, run_device, scaled_error, to_device, torch_dtype

pytestmark = pytest.mark.gpu
ALL = ("simple", "splitk", "batch", "slab", "auto")


@pytest.mark.parametrize("k", [1, 2, 3, 4, 5, 31, 32, 33, 77])
@pytest.mark.parametrize("B", [1, 2, 3, 17])
def test_fan_in_grid_fp32(k, B):
    L = inputs.make_layer(101, 67, k, n_ablated=5, seed=k)
    check_layer(L, inputs.make_x(B, 101, seed=B), "f32", variants=ALL)


@pytest.mark.parametrize("B", [1, 2, 3, 8, 9, 17, 64, 65, 255, 256, 257])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_batch_grid(B, dtype):
    L = inputs.make_layer(768, 200, 77, n_ablated=13, seed=2)
    check_layer(L, inputs.make_x(B, 768, seed=B), dtype, variants=ALL)


@pytest.mark.parametrize("in_f,out_f,k", [(1, 1, 1), (5, 3, 5), (9, 130, 4), (1000, 7, 307), (4096, 33, 819),
                                          (2050, 300, 41), (333, 1025, 100)])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_odd_shapes(in_f, out_f, k, dtype):
    L = inputs.make_layer(in_f, out_f, k, n_ablated=out_f // 7, seed=in_f)
    for B in (1, 5, 70):
        check_layer(L, inputs.make_x(B, in_f, seed=3), dtype, variants=ALL)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("act", ["none", "gelu"])
def test_gelu_and_ablated_rows(dtype, act):
    import torch
    L = inputs.make_layer(256, 96, 20, n_ablated=30, seed=4)
    x = inputs.make_x(33, 256, seed=4)
    y_ref, S = oracle_layer(L, x, dtype, act)
    dl = device_layer(L, dtype, act)
    for v in ALL:
        y = run_device(dl, x, dtype, v)
        assert_parity(y, y_ref, S, dtype)
        # Ablated rows carry act(bias) only, identical for every batch row and rounded once to the storage type.
        expect = torch.tensor(y_ref[0, L.ablated]).to(torch_dtype(dtype)).to(torch.float64).numpy()
        got = y[:, L.ablated]
        if act == "none":
            assert np.array_equal(got, np.tile(expect, (33, 1)))
        else:
            assert np.all(got == got[0:1]) and np.allclose(got[0], expect, rtol=2 ** -7 if dtype == "bf16" else 1e-6, atol=1e-7)
    dl.close()


def test_all_rows_ablated_and_no_bias():
    from paper_2305_02299_b200 import binding as cfi
    dl = cfi.cfi_create(np.zeros((0, 0), np.float32), np.zeros((0, 0), np.int32), np.zeros((0,), np.int32),
                        np.arange(6, dtype=np.float32), 10, 6)
    for v in ALL:
        y = run_device(dl, inputs.make_x(4, 10), "f32", v)
        assert np.array_equal(y, np.tile(np.arange(6.0), (4, 1)))
    dl.close()
    L = inputs.make_layer(40, 12, 6, n_ablated=2, seed=1)
    vv, ix, rows = cfi.cfi_pack(L.w_dense, L.mask)
    dl = cfi.cfi_create(vv, ix, rows, None, 40, 12)          # Algorithm 1 as printed: no bias
    x = inputs.make_x(3, 40, seed=1)
    y_ref, S = oracle.forward(vv, ix, rows, None, 40, 12, x, want_scale=True)
    for v in ALL:
        y = run_device(dl, x, "f32", v)
        assert np.all(y[:, L.ablated] == 0.0)
        assert np.max(np.abs(y - y_ref)) <= 1e-5 * max(1.0, S.max())
    dl.close()


def test_batch_zero_launches_nothing():
    import torch
    from paper_2305_02299_b200 import binding as cfi
    L = inputs.make_layer(16, 8, 2, seed=0)
    dl = device_layer(L)
    y = torch.full((8,), 7.0, device="cuda")
    cfi.cfi_forward(dl, torch.zeros(16, device="cuda"), y, 0)
    torch.cuda.synchronize()
    assert torch.all(y == 7.0)
    assert cfi.cfi_device_status(dl) == 0
    dl.close()


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("B", [1, 6, 40, 130])
def test_exact_integer_arithmetic_is_bit_exact(dtype, B):
    """Small-integer weights and inputs: every partial sum is exact in fp32 (and every output fits bf16
    exactly), so any summation order and tiling must give the oracle's numbers bit for bit."""
    L = inputs.make_layer(512, 150, 24, n_ablated=11, seed=7, integer_valued=True)
    x = inputs.make_x(B, 512, seed=7, integer_valued=True, density=0.15 if dtype == "bf16" else 1.0)
    y_ref, _ = oracle_layer(L, x, dtype)
    if dtype == "bf16":
        assert np.max(np.abs(y_ref)) <= 256          # integers up to 2^8 are exact in bf16
    dl = device_layer(L, dtype)
    for v in ALL:
        assert np.array_equal(run_device(dl, x, dtype, v), y_ref), v
    dl.close()


def test_unsorted_and_duplicate_indices():
    from paper_2305_02299_b200 import binding as cfi
    rng = np.random.default_rng(0)
    vals = rng.standard_normal((20, 9)).astype(np.float32)
    idx = rng.integers(0, 30, size=(20, 9)).astype(np.int32)      # unsorted, with repeats
    rows = rng.permutation(25)[:20].astype(np.int32)              # unsorted rows
    bias = rng.standard_normal(25).astype(np.float32)
    dl = cfi.cfi_create(vals, idx, rows, bias, 30, 25)
    for B in (1, 4, 70):
        x = inputs.make_x(B, 30, seed=B)
        y_ref, S = oracle.forward(vals, idx, rows, bias, 30, 25, x, want_scale=True)
        for v in ALL:
            assert scaled_error(run_device(dl, x, "f32", v), y_ref, S) <= 1e-5
    dl.close()


def test_inf_in_unused_column_does_not_leak():
    """A column no row reads may hold inf/NaN: padding entries must not touch real data."""
    L = inputs.make_layer(64, 10, 3, seed=3)          # 30 of 64 columns used at most
    unused = np.nonzero(L.mask.sum(axis=0) == 0)[0]
    assert unused.size > 0
    x = inputs.make_x(20, 64, seed=3)
    x[:, unused] = np.inf
    x[:, 0] = np.inf if 0 in unused else x[:, 0]
    y_ref, S = oracle_layer(L, x)
    dl = device_layer(L)
    for v in ALL:
        y = run_device(dl, x, "f32", v)
        assert np.all(np.isfinite(y)) and scaled_error(y, y_ref, S) <= 1e-5
    dl.close()


def test_forward_host_matches_device_call():
    import torch
    from paper_2305_02299_b200 import binding as cfi
    L = inputs.make_layer(768, 300, 77, n_ablated=20, seed=6)
    dl = device_layer(L)
    for B in (3, 64, 10):                               # grows, then reuses the staging buffers
        x = inputs.make_x(B, 768, seed=B)
        xh = torch.from_numpy(x).pin_memory()
        yh = torch.empty((B, 300), dtype=torch.float32).pin_memory()
        cfi.cfi_forward_host(dl, xh, yh, B)
        assert np.array_equal(yh.numpy().astype(np.float64), run_device(dl, x, "f32", "auto"))
    dl.close()


def test_misaligned_pointer_is_rejected():
    import torch
    from paper_2305_02299_b200 import binding as cfi
    dl = device_layer(inputs.make_layer(16, 8, 2, seed=0))
    buf = torch.zeros(64, device="cuda")
    with pytest.raises(cfi.CfiError) as e:
        cfi.cfi_forward(dl, buf[1:17], buf[32:40], 1)
    assert e.value.status == 10
    dl.close()


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_stack_matches_chained_oracle(dtype):
    """MLP-shaped chain: per-layer comparison with oracle-supplied inputs, then the library's own chain."""
    import torch
    from paper_2305_02299_b200 import binding as cfi
    s = inputs.StackWorkload(blocks=2, d_model=96, d_hidden=384, k_up=10, k_down=38, batch=70)
    Ls = s.layers(seed=1)
    specs = s.layer_specs()
    packed = [oracle.pack(L.w_dense, L.mask) for L in Ls]
    o_layers = [(p[0], p[1], p[2], L.bias, sp[0], sp[1], sp[4]) for p, L, sp in zip(packed, Ls, specs)]
    x = s.x(seed=1)
    outs, exact, scales = oracle.stack_forward(o_layers, x, dtype=dtype)
    dls = [device_layer(L, dtype, sp[4]) for L, sp in zip(Ls, specs)]
    cur = oracle.round_bf16(x) if dtype == "bf16" else x
    for i, dl in enumerate(dls):                        # teacher-forced: layer i gets the oracle's input
        y = run_device(dl, cur, dtype)
        assert_parity(y, exact[i], scales[i], dtype, str(i))
        cur = outs[i].astype(np.float32)
    st = cfi.cfi_stack_create(dls, 70)
    y_d = torch.empty((70, 96), device="cuda", dtype=torch_dtype(dtype))
    cfi.cfi_stack_forward(st, to_device(x, dtype), y_d, 70)
    torch.cuda.synchronize()
    y = y_d.to(torch.float64).cpu().numpy()
    rel = np.linalg.norm(y - outs[-1]) / np.linalg.norm(outs[-1])
    assert rel <= (1e-5 if dtype == "f32" else 3e-2), rel
    with pytest.raises(cfi.CfiError) as e:
        cfi.cfi_stack_forward(st, to_device(x, dtype), y_d, 71)
    assert e.value.status == 5
    st.close()
    for dl in dls:
        dl.close()


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("B", [8, 16, 24])
def test_splitk_long_rows_full_batch_tile(dtype, B):
    """A long x (4096 columns) with full tiles of eight batch rows: the split-k launch shape with the most threads per
    CTA and the most registers per thread (bf16 widening); it must launch and match on every tile."""
    L = inputs.make_layer(4096, 1024, 205, n_ablated=30, seed=B)
    x = inputs.make_x(B, 4096, seed=B + 3)
    check_layer(L, x, dtype, "gelu", variants=("splitk",))


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("order", ["reversed", "shuffled"])
def test_every_row_active_in_any_row_order(dtype, order):
    """n_active == out_features with active_rows that is not 0, 1, 2, ...: condensed row r belongs to output row
    active_rows[r] in every kernel, the small-batch one included."""
    from paper_2305_02299_b200 import binding as cfi
    out_f, in_f, k = 64, 128, 9
    L = inputs.make_layer(in_f, out_f, k, seed=21)
    v, ix, rows = oracle.pack(L.w_dense, L.mask)
    assert rows.shape[0] == out_f
    perm = np.arange(out_f)[::-1].copy() if order == "reversed" else np.random.default_rng(5).permutation(out_f)
    v2, ix2, rows2 = v[perm], ix[perm], rows[perm].astype(np.int32)
    dl = cfi.cfi_create(v2, ix2, rows2, L.bias, in_f, out_f, dtype=dtype)
    for B in (1, 2, 5, 8, 40, 130):
        x = inputs.make_x(B, in_f, seed=B)
        y_ref, S = oracle_layer(L, x, dtype)
        y_perm, _ = oracle_layer(L, x, dtype, packed=(v2, ix2, rows2))
        assert np.array_equal(y_ref, y_perm)                 # the oracle itself does not care about the row order
        for var in ALL + ("dense_tc",):
            assert_parity(run_device(dl, x, dtype, var), y_ref, S, dtype, f"{var} B={B}")
    dl.close()


@pytest.mark.parametrize("variant", ["simple", "splitk", "batch", "dense_tc", "auto"])
def test_bf16_inputs_are_rounded_to_nearest_even(variant):
    """Weights and activations that lie exactly half-way between two bf16 numbers.  With one-hot partners every
    output is a single product of the rounded numbers, exact in bf16, so the device must return the oracle's
    numbers bit for bit; truncation or round-half-up of either operand gives different bits."""
    from paper_2305_02299_b200 import binding as cfi
    n = 16
    ties = np.array([1 + 1 * 2.0 ** -8, 1 + 3 * 2.0 ** -8, -(1 + 5 * 2.0 ** -8), 2 + 7 * 2.0 ** -7, 0.5 + 9 * 2.0 ** -9,
                     -(1 + 2.0 ** -8 + 2.0 ** -20), 1 + 2.0 ** -8 - 2.0 ** -20, 3.0], dtype=np.float32)
    r = oracle.round_bf16(ties)
    assert r[0] == 1.0 and r[1] == 1 + 2.0 ** -6 and r[2] == -(1 + 2.0 ** -6)     # to even, not down and not up
    assert r[5] == -(1 + 2.0 ** -7) and r[6] == 1.0                               # just past / short of half-way
    # (a) tie-valued weights against one-hot activations.
    vals = np.stack([np.roll(ties, i)[:2] for i in range(n)]).astype(np.float32)           # [16, 2]
    idx = np.stack([[i, (i + 5) % n] for i in range(n)]).astype(np.int32)
    rows = np.arange(n, dtype=np.int32)
    x = np.eye(n, dtype=np.float32)
    dl = cfi.cfi_create(vals, idx, rows, None, n, n, dtype="bf16")
    y_ref = oracle.forward(oracle.round_bf16(vals), idx, rows, None, n, n, x)
    assert np.array_equal(run_device(dl, x, "bf16", variant), y_ref)
    dl.close()
    # (b) tie-valued activations against weights of one.
    ones = np.ones((n, 1), np.float32)
    idx1 = np.arange(n, dtype=np.int32).reshape(n, 1)
    dl = cfi.cfi_create(ones, idx1, rows, None, n, n, dtype="bf16")
    xt = np.stack([np.roll(np.resize(ties, n), b) for b in range(24)]).astype(np.float32)
    y_ref = oracle.forward(ones, idx1, rows, None, n, n, oracle.round_bf16(xt))
    import torch
    x_d = torch.from_numpy(xt).to("cuda", torch.bfloat16)          # torch rounds to nearest even as well
    assert np.array_equal(x_d.float().cpu().numpy(), oracle.round_bf16(xt))
    assert np.array_equal(run_device(dl, xt, "bf16", variant), y_ref)
    dl.close()


def test_wide_layer_small_batch_falls_back_to_a_kernel_that_fits():
    """in_features so large that one row of x does not fit shared memory: the automatic choice must not pick the
    small-batch kernel (which would refuse the shape) but one that can run it."""
    from paper_2305_02299_b200 import binding as cfi
    in_f, out_f, k = 70000, 24, 6
    rng = np.random.default_rng(3)
    idx = np.stack([np.sort(rng.choice(in_f, size=k, replace=False)) for _ in range(out_f)]).astype(np.int32)
    vals = rng.standard_normal((out_f, k)).astype(np.float32)
    rows = np.arange(out_f, dtype=np.int32)
    bias = rng.standard_normal(out_f).astype(np.float32)
    dl = cfi.cfi_create(vals, idx, rows, bias, in_f, out_f)
    for B in (1, 3, 12):
        assert cfi.cfi_choose_variant(dl, B) != 2
        x = inputs.make_x(B, in_f, seed=B)
        y_ref, S = oracle.forward(vals, idx, rows, bias, in_f, out_f, x, want_scale=True)
        assert scaled_error(run_device(dl, x, "f32", "auto"), y_ref, S) <= 1e-5
    with pytest.raises(cfi.CfiError):
        run_device(dl, inputs.make_x(1, in_f), "f32", "splitk")
    dl.close()


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_long_index_stream_with_16_bit_columns(dtype):
    """Above 1.5 M entries (and below 65,536 inputs) the small-batch layout stores its columns in 16 bits: the stream
    is 2 bytes per entry shorter (checked through cfi_layer_info) and every batch tile of the small-batch kernels
    still matches the oracle, ablated rows, odd fan-in and the pad column included."""
    from paper_2305_02299_b200 import binding as cfi
    in_f, out_f, k = 2052, 1100, 1501                                  # 1.6 M entries, k not a multiple of 8
    L = inputs.make_layer(in_f, out_f, k, n_ablated=31, seed=5)
    dl = device_layer(L, dtype, "gelu")
    info = cfi.cfi_layer_info(dl)
    assert info.k_padded == 1504
    assert info.weight_bytes_splitk == info.n_active * info.k_padded * ((4 if dtype == "f32" else 2) + 2)
    packed = oracle.pack(L.w_dense, L.mask)
    for B in (1, 2, 3, 5, 8, 17):
        x = inputs.make_x(B, in_f, seed=B)
        y_ref, S = oracle_layer(L, x, dtype, "gelu", packed=packed)
        for v in ("splitk", "simple", "auto"):
            assert_parity(run_device(dl, x, dtype, v), y_ref, S, dtype, f"{v} B={B}")
    dl.close()
    small = device_layer(inputs.make_layer(64, 40, 7, seed=1), dtype)  # a short stream keeps 32-bit columns
    i2 = cfi.cfi_layer_info(small)
    assert i2.weight_bytes_splitk == i2.n_active * i2.k_padded * ((4 if dtype == "f32" else 2) + 4)
    small.close()


@pytest.mark.parametrize("in_f,out_f,k,nabl", [(4096, 300, 41, 9), (3072, 768, 307, 77), (700, 40, 100, 3), (6000, 64, 13, 0), (20000, 24, 6, 2)])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_slab_kernel_cluster_shapes(in_f, out_f, k, nabl, dtype):
    """The slab kernel with its column slabs on one CTA and divided over clusters of 2, 4 and 8 (by layer width), ragged
    last slab, ragged batch tile, more than one batch tile, ablated rows, bit-identical on a second run."""
    L = inputs.make_layer(in_f, out_f, k, n_ablated=nabl, seed=in_f)
    dl = device_layer(L, dtype, "gelu")
    packed = oracle.pack(L.w_dense, L.mask)
    for B in (9, 16, 37, 64):
        x = inputs.make_x(B, in_f, seed=B)
        y_ref, S = oracle_layer(L, x, dtype, "gelu", packed=packed)
        y = run_device(dl, x, dtype, "slab")
        assert_parity(y, y_ref, S, dtype, f"B={B}")
        assert np.array_equal(y, run_device(dl, x, dtype, "slab"))
    dl.close()


def test_slab_kernel_refuses_a_layer_too_wide_for_a_cluster():
    from paper_2305_02299_b200 import binding as cfi
    dl = device_layer(inputs.make_layer(40000, 24, 6, seed=1))      # an eighth of x for 16 batch rows exceeds shared memory
    with pytest.raises(cfi.CfiError) as e:
        run_device(dl, inputs.make_x(16, 40000), "f32", "slab")
    assert e.value.status == 2
    assert cfi.cfi_choose_variant(dl, 16) != 5
    dl.close()


def test_slab_kernel_exact_integers_and_unused_inf():
    L = inputs.make_layer(1024, 150, 24, n_ablated=11, seed=7, integer_valued=True)
    x = inputs.make_x(40, 1024, seed=7, integer_valued=True)
    y_ref, _ = oracle_layer(L, x, "f32")
    dl = device_layer(L, "f32")
    assert np.array_equal(run_device(dl, x, "f32", "slab"), y_ref)
    dl.close()
    L = inputs.make_layer(900, 20, 3, seed=3)                      # most columns unused; pad entries in every quad
    unused = np.nonzero(L.mask.sum(axis=0) == 0)[0]
    x = inputs.make_x(20, 900, seed=3)
    x[:, unused] = np.inf
    y_ref, S = oracle_layer(L, x)
    dl = device_layer(L)
    y = run_device(dl, x, "f32", "slab")
    assert np.all(np.isfinite(y)) and scaled_error(y, y_ref, S) <= 1e-5
    dl.close()
