"""Layers built with a chosen subset of the device layouts (cfi_create_layouts): every combination must give the
oracle's numbers through the automatic kernel choice at every batch size, hold only what was asked for, and refuse a
variant whose layout is missing."""
import numpy as np
import pytest

import oracle
from paper_2305_02299_b200 import inputs
from parity import TOL, assert_parity, oracle_layer, run_device

pytestmark = pytest.mark.gpu
SMALL, GATHER, DENSE = 1, 2, 4
NEEDS = {"simple": SMALL, "splitk": SMALL, "batch": GATHER, "dense_tc": DENSE, "slab": GATHER}


@pytest.mark.parametrize("layouts", [1, 2, 3, 4, 5, 6, 7])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_every_layout_subset_runs_every_batch(layouts, dtype):
    from paper_2305_02299_b200 import binding as cfi
    L = inputs.make_layer(256, 200, 26, n_ablated=9, seed=layouts)
    v, ix, rows = cfi.cfi_pack(L.w_dense, L.mask)
    dl = cfi.cfi_create(v, ix, rows, L.bias, 256, 200, dtype=dtype, act="gelu", layouts=layouts)
    info = cfi.cfi_layer_info(dl)
    assert info.layouts == layouts
    assert (info.bytes_small_batch > 0) == bool(layouts & SMALL)
    assert (info.bytes_gather > 0) == bool(layouts & GATHER)
    assert (info.bytes_dense > 0) == bool(layouts & DENSE)
    assert info.device_bytes >= info.bytes_small_batch + info.bytes_gather + info.bytes_dense
    for B in (1, 3, 8, 17, 40, 130, 300):
        x = inputs.make_x(B, 256, seed=B)
        y_ref, S = oracle_layer(L, x, dtype, "gelu")
        assert NEEDS[{1: "simple", 2: "splitk", 3: "batch", 4: "dense_tc", 5: "slab"}[cfi.cfi_choose_variant(dl, B)]] & layouts
        assert_parity(run_device(dl, x, dtype, "auto"), y_ref, S, dtype, f"layouts {layouts} B {B}")
    x = inputs.make_x(5, 256)
    for variant, need in NEEDS.items():
        if not (need & layouts):
            with pytest.raises(cfi.CfiError) as e:
                run_device(dl, x, dtype, variant)
            assert e.value.status == 2
    dl.close()


def test_small_batch_only_layer_is_small_and_can_grow():
    """4096 x 4096 at 99 % sparsity for online inference: little more than the condensed arrays on the device; the
    other layouts can be added later and are then used."""
    from paper_2305_02299_b200 import binding as cfi
    w = inputs.workloads()["c4_s99_b1"]
    L = w.layer()
    v, ix, rows = cfi.cfi_pack(L.w_dense, L.mask)
    dl = cfi.cfi_create(v, ix, rows, L.bias, 4096, 4096, layouts=SMALL)
    info = cfi.cfi_layer_info(dl)
    assert info.device_bytes < 2 * 1024 * 1024 and info.bytes_dense == 0 and info.bytes_gather == 0
    x1, x300 = w.x(batch=1), w.x(batch=300)
    packed = oracle.pack(L.w_dense, L.mask)
    y_ref, S = oracle_layer(L, x1, packed=packed)
    assert_parity(run_device(dl, x1, "f32", "auto"), y_ref, S, "f32")
    y_ref, S = oracle_layer(L, x300, packed=packed)
    assert cfi.cfi_choose_variant(dl, 300) == 2                       # the only kernel it has a layout for
    assert_parity(run_device(dl, x300, "f32", "auto"), y_ref, S, "f32")
    cfi.cfi_layer_add_layouts(dl, DENSE | GATHER)
    info = cfi.cfi_layer_info(dl)
    assert info.layouts == 7 and info.bytes_dense >= 4096 * 4096 * 4
    assert cfi.cfi_choose_variant(dl, 300) in (3, 4, 5)
    assert_parity(run_device(dl, x300, "f32", "auto"), y_ref, S, "f32")
    cfi.cfi_layer_add_layouts(dl, 7)                                  # nothing missing: no-op
    assert cfi.cfi_layer_info(dl).device_bytes == info.device_bytes
    dl.close()


def test_dense_only_layer_with_unaddressable_shape_is_refused():
    from paper_2305_02299_b200 import binding as cfi
    L = inputs.make_layer(30, 16, 4, seed=1)                          # fp32 rows of 120 bytes
    v, ix, rows = cfi.cfi_pack(L.w_dense, L.mask)
    with pytest.raises(cfi.CfiError) as e:
        cfi.cfi_create(v, ix, rows, L.bias, 30, 16, layouts=DENSE)
    assert e.value.status == 2
    dl = cfi.cfi_create(v, ix, rows, L.bias, 30, 16, layouts=DENSE | SMALL)   # dense skipped, small built
    assert cfi.cfi_layer_info(dl).layouts == SMALL
    dl.close()
