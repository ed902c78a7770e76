"""The tensor-core variant (dense bf16 copy of the weight, tcgen05) against the oracle, element by element.

It computes the same sums as the condensed forms (exact bf16 products, fp32 accumulation), so the bf16
tolerance of the other parity tests applies and small-integer cases must agree bit for bit.
"""
import numpy as np
import pytest

from paper_2305_02299_b200 import inputs
from parity import TOL, device_layer, oracle_layer, run_device, scaled_error

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("in_f,out_f,k,nabl", [(64, 8, 5, 1), (72, 136, 9, 10), (768, 384, 77, 19), (3072, 200, 307, 20)])
@pytest.mark.parametrize("B", [1, 5, 128, 257])
@pytest.mark.parametrize("act", ["none", "gelu"])
def test_dense_tc_matches_oracle(in_f, out_f, k, nabl, B, act):
    L = inputs.make_layer(in_f, out_f, k, n_ablated=nabl, seed=in_f + B)
    x = inputs.make_x(B, in_f, seed=B)
    y_ref, S = oracle_layer(L, x, "bf16", act)
    dl = device_layer(L, "bf16", act)
    y = run_device(dl, x, "bf16", "dense_tc")
    dl.close()
    assert np.all(np.isfinite(y))
    assert scaled_error(y, y_ref, S) <= TOL["bf16"]


def test_dense_tc_exact_integers_and_agreement_with_gather():
    L = inputs.make_layer(512, 152, 24, n_ablated=11, seed=7, integer_valued=True)
    x = inputs.make_x(200, 512, seed=7, integer_valued=True, density=0.15)
    y_ref, _ = oracle_layer(L, x, "bf16")
    assert np.max(np.abs(y_ref)) <= 256
    dl = device_layer(L, "bf16")
    y_tc = run_device(dl, x, "bf16", "dense_tc")
    y_gather = run_device(dl, x, "bf16", "batch")
    dl.close()
    assert np.array_equal(y_tc, y_ref) and np.array_equal(y_gather, y_ref)


def test_dense_tc_refuses_shapes_it_cannot_address():
    from paper_2305_02299_b200 import binding as cfi
    L = inputs.make_layer(100, 30, 7, seed=1)           # in % 8 != 0
    dl = device_layer(L, "bf16")
    with pytest.raises(cfi.CfiError) as e:
        run_device(dl, inputs.make_x(4, 100), "bf16", "dense_tc")
    assert e.value.status == 2
    dl.close()
    L = inputs.make_layer(64, 16, 4, seed=1)             # fp32 layers have no dense bf16 copy
    dl = device_layer(L, "f32")
    with pytest.raises(cfi.CfiError):
        run_device(dl, inputs.make_x(4, 64), "f32", "dense_tc")
    assert cfi.cfi_device_status(dl) == 0
    dl.close()
