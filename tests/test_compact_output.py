"""The paper's compact output form (Algorithm 1 returns (batch, active_neurons); Sec. 4.4 removes ablated neurons):
cfi_compact_producer / cfi_compact_consumer against the oracle run on the full-width layers.

Pins: (1) the compact producer's output is the full-width output with the ablated columns deleted, bit for bit in
the oracle's doubles; (2) producer -> consumer in compact form equals the full-width pair up to the rounding of
the bias fold (fp32 adds of k-or-fewer constants); (3) the rewritten consumer keeps constant fan-in with distinct,
in-range columns and zero weights exactly where it read an ablated column.
"""
import numpy as np
import pytest

import oracle
from paper_2305_02299_b200 import binding as cfi
from paper_2305_02299_b200 import inputs


def _pair(d_in=96, d_hid=160, d_out=64, k1=10, k2=24, abl1=37, abl2=5, seed=3):
    L1 = inputs.make_layer(d_in, d_hid, k1, n_ablated=abl1, seed=seed, stream=1)
    L2 = inputs.make_layer(d_hid, d_out, k2, n_ablated=abl2, seed=seed, stream=2)
    p1 = cfi.cfi_pack(L1.w_dense, L1.mask)
    p2 = cfi.cfi_pack(L2.w_dense, L2.mask)
    return L1, L2, p1, p2


@pytest.mark.parametrize("act", ["none", "gelu"])
def test_compact_pair_equals_full_width_pair(act):
    L1, L2, (v1, i1, r1), (v2, i2, r2) = _pair()
    x = inputs.make_x(33, L1.in_features, seed=8)
    # full width
    h_full = oracle.forward(v1, i1, r1, L1.bias, L1.in_features, L1.out_features, x, act=act)
    y_full, S = oracle.forward(v2, i2, r2, L2.bias, L2.in_features, L2.out_features, h_full.astype(np.float32), want_scale=True)
    # compact producer
    b1c, r1c = cfi.cfi_compact_producer(L1.bias, r1, L1.out_features)
    assert np.array_equal(r1c, np.arange(r1.shape[0])) and np.array_equal(b1c, L1.bias[r1])
    h_c = oracle.forward(v1, i1, r1c, b1c, L1.in_features, r1.shape[0], x, act=act)
    assert np.array_equal(h_c, h_full[:, r1])                      # pin (1)
    # compact consumer: the constant an ablated producer column emits is act(bias), here in fp32
    const = oracle.forward(v1[:0], i1[:0], r1[:0], L1.bias, L1.in_features, L1.out_features,
                           np.zeros((1, L1.in_features), np.float32), act=act)[0].astype(np.float32)
    v2c, i2c, b2c = cfi.cfi_compact_consumer(r1, L1.out_features, const, v2, i2, r2, L2.bias)
    y_c = oracle.forward(v2c, i2c, r2, b2c, r1.shape[0], L2.out_features, h_c.astype(np.float32))
    assert np.max(np.abs(y_c - y_full) / S) <= 1e-6                # pin (2)
    # pin (3)
    ablated1 = np.setdiff1d(np.arange(L1.out_features), r1)
    read_ablated = np.isin(i2, ablated1)
    assert read_ablated.any()
    assert np.all(v2c[read_ablated] == 0.0) and np.array_equal(v2c[~read_ablated], v2[~read_ablated])
    assert i2c.min() >= 0 and i2c.max() < r1.shape[0]
    assert all(len(set(row)) == row.size for row in i2c)
    rank = -np.ones(L1.out_features, np.int64)
    rank[r1] = np.arange(r1.shape[0])
    assert np.array_equal(i2c[~read_ablated], rank[i2[~read_ablated]])


def test_compact_consumer_without_ablation_is_the_identity():
    L1, L2, (v1, i1, r1), (v2, i2, r2) = _pair(abl1=0)
    v2c, i2c, b2c = cfi.cfi_compact_consumer(r1, L1.out_features, None, v2, i2, r2, L2.bias)
    assert np.array_equal(v2c, v2) and np.array_equal(i2c, i2) and np.array_equal(b2c, L2.bias)


def test_compact_helpers_reject_bad_arguments():
    L1, L2, (v1, i1, r1), (v2, i2, r2) = _pair()
    with pytest.raises(cfi.CfiError) as e:
        cfi.cfi_compact_producer(L1.bias, np.array([0, 0], np.int32), L1.out_features)      # repeated row
    assert e.value.status == 4
    with pytest.raises(cfi.CfiError) as e:
        cfi.cfi_compact_consumer(r1, L1.out_features, None, v2, i2 + 10_000, r2, L2.bias)    # column out of range
    assert e.value.status == 4
    with pytest.raises(cfi.CfiError) as e:
        cfi.cfi_compact_consumer(r1[:5], L1.out_features, None, v2, i2, r2, L2.bias)         # k > producer's n_active
    assert e.value.status == 2


@pytest.mark.gpu
@pytest.mark.parametrize("dtype,B", [("f32", 1), ("f32", 300), ("bf16", 300)])
def test_compact_pair_on_device(dtype, B):
    """The compact pair through the library (stack of two layers) against the oracle's full-width pair."""
    import torch
    from parity import TOL, to_device, torch_dtype
    L1, L2, (v1, i1, r1), (v2, i2, r2) = _pair(d_in=256, d_hid=512, d_out=128, k1=26, k2=51, abl1=100, abl2=9)
    x = inputs.make_x(B, L1.in_features, seed=B)
    rnd = (lambda a: oracle.round_bf16(a)) if dtype == "bf16" else (lambda a: np.asarray(a, np.float32))
    h_full = oracle.forward(rnd(v1), i1, r1, rnd(L1.bias), L1.in_features, L1.out_features, rnd(x), act="gelu")
    y_full, S = oracle.forward(rnd(v2), i2, r2, rnd(L2.bias), L2.in_features, L2.out_features, rnd(h_full), want_scale=True)
    b1c, r1c = cfi.cfi_compact_producer(L1.bias, r1, L1.out_features)
    const = rnd(oracle.forward(v1[:0], i1[:0], r1[:0], rnd(L1.bias), L1.in_features, L1.out_features,
                               np.zeros((1, L1.in_features), np.float32), act="gelu")[0])
    v2c, i2c, b2c = cfi.cfi_compact_consumer(r1, L1.out_features, const, v2, i2, r2, L2.bias)
    l1 = cfi.cfi_create(v1, i1, r1c, b1c, L1.in_features, r1.shape[0], dtype=dtype, act="gelu")
    l2 = cfi.cfi_create(v2c, i2c, r2, b2c, r1.shape[0], L2.out_features, dtype=dtype)
    st = cfi.cfi_stack_create([l1, l2], B)
    y = torch.empty((B, L2.out_features), device="cuda", dtype=torch_dtype(dtype))
    cfi.cfi_stack_forward(st, to_device(x, dtype), y, B)
    torch.cuda.synchronize()
    st.close(); l1.close(); l2.close()
    err = np.max(np.abs(y.float().cpu().numpy().astype(np.float64) - y_full) / S)
    assert err <= TOL[dtype]
