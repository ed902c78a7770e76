"""Pins for the CPU oracle: it is checked against things other than itself.

Brute-force dense products done by numpy in float64 (a library routine), closed
forms, integer arithmetic, a hand-worked fixture, and the identities the paper's
equations imply.  A dropped term, a wrong index or stride, a transposed operand
or a wrong rounding rule in oracle/cfi_oracle.c fails at least one of these.
"""
import itertools
import math

import numpy as np
import pytest

import oracle
from paper_2305_02299_b200 import inputs
from conftest import read_golden


def dense_numpy(layer, x):
    """x (W.M)^T + bias with numpy float64 matmul: independent of the oracle's loops."""
    w = layer.w_dense.astype(np.float64) * layer.mask.astype(np.float64)
    return x.astype(np.float64) @ w.T + layer.bias.astype(np.float64)


# ---------------------------------------------------------------- golden fixture
def test_golden_tiny_layer_forward_and_pack():
    g = read_golden("tiny_layer.txt")
    W = g["W"].astype(np.float32)
    v, ix, rows = oracle.pack(W, None)
    assert np.array_equal(v, g["values"].astype(np.float32))
    assert np.array_equal(ix, g["indices"].astype(np.int32))
    assert np.array_equal(rows, g["active_rows"].astype(np.int32))
    y = oracle.forward(v, ix, rows, g["bias"], 5, 4, g["x"])
    assert np.array_equal(y, g["y"])
    assert np.array_equal(oracle.forward_recombination(v, ix, rows, g["bias"], 5, 4, g["x"]), g["y"])
    assert np.array_equal(oracle.dense_forward(W, None, g["bias"], g["x"]), g["y"])


# ---------------------------------------------------------------- pack
@pytest.mark.parametrize("in_f,out_f,k,nabl", [(16, 8, 3, 2), (33, 17, 33, 0), (7, 5, 1, 4), (64, 40, 20, 7), (5, 3, 2, 3)])
def test_pack_invariants_and_roundtrip(in_f, out_f, k, nabl):
    L = inputs.make_layer(in_f, out_f, k, n_ablated=nabl, seed=3)
    v, ix, rows = oracle.pack(L.w_dense, L.mask)
    n_act = out_f - nabl
    assert v.shape == ix.shape == (n_act, k if n_act else 0)
    assert np.all(np.diff(rows) > 0)                       # rows strictly ascending
    assert np.array_equal(np.setdiff1d(np.arange(out_f), rows), L.ablated)
    if n_act:
        assert np.all(np.diff(ix, axis=1) > 0)             # k distinct ascending columns (Eq. 2)
        assert ix.min() >= 0 and ix.max() < in_f
    back = np.zeros_like(L.w_dense)                        # scatter-back reproduces W.M bit for bit
    for r, o in enumerate(rows):
        back[o, ix[r]] = v[r]
    assert np.array_equal(back.view(np.uint32), (L.w_dense * L.mask).view(np.uint32))


def test_pack_rejects_non_constant_fan_in():
    L = inputs.make_layer(12, 6, 4, seed=1)
    m = L.mask.copy()
    c = np.nonzero(m[2])[0][0]
    m[2, c] = 0                                            # one row now keeps k-1
    with pytest.raises(oracle.NotConstantFanIn):
        oracle.pack(L.w_dense, m)


def test_pack_mask_semantics():
    W = np.array([[0.0, 1.0, -0.0, 2.0], [0.0, 0.0, 3.0, 4.0]], dtype=np.float32)
    v, ix, rows = oracle.pack(W, None)                     # without a mask: w != 0 decides, -0.0 is zero
    assert np.array_equal(ix, [[1, 3], [2, 3]])
    M = np.array([[1, 1, 0, 0], [0, 0, 1, 1]], dtype=np.uint8)
    v, ix, rows = oracle.pack(W, M)                        # with a mask: a kept 0.0 still counts
    assert np.array_equal(ix, [[0, 1], [2, 3]]) and np.array_equal(v, [[0, 1], [3, 4]])


# ---------------------------------------------------------------- forward vs brute force
@pytest.mark.parametrize("in_f,out_f,k,nabl,B", [(16, 8, 3, 2, 3), (40, 24, 7, 0, 5), (9, 6, 9, 1, 2), (128, 50, 31, 5, 4)])
def test_forward_equals_dense_product(in_f, out_f, k, nabl, B):
    L = inputs.make_layer(in_f, out_f, k, n_ablated=nabl, seed=11)
    x = inputs.make_x(B, in_f, seed=11)
    v, ix, rows = oracle.pack(L.w_dense, L.mask)
    y, S = oracle.forward(v, ix, rows, L.bias, in_f, out_f, x, want_scale=True)
    ref = dense_numpy(L, x)
    assert np.max(np.abs(y - ref) / S) < 1e-14
    assert np.max(np.abs(oracle.dense_forward(L.w_dense, L.mask, L.bias, x) - ref) / S) < 1e-14
    assert np.max(np.abs(oracle.forward_recombination(v, ix, rows, L.bias, in_f, out_f, x) - ref) / S) < 1e-14
    S_ref = np.abs(x.astype(np.float64)) @ np.abs(L.w_dense.astype(np.float64) * L.mask).T + np.abs(L.bias.astype(np.float64))
    assert np.allclose(S, S_ref, rtol=1e-13)


def test_forward_all_patterns_tiny():
    """Every choice of k columns out of in <= 6, against the dense definition (Eq. 1)."""
    rng = np.random.default_rng(5)
    for in_f in range(1, 7):
        for k in range(1, in_f + 1):
            pats = list(itertools.combinations(range(in_f), k))
            W = np.zeros((len(pats), in_f), dtype=np.float32)
            for r, p in enumerate(pats):
                W[r, list(p)] = rng.integers(1, 9, size=k) * rng.choice([-1, 1], size=k)
            x = rng.integers(-5, 6, size=(2, in_f)).astype(np.float32)
            bias = rng.integers(-3, 4, size=len(pats)).astype(np.float32)
            v, ix, rows = oracle.pack(W, None)
            assert np.array_equal(ix, np.array(pats, dtype=np.int32))
            y = oracle.forward(v, ix, rows, bias, in_f, len(pats), x)
            assert np.array_equal(y, x.astype(np.float64) @ W.astype(np.float64).T + bias)


def test_dense_limit_is_gemm():
    """k = in with indices 0..in-1: the layer is an ordinary dense linear."""
    rng = np.random.default_rng(2)
    W = rng.standard_normal((10, 12)).astype(np.float32)
    x = rng.standard_normal((4, 12)).astype(np.float32)
    ix = np.tile(np.arange(12, dtype=np.int32), (10, 1))
    y = oracle.forward(W, ix, np.arange(10, dtype=np.int32), None, 12, 10, x)
    assert np.allclose(y, x.astype(np.float64) @ W.astype(np.float64).T, rtol=0, atol=1e-13)


def test_gather_limit_k1():
    rng = np.random.default_rng(4)
    w = rng.standard_normal((9, 1)).astype(np.float32)
    ix = rng.integers(0, 20, size=(9, 1)).astype(np.int32)
    b = rng.standard_normal(9).astype(np.float32)
    x = rng.standard_normal((3, 20)).astype(np.float32)
    y = oracle.forward(w, ix, np.arange(9, dtype=np.int32), b, 20, 9, x)
    expect = b.astype(np.float64)[None, :] + w[:, 0].astype(np.float64)[None, :] * x[:, ix[:, 0]].astype(np.float64)
    assert np.array_equal(y, expect)


def test_index_handling_one_hot_and_ones():
    L = inputs.make_layer(30, 12, 5, n_ablated=2, seed=8)
    v, ix, rows = oracle.pack(L.w_dense, L.mask)
    ones_v = np.ones_like(v)
    eye = np.eye(30, dtype=np.float32)                     # batch of one-hot inputs e_c
    y = oracle.forward(ones_v, ix, rows, None, 30, 12, eye)
    assert np.array_equal(y.T, L.mask.astype(np.float64))  # y[c, o] = [c in idx[o]]
    y1 = oracle.forward(v, ix, rows, None, 30, 12, np.ones((1, 30), dtype=np.float32))
    assert np.allclose(y1[0, rows], v.astype(np.float64).sum(axis=1), atol=1e-14)


def test_unsorted_indices_and_row_order_do_not_matter():
    L = inputs.make_layer(50, 20, 9, n_ablated=3, seed=13)
    x = inputs.make_x(3, 50, seed=13)
    v, ix, rows = oracle.pack(L.w_dense, L.mask)
    y, S = oracle.forward(v, ix, rows, L.bias, 50, 20, x, want_scale=True)
    rng = np.random.default_rng(0)
    perm = np.stack([rng.permutation(9) for _ in range(v.shape[0])])
    v2, ix2 = np.take_along_axis(v, perm, 1), np.take_along_axis(ix, perm, 1)
    rp = rng.permutation(v.shape[0])
    y2 = oracle.forward(v2[rp], ix2[rp], rows[rp], L.bias, 50, 20, x)
    assert np.max(np.abs(y - y2) / S) < 1e-14


def test_duplicate_indices_add():
    v = np.array([[1.5, 2.0, -0.5]], dtype=np.float32)
    ix = np.array([[2, 2, 0]], dtype=np.int32)
    x = np.array([[4.0, 9.0, 3.0]], dtype=np.float32)
    y = oracle.forward(v, ix, np.array([0], dtype=np.int32), None, 3, 1, x)
    assert y[0, 0] == 1.5 * 3 + 2 * 3 - 0.5 * 4


def test_linearity_in_x():
    L = inputs.make_layer(40, 16, 6, seed=21, integer_valued=True)
    v, ix, rows = oracle.pack(L.w_dense, L.mask)
    x1 = inputs.make_x(2, 40, seed=1, integer_valued=True)
    x2 = inputs.make_x(2, 40, seed=2, integer_valued=True)
    f = lambda x: oracle.forward(v, ix, rows, None, 40, 16, x)
    assert np.array_equal(f(2 * x1 - 3 * x2), 2 * f(x1) - 3 * f(x2))


def test_exact_integer_arithmetic():
    L = inputs.make_layer(96, 33, 17, n_ablated=4, seed=17, integer_valued=True)
    x = inputs.make_x(5, 96, seed=17, integer_valued=True)
    v, ix, rows = oracle.pack(L.w_dense, L.mask)
    y = oracle.forward(v, ix, rows, L.bias, 96, 33, x)
    expect = x.astype(np.int64) @ L.w_dense.astype(np.int64).T + L.bias.astype(np.int64)
    assert np.array_equal(y, expect.astype(np.float64))


def test_ablated_rows_return_bias():
    L = inputs.make_layer(32, 20, 4, n_ablated=6, seed=9)
    x = inputs.make_x(4, 32, seed=9)
    v, ix, rows = oracle.pack(L.w_dense, L.mask)
    y = oracle.forward(v, ix, rows, L.bias, 32, 20, x)
    assert np.array_equal(y[:, L.ablated], np.tile(L.bias[L.ablated].astype(np.float64), (4, 1)))
    yg = oracle.forward(v, ix, rows, L.bias, 32, 20, x, act="gelu")
    for o in L.ablated:
        assert np.all(yg[:, o] == oracle.gelu(float(L.bias[o])))
    y0 = oracle.forward(v, ix, rows, None, 32, 20, x)     # Algorithm 1 as printed: no bias, zeros stay
    assert np.all(y0[:, L.ablated] == 0.0)


def test_empty_layer_and_empty_batch():
    y = oracle.forward(np.zeros((0, 0), np.float32), np.zeros((0, 0), np.int32), np.zeros((0,), np.int32),
                       np.array([1.0, 2.0], np.float32), 4, 2, np.ones((3, 4), np.float32))
    assert np.array_equal(y, np.tile([1.0, 2.0], (3, 1)))
    L = inputs.make_layer(8, 4, 2, seed=0)
    v, ix, rows = oracle.pack(L.w_dense, L.mask)
    assert oracle.forward(v, ix, rows, L.bias, 8, 4, np.zeros((0, 8), np.float32)).shape == (0, 4)


# ---------------------------------------------------------------- GELU
def test_gelu_identities_and_values():
    g = oracle.gelu
    assert g(0.0) == 0.0
    for v in (0.1, 0.5, 1.0, 2.5, 4.0):
        assert abs((g(v) - g(-v)) - v) < 1e-15 * max(1, v)           # odd part is v/2 twice
        assert abs((g(v) + g(-v)) - v * math.erf(v / math.sqrt(2))) < 1e-15
    assert abs(g(40.0) - 40.0) < 1e-12 and abs(g(-40.0)) < 1e-12
    # v * Phi(v) with Phi from normal tables: Phi(1) = 0.8413447460685429, Phi(2) = 0.9772498680518208
    assert abs(g(1.0) - 0.8413447460685429) < 1e-15
    assert abs(g(2.0) - 2 * 0.9772498680518208) < 1e-15
    assert abs(g(-1.0) + 0.15865525393145707) < 1e-15
    import torch
    t = torch.linspace(-6, 6, 101, dtype=torch.float64)
    ref = torch.nn.functional.gelu(t, approximate="none").numpy()
    assert np.allclose([g(float(a)) for a in t], ref, rtol=0, atol=1e-14)


def test_gelu_applied_after_bias_and_sum():
    L = inputs.make_layer(24, 10, 5, n_ablated=1, seed=6)
    x = inputs.make_x(3, 24, seed=6)
    v, ix, rows = oracle.pack(L.w_dense, L.mask)
    y = oracle.forward(v, ix, rows, L.bias, 24, 10, x, act="gelu")
    import torch
    ref = torch.nn.functional.gelu(torch.from_numpy(dense_numpy(L, x)), approximate="none").numpy()
    assert np.allclose(y, ref, rtol=0, atol=1e-13)


# ---------------------------------------------------------------- bf16 rounding
def test_bf16_rounding_rule():
    r = lambda f: float(oracle.round_bf16(np.array([f], dtype=np.float32))[0])
    assert r(1.0) == 1.0
    assert r(1.0 + 2.0 ** -8) == 1.0                      # tie -> even mantissa (down)
    assert r(1.0 + 3 * 2.0 ** -8) == 1.0 + 2.0 ** -6      # tie -> even mantissa (up)
    assert r(1.0 + 2.0 ** -8 + 2.0 ** -20) == 1.0 + 2.0 ** -7
    assert r(-1.0 - 2.0 ** -7) == -1.0 - 2.0 ** -7        # representable stays
    assert r(3.3895313892515355e38) == 3.3895313892515355e38   # the largest bf16 stays
    assert r(3.4e38) == float("inf")                      # more than half an ulp above it -> inf
    assert math.isnan(r(float("nan")))
    import torch
    rng = np.random.default_rng(3)
    a = np.concatenate([rng.standard_normal(20000).astype(np.float32) * 10.0 ** rng.integers(-30, 30, 20000),
                        np.array([0.0, -0.0, 1e-45, 1e-40, 65504.0, 3.38e38, -3.4e38], dtype=np.float32)])
    ref = torch.from_numpy(a).to(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(oracle.round_bf16(a).view(np.uint32), ref.view(np.uint32))


# ---------------------------------------------------------------- stack
def test_stack_is_chain_of_layers():
    specs = [(12, 20, 3, 2, "gelu"), (20, 12, 5, 1, "none"), (12, 20, 3, 0, "gelu")]
    layers, dense = [], []
    for li, (i, o, k, na, act) in enumerate(specs):
        L = inputs.make_layer(i, o, k, n_ablated=na, seed=4, stream=li)
        v, ix, rows = oracle.pack(L.w_dense, L.mask)
        layers.append((v, ix, rows, L.bias, i, o, act))
        dense.append((L, act))
    x = inputs.make_x(3, 12, seed=4)
    outs, exact, _ = oracle.stack_forward(layers, x, dtype="f32")
    import torch
    cur = x.astype(np.float64)
    for (L, act), got in zip(dense, exact):
        cur = dense_numpy(L, cur.astype(np.float32))
        if act == "gelu":
            cur = torch.nn.functional.gelu(torch.from_numpy(cur), approximate="none").numpy()
        assert np.allclose(got, cur, rtol=0, atol=1e-12)
        cur = cur.astype(np.float32).astype(np.float64)


def _bf16_torch(a):
    """fp32 -> bf16 -> fp32 through torch's conversion (round to nearest even), independent of the oracle's own."""
    import torch
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(torch.bfloat16).to(torch.float32).numpy()


def _is_bf16(a):
    return bool(np.all((np.ascontiguousarray(a, dtype=np.float32).view(np.uint32) & 0xFFFF) == 0))


def test_stack_bf16_rounds_where_a_bf16_layer_stores():
    """bf16 chain: values and x are rounded when stored, every layer's output once at its store, the bias stays
    fp32, sums are exact products in double.  The chain is written out here with torch's bf16 conversion and numpy
    float64 dense products; a chain with any of the roundings left out must differ from it visibly."""
    import torch
    specs = [(16, 24, 5, 2, "gelu"), (24, 16, 7, 1, "none"), (16, 24, 5, 0, "gelu"), (24, 16, 7, 3, "none")]
    layers, dense = [], []
    for li, (i, o, k, na, act) in enumerate(specs):
        L = inputs.make_layer(i, o, k, n_ablated=na, seed=9, stream=li)
        v, ix, rows = oracle.pack(L.w_dense, L.mask)
        layers.append((v, ix, rows, L.bias, i, o, act))
        dense.append((L, act))
    x = inputs.make_x(5, 16, seed=9)
    outs, exact, scales = oracle.stack_forward(layers, x, dtype="bf16")

    def chain(round_w, round_x, round_y):
        cur = (_bf16_torch(x) if round_x else x).astype(np.float64)
        ys, stored = [], []
        for (L, act) in dense:
            w = (_bf16_torch(L.w_dense) if round_w else L.w_dense).astype(np.float64) * L.mask
            y = cur @ w.T + L.bias.astype(np.float64)[None, :]          # bias is NOT rounded
            if act == "gelu":
                y = torch.nn.functional.gelu(torch.from_numpy(y), approximate="none").numpy()
            ys.append(y)
            cur = (_bf16_torch(y.astype(np.float32)) if round_y else y.astype(np.float32)).astype(np.float64)
            stored.append(cur)
        return ys, stored

    ys, stored = chain(True, True, True)
    for i in range(len(specs)):
        assert np.allclose(exact[i], ys[i], rtol=0, atol=1e-12), i
        assert np.array_equal(outs[i], stored[i]), i                       # the rounded hand-over, bit for bit
        assert _is_bf16(outs[i]), i
        assert np.all(scales[i] >= np.abs(exact[i]) - 1e-12) or specs[i][4] == "gelu"
    # Each rounding matters at this size: leaving one out moves the last layer by far more than 1e-12.
    for flags in ((False, True, True), (True, False, True), (True, True, False)):
        other, _ = chain(*flags)
        assert np.max(np.abs(other[-1] - exact[-1])) > 1e-5, flags
    # A bias that is not bf16-representable must come through unrounded (ablated rows of a no-activation layer).
    L1 = dense[1][0]
    assert not _is_bf16(L1.bias[L1.ablated])
    assert np.array_equal(exact[1][:, L1.ablated], np.tile(L1.bias[L1.ablated].astype(np.float64), (5, 1)))


# ---------------------------------------------------------------- generator
def test_generator_structure_and_moments():
    L = inputs.make_layer(768, 512, 77, n_ablated=51, seed=0, stream=7)
    assert np.array_equal(L.mask.sum(axis=1)[np.setdiff1d(np.arange(512), L.ablated)], np.full(461, 77))
    assert np.all(L.mask[L.ablated] == 0) and np.all(L.w_dense[L.mask == 0] == 0)
    kept = L.w_dense[L.mask == 1].astype(np.float64)
    n = kept.size
    assert abs(kept.mean()) < 4 * (1 / math.sqrt(77)) / math.sqrt(n)
    assert abs(kept.var() * 77 - 1) < 4 * math.sqrt(2 / n)
    assert abs(L.bias.astype(np.float64).var() / 0.01 - 1) < 4 * math.sqrt(2 / 512)
    x = inputs.make_x(64, 768, seed=0)
    assert abs(x.mean()) < 4 / math.sqrt(x.size) and abs(x.var() - 1) < 4 * math.sqrt(2 / x.size)
    col = L.mask.sum(axis=0).astype(np.float64)            # uniform column use: chi-square about its mean
    e = 461 * 77 / 768
    chi2 = ((col - e) ** 2 / (e * (1 - 77 / 768))).sum()
    assert abs(chi2 - 767) < 5 * math.sqrt(2 * 767)
    L2 = inputs.make_layer(768, 512, 77, n_ablated=51, seed=0, stream=7)
    assert np.array_equal(L.w_dense, L2.w_dense) and np.array_equal(L.bias, L2.bias)


def test_named_workloads_match_stated_shapes():
    w = inputs.workloads()
    assert (w["c1"].in_features, w["c1"].out_features, w["c1"].k, w["c1"].batch) == (768, 3072, 77, 1)
    assert w["c2"].batch == 256 and w["c3_b64"].n_ablated == 77 and w["c3_b1"].k == 307
    assert [w[f"c4_s{s}_b1"].k for s in (80, 90, 95, 99)] == [819, 410, 205, 41]
    s = inputs.StackWorkload()
    specs = s.layer_specs()
    assert len(specs) == 24 and specs[0] == (768, 3072, 77, 154, "gelu") and specs[1] == (3072, 768, 307, 38, "none")
    assert s.batch == 50432
