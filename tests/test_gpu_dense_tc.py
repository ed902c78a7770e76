"""The tensor-core variant (dense copy of the weight, tcgen05) against the oracle, element by element.

bf16 layers: exact bf16 products, fp32 accumulation, so the bf16 tolerance of the other parity tests applies.
fp32 layers: three TF32 products of operands split into two TF32-exact parts; what the split drops is below
3 * 2^-20 of each term, so the fp32 tolerance (1e-5 of the sum's scale) applies unchanged, down to a fan-in of one.
Small-integer cases must agree bit for bit in both.
"""
import numpy as np
import pytest

from paper_2305_02299_b200 import inputs
from parity import TOL, assert_parity, device_layer, oracle_layer, run_device, scaled_error

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("in_f,out_f,k,nabl", [(64, 8, 5, 1), (72, 136, 9, 10), (768, 384, 77, 19), (3072, 200, 307, 20),
                                              # few tiles and a long K: K split over a cluster of 4 or 8 CTAs, uneven shares, ragged tail
                                              (1000, 72, 100, 5), (520, 640, 52, 30)])
@pytest.mark.parametrize("B", [1, 5, 128, 257])
@pytest.mark.parametrize("act", ["none", "gelu"])
@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_dense_tc_matches_oracle(in_f, out_f, k, nabl, B, act, dtype):
    L = inputs.make_layer(in_f, out_f, k, n_ablated=nabl, seed=in_f + B)
    x = inputs.make_x(B, in_f, seed=B)
    y_ref, S = oracle_layer(L, x, dtype, act)
    dl = device_layer(L, dtype, act)
    y = run_device(dl, x, dtype, "dense_tc")
    dl.close()
    assert np.all(np.isfinite(y))
    assert_parity(y, y_ref, S, dtype)


# fp32: every batch tile (16, 32, 48, 64, 96, 128 rows; the MMAs are 2 x and 1 x that wide) with and without a K split over a
# thread-block cluster, on shapes with ragged output, batch and K tails, few and many K blocks per CTA (more blocks
# than ring stages, fewer blocks than CTAs of the cluster), ablated rows and both activations.
SPLIT_SHAPES = [(768, 384, 77, 19, 200, "gelu"), (3072, 200, 307, 20, 70, "none"), (1000, 72, 100, 5, 257, "gelu"),
                (520, 640, 52, 30, 129, "none"), (64, 8, 5, 1, 5, "gelu"), (40, 136, 1, 7, 33, "none")]


@pytest.mark.parametrize("tile", [16, 32, 48, 64, 96, 128])
@pytest.mark.parametrize("cluster", [1, 2, 3, 4, 8])
def test_dense_split_tf32_every_launch_shape(tile, cluster):
    from paper_2305_02299_b200 import binding as cfi
    for in_f, out_f, k, nabl, B, act in SPLIT_SHAPES:
        L = inputs.make_layer(in_f, out_f, k, n_ablated=nabl, seed=in_f + out_f)
        x = inputs.make_x(B, in_f, seed=B)
        y_ref, S = oracle_layer(L, x, "f32", act)
        dl = device_layer(L, "f32", act)
        y = run_device(dl, x, "f32", dense_shape=(tile, cluster))
        y2 = run_device(dl, x, "f32", dense_shape=(tile, cluster))
        assert cfi.cfi_device_status(dl) == 0
        dl.close()
        assert scaled_error(y, y_ref, S) <= TOL["f32"], (in_f, out_f, B, tile, cluster)
        assert np.array_equal(y, y2)                      # fixed order of additions: the same bits every time


@pytest.mark.parametrize("tile,cluster", [(16, 4), (48, 4), (64, 8), (96, 2), (128, 2), (32, 1)])
def test_dense_split_tf32_chain_of_launches(tile, cluster):
    """Back-to-back launches (a CUDA graph of 48 calls over 6 rotating layers; each launch lets its successor start
    early and waits for its predecessor before it reads x): a long K, so that the ring wraps several times per CTA.
    No wait may give up (status word), and every call must give the bits of the same call made alone."""
    import torch
    from paper_2305_02299_b200 import binding as cfi
    in_f, out_f, k, B, n = 2048, 640, 64, 24, 6
    layers, xs, ys, alone = [], [], [], []
    for i in range(n):
        L = inputs.make_layer(in_f, out_f, k, n_ablated=5, seed=900 + i)
        x = inputs.make_x(B, in_f, seed=950 + i)
        dl = device_layer(L, "f32", "gelu" if i % 2 else "none")
        if i == 0:
            y_ref, S = oracle_layer(L, x, "f32", "none")
            assert scaled_error(run_device(dl, x, "f32", dense_shape=(tile, cluster)), y_ref, S) <= TOL["f32"]
        alone.append(run_device(dl, x, "f32", dense_shape=(tile, cluster)))
        layers.append(dl)
        xs.append(torch.from_numpy(x).cuda())
        ys.append(torch.empty((B, out_f), device="cuda"))
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        for i in range(n):
            cfi.cfi_forward_dense(layers[i], xs[i], ys[i], B, tile=tile, cluster=cluster)
        stream.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            for j in range(48):
                cfi.cfi_forward_dense(layers[j % n], xs[j % n], ys[j % n], B, tile=tile, cluster=cluster)
        for _ in range(5):
            graph.replay()
        stream.synchronize()
    for i in range(n):
        assert cfi.cfi_device_status(layers[i]) == 0, (i, tile, cluster)
        assert np.array_equal(ys[i].double().cpu().numpy(), alone[i]), (i, tile, cluster)
        layers[i].close()


def test_dense_split_tf32_shape_choice_and_bad_shapes():
    """The shape the library picks is one of the allowed ones and runs; values outside the sets are refused."""
    from paper_2305_02299_b200 import binding as cfi
    L = inputs.make_layer(3072, 768, 307, n_ablated=77, seed=2)
    dl = device_layer(L, "f32")
    seen = set()
    for B in (9, 16, 40, 64, 100, 256, 700):
        tile, cluster = cfi.cfi_dense_tile_shape(dl, B)
        assert tile in (16, 32, 48, 64, 96, 128) and 1 <= cluster <= 8
        seen.add((tile, cluster))
    assert len({c for _, c in seen}) >= 2 and len({t for t, _ in seen}) >= 2, seen   # few output tiles, long K: K is split
    x = inputs.make_x(16, 3072)
    for tile, cluster in ((40, 1), (256, 1), (64, 9), (64, -1)):
        with pytest.raises(cfi.CfiError) as e:
            run_device(dl, x, "f32", dense_shape=(tile, cluster))
        assert e.value.status == 2
    dl.close()


@pytest.mark.parametrize("in_f,out_f,k,nabl,B,act", [(768, 1000, 77, 50, 9601, "gelu"), (1024, 512, 102, 0, 19001, "none"),
                                                     (200, 2048, 20, 100, 4801, "gelu"), (768, 3072, 77, 154, 7000, "gelu"),
                                                     (256, 2120, 26, 60, 2200, "gelu")])
def test_dense_tc_bf16_many_tiles_per_sm(in_f, out_f, k, nabl, B, act):
    """Enough 128 x 256 tiles for the persistent bf16 kernel (at least two per SM): ragged last batch tile and last
    output tile (also one that ends in the first half of a tile, and one whose last 64-column store boxes lie partly
    and wholly past the outputs), ablated rows, more tiles than CTAs so that both accumulator buffers and both store
    boxes are reused.  run_device keeps guard bands around y, so a store that is not clipped at the end of y fails."""
    from paper_2305_02299_b200 import binding as cfi
    L = inputs.make_layer(in_f, out_f, k, n_ablated=nabl, seed=B)
    x = inputs.make_x(B, in_f, seed=B + 1)
    y_ref, S = oracle_layer(L, x, "bf16", act)
    dl = device_layer(L, "bf16", act)
    assert cfi.cfi_dense_tile_shape(dl, B) == (256, 1)
    assert cfi.cfi_dense_tile_shape(dl, 256)[0] == 128   # few tiles: one tile per CTA, K possibly split over a cluster
    y = run_device(dl, x, "bf16", "dense_tc")
    y2 = run_device(dl, x, "bf16", "dense_tc")
    dl.close()
    assert np.all(np.isfinite(y))
    assert_parity(y, y_ref, S, "bf16")
    assert np.array_equal(y, y2)


def test_dense_tc_bf16_cluster_split_is_exercised():
    """bf16, few tiles and a long K: the one-tile kernel with K split over clusters of several sizes (asserted through
    cfi_dense_tile_shape), each case against the oracle; and a case with enough tiles that it does not split."""
    from paper_2305_02299_b200 import binding as cfi
    seen = set()
    for in_f, out_f, k, nabl, B, act in [(3072, 768, 307, 77, 256, "none"), (3072, 768, 307, 77, 64, "gelu"), (4096, 256, 41, 3, 100, "gelu"),
                                          (1000, 72, 100, 5, 257, "none"), (520, 640, 52, 30, 128, "gelu"), (256, 3072, 26, 0, 700, "gelu")]:
        L = inputs.make_layer(in_f, out_f, k, n_ablated=nabl, seed=in_f + B)
        x = inputs.make_x(B, in_f, seed=B)
        y_ref, S = oracle_layer(L, x, "bf16", act)
        dl = device_layer(L, "bf16", act)
        shape = cfi.cfi_dense_tile_shape(dl, B)
        seen.add(shape)
        y = run_device(dl, x, "bf16", "dense_tc")
        dl.close()
        assert_parity(y, y_ref, S, "bf16", str((in_f, out_f, B, shape)))
    clusters = {c for t, c in seen if t == 128}
    assert 1 in clusters and len([c for c in clusters if c > 1]) >= 2, seen


def test_dense_split_tf32_wide_dynamic_range():
    """Inputs spread over many binades: the split must hold for every magnitude, not only for N(0,1)."""
    L = inputs.make_layer(512, 128, 51, n_ablated=7, seed=9)
    rng = np.random.default_rng(4)
    x = (inputs.make_x(130, 512, seed=9) * np.exp2(rng.integers(-20, 20, size=(130, 512)))).astype(np.float32)
    L.w_dense *= np.exp2(rng.integers(-12, 12, size=L.w_dense.shape)).astype(np.float32)
    y_ref, S = oracle_layer(L, x, "f32")
    dl = device_layer(L, "f32")
    y = run_device(dl, x, "f32", "dense_tc")
    dl.close()
    assert scaled_error(y, y_ref, S) <= TOL["f32"]


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_dense_tc_exact_integers_and_agreement_with_gather(dtype):
    L = inputs.make_layer(512, 152, 24, n_ablated=11, seed=7, integer_valued=True)
    x = inputs.make_x(200, 512, seed=7, integer_valued=True, density=0.15 if dtype == "bf16" else 1.0)
    y_ref, _ = oracle_layer(L, x, dtype)
    if dtype == "bf16":
        assert np.max(np.abs(y_ref)) <= 256
    dl = device_layer(L, dtype)
    y_tc = run_device(dl, x, dtype, "dense_tc")
    y_gather = run_device(dl, x, dtype, "batch")
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
    L = inputs.make_layer(30, 16, 4, seed=1)             # fp32 rows of 120 bytes: not a multiple of 16
    dl = device_layer(L, "f32")
    with pytest.raises(cfi.CfiError):
        run_device(dl, inputs.make_x(4, 30), "f32", "dense_tc")
    assert cfi.cfi_device_status(dl) == 0
    dl.close()
