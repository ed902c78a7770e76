"""cfi_srigl_update (device) against the oracle of Sec. 3.1's seven steps: masks and weights bit for bit, k' and the
number of live neurons equal.  Index and integer work: no tolerance."""
import numpy as np
import pytest

from oracle.srigl_update import srigl_update
from paper_2305_02299_b200 import inputs

pytestmark = pytest.mark.gpu


def _layer(out_f, in_f, k, n_abl, seed):
    L = inputs.make_layer(in_f, out_f, k, n_ablated=n_abl, seed=seed, bias=False)
    g = inputs.make_x(out_f, in_f, seed=seed + 77)
    return L.w_dense.copy(), L.mask.copy(), g


def _run_device(w, m, g, K, gamma):
    import torch
    from paper_2305_02299_b200 import binding as cfi
    wd, md, gd = torch.from_numpy(w).cuda(), torch.from_numpy(m).cuda(), torch.from_numpy(g).cuda()
    k_new, n_act = cfi.cfi_srigl_update(wd, md, gd, K, gamma)
    torch.cuda.synchronize()
    return wd.cpu().numpy(), md.cpu().numpy(), k_new, n_act


def _compare(w, m, g, K, gamma):
    gamma = float(np.float32(gamma))
    w_ref, m_ref, k_ref, abl = srigl_update(w, m, g, K, gamma)
    w_dev, m_dev, k_dev, n_dev = _run_device(w, m, g, K, gamma)
    assert k_dev == k_ref
    assert n_dev == int((m_ref.sum(1) > 0).sum())
    assert np.array_equal(m_dev, m_ref)
    assert np.array_equal(w_dev, w_ref)
    return k_ref, abl


@pytest.mark.parametrize("out_f,in_f,k,n_abl,K,gamma", [
    (24, 40, 6, 0, 30, 0.3), (24, 40, 6, 3, 60, 0.5), (16, 16, 2, 0, 8, 1.0), (64, 96, 10, 5, 200, 0.3),
    (8, 8, 8, 0, 0, 0.3), (12, 30, 3, 0, 36, 0.0), (1, 5, 2, 0, 1, 0.5), (7, 4099, 33, 1, 100, 0.25),
    (768, 3072, 307, 38, 70_000, 0.3), (3072, 768, 77, 154, 60_000, 0.3), (300, 1000, 10, 0, 2990, 0.9),
    (6, 9000, 50, 1, 120, 0.25), (5, 9001, 40, 0, 199, 0.5)])   # rows too long for the shared-memory copy of the keys
def test_matches_oracle(out_f, in_f, k, n_abl, K, gamma):
    w, m, g = _layer(out_f, in_f, k, n_abl, seed=out_f + in_f)
    _compare(w, m, g, K, gamma)


def test_matches_oracle_at_the_benchmarked_size():
    """4096 x 4096 at 80 % sparsity with K = 30 % of the active weights (about 1.0 M): the size and K the benchmark's
    mask-update leg times."""
    w, m, g = _layer(4096, 4096, 819, 0, seed=11)
    _compare(w, m, g, int(0.3 * 4096 * 819), 0.3)


def test_ablation_case_and_chained_updates():
    """A neuron with tiny weights and gradients is ablated and k' rises; a second update on the result still matches."""
    w, m, g = _layer(64, 256, 16, 0, seed=9)
    w[5] *= 1e-6
    g[5] *= 1e-6
    w[40] *= 1e-6
    g[40] *= 1e-6
    k2, abl = _compare(w, m, g, 32, 0.3)
    assert set(abl) == {5, 40} and k2 == (16 * 64) // 62
    w2, m2, _, _ = srigl_update(w, m, g, 32, float(np.float32(0.3)))
    g2 = inputs.make_x(64, 256, seed=123)
    _compare(w2, m2, g2, 50, 0.3)


@pytest.mark.parametrize("seed", range(6))
def test_many_ties(seed):
    """Quantised magnitudes and gradients: most selections are decided by position."""
    rng = np.random.default_rng(seed)
    out_f, in_f, k = int(rng.integers(3, 40)), int(rng.integers(8, 300)), 0
    k = int(rng.integers(1, min(in_f, 20)))
    w, m, g = _layer(out_f, in_f, k, int(rng.integers(0, out_f // 3 + 1)), seed=200 + seed)
    w = (np.round(w * 2) / 2 * (m == 1)).astype(np.float32)
    g = np.round(g).astype(np.float32)
    _compare(w, m, g, int(rng.integers(0, out_f * k + 1)), float(rng.choice([0.0, 0.25, 0.5, 1.0])))


@pytest.mark.parametrize("levels", [3, 4096])
def test_ties_with_and_without_room_in_the_candidate_list(levels):
    """300 x 1024 with magnitudes and gradients quantised to `levels` values.  With 3 levels a third of the layer
    equals the cut key: far more than the list of the last digit's candidates holds (4800 entries), so ties are ranked
    by the counting path; with 4096 levels the ties at the cut fit the list and the marking takes them up to a position.
    Both must equal the oracle bit for bit."""
    w, m, g = _layer(300, 1024, 100, 7, seed=77)
    q = float(levels)
    w = (np.ceil(np.abs(w) * q / 4) * 4 / q * np.sign(w) * (m == 1)).astype(np.float32)
    g = (np.round(g * q / 8) * 8 / q).astype(np.float32)
    _compare(w, m, g, 9000, 0.3)


def test_workspace_and_argument_checks():
    import ctypes
    import torch
    from paper_2305_02299_b200 import binding as cfi
    w = torch.zeros((4, 8), device="cuda")
    m = torch.zeros((4, 8), device="cuda", dtype=torch.uint8)
    with pytest.raises(cfi.CfiError) as e:
        cfi.cfi_srigl_update(w, m, w, 1, -0.5)
    assert e.value.status == 2
    k_new, n_act = cfi.cfi_srigl_update(w, m, w, 3, 0.3)      # a layer with no active weight stays empty
    assert (k_new, n_act) == (0, 0) and int(m.sum()) == 0


def test_update_then_pack_create_forward():
    """The update's output is a constant-fan-in mask that the forward path accepts as is: cfi_pack (mask given, so grown
    weights with value 0 count), cfi_create, cfi_forward, against the oracle forward on the oracle's updated layer."""
    import torch
    import oracle
    from paper_2305_02299_b200 import binding as cfi
    from parity import TOL, scaled_error
    w, m, g = _layer(384, 512, 51, 20, seed=31)
    w[7] *= 1e-6
    g[7] *= 1e-6
    gamma = float(np.float32(0.3))
    w_ref, m_ref, k_ref, _ = srigl_update(w, m, g, 3000, gamma)
    w_dev, m_dev, k_dev, n_dev = _run_device(w, m, g, 3000, gamma)
    assert k_dev == k_ref and np.array_equal(m_dev, m_ref)
    v, ix, rows = cfi.cfi_pack(w_dev, m_dev)
    assert v.shape == (n_dev, k_dev) and np.any(v == 0.0)            # freshly grown weights are kept entries of value 0
    bias = inputs.make_layer(512, 384, 51, seed=32).bias
    x = inputs.make_x(40, 512, seed=33)
    vr, ir, rr = oracle.pack(w_ref, m_ref)
    y_ref, S = oracle.forward(vr, ir, rr, bias, 512, 384, x, want_scale=True)
    layer = cfi.cfi_create(v, ix, rows, bias, 512, 384)
    y = torch.empty((40, 384), device="cuda")
    cfi.cfi_forward(layer, torch.from_numpy(x).cuda(), y, 40)
    torch.cuda.synchronize()
    layer.close()
    assert scaled_error(y.cpu().numpy(), y_ref, S) <= TOL["f32"]


@pytest.mark.parametrize("out_f,in_f,k,n_abl", [(24, 40, 6, 0), (300, 1000, 10, 37), (7, 4099, 33, 1), (768, 3072, 307, 38), (5, 9, 9, 0)])
def test_pack_device_equals_host_pack(out_f, in_f, k, n_abl):
    """cfi_pack_device on device-resident w and mask gives exactly cfi_pack's arrays (and the oracle's)."""
    import torch
    import oracle
    from paper_2305_02299_b200 import binding as cfi
    w, m, _ = _layer(out_f, in_f, k, n_abl, seed=out_f)
    zr, zc = np.nonzero(m == 1)
    w[zr[::7], zc[::7]] = 0.0                                    # kept entries of value 0 still count (the mask decides)
    v, ix, rows = cfi.cfi_pack_device(torch.from_numpy(w).cuda(), torch.from_numpy(m).cuda())
    vh, ih, rh = cfi.cfi_pack(w, m)
    vo, io, ro = oracle.pack(w, m)
    assert np.array_equal(v.cpu().numpy(), vh) and np.array_equal(ix.cpu().numpy(), ih) and np.array_equal(rows.cpu().numpy(), rh)
    assert np.array_equal(vh, vo) and np.array_equal(ih, io) and np.array_equal(rh, ro)


def test_pack_device_errors_and_empty():
    import torch
    from paper_2305_02299_b200 import binding as cfi
    w, m, _ = _layer(10, 20, 4, 2, seed=3)
    m2 = m.copy()
    row = int(np.nonzero(m2.sum(1))[0][0])
    m2[row, np.nonzero(m2[row])[0][0]] = 0                        # one row keeps one entry fewer
    with pytest.raises(cfi.CfiError) as e:
        cfi.cfi_pack_device(torch.from_numpy(w).cuda(), torch.from_numpy(m2).cuda())
    assert e.value.status == 3
    v, ix, rows = cfi.cfi_pack_device(torch.zeros((4, 8), device="cuda"), torch.zeros((4, 8), device="cuda", dtype=torch.uint8))
    assert v.shape == (0, 0) and rows.shape == (0,)
