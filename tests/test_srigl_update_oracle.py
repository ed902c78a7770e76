"""Pins of the SRigL mask-update oracle (Sec. 3.1, steps 1-7), none of which re-use its code: invariants the method
fixes, special cases with known answers, and a brute-force restatement with Python loops on tiny layers."""
import itertools

import numpy as np
import pytest

from oracle.srigl_update import srigl_update
from paper_2305_02299_b200 import inputs


def _layer(out_f, in_f, k, n_abl, seed):
    L = inputs.make_layer(in_f, out_f, k, n_ablated=n_abl, seed=seed, bias=False)
    g = inputs.make_x(out_f, in_f, seed=seed + 77)          # any seeded dense array serves as the gradient
    return L.w_dense, L.mask, g


def _check_invariants(w, m, g, K, gamma, w2, m2, k2, abl):
    out_f, in_f = w.shape
    rows_before = np.nonzero(m.sum(1) > 0)[0]
    k = int(m[rows_before[0]].sum())
    counts = m2.sum(1)
    live = np.nonzero(counts > 0)[0]
    assert set(live) | set(abl) == set(rows_before) and not (set(live) & set(abl))       # ablated rows stay out
    assert np.all(counts[live] == k2)                                                    # constant fan-in k'
    assert np.all(m2[abl] == 0) and np.all(w2[m2 == 0] == 0)
    if live.size:
        assert k2 == min(in_f, (k * rows_before.size) // live.size)                      # step 5
        assert live.size * k2 <= rows_before.size * k                                    # budget not exceeded
    both = (m2 == 1) & (m == 1)
    assert np.all((w2[both] == w[both]) | (w2[both] == 0))        # a survivor keeps its value (or was pruned and regrown at 0)
    assert np.all(w2[(m2 == 1) & (m == 0)] == 0)                  # grown weights start at 0


@pytest.mark.parametrize("out_f,in_f,k,n_abl,K,gamma", [(24, 40, 6, 0, 30, 0.3), (24, 40, 6, 3, 60, 0.5), (16, 16, 2, 0, 8, 1.0),
                                                        (64, 96, 10, 5, 200, 0.3), (8, 8, 8, 0, 0, 0.3), (12, 30, 3, 0, 36, 0.0)])
def test_invariants(out_f, in_f, k, n_abl, K, gamma):
    w, m, g = _layer(out_f, in_f, k, n_abl, seed=out_f + K)
    w2, m2, k2, abl = srigl_update(w, m, g, K, gamma)
    _check_invariants(w, m, g, K, gamma, w2, m2, k2, abl)


def test_nothing_to_prune_changes_nothing():
    w, m, g = _layer(20, 30, 5, 2, seed=1)
    w2, m2, k2, abl = srigl_update(w, m, g, 0, 0.3)          # every weight is salient, nothing is pruned or grown
    assert np.array_equal(m2, m) and np.array_equal(w2, w) and k2 == 5 and abl.size == 0


def test_without_ablation_each_row_regrows_what_it_lost():
    """gamma_sal = 0 ablates nobody (threshold max(1, 0) = 1 and every row keeps a salient weight here), so k' = k:
    the K globally smallest weights go, and each row regrows exactly as many as it lost, at its largest gradients."""
    w, m, g = _layer(10, 24, 6, 0, seed=3)
    K = 12
    w2, m2, k2, abl = srigl_update(w, m, g, K, 0.0)
    assert k2 == 6 and abl.size == 0
    mags = np.where(m == 1, np.abs(w), np.inf).ravel()
    cut = np.sort(mags)[K - 1]
    pruned = (m == 1) & (np.abs(w) <= cut)
    assert pruned.sum() == K                                  # no ties in these draws
    for r in range(10):
        lost = int(pruned[r].sum())
        new_cols = np.nonzero((m2[r] == 1) & ((m[r] == 0) | pruned[r]))[0]
        assert new_cols.size == lost and np.all(w2[r, new_cols] == 0)
        if lost:
            free = np.nonzero((m[r] == 0) | pruned[r])[0]
            best = free[np.argsort(-np.abs(g[r, free]), kind="stable")[:lost]]
            assert set(new_cols) == set(best)


def test_ablation_raises_the_fan_in():
    """A neuron whose weights are all tiny and whose gradients are all tiny has no salient weight and is ablated;
    its budget goes to the others: k' = floor(k n / (n - 1))."""
    w, m, g = _layer(8, 32, 4, 0, seed=5)
    w[3] *= 1e-6
    g[3] *= 1e-6
    K = 4                                                     # exactly row 3's four weights are the smallest
    w2, m2, k2, abl = srigl_update(w, m, g, K, 0.3)
    assert list(abl) == [3] and k2 == (4 * 8) // 7 and m2[3].sum() == 0
    assert np.all(m2.sum(1)[[0, 1, 2, 4, 5, 6, 7]] == k2)


def test_ties_go_to_the_smaller_position():
    m = np.zeros((2, 6), np.uint8)
    m[:, :3] = 1
    w = np.where(m == 1, 1.0, 0.0).astype(np.float32)         # all magnitudes equal
    g = np.ones((2, 6), np.float32)                           # all gradients equal
    w2, m2, k2, abl = srigl_update(w, m, g, 2, 0.0)
    # the two smallest flat positions (row 0, columns 0 and 1) are pruned; row 0 regrows two at the smallest free columns,
    # which are the ones just pruned (they restart at 0)
    assert k2 == 3 and np.array_equal(m2, m)
    assert list(w2[0]) == [0, 0, 1, 0, 0, 0] and list(w2[1]) == [1, 1, 1, 0, 0, 0]


def _brute_force(w, m, g, K, gamma):
    """The seven steps with Python lists and explicit loops (tiny layers only)."""
    out_f, in_f = w.shape
    act = [(abs(float(w[r, c])), r * in_f + c) for r in range(out_f) for c in range(in_f) if m[r, c]]
    live_rows = [r for r in range(out_f) if m[r].any()]
    ina = [(-abs(float(g[r, c])), r * in_f + c) for r in live_rows for c in range(in_f) if not m[r, c]]
    k = int(m[live_rows[0]].sum())
    K = max(0, min(K, len(act), len(ina)))
    drop = {p for _, p in sorted(act)[:K]}
    top = {p for _, p in sorted(ina)[:K]}
    sal = {r: 0 for r in live_rows}
    for _, p in act:
        if p not in drop:
            sal[p // in_f] += 1
    for p in top:
        sal[p // in_f] += 1
    thr = max(1.0, gamma * k)
    surv = [r for r in live_rows if sal[r] >= thr]
    m2 = np.zeros_like(m)
    w2 = np.zeros_like(w)
    if not surv:
        return w2, m2, 0
    k2 = min(in_f, (k * len(live_rows)) // len(surv))
    for r in surv:
        kept = sorted([(abs(float(w[r, c])), c) for c in range(in_f) if m[r, c] and (r * in_f + c) not in drop])
        while len(kept) > k2:
            kept.pop(0)
        cols = [c for _, c in kept]
        free = sorted([(-abs(float(g[r, c])), c) for c in range(in_f) if c not in cols])
        grown = [c for _, c in free[:k2 - len(cols)]]
        for c in cols:
            m2[r, c], w2[r, c] = 1, w[r, c]
        for c in grown:
            m2[r, c] = 1
    return w2, m2, k2


@pytest.mark.parametrize("seed", range(12))
def test_against_brute_force_on_tiny_layers(seed):
    rng = np.random.default_rng(seed)
    out_f, in_f = int(rng.integers(2, 7)), int(rng.integers(3, 9))
    k = int(rng.integers(1, in_f))
    w, m, g = _layer(out_f, in_f, k, int(rng.integers(0, max(1, out_f // 2))), seed=100 + seed)
    if seed % 3 == 0:                                         # quantised values: many ties
        w = np.round(w * 2) / 2 * (m == 1)
        g = np.round(g)
    K = int(rng.integers(0, out_f * k + 1))
    gamma = float(rng.choice([0.0, 0.3, 0.6, 1.0]))
    w2, m2, k2, _ = srigl_update(w, m, g, K, gamma)
    wb, mb, kb = _brute_force(w, m, g, K, gamma)
    assert k2 == kb and np.array_equal(m2, mb) and np.array_equal(w2, wb)
