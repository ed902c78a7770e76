"""CPU oracle of one SRigL mask update of one layer (Sec. 3.1, the seven numbered steps "for each layer").

TEST INFRASTRUCTURE ONLY, like the rest of this package: plain numpy, whole-array sorts, no attempt at speed, and no
code shared with the CUDA library.  Steps are taken in the paper's order and notation (K = weights pruned and grown
in this step, k = fan-in before, k' = fan-in after, gamma_sal = ablation threshold).

Where the paper leaves a choice open, the reading taken is:
  * ties in magnitude are broken by position: among equal magnitudes the entry with the smaller flat index
    (row * in + column) counts as the smaller weight when pruning and as the larger gradient when growing;
  * "salient" (step 3): an active weight that is NOT among the K smallest magnitudes of the layer, or an inactive
    position that IS among the K largest gradient magnitudes of the layer;
  * rows that are already ablated (no active weight) stay ablated and take no part;
  * ablation threshold (step 4): a neuron is ablated if its salient count is below max(1, gamma_sal * k);
  * k' (step 5): floor(k * n_active_before / n_active_after), at most in_features: the layer's budget of weights is
    kept up to rounding;
  * the gradient top-K of step 3 is taken over the positions that were inactive before the update (step 1); the
    regrowth of step 7 may use any position of the neuron that is not active at that moment, which includes a
    weight pruned in step 6 (it restarts at 0, like every grown weight, as in RigL) -- so a neuron can always reach
    k' <= in_features;
  * a neuron left with more than k' weights after the global pruning of step 6 loses its smallest ones down to k'.
"""
from __future__ import annotations

import numpy as np


def _smallest(flat_keys: np.ndarray, candidates: np.ndarray, count: int) -> np.ndarray:
    """Flat positions of the `count` smallest keys among `candidates` (flat positions), ties to the smaller position."""
    if count <= 0 or candidates.size == 0:
        return candidates[:0]
    order = np.lexsort((candidates, flat_keys[candidates]))      # primary: key, secondary: position
    return candidates[order[:count]]


def _largest(flat_keys: np.ndarray, candidates: np.ndarray, count: int) -> np.ndarray:
    """Flat positions of the `count` largest keys among `candidates`, ties to the smaller position."""
    if count <= 0 or candidates.size == 0:
        return candidates[:0]
    order = np.lexsort((candidates, -flat_keys[candidates].astype(np.float64)))
    return candidates[order[:count]]


def srigl_update(w, mask, grad, K: int, gamma_sal: float):
    """One update.  w, grad: float32 [out, in]; mask: uint8 [out, in] with the same number k of ones in every non-empty
    row.  Returns (w_new float32, mask_new uint8, k_new int, ablated_now int32 rows ablated by this update)."""
    w = np.asarray(w, dtype=np.float32)
    g = np.asarray(grad, dtype=np.float32)
    m = np.asarray(mask, dtype=np.uint8) != 0
    out_f, in_f = w.shape
    row_counts = m.sum(axis=1)
    active_rows = np.nonzero(row_counts > 0)[0]
    if active_rows.size == 0:
        return np.zeros_like(w), np.zeros((out_f, in_f), np.uint8), 0, np.zeros(0, np.int32)
    k = int(row_counts[active_rows[0]])
    assert np.all(row_counts[active_rows] == k), "constant fan-in expected"
    row_is_active = row_counts > 0

    # Step 1: prune criterion = |w| of active weights; growth criterion = |grad| of inactive positions (of live rows).
    mag_w = np.abs(w).ravel()
    mag_g = np.abs(g).ravel()
    flat = np.arange(out_f * in_f)
    active_pos = flat[m.ravel()]
    inactive_pos = flat[(~m & row_is_active[:, None]).ravel()]
    # Step 2: K is given (the schedule that produces it is outside this function); it cannot exceed either pool.
    K = int(max(0, min(K, active_pos.size, inactive_pos.size)))
    # Step 3: salient weights per neuron.
    drop = _smallest(mag_w, active_pos, K)                  # the K smallest active magnitudes of the layer
    grow_top = _largest(mag_g, inactive_pos, K)             # the K largest gradient magnitudes of the layer
    dropped = np.zeros(out_f * in_f, bool)
    dropped[drop] = True
    grow_flag = np.zeros(out_f * in_f, bool)
    grow_flag[grow_top] = True
    salient = ((m.ravel() & ~dropped) | grow_flag).reshape(out_f, in_f).sum(axis=1)
    # Step 4: ablate neurons with too few salient weights.
    threshold = max(1.0, gamma_sal * k)
    ablate = row_is_active & (salient < threshold)
    survivors = row_is_active & ~ablate
    n_before, n_after = int(row_is_active.sum()), int(survivors.sum())
    w_new = np.zeros_like(w)
    m_new = np.zeros((out_f, in_f), bool)
    if n_after == 0:
        return w_new, m_new.astype(np.uint8), 0, np.nonzero(ablate)[0].astype(np.int32)
    # Step 5: the new fan-in.
    k_new = min(in_f, (k * n_before) // n_after)
    # Step 6: prune the K smallest magnitudes of the layer (the set of step 3); ablated neurons lose everything.
    kept = (m.ravel() & ~dropped).reshape(out_f, in_f)
    # Step 7: every surviving neuron is brought to exactly k' weights.
    for r in np.nonzero(survivors)[0]:
        base = r * in_f
        cols_kept = np.nonzero(kept[r])[0]
        if cols_kept.size > k_new:                          # too many left: drop the smallest down to k'
            extra = _smallest(mag_w, base + cols_kept, cols_kept.size - k_new) - base
            cols_kept = np.setdiff1d(cols_kept, extra)
        m_new[r, cols_kept] = True
        w_new[r, cols_kept] = w[r, cols_kept]
        need = k_new - cols_kept.size
        if need > 0:                                        # regrow in order of decreasing gradient magnitude
            cand = base + np.nonzero(~m_new[r])[0]          # every position of the neuron that is not active now
            grown = _largest(mag_g, cand, need) - base
            m_new[r, grown] = True                          # value 0
    return w_new, m_new.astype(np.uint8), int(k_new), np.nonzero(ablate)[0].astype(np.int32)
