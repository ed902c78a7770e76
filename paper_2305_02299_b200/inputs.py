"""Seeded synthetic inputs for the condensed constant-fan-in linear layer.

This module only draws random numbers and lays them out; it performs none of
the layer's arithmetic (no packing, no products, no rounding to bf16).  Both
the CPU oracle's tests and the CUDA library's tests/benchmarks take their
inputs from here, so that the two sides see bit-identical arrays without
sharing any code of the method itself.

What is generated mirrors the layers the paper benchmarks (Sec. 4.4 and the
appendix "Condensed linear CPU benchmark details": the two linear layers of a
ViT-B/16 MLP block, 768 <-> 3072 features, fp32, 80-99 % sparsity): a dense
weight matrix with a mask that keeps exactly k entries in every non-ablated
row and none in an ablated row.  The paper's layers come from a trained
model; here the kept columns are uniform random, which is stated wherever a
number measured on these inputs is reported.

Every tensor has its own Philox stream keyed by (seed, stream id, tensor id),
so a tensor does not change when another one is added or resized.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional, Tuple

import numpy as np

_T_MASK, _T_WEIGHT, _T_BIAS, _T_ABLATE, _T_X, _T_XI = 1, 2, 3, 4, 5, 6


def _rng(seed: int, stream: int, tensor: int) -> np.random.Generator:
    key = (int(seed) & 0xFFFFFFFF) | ((int(stream) & 0xFFFFFF) << 32) | ((int(tensor) & 0xFF) << 56)
    return np.random.Generator(np.random.Philox(key=key))


@dataclass
class DenseMaskedLayer:
    """A dense weight with its keep-mask, as a trained layer would be handed over.

    w_dense : float32 [out_features, in_features], zero wherever mask == 0
    mask    : uint8   [out_features, in_features], 1 = kept weight
    bias    : float32 [out_features]
    k       : kept entries in every non-ablated row
    ablated : sorted int32 row numbers whose mask row is all zero
    """
    w_dense: np.ndarray
    mask: np.ndarray
    bias: np.ndarray
    k: int
    ablated: np.ndarray
    in_features: int = field(init=False)
    out_features: int = field(init=False)

    def __post_init__(self):
        self.out_features, self.in_features = self.w_dense.shape

    @property
    def n_active(self) -> int:
        return self.out_features - int(self.ablated.size)


def _choose_columns(rng: np.random.Generator, rows: int, in_features: int, k: int) -> np.ndarray:
    """k distinct uniform-random columns per row (unsorted), shape [rows, k]."""
    if k == in_features:
        return np.tile(np.arange(in_features, dtype=np.int64), (rows, 1))
    out = np.empty((rows, k), dtype=np.int64)
    step = max(1, (1 << 24) // max(in_features, 1))
    for r0 in range(0, rows, step):
        r1 = min(rows, r0 + step)
        u = rng.random((r1 - r0, in_features), dtype=np.float32)
        out[r0:r1] = np.argpartition(u, k - 1, axis=1)[:, :k]
    return out


def make_layer(in_features: int, out_features: int, k: int, *, n_ablated: int = 0, seed: int = 0,
               stream: int = 0, integer_valued: bool = False, bias: bool = True) -> DenseMaskedLayer:
    """Draw one masked dense layer.

    Kept weights ~ N(0, variance 1/k), bias ~ N(0, variance 0.01).  With
    integer_valued=True weights and bias are small integers in [-4, 4]
    (weights never 0), so that sums of products with integer x are exact in
    fp32 whatever the order of summation.
    """
    if not (1 <= k <= in_features) and not (out_features == n_ablated):
        raise ValueError("need 1 <= k <= in_features")
    if not (0 <= n_ablated <= out_features):
        raise ValueError("need 0 <= n_ablated <= out_features")
    abl = np.sort(_rng(seed, stream, _T_ABLATE).permutation(out_features)[:n_ablated]).astype(np.int32)
    active = np.ones(out_features, dtype=bool)
    active[abl] = False
    n_act = int(active.sum())

    mask = np.zeros((out_features, in_features), dtype=np.uint8)
    w = np.zeros((out_features, in_features), dtype=np.float32)
    if n_act:
        cols = _choose_columns(_rng(seed, stream, _T_MASK), n_act, in_features, k)
        rows = np.repeat(np.nonzero(active)[0], k)
        mask[rows, cols.ravel()] = 1
        wr = _rng(seed, stream, _T_WEIGHT)
        if integer_valued:
            vals = wr.integers(1, 5, size=n_act * k).astype(np.float32)
            vals *= wr.choice(np.array([-1.0, 1.0], dtype=np.float32), size=n_act * k)
        else:
            vals = (wr.standard_normal(n_act * k) / np.sqrt(float(k))).astype(np.float32)
        w[rows, cols.ravel()] = vals
    br = _rng(seed, stream, _T_BIAS)
    if not bias:
        b = np.zeros(out_features, dtype=np.float32)
    elif integer_valued:
        b = br.integers(-4, 5, size=out_features).astype(np.float32)
    else:
        b = (br.standard_normal(out_features) * 0.1).astype(np.float32)
    return DenseMaskedLayer(w_dense=w, mask=mask, bias=b, k=int(k), ablated=abl)


def make_x(batch: int, in_features: int, *, seed: int = 0, stream: int = 0,
           integer_valued: bool = False, density: float = 1.0) -> np.ndarray:
    """x ~ N(0,1), float32 [batch, in_features]; or small integers in [-3,3].

    density < 1 zeroes a random subset of entries (used by the exact-integer
    bf16 cases, which need every partial sum to stay small).
    """
    r = _rng(seed, stream, _T_X)
    if integer_valued:
        x = r.integers(-3, 4, size=(batch, in_features)).astype(np.float32)
    else:
        x = r.standard_normal((batch, in_features), dtype=np.float32)
    if density < 1.0:
        x *= (r.random((batch, in_features), dtype=np.float32) < density)
    return np.ascontiguousarray(x, dtype=np.float32)


# ----------------------------------------------------------------------------
# Named workloads.  Layer shapes are the ViT-B/16 MLP linears the paper times
# (Sec. 4.4; appendix "Condensed linear CPU benchmark details"); sparsities are
# the paper's sweep 80/90/95/99 %; batch sizes 1 and 256 are those of its
# CPU-online and GPU figures.  k = round((1 - sparsity) * in_features).
# ----------------------------------------------------------------------------
@dataclass(frozen=True)
class Workload:
    name: str
    in_features: int
    out_features: int
    k: int
    n_ablated: int
    batch: int
    dtype: str = "f32"       # storage type of values / x / y ("f32" or "bf16")
    act: str = "none"        # "none" or "gelu"
    stream: int = 0

    def layer(self, seed: int = 0, replica: int = 0) -> DenseMaskedLayer:
        return make_layer(self.in_features, self.out_features, self.k, n_ablated=self.n_ablated,
                          seed=seed, stream=self.stream + 1000 * replica)

    def x(self, seed: int = 0, replica: int = 0, batch: Optional[int] = None) -> np.ndarray:
        return make_x(self.batch if batch is None else batch, self.in_features, seed=seed,
                      stream=self.stream + 1000 * replica)


def n_ablated_for(out_features: int, fraction: float) -> int:
    return int(np.floor(fraction * out_features + 0.5))


def workloads() -> Dict[str, Workload]:
    w: Dict[str, Workload] = {}
    w["c1"] = Workload("c1", 768, 3072, 77, 0, 1, stream=1)
    w["c2"] = Workload("c2", 768, 3072, 77, 0, 256, stream=1)
    for b in (1, 64, 256):
        w[f"c3_b{b}"] = Workload(f"c3_b{b}", 3072, 768, 307, n_ablated_for(768, 0.10), b, stream=3)
    for sp, k in ((80, 819), (90, 410), (95, 205), (99, 41)):
        for b in (1, 16, 256):
            w[f"c4_s{sp}_b{b}"] = Workload(f"c4_s{sp}_b{b}", 4096, 4096, k, 0, b, stream=40 + sp)
    return w


@dataclass(frozen=True)
class StackWorkload:
    """ViT-B/16-shaped MLP stack: blocks of 768->3072 (GELU) -> 3072->768."""
    name: str = "c5"
    blocks: int = 12
    d_model: int = 768
    d_hidden: int = 3072
    k_up: int = 77
    k_down: int = 307
    ablate_fraction: float = 0.05
    batch: int = 256 * 197
    dtype: str = "bf16"
    stream: int = 500

    def layer_specs(self) -> List[Tuple[int, int, int, int, str]]:
        """(in, out, k, n_ablated, act) for each of the 2*blocks layers in order."""
        specs = []
        for _ in range(self.blocks):
            specs.append((self.d_model, self.d_hidden, self.k_up,
                          n_ablated_for(self.d_hidden, self.ablate_fraction), "gelu"))
            specs.append((self.d_hidden, self.d_model, self.k_down,
                          n_ablated_for(self.d_model, self.ablate_fraction), "none"))
        return specs

    def layers(self, seed: int = 0) -> List[DenseMaskedLayer]:
        return [make_layer(i, o, k, n_ablated=na, seed=seed, stream=self.stream + li)
                for li, (i, o, k, na, _) in enumerate(self.layer_specs())]

    def x(self, seed: int = 0, batch: Optional[int] = None) -> np.ndarray:
        return make_x(self.batch if batch is None else batch, self.d_model, seed=seed, stream=self.stream)


# ----------------------------------------------------------------------------
# Draws for the output-norm-variance simulation (Sec. 3, "Constant Fan-In
# sparsity"; appendix "Computing the output norm variance", Definition 1):
# many independent square layers with W ~ N(0,1) iid, exactly k ones per row of
# I (rows independent, uniform over the k-subsets), xi ~ Ber(1/2)^n and u
# uniform on the unit sphere.  Only the draws; the scaling sqrt(2/k), the
# products and the norms are the caller's.
# ----------------------------------------------------------------------------
def make_norm_variance_draws(n: int, k: int, layers: int, batch: int, *, seed: int = 0, stream: int = 900):
    """Returns (w [layers,n,k] f32 ~ N(0,1), cols [layers,n,k] int32 distinct per row and ascending,
    xi [layers,batch,n] f32 in {0,1}, u [layers,batch,n] f32 with unit rows)."""
    if not (1 <= k <= n):
        raise ValueError("need 1 <= k <= n")
    cols = _choose_columns(_rng(seed, stream, _T_MASK), layers * n, n, k).reshape(layers, n, k)
    cols = np.sort(cols, axis=2).astype(np.int32)
    w = _rng(seed, stream, _T_WEIGHT).standard_normal((layers, n, k), dtype=np.float32)
    xi = (_rng(seed, stream, _T_XI).random((layers, batch, n), dtype=np.float32) < 0.5).astype(np.float32)
    g = _rng(seed, stream, _T_X).standard_normal((layers, batch, n))
    u = (g / np.linalg.norm(g, axis=2, keepdims=True)).astype(np.float32)
    return w, cols, xi, u
