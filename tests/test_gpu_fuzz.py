"""cfi_forward (automatic kernel choice) against the oracle on seeded random shapes: odd and aligned feature counts,
batches on both sides of every switch-over point, both dtypes and activations.  Whatever kernel and launch shape the
library picks for a case must launch and match."""
import numpy as np
import pytest

from paper_2305_02299_b200 import inputs
from parity import check_layer

pytestmark = pytest.mark.gpu


def _cases(n, seed):
    rng = np.random.default_rng(seed)
    out = []
    for i in range(n):
        align = int(rng.choice([1, 4, 8, 8, 16]))
        in_f = int(rng.integers(1, 260)) * align
        out_f = int(rng.integers(1, 200)) * int(rng.choice([1, 4, 8, 8]))
        k = int(rng.integers(1, min(in_f, 96) + 1))
        n_abl = int(rng.integers(0, max(1, out_f // 3)))
        B = int(rng.choice([1, 2, 3, 7, 8, 9, 16, 23, 24, 25, 40, 63, 64, 95, 96, 127, 128, 129, 200, 300, 513]))
        dtype = str(rng.choice(["f32", "bf16"]))
        act = str(rng.choice(["none", "gelu"]))
        out.append((in_f, out_f, k, n_abl, B, dtype, act, 1000 + i))
    return out


@pytest.mark.parametrize("in_f,out_f,k,n_abl,B,dtype,act,seed", _cases(60, 20230502))
def test_random_shape(in_f, out_f, k, n_abl, B, dtype, act, seed):
    L = inputs.make_layer(in_f, out_f, k, n_ablated=n_abl, seed=seed)
    x = inputs.make_x(B, in_f, seed=seed + 1)
    check_layer(L, x, dtype, act, variants=("auto",))


def _large_cases(n, seed):
    rng = np.random.default_rng(seed)
    out = []
    for i in range(n):
        in_f = int(rng.integers(128, 513)) * 8
        out_f = int(rng.integers(8, 513)) * 8
        k = int(rng.integers(1, 401))
        n_abl = int(rng.integers(0, out_f // 4))
        B = int(rng.choice([1, 5, 8, 12, 16, 24, 31, 64, 100, 128, 256, 300, 700]))
        dtype = str(rng.choice(["f32", "bf16"]))
        act = str(rng.choice(["none", "gelu"]))
        out.append((in_f, out_f, k, n_abl, B, dtype, act, 2000 + i))
    return out


@pytest.mark.parametrize("in_f,out_f,k,n_abl,B,dtype,act,seed", _large_cases(24, 4096))
def test_random_large_shape(in_f, out_f, k, n_abl, B, dtype, act, seed):
    """Long rows and wide layers: the launch shapes with the most threads, shared memory and cluster splits."""
    L = inputs.make_layer(in_f, out_f, k, n_ablated=n_abl, seed=seed)
    x = inputs.make_x(B, in_f, seed=seed + 1)
    check_layer(L, x, dtype, act, variants=("auto",))
