"""Seeded random layer shapes (ragged token counts, feature counts that are odd multiples of 8, ranks from 16 up to
min(K, N)) through every path the library may take for them, against the oracle.  The draws are fixed by the seed, so
a failure names a shape that can be re-run on its own."""
import numpy as np
import pytest

from paper_2309_03824_b200 import binding as b
from paper_2309_03824_b200 import workloads as wl

from helpers import check_linear

pytestmark = pytest.mark.gpu


def _shapes(n, seed):
    rng = np.random.Generator(np.random.PCG64(seed))
    out = []
    for _ in range(n):
        M = int(rng.integers(1, 1400))
        K = 8 * int(rng.integers(2, 140))
        N = 8 * int(rng.integers(2, 140))
        r = min(16 * int(rng.integers(1, 33)), min(K, N) // 8 * 8)
        out.append((M, K, N, r))
    return out


SHAPES = _shapes(24, 20240)


@pytest.mark.parametrize("shape", SHAPES, ids=["x".join(map(str, s)) for s in SHAPES])
def test_random_shape_every_mask_automatic_path(shape):
    M, K, N, r = shape
    for freeze in (b.LRD_FREEZE_NONE, b.LRD_FREEZE_U, b.LRD_FREEZE_V):
        check_linear(wl.random_factor_case(M, K, N, r, "bf16", 7000 + M + K), freeze)


@pytest.mark.parametrize("shape", SHAPES[:10], ids=["x".join(map(str, s)) for s in SHAPES[:10]])
@pytest.mark.parametrize("path", [b.LRD_PATH_FUSED, b.LRD_PATH_UNFUSED])
def test_random_shape_forced_paths(shape, path):
    M, K, N, r = shape
    check_linear(wl.random_factor_case(M, K, N, r, "bf16", 7100 + M + N), b.LRD_FREEZE_NONE, path=path)
