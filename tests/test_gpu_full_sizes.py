"""Parity at the full sizes of the rank-sweep (M = 8192, 4096 x 4096) and GPT-2-medium-shaped
(M = 8192, hidden 1024, FFN 4096) workloads.  The oracle evaluates sampled rows of Y and dX one by one
(each output row is an independent product) and the whole of dU, dV and db."""
import numpy as np
import pytest
import torch

from oracle import lrd_oracle as o
from paper_2309_03824_b200 import binding as b
from paper_2309_03824_b200 import workloads as wl

from helpers import host, run_linear

pytestmark = pytest.mark.gpu


def check_sampled(case, freeze, tol=2e-2, n_rows=192):
    got = run_linear(case, freeze)
    X, V, U, bias, dY = (case[k].astype(np.float64) for k in ("X", "V", "U", "b", "dY"))
    rows = wl.sample_rows(case["M"] + case["r"], case["M"], n_rows)
    Zs, Ys = o.linear_fwd(X[rows], V, U, bias)
    errs = {"Y": np.abs(host(got["Y"])[rows] - Ys).max() / np.abs(Ys).max()}
    dXs = o.linear_bwd(dY[rows], X[rows], V, U, Zs, o.FREEZE_NONE)["dX"]
    errs["dX"] = np.abs(host(got["dX"])[rows] - dXs).max() / np.abs(dXs).max()
    if freeze != b.LRD_FREEZE_U:
        Z = X @ V
        errs["Z"] = np.abs(host(got["Z"])[rows] - Z[rows]).max() / np.abs(Z[rows]).max()
        dU = dY.T @ Z
        errs["dU"] = np.abs(host(got["dU"]) - dU).max() / np.abs(dU).max()
        db = dY.sum(axis=0)
        errs["db"] = np.abs(host(got["db"]) - db).max() / np.abs(db).max()
    else:
        assert not host(got["dU"]).any() and not host(got["db"]).any()
    if freeze != b.LRD_FREEZE_V:
        dV = X.T @ (dY @ U)
        errs["dV"] = np.abs(host(got["dV"]) - dV).max() / np.abs(dV).max()
    else:
        assert not host(got["dV"]).any()
    bad = {k: v for k, v in errs.items() if not v <= tol}
    assert not bad, (bad, errs)


@pytest.mark.parametrize("r,freeze", [(100, b.LRD_FREEZE_V), (104, b.LRD_FREEZE_NONE), (128, b.LRD_FREEZE_NONE),
                                      (256, b.LRD_FREEZE_V), (512, b.LRD_FREEZE_NONE), (1024, b.LRD_FREEZE_V)])
def test_rank_sweep_layer_full_size(r, freeze):
    c = wl.C2_SWEEP
    check_sampled(wl.random_factor_case(c["M"], c["K"], c["N"], r, "bf16", 2000 + r), freeze)


@pytest.mark.parametrize("r", [100, 250, 500, 750, 1000, 504, 752])
@pytest.mark.parametrize("freeze", [b.LRD_FREEZE_NONE, b.LRD_FREEZE_V])
def test_rank_sweep_packed_and_rounded_to_8_full_size(r, freeze):
    """The sweep's unquantized ranks stored packed (leading dimension = r: rows of V, U, Z, dU, dV start at
    addresses that are not multiples of 16 bytes) and the ranks rounded up to a multiple of 8 that are not
    multiples of 16, under both masks the workload names."""
    c = wl.C2_SWEEP
    check_sampled(wl.random_factor_case(c["M"], c["K"], c["N"], r, "bf16", 2100 + r), freeze)


@pytest.mark.parametrize("layer", wl.C4_GPT_LAYERS[3:], ids=[l[0] for l in wl.C4_GPT_LAYERS[3:]])
@pytest.mark.parametrize("freeze", [b.LRD_FREEZE_U, b.LRD_FREEZE_V])
def test_gpt2_medium_shaped_layers_full_size(layer, freeze):
    name, K, N, r = layer
    check_sampled(wl.random_factor_case(wl.C4_M, K, N, r, "bf16", 4000 + K + r), freeze)


@pytest.mark.parametrize("r", [64, 72])
def test_quarter_of_a_million_tokens(r):
    """2049 row tiles with a ragged last one, weight gradients summed over 262 221 tokens (4098 k-blocks of 64):
    r = 64 takes the fused chain, r = 72 (not a multiple of 16) the separate products on pairs of SMs."""
    check_sampled(wl.random_factor_case(262221, 136, 264, r, "bf16", 5000 + r), b.LRD_FREEZE_NONE)
