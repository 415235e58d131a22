"""Parity of the fused chain kernel under every launch shape it can be forced into, of the cluster-split weight
gradients where some blocks of a cluster get no share of the reduction, and of layers launched back to back
whose inputs are the previous launch's outputs (the kernels start early under programmatic dependent launch and
must still wait for their producers)."""
import numpy as np
import pytest
import torch

from oracle import lrd_oracle as o
from paper_2309_03824_b200 import binding as b
from paper_2309_03824_b200 import workloads as wl

from helpers import check_linear, dev, host, rel_err, workspace

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True)
def _restore_tuning():
    yield
    b.lrd_chain_tuning(0, 0, 0)
    b.lrd_chain_pair_tuning(0, 0, 0, 0)
    b.lrd_gemm_tuning(0)
    b.lrd_set_path(b.LRD_PATH_AUTO)


@pytest.mark.parametrize("tune", [(1, 0, 0), (2, 0, 0), (4, 0, 0), (0, 1, 0), (0, 2, 0), (0, 3, 0), (0, 0, 64), (0, 0, 128), (0, 0, 192),
                                  (0, 0, 256), (2, 2, 128), (4, 1, 64)])
@pytest.mark.parametrize("shape", [(400, 776, 520, 192), (300, 200, 1000, 128)])
def test_chain_kernel_launch_shape_overrides(tune, shape):
    M, K, N, r = shape
    b.lrd_chain_tuning(*tune)
    case = wl.random_factor_case(M, K, N, r, "bf16", 900 + M + tune[0] + tune[1] + tune[2])
    n0 = b.lrd_launch_count()
    check_linear(case, b.LRD_FREEZE_NONE, path=b.LRD_PATH_FUSED)
    assert b.lrd_launch_count() - n0 == 4          # fused forward, fused dZ -> dX, dU (+ db), dV: the override stayed feasible


@pytest.mark.parametrize("shape", [(400, 776, 520, 192), (640, 768, 768, 96), (300, 776, 1000, 384)])
def test_chain_kernel_clusters_of_three(shape):
    M, K, N, r = shape
    b.lrd_chain_tuning(3, 0, 0)
    b.lrd_chain_pair_tuning(1, 0, 0, 0)
    try:
        n0 = b.lrd_launch_count()
        check_linear(wl.random_factor_case(M, K, N, r, "bf16", 930 + M), b.LRD_FREEZE_NONE, path=b.LRD_PATH_FUSED)
        assert b.lrd_launch_count() - n0 == 4
    finally:
        b.lrd_chain_pair_tuning(0, 0, 0, 0)


@pytest.mark.parametrize("mode", [(2, 1, 0, 0), (2, 2, 0, 0), (2, 3, 0, 0), (2, 4, 0, 0), (2, 0, 1, 0), (2, 0, 2, 0), (2, 2, 1, 128), (2, 1, 3, 64),
                                  (2, 0, 0, 192)])
@pytest.mark.parametrize("shape", [(400, 776, 520, 192), (300, 520, 1000, 384), (1100, 3072, 136, 128)])
def test_chain_on_pairs_of_sms_launch_shape_overrides(mode, shape):
    """The chain on pairs of SMs under forced pairs per cluster, k-blocks per stage and chunk widths (a shape an override
    makes infeasible runs the unfused products instead: parity must hold either way)."""
    M, K, N, r = shape
    b.lrd_chain_pair_tuning(*mode)
    try:
        for freeze in (b.LRD_FREEZE_NONE, b.LRD_FREEZE_U):
            check_linear(wl.random_factor_case(M, K, N, r, "bf16", 940 + M + mode[1]), freeze)
    finally:
        b.lrd_chain_pair_tuning(0, 0, 0, 0)


def test_chain_tuning_rejects_values_outside_the_lists():
    for bad in ((5, 0, 0), (-1, 0, 0), (0, 5, 0), (0, -1, 0), (0, 0, 100), (0, 0, 512)):
        with pytest.raises(b.LrdError):
            b.lrd_chain_tuning(*bad)
    b.lrd_chain_tuning(0, 0, 0)


@pytest.mark.parametrize("shape", [(576, 136, 200, 64), (520, 264, 328, 192), (1100, 136, 200, 128), (130, 64, 64, 64)])
def test_weight_gradients_when_the_reduction_does_not_fill_the_cluster(shape):
    # M = 576, 520, 1100 tokens = 9, 9, 18 k-blocks of 64: split over a cluster of 8 (or 4) some blocks get none
    # and contribute zeros; M = 130 is three k-blocks for clusters that want more.
    M, K, N, r = shape
    for freeze in (b.LRD_FREEZE_NONE, b.LRD_FREEZE_U, b.LRD_FREEZE_V):
        check_linear(wl.random_factor_case(M, K, N, r, "bf16", 950 + M), freeze)


def test_dependent_launches_back_to_back():
    """Two layers, the second fed by the first, forward then backward through both, enqueued without any host
    synchronisation and repeated: every kernel reads what the previous kernel in the stream wrote."""
    M, K, H, N, r1, r2 = 640, 256, 384, 264, 64, 128
    c1 = wl.random_factor_case(M, K, H, r1, "bf16", 981)
    c2 = wl.random_factor_case(M, H, N, r2, "bf16", 982)
    bf = torch.bfloat16
    X, V1, U1, b1 = (dev(c1[k], "bf16") for k in ("X", "V", "U", "b"))
    V2, U2, b2, dY = (dev(c2[k], "bf16") for k in ("V", "U", "b", "dY"))
    d1, d2 = b.linear_desc(M, K, H, r1, b.LRD_BF16), b.linear_desc(M, H, N, r2, b.LRD_BF16)
    ws1 = workspace(max(b.lrd_linear_workspace_bytes(d1, 0, 0), b.lrd_linear_workspace_bytes(d1, 0, 1)))
    ws2 = workspace(max(b.lrd_linear_workspace_bytes(d2, 0, 0), b.lrd_linear_workspace_bytes(d2, 0, 1)))
    Y1, Z1 = torch.empty(M, H, dtype=bf, device="cuda"), torch.empty(M, r1, dtype=bf, device="cuda")
    Y2, Z2 = torch.empty(M, N, dtype=bf, device="cuda"), torch.empty(M, r2, dtype=bf, device="cuda")
    dY1, dX = torch.empty(M, H, dtype=bf, device="cuda"), torch.empty(M, K, dtype=bf, device="cuda")
    g = {n: torch.empty(s, dtype=bf, device="cuda") for n, s in (("dU1", (H, r1)), ("dV1", (K, r1)), ("db1", (H,)), ("dU2", (N, r2)),
                                                                 ("dV2", (H, r2)), ("db2", (N,)))}
    first = None
    for it in range(6):
        for t in (Y1, Z1, Y2, Z2, dY1, dX, *g.values()):
            t.fill_(float("nan"))
        b.lrd_linear_fwd(d1, X, V1, U1, b1, Y1, Z1, b.LRD_FREEZE_NONE, ws1)
        b.lrd_linear_fwd(d2, Y1, V2, U2, b2, Y2, Z2, b.LRD_FREEZE_NONE, ws2)
        b.lrd_linear_bwd(d2, dY, Y1, V2, U2, Z2, dY1, g["dU2"], g["dV2"], g["db2"], b.LRD_FREEZE_NONE, ws2)
        b.lrd_linear_bwd(d1, dY1, X, V1, U1, Z1, dX, g["dU1"], g["dV1"], g["db1"], b.LRD_FREEZE_NONE, ws1)
        torch.cuda.synchronize()
        now = {n: t.clone() for n, t in (("Y2", Y2), ("dX", dX), *g.items())}
        if first is None:
            first = now
        else:
            for n in now:
                assert torch.equal(now[n], first[n]), n          # same inputs, same order of additions: same bits
    assert b.lrd_check_device_status() == b.LRD_OK
    # the oracle on the same chain; Y1 and dY1 cross the layer boundary rounded to bf16, as on the device
    _, Y1r = o.linear_fwd(c1["X"], c1["V"], c1["U"], c1["b"])
    Y1b = host(Y1)
    assert rel_err(Y1, Y1r) <= 2e-2
    Z2r, Y2r = o.linear_fwd(Y1b, c2["V"], c2["U"], c2["b"])
    r2g = o.linear_bwd(c2["dY"], Y1b, c2["V"], c2["U"], Z2r, o.FREEZE_NONE)
    Z1r, _ = o.linear_fwd(c1["X"], c1["V"], c1["U"], c1["b"])
    r1g = o.linear_bwd(host(dY1), c1["X"], c1["V"], c1["U"], Z1r, o.FREEZE_NONE)
    errs = {"Y2": rel_err(Y2, Y2r), "dY1": rel_err(dY1, r2g["dX"]), "dU2": rel_err(g["dU2"], r2g["dU"]), "dV2": rel_err(g["dV2"], r2g["dV"]),
            "db2": rel_err(g["db2"], r2g["db"]), "dX": rel_err(dX, r1g["dX"]), "dU1": rel_err(g["dU1"], r1g["dU"]),
            "dV1": rel_err(g["dV1"], r1g["dV"]), "db1": rel_err(g["db1"], r1g["db"])}
    assert all(v <= 2e-2 for v in errs.values()), errs


def _dense_run(M, K, N, seed):
    bf = torch.bfloat16
    X = wl.round_to(wl.normal(seed, (M, K)), "bf16")
    W = wl.round_to(wl.normal(seed + 1, (N, K), 0.02), "bf16")
    bias = wl.round_to(wl.normal(seed + 2, (N,), 0.1), "bf16")
    dY = wl.round_to(wl.normal(seed + 3, (M, N)), "bf16")
    desc = b.linear_desc(M, K, N, 0, b.LRD_BF16)
    ws = workspace(b.lrd_dense_workspace_bytes(desc, 1))
    Y = torch.full((M, N), float("nan"), dtype=bf, device="cuda")
    dX = torch.full((M, K), float("nan"), dtype=bf, device="cuda")
    dW, db = torch.empty(N, K, dtype=bf, device="cuda"), torch.empty(N, dtype=bf, device="cuda")
    b.lrd_dense_fwd(desc, dev(X, "bf16"), dev(W, "bf16"), dev(bias, "bf16"), Y, ws)
    b.lrd_dense_bwd(desc, dev(dY, "bf16"), dev(X, "bf16"), dev(W, "bf16"), dX, dW, db, ws)
    torch.cuda.synchronize()
    assert b.lrd_check_device_status() == b.LRD_OK
    return (X, W, bias, dY), (Y, dX)


# 129 rows: the odd block of the only pair holds one row; 300 / 1300: an odd number of 128-row tiles, so the last
# pair's odd block hangs over the edge entirely; 2304 x 2100: several tiles per pair, both accumulator buffers reused
@pytest.mark.parametrize("shape", [(129, 64, 72), (300, 200, 136), (1300, 328, 520), (2304, 264, 2100), (512, 1096, 256)])
def test_products_on_pairs_of_sms_match_the_oracle_and_single_blocks(shape):
    M, K, N = shape
    b.lrd_gemm_tuning(1)
    _, (Y1, dX1) = _dense_run(M, K, N, 700 + M)
    b.lrd_gemm_tuning(2)
    (X, W, bias, dY), (Y2, dX2) = _dense_run(M, K, N, 700 + M)
    assert rel_err(Y2, o.dense_fwd(X, W, bias)) <= 2e-2
    assert rel_err(dX2, o.dense_bwd(dY, X, W)["dX"]) <= 2e-2
    # same products summed in the same order, whichever SM holds which rows
    assert torch.equal(Y1, Y2) and torch.equal(dX1, dX2)


@pytest.mark.parametrize("cg", [1, 2])
@pytest.mark.parametrize("shape", [(700, 520, 776, 512), (1500, 264, 200, 72)])
def test_unfused_layer_with_products_on_single_blocks_and_on_pairs(cg, shape):
    M, K, N, r = shape
    b.lrd_gemm_tuning(cg)
    for freeze in (b.LRD_FREEZE_NONE, b.LRD_FREEZE_U):
        check_linear(wl.random_factor_case(M, K, N, r, "bf16", 760 + M + cg), freeze, path=b.LRD_PATH_UNFUSED)


def test_gemm_tuning_rejects_values_outside_the_list():
    for bad in (-1, 3, 4):
        with pytest.raises(b.LrdError):
            b.lrd_gemm_tuning(bad)
    b.lrd_gemm_tuning(0)
