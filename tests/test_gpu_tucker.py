"""GPU parity of the Tucker-2 decomposed convolution against the CPU oracle, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import lrd_oracle as o
from paper_2309_03824_b200 import binding as b
from paper_2309_03824_b200 import decompose
from paper_2309_03824_b200 import workloads as wl

from helpers import DT, TOL, dev, host, rel_err, workspace

pytestmark = pytest.mark.gpu
MASKS = [b.LRD_TK_FREEZE_NONE, b.LRD_TK_FREEZE_FACTORS, b.LRD_TK_FREEZE_CORE]


def run_tucker(case, freeze, path=b.LRD_PATH_AUTO, want_dx=True):
    dt = case["dtype"]
    code, tdt = DT[dt]
    B, H, W, C, S, r1, r2 = (case[k] for k in ("B", "H", "W", "C", "S", "r1", "r2"))
    k, stride = case.get("k", 3), case.get("stride", 1)
    Ho, Wo = (H - 1) // stride + 1, (W - 1) // stride + 1
    desc = b.tucker2_desc(B, H, W, C, S, r1, r2, code, k=k, stride=stride, pad=(k - 1) // 2)
    X, A, G, Bm, bias, dY = (dev(case[k], dt) for k in ("X", "A", "G", "Bm", "b", "dY"))
    ws = workspace(max(b.lrd_tucker2_workspace_bytes(desc, freeze, 0), b.lrd_tucker2_workspace_bytes(desc, freeze, 1)))
    b.lrd_set_path(path)
    try:
        Y = torch.empty(B, Ho, Wo, S, dtype=tdt, device="cuda")
        Z1 = None if freeze == b.LRD_TK_FREEZE_CORE else torch.empty(B, H, W, r1, dtype=tdt, device="cuda")
        Z2 = None if freeze == b.LRD_TK_FREEZE_FACTORS else torch.empty(B, Ho, Wo, r2, dtype=tdt, device="cuda")
        b.lrd_tucker2_fwd(desc, X, A, G, Bm, bias, Y, Z1, Z2, freeze, ws)
        nan = float("nan")
        dX = torch.full((B, H, W, C), nan, dtype=tdt, device="cuda") if want_dx else None
        dA = torch.full((C, r1), nan, dtype=tdt, device="cuda")
        dG = torch.full((r2, k, k, r1), nan, dtype=tdt, device="cuda")
        dB = torch.full((S, r2), nan, dtype=tdt, device="cuda")
        db = torch.full((S,), nan, dtype=tdt, device="cuda")
        b.lrd_tucker2_bwd(desc, dY, None if freeze == b.LRD_TK_FREEZE_FACTORS else X, A, G, Bm, Z1, Z2, dX, dA, dG, dB, db,
                          freeze, ws)
        torch.cuda.synchronize()
        assert b.lrd_check_device_status() == b.LRD_OK
    finally:
        b.lrd_set_path(b.LRD_PATH_AUTO)
    return {"Y": Y, "Z1": Z1, "Z2": Z2, "dX": dX, "dA": dA, "dG": dG, "dB": dB, "db": db}


def check_tucker(case, freeze, path=b.LRD_PATH_AUTO, tol=None):
    got = run_tucker(case, freeze, path)
    stride = case.get("stride", 1)
    Z1, Z2, Y = o.tucker2_fwd(case["X"], case["A"], case["G"], case["Bm"], case["b"], stride)
    ref = o.tucker2_bwd(case["dY"], case["X"], case["A"], case["G"], case["Bm"], Z1, Z2, freeze, stride)
    ref.update({"Y": Y, "Z1": Z1, "Z2": Z2})
    tol = TOL[case["dtype"]] if tol is None else tol
    errs = {k: rel_err(v, ref[k]) for k, v in got.items() if v is not None}
    if freeze == b.LRD_TK_FREEZE_FACTORS:
        assert not host(got["dA"]).any() and not host(got["dB"]).any() and not host(got["db"]).any()
    if freeze == b.LRD_TK_FREEZE_CORE:
        assert not host(got["dG"]).any()
    bad = {k: v for k, v in errs.items() if not v <= tol}
    assert not bad, (bad, errs)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("geom", [(2, 5, 7, 12, 10, 5, 6), (1, 1, 1, 4, 4, 2, 3), (3, 14, 14, 40, 48, 24, 16)])
@pytest.mark.parametrize("freeze", MASKS)
def test_general_path_small_geometries(dtype, geom, freeze):
    B, H, W, C, S, r1, r2 = geom
    check_tucker(wl.random_tucker_case(B, H, W, C, S, r1, r2, 3, dtype, 400 + H), freeze, path=b.LRD_PATH_GENERAL)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("geom", [(2, 8, 8, 16, 24, 8, 16, 3, 2), (2, 7, 9, 12, 10, 5, 6, 3, 2), (1, 1, 1, 4, 4, 2, 3, 3, 2), (2, 6, 5, 16, 16, 8, 8, 5, 1),
                                  (2, 9, 7, 12, 20, 6, 7, 5, 2), (2, 5, 6, 24, 16, 8, 16, 1, 1), (3, 7, 7, 16, 24, 16, 8, 1, 2),
                                  (1, 8, 9, 8, 8, 4, 4, 7, 1), (4, 14, 14, 64, 128, 32, 40, 3, 2)])
@pytest.mark.parametrize("freeze", MASKS)
def test_strided_and_wider_cores(dtype, geom, freeze):
    """k x k cores with k = 1, 3, 5, 7 and stride 1 or 2 (the downsampling blocks of a residual network carry their
    stride on the 3 x 3 convolution): the 1 x 1 products run wherever their shapes allow, the core on the general
    kernels; Z2, Y and dY live on the strided output grid."""
    B, H, W, C, S, r1, r2, k, stride = geom
    check_tucker(wl.random_tucker_case(B, H, W, C, S, r1, r2, k, dtype, 470 + H + k + stride, stride=stride), freeze)


def test_geometries_outside_the_supported_set_are_refused():
    t = torch.zeros(1 << 12, dtype=torch.float32, device="cuda")
    ws = workspace(1 << 16)
    for k, stride, pad, want in ((4, 1, 1, b.LRD_ERR_UNSUPPORTED), (9, 1, 4, b.LRD_ERR_UNSUPPORTED), (3, 3, 1, b.LRD_ERR_UNSUPPORTED),
                                 (3, 1, 0, b.LRD_ERR_UNSUPPORTED), (5, 1, 1, b.LRD_ERR_UNSUPPORTED), (0, 1, 0, b.LRD_ERR_INVALID_ARG),
                                 (3, 0, 1, b.LRD_ERR_INVALID_ARG)):
        d = b.tucker2_desc(1, 4, 4, 4, 4, 2, 2, b.LRD_F32, k=k, stride=stride, pad=pad)
        assert b.lrd_tucker2_fwd(d, t, t, t, t, None, t, t, t, 0, ws, check=False) == want, (k, stride, pad)
        assert b.lrd_tucker2_workspace_bytes(d, 0, 0) == 0


@pytest.mark.parametrize("geom", [(4, 14, 14, 64, 72, 32, 40), (2, 9, 11, 128, 136, 96, 104), (5, 14, 14, 256, 256, 96, 96),
                                  (3, 10, 12, 72, 200, 48, 64), (2, 7, 9, 40, 24, 16, 16), (1, 14, 14, 256, 248, 128, 112),
                                  (2, 9, 11, 256, 256, 144, 160), (1, 14, 14, 256, 256, 256, 256), (2, 6, 50, 64, 64, 32, 48)])
@pytest.mark.parametrize("freeze", MASKS)
def test_tensor_core_path(geom, freeze):
    B, H, W, C, S, r1, r2 = geom
    check_tucker(wl.random_tucker_case(B, H, W, C, S, r1, r2, 3, "bf16", 500 + C), freeze)


@pytest.mark.parametrize("geom", [(2, 14, 14, 256, 256, 96, 96), (2, 20, 14, 64, 64, 32, 32), (1, 5, 40, 16, 16, 16, 16), (1, 33, 3, 24, 40, 16, 16),
                                  (3, 9, 11, 72, 200, 48, 64), (2, 4, 1, 16, 16, 16, 16), (2, 13, 30, 136, 256, 128, 128),
                                  (1, 16, 16, 264, 88, 112, 80)])
@pytest.mark.parametrize("freeze", MASKS)
def test_whole_pass_in_one_launch(geom, freeze):
    """Shapes the one-launch data passes take (ranks multiples of 16 up to 128, at most 256 output channels): tiles
    of 7, 9, 1, 25 ... image rows with a ragged last tile, images 1 to 40 pixels wide, input channels off a multiple
    of 64; the forward is then ONE launch, and the separate launches (forced through the unfused path) agree with
    the oracle on the same inputs."""
    B, H, W, C, S, r1, r2 = geom
    case = wl.random_tucker_case(B, H, W, C, S, r1, r2, 3, "bf16", 600 + H + W)
    desc = b.tucker2_desc(B, H, W, C, S, r1, r2, b.LRD_BF16)
    X, A, G, Bm, bias = (dev(case[k], "bf16") for k in ("X", "A", "G", "Bm", "b"))
    ws = workspace(b.lrd_tucker2_workspace_bytes(desc, b.LRD_TK_FREEZE_FACTORS, 0))
    Y = torch.empty(B, H, W, S, dtype=torch.bfloat16, device="cuda")
    Z1 = torch.empty(B, H, W, r1, dtype=torch.bfloat16, device="cuda")
    n0 = b.lrd_launch_count()
    b.lrd_tucker2_fwd(desc, X, A, G, Bm, bias, Y, Z1, None, b.LRD_TK_FREEZE_FACTORS, ws)
    assert b.lrd_launch_count() - n0 == 1
    check_tucker(case, freeze)
    check_tucker(case, freeze, path=b.LRD_PATH_UNFUSED)


@pytest.mark.parametrize("geom", [(2, 7, 7, 512, 512, 136, 136), (2, 7, 7, 512, 512, 256, 256), (1, 7, 7, 512, 512, 304, 248),
                                  (3, 7, 7, 512, 512, 312, 312)])
@pytest.mark.parametrize("freeze", MASKS)
def test_tensor_core_path_ranks_above_128(geom, freeze):
    """The [512, 512, 3, 3] layer on 7 x 7 images at ranks between Eq. 6's and Eq. 5's: several 128-column output
    tiles of the core and three to five 64-channel blocks per filter tap."""
    B, H, W, C, S, r1, r2 = geom
    check_tucker(wl.random_tucker_case(B, H, W, C, S, r1, r2, 3, "bf16", 700 + r1), freeze)


@pytest.mark.parametrize("geom", [(2, 7, 7, 512, 512, 309, 309), (3, 14, 14, 64, 72, 33, 41), (2, 9, 11, 128, 136, 100, 96)])
@pytest.mark.parametrize("freeze", MASKS)
def test_ranks_off_a_multiple_of_8_run_on_the_tensor_cores(geom, freeze):
    """Packed factors with odd ranks (Eq. 5's own 309 among them): repacked into the workspace with padded ranks."""
    B, H, W, C, S, r1, r2 = geom
    check_tucker(wl.random_tucker_case(B, H, W, C, S, r1, r2, 3, "bf16", 750 + r1), freeze)


@pytest.mark.parametrize("geom", [(4, 14, 14, 64, 72, 32, 40), (2, 5, 7, 12, 10, 5, 6)])
@pytest.mark.parametrize("freeze", MASKS)
def test_backward_launches_side_by_side_or_in_a_row_give_the_same_bits(geom, freeze):
    """The weight-gradient launches run beside the data path by default; in a row they must give the same results,
    and a backward repeated back to back (each call joins its side streams before it returns) must not change them."""
    B, H, W, C, S, r1, r2 = geom
    case = wl.random_tucker_case(B, H, W, C, S, r1, r2, 3, "bf16", 600 + C)
    try:
        b.lrd_tucker2_overlap(False)
        row = run_tucker(case, freeze)
    finally:
        b.lrd_tucker2_overlap(True)
    check_tucker(case, freeze)
    for _ in range(3):
        side = run_tucker(case, freeze)
        for k, v in side.items():
            if v is not None:
                assert torch.equal(v, row[k]), k


@pytest.mark.parametrize("freeze", [b.LRD_TK_FREEZE_CORE, b.LRD_TK_FREEZE_FACTORS])
def test_c3_resnet_stage3_shape_full_size(freeze):
    c = wl.C3_TUCKER
    case = wl.tucker_case(c["B"], c["H"], c["W"], c["C"], c["S"], c["r1"], c["r2"], c["k"], "bf16", 3000,
                          decompose.tucker2_factors)
    check_tucker(case, freeze)


@pytest.mark.parametrize("dtype,geom", [("bf16", (2, 7, 7, 64, 72)), ("bf16", (3, 14, 14, 256, 256)), ("bf16", (1, 7, 7, 512, 512)),
                                        ("f32", (2, 5, 7, 12, 10))])
def test_undecomposed_3x3_convolution(dtype, geom):
    """The comparison layer (the convolution a Tucker-2 layer replaces): forward, input gradient and filter gradient
    against the oracle's direct convolution."""
    B, H, W, C, S = geom
    code, tdt = DT[dtype]
    X = wl.round_to(wl.normal(801, (B, H, W, C)), dtype)
    Wk = wl.round_to(wl.normal(802, (S, 3, 3, C), (9 * C) ** -0.5), dtype)
    dY = wl.round_to(wl.normal(803, (B, H, W, S)), dtype)
    Xd, Wd, dYd = dev(X, dtype), dev(Wk, dtype), dev(dY, dtype)
    Y = torch.full((B, H, W, S), float("nan"), dtype=tdt, device="cuda")
    dX = torch.full((B, H, W, C), float("nan"), dtype=tdt, device="cuda")
    dW = torch.full((S, 3, 3, C), float("nan"), dtype=tdt, device="cuda")
    ws = workspace(b.lrd_conv3x3_workspace_bytes(B, H, W, C, S, code))
    b.lrd_conv3x3_fwd(B, H, W, C, S, code, Xd, Wd, Y)
    b.lrd_conv3x3_bwd(B, H, W, C, S, code, dYd, Xd, Wd, dX, dW, ws)
    torch.cuda.synchronize()
    assert b.lrd_check_device_status() == b.LRD_OK
    assert rel_err(Y, o.conv2d_nhwc_fwd(X, Wk, 1)) <= TOL[dtype]
    assert rel_err(dX, o.conv2d_nhwc_bwd_data(dY, Wk, 1, (H, W))) <= TOL[dtype]
    assert rel_err(dW, o.conv2d_nhwc_bwd_filter(dY, X, 3, 1)) <= TOL[dtype]


def test_argument_checks():
    code, tdt = DT["bf16"]
    d = b.tucker2_desc(1, 4, 4, 8, 8, 4, 4, code)
    t = torch.zeros(4096, dtype=tdt, device="cuda")
    ws = workspace(b.lrd_tucker2_workspace_bytes(d, 0, 1))
    # Z1_save is refused when the core is frozen and required otherwise
    assert b.lrd_tucker2_fwd(d, t, t, t, t, None, t, t, t, b.LRD_TK_FREEZE_CORE, ws, check=False) == b.LRD_ERR_INVALID_ARG
    assert b.lrd_tucker2_fwd(d, t, t, t, t, None, t, None, t, b.LRD_TK_FREEZE_NONE, ws, check=False) == b.LRD_ERR_INVALID_ARG
    assert b.lrd_tucker2_fwd(d, t, t, t, t, None, t, t, t, b.LRD_TK_FREEZE_FACTORS, ws, check=False) == b.LRD_ERR_INVALID_ARG
    bad = b.tucker2_desc(1, 4, 4, 8, 8, 4, 4, code, k=4, pad=1)
    assert b.lrd_tucker2_fwd(bad, t, t, t, t, None, t, t, t, 0, ws, check=False) == b.LRD_ERR_UNSUPPORTED
    bad = b.tucker2_desc(1, 4, 4, 8, 8, 9, 4, code)
    assert b.lrd_tucker2_fwd(bad, t, t, t, t, None, t, t, t, 0, ws, check=False) == b.LRD_ERR_BAD_RANK
