"""GPU parity of the decomposed linear layer against the CPU oracle, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import lrd_oracle as o
from paper_2309_03824_b200 import binding as b
from paper_2309_03824_b200 import workloads as wl

from helpers import DT, TOL, check_linear, dev, host, oracle_linear, rel_err, run_linear, workspace

pytestmark = pytest.mark.gpu
MASKS = [b.LRD_FREEZE_NONE, b.LRD_FREEZE_U, b.LRD_FREEZE_V]


@pytest.fixture(scope="module")
def c0_case():
    c = wl.C0_LINEAR
    return wl.linear_case(c["M"], c["K"], c["N"], c["r"], "f32", 0, c["w_std"], o.factorize, w_seed=0)


@pytest.mark.parametrize("freeze", MASKS)
def test_c0_fp32_single_layer(c0_case, freeze):
    check_linear(c0_case, freeze)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("shape", [(77, 50, 37, 5), (1, 3, 2, 1), (130, 65, 129, 33), (64, 64, 64, 64)])
@pytest.mark.parametrize("freeze", MASKS)
def test_general_path_odd_shapes(dtype, shape, freeze):
    M, K, N, r = shape
    check_linear(wl.random_factor_case(M, K, N, r, dtype, 100 + M), freeze, path=b.LRD_PATH_GENERAL)


@pytest.mark.parametrize("shape", [(300, 200, 136, 72), (128, 64, 64, 64), (513, 776, 264, 200), (1000, 328, 520, 8),
                                   (257, 1032, 72, 64)])
@pytest.mark.parametrize("freeze", MASKS)
def test_tensor_core_unfused_ragged_tiles(shape, freeze):
    M, K, N, r = shape
    check_linear(wl.random_factor_case(M, K, N, r, "bf16", 200 + M), freeze, path=b.LRD_PATH_UNFUSED)


@pytest.mark.parametrize("shape", [(300, 200, 136, 72), (128, 64, 64, 64), (513, 776, 264, 200), (640, 768, 768, 192),
                                   (256, 3072, 768, 384), (384, 768, 3072, 384), (200, 1024, 1024, 256),
                                   (5120, 256, 264, 128), (9728, 128, 136, 64), (256, 200, 136, 64), (256, 128, 128, 48),
                                   (130, 512, 520, 512), (257, 96, 1000, 32)])
@pytest.mark.parametrize("freeze", MASKS)
def test_tensor_core_fused_or_auto(shape, freeze):
    M, K, N, r = shape
    check_linear(wl.random_factor_case(M, K, N, r, "bf16", 300 + M), freeze, path=b.LRD_PATH_FUSED)


@pytest.mark.parametrize("shape", [(300, 200, 136, 5), (513, 776, 264, 33), (640, 768, 768, 100), (1100, 1032, 520, 250),
                                   (384, 768, 3072, 390)])
@pytest.mark.parametrize("freeze", MASKS)
def test_packed_ranks_off_a_multiple_of_8(shape, freeze):
    """Factors stored packed with a rank that is not a multiple of 8 (rows of V, U, Z, dU, dV start off 16-byte
    boundaries): the factors are repacked into the workspace and the layer still runs on the tensor-core kernels."""
    M, K, N, r = shape
    check_linear(wl.random_factor_case(M, K, N, r, "bf16", 350 + M), freeze)


def test_odd_factor_strides_leave_the_padding_alone():
    M, K, N, r = 260, 136, 200, 40
    ldv, ldu, ldz = 43, 45, 41
    case = wl.random_factor_case(M, K, N, r, "bf16", 360)
    code, tdt = DT["bf16"]
    desc = b.linear_desc(M, K, N, r, code, 0, ldv, ldu, 0, ldz)

    def padded(a, ld, fill=float("nan")):
        t = torch.full((a.shape[0], ld), fill, dtype=tdt, device="cuda")
        t[:, : a.shape[1]] = dev(a, "bf16")
        return t

    X, dY, bias = dev(case["X"], "bf16"), dev(case["dY"], "bf16"), dev(case["b"], "bf16")
    V, U = padded(case["V"], ldv), padded(case["U"], ldu)
    Y = torch.empty(M, N, dtype=tdt, device="cuda")
    Z = torch.full((M, ldz), 3.0, dtype=tdt, device="cuda")
    dX = torch.empty(M, K, dtype=tdt, device="cuda")
    dU = torch.full((N, ldu), 3.0, dtype=tdt, device="cuda")
    dV = torch.full((K, ldv), 3.0, dtype=tdt, device="cuda")
    db = torch.empty(N, dtype=tdt, device="cuda")
    ws = workspace(max(b.lrd_linear_workspace_bytes(desc, 0, 0), b.lrd_linear_workspace_bytes(desc, 0, 1)))
    b.lrd_linear_fwd(desc, X, V, U, bias, Y, Z, b.LRD_FREEZE_NONE, ws)
    b.lrd_linear_bwd(desc, dY, X, V, U, Z, dX, dU, dV, db, b.LRD_FREEZE_NONE, ws)
    torch.cuda.synchronize()
    assert b.lrd_check_device_status() == b.LRD_OK
    ref = oracle_linear(case, b.LRD_FREEZE_NONE)
    for got, name, w in ((Y, "Y", N), (Z, "Z", r), (dX, "dX", K), (dU, "dU", r), (dV, "dV", r), (db.reshape(1, -1), "db", N)):
        assert rel_err(got[:, :w], np.asarray(ref[name]).reshape(got.shape[0], -1)) <= TOL["bf16"], name
    for got, w in ((Z, r), (dU, r), (dV, r)):
        assert (got[:, w:] == 3.0).all()                      # columns past the rank are never written


@pytest.mark.parametrize("shape", [(520, 264, 328, 64), (640, 768, 768, 192), (300, 200, 136, 33), (384, 3072, 768, 384)])
@pytest.mark.parametrize("freeze", MASKS)
def test_backward_in_two_calls_on_two_streams(shape, freeze):
    """The data half on one stream, the weight-gradient half on another (ordered by an event, as a caller that runs the
    weight gradients beside the next layer's data call would): both halves take launch shapes that leave room for each
    other (the data pass on pairs of SMs, the weight gradients reduced in fewer, larger shares), so the results agree with
    lrd_linear_bwd to rounding, with the oracle within the bound, and with themselves bit for bit when repeated."""
    M, K, N, r = shape
    case = wl.random_factor_case(M, K, N, r, "bf16", 380 + M)
    one = run_linear(case, freeze)
    code, tdt = DT["bf16"]
    X, V, U, bias, dY = (dev(case[k], "bf16") for k in ("X", "V", "U", "b", "dY"))
    desc = b.linear_desc(M, K, N, r, code)
    ws = workspace(max(b.lrd_linear_workspace_bytes(desc, freeze, 0), b.lrd_linear_workspace_bytes(desc, freeze, 1)))
    Z = one["Z"]
    nan = float("nan")
    dX, dU, dV, db = (torch.full(sh, nan, dtype=tdt, device="cuda") for sh in ((M, K), (N, r), (K, r), (N,)))
    main, side = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    with torch.cuda.stream(main):
        b.lrd_linear_bwd_data(desc, dY, V, U, dX, freeze, ws)
        ev = torch.cuda.Event()
        ev.record(main)
    with torch.cuda.stream(side):
        side.wait_event(ev)
        b.lrd_linear_bwd_weights(desc, dY, None if freeze == b.LRD_FREEZE_V else X, Z, dU, dV, db, freeze, ws)
    torch.cuda.synchronize()
    assert b.lrd_check_device_status() == b.LRD_OK
    ref = oracle_linear(case, freeze)
    first = {}
    for name, got in (("dX", dX), ("dU", dU), ("dV", dV), ("db", db)):
        assert rel_err(got, ref[name]) <= TOL["bf16"], name
        assert rel_err(got, host(one[name])) <= 2.0 ** -7, name
        first[name] = got.clone()
    with torch.cuda.stream(main):
        b.lrd_linear_bwd_data(desc, dY, V, U, dX, freeze, ws)
    torch.cuda.synchronize()
    with torch.cuda.stream(side):
        b.lrd_linear_bwd_weights(desc, dY, None if freeze == b.LRD_FREEZE_V else X, Z, dU, dV, db, freeze, ws)
    torch.cuda.synchronize()
    for name, got in (("dX", dX), ("dU", dU), ("dV", dV), ("db", db)):
        assert torch.equal(got, first[name]), name


def test_a_bounded_wait_that_runs_out_is_reported_once():
    """The self-test block waits on a barrier nothing arrives at; its wait gives up at the limit every pipeline wait
    has, the status check reports LRD_ERR_TIMEOUT exactly once, and the library keeps working afterwards."""
    assert b.lrd_check_device_status() == b.LRD_OK
    b.lrd_selftest_wait_timeout()
    assert b.lrd_check_device_status() == b.LRD_ERR_TIMEOUT
    assert b.lrd_check_device_status() == b.LRD_OK
    check_linear(wl.random_factor_case(300, 200, 136, 64, "bf16", 370), b.LRD_FREEZE_NONE)


def test_debug_mode_reports_at_the_call():
    """LRD_DEBUG=1: an entry point waits for its own work, so a device wait that ran out before it is reported (and
    cleared) by the next compute call itself, and a clean call returns LRD_OK with its results complete."""
    import os
    import subprocess
    import sys
    code = """
import torch
from paper_2309_03824_b200 import binding as b, workloads as wl
from helpers import check_linear
check_linear(wl.random_factor_case(300, 200, 136, 64, "bf16", 371), b.LRD_FREEZE_NONE)
b.lrd_selftest_wait_timeout()
case = wl.random_factor_case(300, 200, 136, 64, "bf16", 372)
bf = torch.bfloat16
X, V, U, bias = (torch.from_numpy(case[k]).to("cuda", bf) for k in ("X", "V", "U", "b"))
desc = b.linear_desc(300, 200, 136, 64, b.LRD_BF16)
Y = torch.empty(300, 136, dtype=bf, device="cuda")
ws = torch.empty(max(b.lrd_linear_workspace_bytes(desc, 1, 0), 256), dtype=torch.uint8, device="cuda")
st = b.lrd_linear_fwd(desc, X, V, U, bias, Y, None, b.LRD_FREEZE_U, ws, check=False)
assert st == b.LRD_ERR_TIMEOUT, st
assert b.lrd_linear_fwd(desc, X, V, U, bias, Y, None, b.LRD_FREEZE_U, ws, check=False) == b.LRD_OK
assert b.lrd_check_device_status() == b.LRD_OK
print("debug mode ok")
"""
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = dict(os.environ, LRD_DEBUG="1", PYTHONPATH=os.pathsep.join([root, os.path.join(root, "tests")]))
    out = subprocess.run([sys.executable, "-c", code], env=env, capture_output=True, text=True, timeout=300)
    assert out.returncode == 0 and "debug mode ok" in out.stdout, out.stderr[-2000:]


def _svd_factors(W, r):
    Uf, s, Vt = np.linalg.svd(W, full_matrices=False)     # input construction only
    root = np.sqrt(s[:r])
    return Vt[:r].T * root, Uf[:, :r] * root


@pytest.mark.parametrize("layer", wl.C1_BERT_LAYERS, ids=[l[0] for l in wl.C1_BERT_LAYERS])
@pytest.mark.parametrize("freeze", [b.LRD_FREEZE_U, b.LRD_FREEZE_V])
def test_c1_bert_base_layers_full_size(layer, freeze):
    name, K, N, r = layer
    idx = [l[0] for l in wl.C1_BERT_LAYERS].index(name)
    case = wl.linear_case(wl.C1_M, K, N, r, "bf16", 1000 + 10 * idx, wl.W_STD_TRANSFORMER, _svd_factors)
    check_linear(case, freeze)


def test_results_are_bit_identical_across_runs_and_paths_agree():
    case = wl.random_factor_case(700, 392, 264, 136, "bf16", 41)
    a = run_linear(case, b.LRD_FREEZE_NONE)
    c = run_linear(case, b.LRD_FREEZE_NONE)
    for k in a:
        assert torch.equal(a[k], c[k]), k
    g = run_linear(case, b.LRD_FREEZE_NONE, path=b.LRD_PATH_GENERAL)
    for k in ("Y", "dX", "dU", "dV", "db"):
        assert rel_err(a[k], host(g[k])) <= 2e-2, k


def test_freeze_dispatch_never_touches_what_it_must_not():
    case = wl.random_factor_case(256, 128, 128, 64, "bf16", 55)
    code, tdt = DT["bf16"]
    desc = b.linear_desc(256, 128, 128, 64, code)
    X, V, U, bias, dY = (dev(case[k], "bf16") for k in ("X", "V", "U", "b", "dY"))
    ws = workspace(b.lrd_linear_workspace_bytes(desc, 0, 1))
    Y = torch.empty(256, 128, dtype=tdt, device="cuda")
    Z = torch.empty(256, 64, dtype=tdt, device="cuda")
    # U frozen: a Z_save buffer is refused; V frozen or none: it is required
    assert b.lrd_linear_fwd(desc, X, V, U, bias, Y, Z, b.LRD_FREEZE_U, ws, check=False) == b.LRD_ERR_INVALID_ARG
    assert b.lrd_linear_fwd(desc, X, V, U, bias, Y, None, b.LRD_FREEZE_V, ws, check=False) == b.LRD_ERR_INVALID_ARG
    assert b.lrd_linear_fwd(desc, X, V, U, bias, Y, None, b.LRD_FREEZE_NONE, ws, check=False) == b.LRD_ERR_INVALID_ARG
    b.lrd_linear_fwd(desc, X, V, U, bias, Y, Z, b.LRD_FREEZE_NONE, ws)
    # frozen gradient pointers may be NULL; then nothing is written anywhere for them.  X may be NULL when V is frozen.
    dX = torch.empty(256, 128, dtype=tdt, device="cuda")
    dU = torch.full((128, 64), 7.0, dtype=tdt, device="cuda")
    dV = torch.full((128, 64), 7.0, dtype=tdt, device="cuda")
    b.lrd_linear_bwd(desc, dY, None, V, U, Z, dX, dU, None, None, b.LRD_FREEZE_V, ws)
    b.lrd_linear_bwd(desc, dY, X, V, U, None, dX, None, dV, None, b.LRD_FREEZE_U, ws)
    torch.cuda.synchronize()
    assert (dU != 7.0).any() and (dV != 7.0).any()
    # an unfrozen factor needs its inputs and its gradient buffer
    assert b.lrd_linear_bwd(desc, dY, X, V, U, None, dX, dU, dV, None, b.LRD_FREEZE_NONE, ws, check=False) == b.LRD_ERR_INVALID_ARG
    assert b.lrd_linear_bwd(desc, dY, None, V, U, Z, dX, dU, dV, None, b.LRD_FREEZE_NONE, ws, check=False) == b.LRD_ERR_INVALID_ARG
    assert b.lrd_linear_bwd(desc, dY, X, V, U, Z, dX, dU, None, None, b.LRD_FREEZE_NONE, ws, check=False) == b.LRD_ERR_INVALID_ARG
    # workspace too small / misaligned
    assert b.lrd_linear_bwd(desc, dY, X, V, U, Z, dX, dU, dV, None, 0, ws[:128], check=False) == b.LRD_ERR_WORKSPACE
    assert b.lrd_linear_bwd(desc, dY, X, V, U, Z, dX, dU, dV, None, 0, ws[8:], check=False) in (b.LRD_ERR_ALIGNMENT, b.LRD_ERR_WORKSPACE)
    # dX = NULL skips the second data product; weight gradients are unchanged
    dU2 = torch.empty_like(dU)
    dV2 = torch.empty_like(dV)
    b.lrd_linear_bwd(desc, dY, X, V, U, Z, None, dU2, dV2, None, b.LRD_FREEZE_NONE, ws)
    b.lrd_linear_bwd(desc, dY, X, V, U, Z, dX, dU, dV, None, b.LRD_FREEZE_NONE, ws)
    torch.cuda.synchronize()
    assert torch.equal(dU, dU2) and torch.equal(dV, dV2)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_leading_dimensions_and_empty_batch(dtype):
    code, tdt = DT[dtype]
    M, K, N, r = 200, 96, 80, 40
    case = wl.random_factor_case(M, K, N, r, dtype, 77)
    ref_Z, ref_Y = o.linear_fwd(case["X"], case["V"], case["U"], case["b"])
    ldx, ldv, ldu, ldy, ldz = K + 8, r + 16, r + 8, N + 24, r + 8
    desc = b.linear_desc(M, K, N, r, code, ldx, ldv, ldu, ldy, ldz)

    def padded(a, ld):
        t = torch.full((a.shape[0], ld), float("nan"), dtype=tdt, device="cuda")
        t[:, : a.shape[1]] = dev(a, dtype)
        return t

    X, V, U, dY = padded(case["X"], ldx), padded(case["V"], ldv), padded(case["U"], ldu), padded(case["dY"], ldy)
    Y = torch.full((M, ldy), 3.0, dtype=tdt, device="cuda")
    Z = torch.full((M, ldz), 3.0, dtype=tdt, device="cuda")
    ws = workspace(b.lrd_linear_workspace_bytes(desc, 0, 1))
    b.lrd_linear_fwd(desc, X, V, U, dev(case["b"], dtype), Y, Z, b.LRD_FREEZE_NONE, ws)
    dX = torch.full((M, ldx), 3.0, dtype=tdt, device="cuda")
    dU = torch.full((N, ldu), 3.0, dtype=tdt, device="cuda")
    dV = torch.full((K, ldv), 3.0, dtype=tdt, device="cuda")
    db = torch.empty(N, dtype=tdt, device="cuda")
    b.lrd_linear_bwd(desc, dY, X, V, U, Z, dX, dU, dV, db, b.LRD_FREEZE_NONE, ws)
    torch.cuda.synchronize()
    ref = o.linear_bwd(case["dY"], case["X"], case["V"], case["U"], ref_Z, 0)
    tol = 1e-5 if dtype == "f32" else 2e-2
    for got, want, w in ((Y, ref_Y, N), (Z, ref_Z, r), (dX, ref["dX"], K), (dU, ref["dU"], r), (dV, ref["dV"], r)):
        assert rel_err(got[:, :w], want) <= tol
        assert (got[:, w:] == 3.0).all()                      # padding columns are never written
    # no tokens: nothing to do forward; weight gradients are sums over nothing
    d0 = b.linear_desc(0, K, N, r, code)
    e = torch.empty(0, dtype=tdt, device="cuda")
    b.lrd_linear_fwd(d0, X, V[:, :r].contiguous(), U[:, :r].contiguous(), None, Y, Z, 0, ws)
    dU0 = torch.full((N, r), 5.0, dtype=tdt, device="cuda")
    dV0 = torch.full((K, r), 5.0, dtype=tdt, device="cuda")
    b.lrd_linear_bwd(d0, dY, X, V, U, Z, None, dU0, dV0, None, 0, ws)
    torch.cuda.synchronize()
    assert not dU0.any() and not dV0.any()


@pytest.mark.parametrize("shape", [(333, 200, 136), (1024, 768, 3072)])
def test_dense_layer_comparison_case(shape):
    M, K, N = shape
    code, tdt = DT["bf16"]
    X = wl.round_to(wl.normal(1, (M, K)), "bf16")
    W = wl.round_to(wl.normal(2, (N, K), 0.02), "bf16")
    bias = wl.round_to(wl.normal(3, (N,), 0.1), "bf16")
    dY = wl.round_to(wl.normal(4, (M, N)), "bf16")
    desc = b.linear_desc(M, K, N, 0, code)
    ws = workspace(b.lrd_dense_workspace_bytes(desc, 1))
    Y = torch.empty(M, N, dtype=tdt, device="cuda")
    dX = torch.empty(M, K, dtype=tdt, device="cuda")
    dW = torch.empty(N, K, dtype=tdt, device="cuda")
    db = torch.empty(N, dtype=tdt, device="cuda")
    b.lrd_dense_fwd(desc, dev(X, "bf16"), dev(W, "bf16"), dev(bias, "bf16"), Y, ws)
    b.lrd_dense_bwd(desc, dev(dY, "bf16"), dev(X, "bf16"), dev(W, "bf16"), dX, dW, db, ws)
    torch.cuda.synchronize()
    ref = o.dense_bwd(dY, X, W)
    assert rel_err(Y, o.dense_fwd(X, W, bias)) <= 2e-2
    assert rel_err(dX, ref["dX"]) <= 2e-2 and rel_err(dW, ref["dW"]) <= 2e-2 and rel_err(db, ref["db"]) <= 2e-2


def test_fused_forward_is_one_kernel_and_keeps_z_on_chip():
    """With U frozen the forward is a single launch (the rank-r intermediate never leaves the chip);
    the unfused path needs two and a scratch buffer for Z."""
    M, K, N, r = 512, 768, 768, 192
    case = wl.random_factor_case(M, K, N, r, "bf16", 91)
    code, tdt = DT["bf16"]
    desc = b.linear_desc(M, K, N, r, code)
    X, V, U, bias = (dev(case[k], "bf16") for k in ("X", "V", "U", "b"))
    Y = torch.empty(M, N, dtype=tdt, device="cuda")
    ws = workspace(b.lrd_linear_workspace_bytes(desc, b.LRD_FREEZE_U, 0))
    ws.fill_(0x5A)
    before = ws.clone()
    b.lrd_set_path(b.LRD_PATH_FUSED)
    try:
        n0 = b.lrd_launch_count()
        b.lrd_linear_fwd(desc, X, V, U, bias, Y, None, b.LRD_FREEZE_U, ws)
        assert b.lrd_launch_count() - n0 == 1
        torch.cuda.synchronize()
        assert torch.equal(ws, before)                     # the workspace was not used: Z stayed on chip
        b.lrd_set_path(b.LRD_PATH_UNFUSED)
        n0 = b.lrd_launch_count()
        b.lrd_linear_fwd(desc, X, V, U, bias, Y, None, b.LRD_FREEZE_U, ws)
        assert b.lrd_launch_count() - n0 == 2
    finally:
        b.lrd_set_path(b.LRD_PATH_AUTO)
    torch.cuda.synchronize()
    assert b.lrd_check_device_status() == b.LRD_OK


@pytest.mark.parametrize("dtype,shape", [("bf16", (520, 264, 328, 64)), ("bf16", (300, 200, 136, 72)), ("f32", (256, 96, 80, 24))])
@pytest.mark.parametrize("freeze", MASKS)
def test_backward_accumulates_over_micro_batches(dtype, shape, freeze):
    """Two micro-batches through the same layer: the accumulating backward adds each one's gradients to the buffers
    (the oracle's two gradients summed in fp64); a frozen factor's buffers keep whatever they held."""
    M, K, N, r = shape
    code, tdt = DT[dtype]
    A = wl.random_factor_case(M, K, N, r, dtype, 8100 + M)
    Bc = wl.random_factor_case(M + 40, K, N, r, dtype, 8200 + M)
    Bc["V"], Bc["U"], Bc["b"] = A["V"], A["U"], A["b"]
    V, U, bias = (dev(A[k], dtype) for k in ("V", "U", "b"))
    start = {"dU": wl.round_to(wl.normal(8301, (N, r), 0.5), dtype), "dV": wl.round_to(wl.normal(8302, (K, r), 0.5), dtype),
             "db": wl.round_to(wl.normal(8303, (N,), 0.5), dtype)}
    dU, dV, db = (dev(start[k], dtype) for k in ("dU", "dV", "db"))
    want = {k: v.astype(np.float64).copy() for k, v in start.items()}
    for case in (A, Bc):
        m = case["M"]
        desc = b.linear_desc(m, K, N, r, code)
        ws = workspace(max(b.lrd_linear_workspace_bytes(desc, freeze, 0), b.lrd_linear_workspace_bytes(desc, freeze, 2)))
        X, dY = dev(case["X"], dtype), dev(case["dY"], dtype)
        Y = torch.empty(m, N, dtype=tdt, device="cuda")
        Z = None if freeze == b.LRD_FREEZE_U else torch.empty(m, r, dtype=tdt, device="cuda")
        dX = torch.empty(m, K, dtype=tdt, device="cuda")
        b.lrd_linear_fwd(desc, X, V, U, bias, Y, Z, freeze, ws)
        b.lrd_linear_bwd_accumulate(desc, dY, None if freeze == b.LRD_FREEZE_V else X, V, U, Z, dX, dU, dV, db, freeze, ws)
        torch.cuda.synchronize()
        ref = oracle_linear(case, freeze)
        assert rel_err(dX, ref["dX"]) <= TOL[dtype]
        for k in want:
            want[k] += ref[k]                       # zero for a frozen factor
    assert b.lrd_check_device_status() == b.LRD_OK
    tol = TOL[dtype]
    assert rel_err(dU, want["dU"]) <= tol and rel_err(dV, want["dV"]) <= tol and rel_err(db, want["db"]) <= tol
    if freeze == b.LRD_FREEZE_U:
        assert np.array_equal(host(dU), start["dU"].astype(np.float64)) and np.array_equal(host(db), start["db"].astype(np.float64))
    if freeze == b.LRD_FREEZE_V:
        assert np.array_equal(host(dV), start["dV"].astype(np.float64))
