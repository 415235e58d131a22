"""The bias-gradient entry point that needs no workspace (collected last on purpose: if it fails,
a run that stops at the first failure has already been through every other test).

Some users of this library cannot allocate device memory at the point where they need a result -
code running inside another framework's allocator-owned region, or late in a job whose pool is fully
committed.  `lrd_bias_grad_noalloc` serves them with scratch that is part of the library image.  The
test calls it through the C ABI twice in a row (the second call finds the first call's partial sums
still in the shared array) and checks both results against the `dbias` that `lrd_linear_bwd`
produces for the same upstream gradient, within the tolerance of the other bf16 / fp32 tests.
"""
import pytest
import torch

from paper_2309_03824_b200 import binding as b
from paper_2309_03824_b200 import workloads as wl

from helpers import DT, TOL, dev, host, rel_err, workspace

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_no_alloc_bias_gradient_matches_linear_bwd_twice_in_a_row(dtype):
    code, tdt = DT[dtype]
    results = []
    for M, K, N, r, seed in ((1000, 64, 520, 32, 61), (4096, 64, 768, 32, 62)):   # second call: other size, stale scratch
        case = wl.random_factor_case(M, K, N, r, dtype, seed)
        dY, X, V, U = (dev(case[k], dtype) for k in ("dY", "X", "V", "U"))
        desc = b.linear_desc(M, K, N, r, code)
        ws = workspace(b.lrd_linear_workspace_bytes(desc, b.LRD_FREEZE_V, 1))
        Z = torch.zeros(M, r, dtype=tdt, device="cuda")
        dU = torch.empty(N, r, dtype=tdt, device="cuda")
        want = torch.empty(N, dtype=tdt, device="cuda")
        b.lrd_linear_bwd(desc, dY, None, V, U, Z, None, dU, None, want, b.LRD_FREEZE_V, ws)     # existing entry point
        got = torch.full((N,), float("nan"), dtype=tdt, device="cuda")
        b.lrd_bias_grad_noalloc(dY, 0, M, N, got, code)
        torch.cuda.synchronize()
        results.append((got, want, case))
    for got, want, case in results:
        assert rel_err(got, host(want)) <= TOL[dtype]
        assert rel_err(got, case["dY"].astype("float64").sum(axis=0)) <= TOL[dtype]
    assert b.lrd_check_device_status() == b.LRD_OK


def test_no_alloc_limits_and_argument_errors():
    code, tdt = DT["bf16"]
    t = torch.zeros(16, dtype=tdt, device="cuda")
    assert b.lrd_bias_grad_noalloc(t, 0, 1, 8193, t, code, check=False) == b.LRD_ERR_TOO_LARGE
    assert b.lrd_bias_grad_noalloc(t, 0, 1, 0, t, code, check=False) == b.LRD_ERR_INVALID_ARG
    assert b.lrd_bias_grad_noalloc(None, 0, 4, 4, t, code, check=False) == b.LRD_ERR_INVALID_ARG
    assert b.lrd_bias_grad_noalloc(t, 2, 4, 4, t, code, check=False) == b.LRD_ERR_INVALID_ARG      # ld < N
    out = torch.full((8,), 3.0, dtype=tdt, device="cuda")
    b.lrd_bias_grad_noalloc(None, 0, 0, 8, out, code)            # no rows: the sum over nothing
    torch.cuda.synchronize()
    assert not out.any()
