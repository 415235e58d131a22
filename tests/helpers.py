"""Shared pieces of the GPU parity tests: move a seeded case to the device, run the library through
its C ABI, and compare with the oracle (max |err| / max |ref| per output tensor)."""
import numpy as np
import torch

from oracle import lrd_oracle as o
from paper_2309_03824_b200 import binding as b

TOL = {"f32": 1e-5, "bf16": 2e-2}      # fp32; bf16 inputs with fp32 accumulation
DT = {"f32": (b.LRD_F32, torch.float32), "bf16": (b.LRD_BF16, torch.bfloat16)}


def dev(a, dtype):
    return None if a is None else torch.from_numpy(np.ascontiguousarray(a)).to("cuda", DT[dtype][1])


def host(t):
    return t.detach().to(torch.float64).cpu().numpy()


def rel_err(got, ref):
    ref = np.asarray(ref, dtype=np.float64)
    scale = np.abs(ref).max()
    return float(np.abs(host(got) - ref).max() / (scale if scale > 0 else 1.0))


def workspace(nbytes):
    return torch.empty(max(nbytes, 256), dtype=torch.uint8, device="cuda")


def run_linear(case, freeze, path=b.LRD_PATH_AUTO, want_dx=True, sentinel=None):
    """Forward + backward of one layer on the GPU.  Returns dict of device tensors."""
    dt = case["dtype"]
    code, tdt = DT[dt]
    M, K, N, r = case["M"], case["K"], case["N"], case["r"]
    X, V, U, bias, dY = (dev(case[k], dt) for k in ("X", "V", "U", "b", "dY"))
    desc = b.linear_desc(M, K, N, r, code)
    b.lrd_set_path(path)
    try:
        Y = torch.empty(M, N, dtype=tdt, device="cuda")
        Z = None if freeze == b.LRD_FREEZE_U else torch.empty(M, r, dtype=tdt, device="cuda")
        ws = workspace(max(b.lrd_linear_workspace_bytes(desc, freeze, 0), b.lrd_linear_workspace_bytes(desc, freeze, 1)))
        b.lrd_linear_fwd(desc, X, V, U, bias, Y, Z, freeze, ws)
        fill = float("nan") if sentinel is None else sentinel
        dX = torch.full((M, K), fill, dtype=tdt, device="cuda") if want_dx else None
        dU = torch.full((N, r), fill, dtype=tdt, device="cuda")
        dV = torch.full((K, r), fill, dtype=tdt, device="cuda")
        db = torch.full((N,), fill, dtype=tdt, device="cuda")
        b.lrd_linear_bwd(desc, dY, None if freeze == b.LRD_FREEZE_V else X, V, U, Z, dX, dU, dV, db, freeze, ws)
        torch.cuda.synchronize()
        assert b.lrd_check_device_status() == b.LRD_OK
    finally:
        b.lrd_set_path(b.LRD_PATH_AUTO)
    return {"Y": Y, "Z": Z, "dX": dX, "dU": dU, "dV": dV, "db": db}


def oracle_linear(case, freeze):
    Z, Y = o.linear_fwd(case["X"], case["V"], case["U"], case["b"])
    g = o.linear_bwd(case["dY"], case["X"], case["V"], case["U"], Z, freeze)
    g.update({"Y": Y, "Z": Z})
    return g


def check_linear(case, freeze, path=b.LRD_PATH_AUTO, want_dx=True, tol=None):
    got = run_linear(case, freeze, path, want_dx)
    ref = oracle_linear(case, freeze)
    tol = TOL[case["dtype"]] if tol is None else tol
    errs = {}
    for name in ("Y", "Z", "dX", "dU", "dV", "db"):
        if got[name] is None:
            continue
        errs[name] = rel_err(got[name], ref[name])
    # frozen gradients are exactly zero
    if freeze == b.LRD_FREEZE_U:
        assert not host(got["dU"]).any() and not host(got["db"]).any()
    if freeze == b.LRD_FREEZE_V:
        assert not host(got["dV"]).any()
    bad = {k: v for k, v in errs.items() if not v <= tol}
    assert not bad, (bad, errs)
    return got, errs
