"""Run one decomposed linear layer on the GPU a few times: the smallest driver of the C ABI, for
profilers and quick timing.

    python -m paper_2309_03824_b200.run_case --M 4096 --K 768 --N 768 --r 192 --freeze U --what fwd --iters 5

--r 0 runs the undecomposed layer (lrd_dense_fwd / lrd_dense_bwd) instead.  --tucker B,H,W,C,S,r1,r2 runs a Tucker-2
decomposed 3 x 3 convolution (lrd_tucker2_fwd / lrd_tucker2_bwd; --freeze none | factors | core).  --dtype f32 runs
the linear layer in fp32 (the general fp32-FMA kernels).  Factors are stored packed, so a rank that is not a multiple
of 8 (--r 250) takes the repacking path.  --accumulate runs the backward pass through lrd_linear_bwd_accumulate (the
gradients are added to what the buffers hold).
"""
from __future__ import annotations

import argparse

import torch

from . import binding as b
from . import workloads as wl


def run_tucker(a):
    B, H, W, C, S, r1, r2 = (int(x) for x in a.tucker.split(","))
    f = {"none": 0, "factors": 1, "core": 2}[a.freeze]
    bf = torch.bfloat16
    case = wl.random_tucker_case(B, H, W, C, S, r1, r2, 3, "bf16", 7)
    A, G, Bm, bias = (torch.from_numpy(case[k]).to("cuda", bf) for k in ("A", "G", "Bm", "b"))
    desc = b.tucker2_desc(B, H, W, C, S, r1, r2, b.LRD_BF16)
    ws = torch.empty(max(b.lrd_tucker2_workspace_bytes(desc, f, 0), b.lrd_tucker2_workspace_bytes(desc, f, 1), 256), dtype=torch.uint8, device="cuda")
    sets = [dict(X=torch.from_numpy(case["X"]).to("cuda", bf), dY=torch.from_numpy(case["dY"]).to("cuda", bf),
                 Y=torch.empty(B, H, W, S, dtype=bf, device="cuda"), Z1=torch.empty(B, H, W, r1, dtype=bf, device="cuda"),
                 Z2=torch.empty(B, H, W, r2, dtype=bf, device="cuda"), dX=torch.empty(B, H, W, C, dtype=bf, device="cuda")) for _ in range(a.sets)]
    dA, dG, dB, db = (torch.empty(*sh, dtype=bf, device="cuda") for sh in ((C, r1), (r2, 3, 3, r1), (S, r2), (S,)))
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for phase in ("warm", "timed"):
        torch.cuda.synchronize()
        e0.record()
        for i in range(a.iters):
            s = sets[i % a.sets]
            if a.what in ("fwd", "both"):
                b.lrd_tucker2_fwd(desc, s["X"], A, G, Bm, bias, s["Y"], None if f == 2 else s["Z1"], None if f == 1 else s["Z2"], f, ws)
            if a.what in ("bwd", "both"):
                b.lrd_tucker2_bwd(desc, s["dY"], None if f == 1 else s["X"], A, G, Bm, None if f == 2 else s["Z1"], None if f == 1 else s["Z2"],
                                  s["dX"], None if f == 1 else dA, None if f == 2 else dG, None if f == 1 else dB, None if f == 1 else db, f, ws)
        e1.record()
        torch.cuda.synchronize()
    st = b.lrd_check_device_status()
    print(f"tucker {a.what} {a.tucker} freeze={a.freeze}: {e0.elapsed_time(e1) * 1e3 / a.iters:.2f} us per iteration (eager launches), device status {st}")
    if st != b.LRD_OK:
        raise SystemExit(1)


def main():
    ap = argparse.ArgumentParser()
    for n, d in (("M", 4096), ("K", 768), ("N", 768), ("r", 192), ("iters", 5), ("sets", 8)):
        ap.add_argument(f"--{n}", type=int, default=d)
    ap.add_argument("--freeze", default="U", choices=["none", "U", "V", "factors", "core"])
    ap.add_argument("--tucker", default="", help="B,H,W,C,S,r1,r2")
    ap.add_argument("--dtype", default="bf16", choices=["bf16", "f32"])
    ap.add_argument("--what", default="both", choices=["fwd", "bwd", "both"])
    ap.add_argument("--path", default="auto", choices=["auto", "general", "unfused", "fused"])
    ap.add_argument("--accumulate", action="store_true")
    a = ap.parse_args()
    b.lrd_set_path({"auto": 0, "general": 1, "unfused": 2, "fused": 3}[a.path])
    if a.tucker:
        return run_tucker(a)
    freeze = {"none": 0, "U": 1, "V": 2}[a.freeze]
    bf = torch.bfloat16 if a.dtype == "bf16" else torch.float32
    code = b.LRD_BF16 if a.dtype == "bf16" else b.LRD_F32
    dense = a.r == 0
    case = wl.random_factor_case(a.M, a.K, a.N, 64 if dense else a.r, a.dtype, 7)
    V, U, bias = (torch.from_numpy(case[k]).to("cuda", bf) for k in ("V", "U", "b"))
    desc = b.linear_desc(a.M, a.K, a.N, a.r, code)
    if dense:
        W = (U.float() @ V.float().T).to(bf)                 # [N x K]
        dW = torch.empty(a.N, a.K, dtype=bf, device="cuda")
        ws = torch.empty(max(b.lrd_dense_workspace_bytes(desc, 1), 256), dtype=torch.uint8, device="cuda")
    else:
        ws = torch.empty(max(b.lrd_linear_workspace_bytes(desc, freeze, 1), 256), dtype=torch.uint8, device="cuda")
    sets = []
    for _ in range(a.sets):        # distinct buffers so that consecutive launches do not hit in L2
        sets.append(dict(X=torch.from_numpy(case["X"]).to("cuda", bf), dY=torch.from_numpy(case["dY"]).to("cuda", bf),
                         Y=torch.empty(a.M, a.N, dtype=bf, device="cuda"), Z=torch.empty(a.M, max(a.r, 8), dtype=bf, device="cuda"),
                         dX=torch.empty(a.M, a.K, dtype=bf, device="cuda")))
    dU = torch.zeros(a.N, a.r, dtype=bf, device="cuda")
    dV = torch.zeros(a.K, a.r, dtype=bf, device="cuda")
    db = torch.zeros(a.N, dtype=bf, device="cuda")
    if a.accumulate and not dense:
        ws = torch.empty(max(b.lrd_linear_workspace_bytes(desc, freeze, 2), 256), dtype=torch.uint8, device="cuda")
    bwd = b.lrd_linear_bwd_accumulate if a.accumulate else b.lrd_linear_bwd
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for phase in ("warm", "timed"):
        torch.cuda.synchronize()
        e0.record()
        for i in range(a.iters):
            s = sets[i % a.sets]
            if dense:
                if a.what in ("fwd", "both"):
                    b.lrd_dense_fwd(desc, s["X"], W, bias, s["Y"], ws)
                if a.what in ("bwd", "both"):
                    b.lrd_dense_bwd(desc, s["dY"], s["X"], W, s["dX"], dW, db, ws)
                continue
            if a.what in ("fwd", "both"):
                b.lrd_linear_fwd(desc, s["X"], V, U, bias, s["Y"], None if freeze == 1 else s["Z"], freeze, ws)
            if a.what in ("bwd", "both"):
                bwd(desc, s["dY"], None if freeze == 2 else s["X"], V, U, None if freeze == 1 else s["Z"],
                    s["dX"], None if freeze == 1 else dU, None if freeze == 2 else dV,
                    None if freeze == 1 else db, freeze, ws)
        e1.record()
        torch.cuda.synchronize()
    st = b.lrd_check_device_status()
    print(f"{a.what} M={a.M} K={a.K} N={a.N} r={a.r} freeze={a.freeze} path={a.path}: "
          f"{e0.elapsed_time(e1) * 1e3 / a.iters:.2f} us per iteration (eager launches), device status {st}")
    if st != b.LRD_OK:
        raise SystemExit(1)


if __name__ == "__main__":
    main()
