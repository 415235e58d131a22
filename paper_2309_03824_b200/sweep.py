"""Rank-quantization sweep on one square layer (M = 8192 tokens, K = N = 4096, bf16): every rank of the
list unquantized (factors stored packed, leading dimension = r) and rounded up to multiples of 8, 64 and
128, forward + backward with no freezing and with V frozen, beside the undecomposed dense layer.

    python -m paper_2309_03824_b200.sweep [--M 8192] [--K 4096] [--N 4096] [--ranks 100,250,500,750,1000]

Prints a markdown table: time per forward + backward, tokens/s, useful TFLOP/s (the products actually
executed), fraction of the roofline (the slower of those flops at the bf16 tensor peak and the algorithmic
bytes at the HBM peak), and which kernels ran.  Inputs are seeded normal draws made on the device (timing
only; parity of these shapes is covered by the sampled full-size tests).
"""
from __future__ import annotations

import argparse
import json
import os

import torch

from . import binding as b

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def peaks():
    try:
        d = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
        return float(d["bf16_tflops"]) * 1e12, float(d["hbm_gbs"]) * 1e9, "measured"
    except Exception:
        return 1590e12, 6650e9, "fallback"


def lrd_work(M, K, N, r, freeze):
    fl = 2 * M * r * (K + N) + 2 * M * N * r + 2 * M * r * K + (0 if freeze == 1 else 2 * M * N * r) + (0 if freeze == 2 else 2 * M * K * r)
    by = 2 * (M * K + K * r + N * r + N + M * N + (0 if freeze == 1 else M * r)) + 2 * (M * N + N * r + K * r + M * K)
    if freeze != 1:
        by += 2 * (M * r + N * r + N)
    if freeze != 2:
        by += 2 * (M * K + K * r)
    return fl, by


def dense_work(M, K, N):
    return 6 * M * K * N, 2 * (M * K + K * N + N + M * N) + 2 * (M * N + K * N + M * K) + 2 * (M * K + K * N + N)


def time_graph(fn, sets, reps, rounds=1):
    for s in range(sets):
        fn(s)
    torch.cuda.synchronize()
    side, g = torch.cuda.Stream(), torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(g, stream=side):
            for _ in range(rounds):          # a graph launch leaves the device idle for ~14 us: more rounds per graph for short steps
                for s in range(sets):
                    fn(s)
    torch.cuda.synchronize()
    g.replay()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    for _ in range(reps):
        g.replay()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) * 1e-3 / (reps * rounds * sets)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--M", type=int, default=8192)
    ap.add_argument("--K", type=int, default=4096)
    ap.add_argument("--N", type=int, default=4096)
    ap.add_argument("--ranks", default="100,250,500,750,1000")
    ap.add_argument("--sets", type=int, default=2, help="activation buffer sets cycled through (2 x 270 MB > L2)")
    ap.add_argument("--reps", type=int, default=5)
    a = ap.parse_args()
    M, K, N = a.M, a.K, a.N
    bf = torch.bfloat16
    P_t, P_h, src = peaks()
    gen = torch.Generator(device="cuda").manual_seed(2000)
    sets = [dict(X=torch.randn(M, K, device="cuda", generator=gen).to(bf), dY=torch.randn(M, N, device="cuda", generator=gen).to(bf),
                 Y=torch.empty(M, N, dtype=bf, device="cuda"), dX=torch.empty(M, K, dtype=bf, device="cuda"))
            for _ in range(a.sets)]
    bias = (torch.randn(N, device="cuda", generator=gen) * 0.1).to(bf)
    rows = []

    def report(name, r, freeze, sec, fl, by, kernels):
        roof = max(fl / P_t, by / P_h)
        rows.append((name, r, {0: "none", 1: "U", 2: "V"}.get(freeze, "-"), sec * 1e6, M / sec / 1e6, fl / sec / 1e12, roof / sec, kernels))

    ranks = [int(x) for x in a.ranks.split(",")]
    variants = []
    for r0 in ranks:
        seen = set()
        for label, mult in (("unquantized", 1), ("up to x8", 8), ("up to x64", 64), ("up to x128", 128)):
            r = r0 if mult == 1 else b.lrd_rank_quantize(r0, mult, b.LRD_ROUND_UP, K, N)
            if r in seen:
                continue
            seen.add(r)
            variants.append((f"r={r0} {label}", r))
    for name, r in variants:
        V = (torch.randn(K, r, device="cuda", generator=gen) * 0.02).to(bf)
        U = (torch.randn(N, r, device="cuda", generator=gen) * 0.02).to(bf)
        desc = b.linear_desc(M, K, N, r, b.LRD_BF16)
        ws = torch.empty(max(b.lrd_linear_workspace_bytes(desc, 0, 0), b.lrd_linear_workspace_bytes(desc, 0, 1), 256), dtype=torch.uint8, device="cuda")
        Z = [torch.empty(M, r, dtype=bf, device="cuda") for _ in range(a.sets)]
        dU, dV, db = torch.empty(N, r, dtype=bf, device="cuda"), torch.empty(K, r, dtype=bf, device="cuda"), torch.empty(N, dtype=bf, device="cuda")
        for freeze in (b.LRD_FREEZE_NONE, b.LRD_FREEZE_V):
            def step(s, freeze=freeze):
                st = sets[s]
                b.lrd_linear_fwd(desc, st["X"], V, U, bias, st["Y"], Z[s], freeze, ws)
                b.lrd_linear_bwd(desc, st["dY"], None if freeze == b.LRD_FREEZE_V else st["X"], V, U, Z[s], st["dX"], dU,
                                 None if freeze == b.LRD_FREEZE_V else dV, db, freeze, ws)
            n0 = b.lrd_launch_count()
            step(0)
            nk = b.lrd_launch_count() - n0
            sec = time_graph(step, a.sets, a.reps)
            fl, by = lrd_work(M, K, N, r, freeze)
            report(name, r, freeze, sec, fl, by, nk)
        del V, U, Z, ws
    # the undecomposed layer
    W = (torch.randn(N, K, device="cuda", generator=gen) * 0.02).to(bf)
    dW = torch.empty(N, K, dtype=bf, device="cuda")
    db = torch.empty(N, dtype=bf, device="cuda")
    desc = b.linear_desc(M, K, N, 0, b.LRD_BF16)
    ws = torch.empty(max(b.lrd_dense_workspace_bytes(desc, 1), 256), dtype=torch.uint8, device="cuda")

    def dense_step(s):
        st = sets[s]
        b.lrd_dense_fwd(desc, st["X"], W, bias, st["Y"], ws)
        b.lrd_dense_bwd(desc, st["dY"], st["X"], W, st["dX"], dW, db, ws)
    n0 = b.lrd_launch_count()
    dense_step(0)
    nk = b.lrd_launch_count() - n0
    sec = time_graph(dense_step, a.sets, a.reps)
    fl, by = dense_work(M, K, N)
    report("dense 4096x4096", 0, -1, sec, fl, by, nk)
    if b.lrd_check_device_status() != b.LRD_OK:
        raise SystemExit("device-side wait timed out")

    print(f"M={M} K={K} N={N}, bf16, forward + backward, CUDA-graph replay over {a.sets} buffer sets; peaks: {src} "
          f"({P_t / 1e12:.0f} TFLOP/s, {P_h / 1e9:.0f} GB/s)\n")
    print("| variant | r | frozen | us fwd+bwd | M tokens/s | useful TFLOP/s | roofline frac | kernels |")
    print("|---|---|---|---|---|---|---|---|")
    for name, r, fz, us, mtok, tf, frac, nk in rows:
        print(f"| {name} | {r} | {fz} | {us:.1f} | {mtok:.2f} | {tf:.1f} | {frac:.3f} | {nk} |")


if __name__ == "__main__":
    main()
