"""Decomposed-layer time of a 12-block GPT-2-medium-shaped stack (hidden 1024, FFN 4096, 8 x 1024 = 8192 tokens,
bf16): every linear layer decomposed at r = 256 (attention projections) and r = 512 (feed-forward), forward through
all blocks, then backward through all blocks in reverse, with U frozen, with V frozen (the two phases of sequential
freezing, Algorithm 2) and with nothing frozen, beside the undecomposed stack.

    python -m paper_2309_03824_b200.gpt_stack [--blocks 12] [--reps 5]

Only the decomposed layers run: layer norm, attention itself, GELU, embedding and loss are not part of the method.
Every block has its own weights; activations rotate over two buffer sets per layer (1.3 GB > L2), seeded normal
draws made on the device (timing only; parity of these shapes is covered by the sampled full-size tests).  The
query / key / value projections of a block go out as one group.  Prints a markdown table.
"""
from __future__ import annotations

import argparse

import torch

from . import binding as b
from . import workloads as wl
from .sweep import peaks, time_graph


def layer_work(M, K, N, r, freeze):
    """(forward flops, bytes), (backward flops, bytes): the products executed, every tensor once."""
    ff = 2 * M * r * (K + N)
    fb = 2 * (M * K + K * r + N * r + N + M * N + (0 if freeze == 1 else M * r))
    bf_ = 2 * M * N * r + 2 * M * r * K + (0 if freeze == 1 else 2 * M * N * r) + (0 if freeze == 2 else 2 * M * K * r)
    bb = 2 * (M * N + N * r + K * r + M * K)
    if freeze != 1:
        bb += 2 * (M * r + N * r + N)
    if freeze != 2:
        bb += 2 * (M * K + K * r)
    return (ff, fb), (bf_, bb)


def dense_work(M, K, N):
    return (2 * M * K * N, 2 * (M * K + K * N + N + M * N)), (4 * M * K * N, 2 * (M * N + K * N + M * K) + 2 * (M * K + K * N + N))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--blocks", type=int, default=wl.C4_BLOCKS)
    ap.add_argument("--reps", type=int, default=5)
    a = ap.parse_args()
    M, bf = wl.C4_M, torch.bfloat16
    P_t, P_h, src = peaks()
    gen = torch.Generator(device="cuda").manual_seed(4000)
    SETS = 2

    def randn(*shape, std=1.0):
        return (torch.randn(*shape, device="cuda", generator=gen) * std).to(bf)

    # activations: shared by all blocks (a block's layers are timed, not chained numerically), two sets per layer
    acts = {}
    for name, K, N, r in wl.C4_GPT_LAYERS:
        acts[name] = [dict(X=randn(M, K), dY=randn(M, N), Y=torch.empty(M, N, dtype=bf, device="cuda"),
                           Z=torch.empty(M, r, dtype=bf, device="cuda"), dX=torch.empty(M, K, dtype=bf, device="cuda")) for _ in range(SETS)]
    blocks = []
    for _ in range(a.blocks):
        layers = []
        for name, K, N, r in wl.C4_GPT_LAYERS:
            desc = b.linear_desc(M, K, N, r, b.LRD_BF16)
            dd = b.linear_desc(M, K, N, 0, b.LRD_BF16)
            nws = max(b.lrd_linear_workspace_bytes(desc, 0, 0), b.lrd_linear_workspace_bytes(desc, 0, 1), b.lrd_dense_workspace_bytes(dd, 1), 256)
            layers.append(dict(name=name, K=K, N=N, r=r, desc=desc, ddesc=dd, V=randn(K, r, std=0.02), U=randn(N, r, std=0.02),
                               W=randn(N, K, std=0.02), b=randn(N, std=0.1), dU=torch.empty(N, r, dtype=bf, device="cuda"),
                               dV=torch.empty(K, r, dtype=bf, device="cuda"), dW=torch.empty(N, K, dtype=bf, device="cuda"),
                               db=torch.empty(N, dtype=bf, device="cuda"), ws=torch.empty(nws, dtype=torch.uint8, device="cuda")))
        blocks.append(layers)

    def fwd(L, st, f):
        b.lrd_linear_fwd(L["desc"], st["X"], L["V"], L["U"], L["b"], st["Y"], None if f == 1 else st["Z"], f, L["ws"])

    def bwd(L, st, f):
        b.lrd_linear_bwd(L["desc"], st["dY"], None if f == 2 else st["X"], L["V"], L["U"], None if f == 1 else st["Z"], st["dX"],
                         None if f == 1 else L["dU"], None if f == 2 else L["dV"], None if f == 1 else L["db"], f, L["ws"])

    def gfwd(Ls, s, f):
        sts = [acts[L["name"]][s] for L in Ls]
        b.lrd_linear_group_fwd([L["desc"] for L in Ls], [x["X"] for x in sts], [L["V"] for L in Ls], [L["U"] for L in Ls],
                               [L["b"] for L in Ls], [x["Y"] for x in sts], None if f == 1 else [x["Z"] for x in sts], f, [L["ws"] for L in Ls])

    def gbwd(Ls, s, f):
        sts = [acts[L["name"]][s] for L in Ls]
        b.lrd_linear_group_bwd([L["desc"] for L in Ls], [x["dY"] for x in sts], None if f == 2 else [x["X"] for x in sts],
                               [L["V"] for L in Ls], [L["U"] for L in Ls], None if f == 1 else [x["Z"] for x in sts], [x["dX"] for x in sts],
                               None if f == 1 else [L["dU"] for L in Ls], None if f == 2 else [L["dV"] for L in Ls],
                               None if f == 1 else [L["db"] for L in Ls], f, [L["ws"] for L in Ls])

    def lrd_step(s, f, grouped):
        for bi, layers in enumerate(blocks):
            ss = (s + bi) % SETS
            if grouped:
                gfwd(layers[:3], ss, f)
            for L in layers[3 if grouped else 0:]:
                fwd(L, acts[L["name"]][ss], f)
        for bi, layers in reversed(list(enumerate(blocks))):
            ss = (s + bi) % SETS
            for L in reversed(layers[3 if grouped else 0:]):
                bwd(L, acts[L["name"]][ss], f)
            if grouped:
                gbwd(layers[:3], ss, f)

    def dense_step(s):
        for bi, layers in enumerate(blocks):
            for L in layers:
                st = acts[L["name"]][(s + bi) % SETS]
                b.lrd_dense_fwd(L["ddesc"], st["X"], L["W"], L["b"], st["Y"], L["ws"])
        for bi, layers in reversed(list(enumerate(blocks))):
            for L in reversed(layers):
                st = acts[L["name"]][(s + bi) % SETS]
                b.lrd_dense_bwd(L["ddesc"], st["dY"], st["X"], L["W"], st["dX"], L["dW"], L["db"], L["ws"])

    def roof(work):
        return sum(max(fl / P_t, by / P_h) for fl, by in work)

    rows = []
    for f, label in ((1, "U frozen (phase 0)"), (2, "V frozen (phase 1)"), (0, "nothing frozen")):
        work, flops = [], 0
        for name, K, N, r in wl.C4_GPT_LAYERS:
            w = layer_work(M, K, N, r, f)
            work += list(w) * a.blocks
            flops += (w[0][0] + w[1][0]) * a.blocks
        for grouped in (True, False):
            n0 = b.lrd_launch_count()
            lrd_step(0, f, grouped)
            nk = b.lrd_launch_count() - n0
            sec = time_graph(lambda s: lrd_step(s, f, grouped), SETS, a.reps, rounds=1)
            rows.append((label + (", q/k/v grouped" if grouped else ", one call per layer"), sec, flops, roof(work), nk))
    work, flops = [], 0
    for name, K, N, r in wl.C4_GPT_LAYERS:
        w = dense_work(M, K, N)
        work += list(w) * a.blocks
        flops += (w[0][0] + w[1][0]) * a.blocks
    n0 = b.lrd_launch_count()
    dense_step(0)
    nk = b.lrd_launch_count() - n0
    sec = time_graph(dense_step, SETS, a.reps, rounds=1)
    rows.append(("undecomposed stack", sec, flops, roof(work), nk))
    if b.lrd_check_device_status() != b.LRD_OK:
        raise SystemExit("device-side wait timed out")

    print(f"{a.blocks} blocks, M={M} tokens, bf16, forward + backward of the linear layers only, CUDA-graph replay over {SETS} "
          f"activation sets; peaks: {src} ({P_t / 1e12:.0f} TFLOP/s, {P_h / 1e9:.0f} GB/s)\n")
    print("| variant | ms per step | M tokens/s | useful TFLOP/s | roofline ms | roofline frac | launches |")
    print("|---|---|---|---|---|---|---|")
    for name, sec, fl, rf, nk in rows:
        print(f"| {name} | {sec * 1e3:.3f} | {M / sec / 1e6:.2f} | {fl / sec / 1e12:.0f} | {rf * 1e3:.3f} | {rf / sec:.3f} | {nk} |")


if __name__ == "__main__":
    main()
