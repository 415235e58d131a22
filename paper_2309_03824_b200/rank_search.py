"""Algorithm 1 on this GPU: the timing-driven rank search.

For a layer of shape (K inputs, N outputs) at M tokens, every rank from the starting rank R (from the
compression ratio, Eq. 5 / its fully-connected analogue) down to R_min (the same formula at ratio + 1) is
timed through the library's own forward + backward (factors stored packed, leading dimension = r, so that a
rank the tensor-core path cannot address runs on the general path — that is the effect the algorithm looks
for), the undecomposed layer is timed the same way, and `lrd_rank_search` picks R_opt and decides whether
the decomposed layer is kept.

    python -m paper_2309_03824_b200.rank_search --M 4096 --K 768 --N 768 --alpha 2

With --tucker the layer is a Tucker-2 decomposed 3x3 convolution (Eq. 4) with ranks r1 = r2 = r running from the
rank of Eq. 5 at the compression ratio down to the rank at ratio + 1 (Eq. 6):

    python -m paper_2309_03824_b200.rank_search --tucker --B 64 --H 14 --C 512 --S 512 --alpha 2
"""
from __future__ import annotations

import argparse

import torch

from . import binding as b


def fc_rank(K, N, alpha):
    """Rank of a fully connected layer for a parameter ratio alpha: r (K + N) <= K N / alpha."""
    return max(1, (K * N) // (alpha * (K + N)))


def tucker_rank(C, S, k, alpha):
    """Eq. 5 with r2 = r1: the largest r whose parameter count C r + k^2 r^2 + S r stays within C S k^2 / alpha
    (the paper's [512, 512, 3, 3] example at alpha = 2 gives 309)."""
    budget = C * S * k * k / alpha
    b_, a_ = C + S, k * k
    r = int((-b_ + (b_ * b_ + 4.0 * a_ * budget) ** 0.5) / (2.0 * a_))
    while (r + 1) * (C + S) + a_ * (r + 1) * (r + 1) <= budget:      # settle the float root on the integer condition
        r += 1
    while r > 1 and r * (C + S) + a_ * r * r > budget:
        r -= 1
    return max(r, 1)


def _time(fn, iters):
    for _ in range(3):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(iters):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) * 1e-3 / iters


def time_decomposed(M, K, N, r, freeze=b.LRD_FREEZE_NONE, iters=10, seed=0):
    """Seconds per forward + backward of the layer decomposed at rank r (synthetic normal inputs)."""
    bf = torch.bfloat16
    g = torch.Generator(device="cuda").manual_seed(seed)
    X = torch.randn(M, K, device="cuda", generator=g).to(bf)
    dY = torch.randn(M, N, device="cuda", generator=g).to(bf)
    V = (torch.randn(K, r, device="cuda", generator=g) * 0.02).to(bf)
    U = (torch.randn(N, r, device="cuda", generator=g) * 0.02).to(bf)
    bias = torch.zeros(N, dtype=bf, device="cuda")
    Y, Z, dX = torch.empty(M, N, dtype=bf, device="cuda"), torch.empty(M, r, dtype=bf, device="cuda"), torch.empty(M, K, dtype=bf, device="cuda")
    dU, dV, db = torch.empty(N, r, dtype=bf, device="cuda"), torch.empty(K, r, dtype=bf, device="cuda"), torch.empty(N, dtype=bf, device="cuda")
    desc = b.linear_desc(M, K, N, r, b.LRD_BF16)
    ws = torch.empty(max(b.lrd_linear_workspace_bytes(desc, freeze, 0), b.lrd_linear_workspace_bytes(desc, freeze, 1), 256),
                     dtype=torch.uint8, device="cuda")
    fU, fV = freeze == b.LRD_FREEZE_U, freeze == b.LRD_FREEZE_V

    def step():
        b.lrd_linear_fwd(desc, X, V, U, bias, Y, None if fU else Z, freeze, ws)
        b.lrd_linear_bwd(desc, dY, None if fV else X, V, U, None if fU else Z, dX, None if fU else dU, None if fV else dV,
                         None if fU else db, freeze, ws)
    return _time(step, iters)


def time_dense(M, K, N, iters=10, seed=0):
    bf = torch.bfloat16
    g = torch.Generator(device="cuda").manual_seed(seed)
    X = torch.randn(M, K, device="cuda", generator=g).to(bf)
    dY = torch.randn(M, N, device="cuda", generator=g).to(bf)
    W = (torch.randn(N, K, device="cuda", generator=g) * 0.02).to(bf)
    bias = torch.zeros(N, dtype=bf, device="cuda")
    Y, dX, dW, db = (torch.empty(M, N, dtype=bf, device="cuda"), torch.empty(M, K, dtype=bf, device="cuda"),
                     torch.empty(N, K, dtype=bf, device="cuda"), torch.empty(N, dtype=bf, device="cuda"))
    desc = b.linear_desc(M, K, N, 0, b.LRD_BF16)
    ws = torch.empty(max(b.lrd_dense_workspace_bytes(desc, 1), 256), dtype=torch.uint8, device="cuda")

    def step():
        b.lrd_dense_fwd(desc, X, W, bias, Y, ws)
        b.lrd_dense_bwd(desc, dY, X, W, dX, dW, db, ws)
    return _time(step, iters)


def time_tucker(B, H, W, C, S, r, iters=10, seed=0):
    """Seconds per forward + backward of the Tucker-2 layer at r1 = r2 = r (nothing frozen, synthetic inputs)."""
    bf = torch.bfloat16
    g = torch.Generator(device="cuda").manual_seed(seed)
    rn = lambda *shape, sc=1.0: (torch.randn(*shape, device="cuda", generator=g) * sc).to(bf)
    X, dY = rn(B, H, W, C), rn(B, H, W, S)
    A, G, Bm, bias = rn(C, r, sc=C ** -0.5), rn(r, 3, 3, r, sc=(9 * r) ** -0.5), rn(S, r, sc=r ** -0.5), rn(S, sc=0.1)
    e = lambda *shape: torch.empty(*shape, dtype=bf, device="cuda")
    Y, Z1, Z2, dX, dA, dG, dB, db = e(B, H, W, S), e(B, H, W, r), e(B, H, W, r), e(B, H, W, C), e(C, r), e(r, 3, 3, r), e(S, r), e(S)
    desc = b.tucker2_desc(B, H, W, C, S, r, r, b.LRD_BF16)
    ws = torch.empty(max(b.lrd_tucker2_workspace_bytes(desc, 0, 0), b.lrd_tucker2_workspace_bytes(desc, 0, 1), 256),
                     dtype=torch.uint8, device="cuda")

    def step():
        b.lrd_tucker2_fwd(desc, X, A, G, Bm, bias, Y, Z1, Z2, b.LRD_TK_FREEZE_NONE, ws)
        b.lrd_tucker2_bwd(desc, dY, X, A, G, Bm, Z1, Z2, dX, dA, dG, dB, db, b.LRD_TK_FREEZE_NONE, ws)
    return _time(step, iters)


def search_tucker(B, H, W, C, S, R, R_min, iters=10):
    """Algorithm 1 for a Tucker-2 layer; the original layer is not timed here (no dense 3x3 kernel in this library),
    so the closing test is left open: returns (R_opt, {rank: seconds})."""
    if not (1 <= R_min <= R <= min(C, S)):
        raise ValueError("need 1 <= R_min <= R <= min(C, S)")
    curve = {r: time_tucker(B, H, W, C, S, r, iters) for r in range(R, R_min - 1, -1)}
    r_opt, _ = b.lrd_rank_search([curve[r] for r in range(R_min, R + 1)], R_min, float("inf"))
    return r_opt, curve


def search(M, K, N, R, R_min, freeze=b.LRD_FREEZE_NONE, iters=10):
    """Algorithm 1: returns (R_opt, use_decomposed, {rank: seconds}, seconds of the dense layer)."""
    if not (1 <= R_min <= R <= min(K, N)):
        raise ValueError("need 1 <= R_min <= R <= min(K, N)")
    T = time_dense(M, K, N, iters)
    curve = {r: time_decomposed(M, K, N, r, freeze, iters) for r in range(R, R_min - 1, -1)}   # R down to R_min, as the paper does
    t = [curve[r] for r in range(R_min, R + 1)]
    r_opt, use = b.lrd_rank_search(t, R_min, T)
    return r_opt, use, curve, T


def main():
    ap = argparse.ArgumentParser()
    for n, d in (("M", 4096), ("K", 768), ("N", 768), ("alpha", 2), ("iters", 10)):
        ap.add_argument(f"--{n}", type=int, default=d)
    ap.add_argument("--R", type=int, default=0, help="starting rank (default: from --alpha)")
    ap.add_argument("--Rmin", type=int, default=0, help="lowest rank (default: the rank at alpha + 1)")
    ap.add_argument("--tucker", action="store_true", help="Tucker-2 decomposed 3x3 convolution instead of a linear layer")
    for n, d in (("B", 64), ("H", 14), ("C", 512), ("S", 512)):
        ap.add_argument(f"--{n}", type=int, default=d)
    a = ap.parse_args()
    if a.tucker:
        R = a.R or tucker_rank(a.C, a.S, 3, a.alpha)
        R_min = a.Rmin or tucker_rank(a.C, a.S, 3, a.alpha + 1)
        r_opt, curve = search_tucker(a.B, a.H, a.H, a.C, a.S, R, R_min, iters=a.iters)
        print(f"Tucker-2 3x3 conv {a.C}->{a.S}, {a.B} x {a.H} x {a.H}: ranks {R}..{R_min}")
        for r in sorted(curve, reverse=True):
            print(f"  r={r:4d}  {curve[r] * 1e6:9.1f} us{'   <- R_opt' if r == r_opt else ''}")
        print(f"R_opt = {r_opt}")
        if b.lrd_check_device_status() != b.LRD_OK:
            raise SystemExit("device-side wait timed out")
        return
    R = a.R or fc_rank(a.K, a.N, a.alpha)
    R_min = a.Rmin or fc_rank(a.K, a.N, a.alpha + 1)
    r_opt, use, curve, T = search(a.M, a.K, a.N, R, R_min, iters=a.iters)
    print(f"layer {a.K}->{a.N}, M={a.M}: dense {T * 1e6:.1f} us; ranks {R}..{R_min}")
    for r in sorted(curve, reverse=True):
        print(f"  r={r:4d}  {curve[r] * 1e6:9.1f} us{'   <- R_opt' if r == r_opt else ''}")
    print(f"R_opt = {r_opt}; {'use the decomposed layer' if use else 'keep the original layer'}")
    if b.lrd_check_device_status() != b.LRD_OK:
        raise SystemExit("device-side wait timed out")


if __name__ == "__main__":
    main()
