"""Algorithm 1 on this GPU: the timing-driven rank search.

For a layer of shape (K inputs, N outputs) at M tokens, every rank from the starting rank R (from the
compression ratio, Eq. 5 / its fully-connected analogue) down to R_min (the same formula at ratio + 1) is
timed through the library's own forward + backward (factors stored packed, leading dimension = r), three times
each (the minimum is the curve, the spread between the repeats sets the noise floor), the undecomposed layer is
timed the same way, and `lrd_rank_search` picks R_opt -- a peak of the difference curve counts only if it drops
by at least NOISE_MULTIPLE x the median relative spread (and at least MIN_DROP of the step time) -- and decides
whether the decomposed layer is kept; `lrd_rank_multiple` reports the spacing of the fast ranks the curve shows.

    python -m paper_2309_03824_b200.rank_search --M 4096 --K 768 --N 768 --alpha 2

With --tucker the layer is a Tucker-2 decomposed 3x3 convolution (Eq. 4) with ranks r1 = r2 = r running from the
rank of Eq. 5 at the compression ratio down to the rank at ratio + 1 (Eq. 6):

    python -m paper_2309_03824_b200.rank_search --tucker --B 64 --H 14 --C 512 --S 512 --alpha 2
"""
from __future__ import annotations

import argparse

import torch

from . import binding as b


NOISE_MULTIPLE = 4.0     # a drop counts as a peak from this many times the timer's median relative spread ...
MIN_DROP = 0.02          # ... and from this fraction of the step time


def fc_rank(K, N, alpha):
    """Rank of a fully connected layer for a parameter ratio alpha: r (K + N) <= K N / alpha (the library's routine)."""
    return max(1, b.lrd_svd_rank(K, N, alpha))


def tucker_rank(C, S, k, alpha):
    """Eq. 5 with r2 = r1 (the library's routine; the paper's [512, 512, 3, 3] example at alpha = 2 gives 309)."""
    return max(1, b.lrd_tucker_rank(C, S, k, alpha, 1.0)[0])


class Timing(float):
    """Seconds (the minimum over the repeats) that also carry the relative spread of the repeats."""
    spread = 0.0


def _time(fn, iters, repeats=3):
    """Seconds per call of fn: `iters` calls captured into one CUDA graph (what is timed is then the GPU's time, not
    the host's launch path, which at these sizes is the longer of the two and the noisier), replayed `repeats` times
    after a warm-up replay; the fastest replay counts, the spread of the replays is kept beside it."""
    for _ in range(3):                      # eager first: the library creates its side streams outside a capture
        fn()
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            for _ in range(iters):
                fn()
    torch.cuda.synchronize()
    graph.replay()
    out = []
    for _ in range(repeats):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        graph.replay()
        e1.record()
        torch.cuda.synchronize()
        out.append(e0.elapsed_time(e1) * 1e-3 / iters)
    t = Timing(min(out))
    t.spread = (max(out) - min(out)) / min(out)
    return t


def noise_floor(curve):
    """The relative drop from which a step of the curve counts: NOISE_MULTIPLE x the median relative spread of the
    repeats, at least MIN_DROP."""
    spreads = sorted(getattr(v, "spread", 0.0) for v in curve.values())
    med = spreads[len(spreads) // 2] if spreads else 0.0
    return max(NOISE_MULTIPLE * med, MIN_DROP)


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


def time_dense_conv(B, H, W, C, S, iters=10, seed=0):
    """Seconds per forward + backward of the undecomposed 3 x 3 convolution (the T of the closing test)."""
    bf = torch.bfloat16
    g = torch.Generator(device="cuda").manual_seed(seed)
    rn = lambda *shape, sc=1.0: (torch.randn(*shape, device="cuda", generator=g) * sc).to(bf)
    X, dY, Wk = rn(B, H, W, C), rn(B, H, W, S), rn(S, 3, 3, C, sc=(9 * C) ** -0.5)
    e = lambda *shape: torch.empty(*shape, dtype=bf, device="cuda")
    Y, dX, dW = e(B, H, W, S), e(B, H, W, C), e(S, 3, 3, C)
    ws = torch.empty(max(b.lrd_conv3x3_workspace_bytes(B, H, W, C, S, b.LRD_BF16), 256), dtype=torch.uint8, device="cuda")

    def step():
        b.lrd_conv3x3_fwd(B, H, W, C, S, b.LRD_BF16, X, Wk, Y)
        b.lrd_conv3x3_bwd(B, H, W, C, S, b.LRD_BF16, dY, X, Wk, dX, dW, ws)
    return _time(step, iters)


def search_tucker(B, H, W, C, S, R, R_min, iters=10):
    """Algorithm 1 for a Tucker-2 layer: returns (R_opt, use_decomposed, {rank: seconds}, seconds of the dense 3 x 3
    convolution, noise floor, multiple)."""
    if not (1 <= R_min <= R <= min(C, S)):
        raise ValueError("need 1 <= R_min <= R <= min(C, S)")
    T = time_dense_conv(B, H, W, C, S, iters)
    curve = {r: time_tucker(B, H, W, C, S, r, iters) for r in range(R, R_min - 1, -1)}
    t = [curve[r] for r in range(R_min, R + 1)]
    floor = noise_floor(curve)
    r_opt, use = b.lrd_rank_search(t, R_min, T, floor)
    return r_opt, use, curve, T, floor, b.lrd_rank_multiple(t, R_min, floor)


def search(M, K, N, R, R_min, freeze=b.LRD_FREEZE_NONE, iters=10):
    """Algorithm 1: returns (R_opt, use_decomposed, {rank: seconds}, seconds of the dense layer, noise floor, multiple)."""
    if not (1 <= R_min <= R <= min(K, N)):
        raise ValueError("need 1 <= R_min <= R <= min(K, N)")
    T = time_dense(M, K, N, iters)
    curve = {r: time_decomposed(M, K, N, r, freeze, iters) for r in range(R, R_min - 1, -1)}   # R down to R_min, as the paper does
    t = [curve[r] for r in range(R_min, R + 1)]
    floor = noise_floor(curve)
    r_opt, use = b.lrd_rank_search(t, R_min, T, floor)
    return r_opt, use, curve, T, floor, b.lrd_rank_multiple(t, R_min, floor)


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
        r_opt, use, curve, T, floor, mult = search_tucker(a.B, a.H, a.H, a.C, a.S, R, R_min, iters=a.iters)
        print(f"Tucker-2 3x3 conv {a.C}->{a.S}, {a.B} x {a.H} x {a.H}: dense 3x3 conv {T * 1e6:.1f} us; ranks {R}..{R_min}; "
              f"a drop counts from {floor * 100:.1f} % of the step time")
        for r in sorted(curve, reverse=True):
            print(f"  r={r:4d}  {curve[r] * 1e6:9.1f} us  (spread {curve[r].spread * 100:4.1f} %){'   <- R_opt' if r == r_opt else ''}")
        print(f"R_opt = {r_opt}; fast ranks are multiples of {mult}; {'use the decomposed layer' if use else 'keep the original layer'}")
        if b.lrd_check_device_status() != b.LRD_OK:
            raise SystemExit("device-side wait timed out")
        return
    R = a.R or fc_rank(a.K, a.N, a.alpha)
    R_min = a.Rmin or fc_rank(a.K, a.N, a.alpha + 1)
    r_opt, use, curve, T, floor, mult = search(a.M, a.K, a.N, R, R_min, iters=a.iters)
    print(f"layer {a.K}->{a.N}, M={a.M}: dense {T * 1e6:.1f} us; ranks {R}..{R_min}; a drop counts from {floor * 100:.1f} % of the step time")
    for r in sorted(curve, reverse=True):
        print(f"  r={r:4d}  {curve[r] * 1e6:9.1f} us  (spread {curve[r].spread * 100:4.1f} %){'   <- R_opt' if r == r_opt else ''}")
    print(f"R_opt = {r_opt}; fast ranks are multiples of {mult}; {'use the decomposed layer' if use else 'keep the original layer'}")
    if b.lrd_check_device_status() != b.LRD_OK:
        raise SystemExit("device-side wait timed out")


if __name__ == "__main__":
    main()
