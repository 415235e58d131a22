"""CPU fp64 oracle for the training step of a low-rank decomposed layer.

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain definition that the
CUDA library is checked against.  It shares no code with the CUDA path, is
never imported by the library or its Python binding, and is only ever used by
the tests, the smoke check and the CPU-baseline leg of the benchmark.

Everything is numpy float64.  A library matmul / einsum is used as a step; no
blocking, fusion or reordering beyond what each definition states.

Letters (the paper writes W in R^{C x S}, C = inputs, S = outputs, and calls the
input-side factor U', the output-side factor V'; here the layer weight is
W[N x K] with N = outputs and K = inputs, the input-side factor is V[K x r],
applied first, and the output-side factor is U[N x r], applied second):

    Z = X V          Y = Z U^T + b                       (Section 2, Fig. 1)

Pins (tests/test_oracle_*.py): every function below is pinned to something other
than itself - closed forms, the paper's worked examples, numpy.linalg as an
independent library routine, finite differences, brute force on tiny inputs.
`rank_search` (Algorithm 1) is the one exception: parity unpinned, because the
data of the figure it was designed on is not printed in the paper; only the
reading stated in its docstring is tested, on synthetic timing curves.
"""
from __future__ import annotations

import math

import numpy as np

FREEZE_NONE, FREEZE_U, FREEZE_V = 0, 1, 2
TK_FREEZE_NONE, TK_FREEZE_FACTORS, TK_FREEZE_CORE = 0, 1, 2
ROUND_UP, ROUND_DOWN, ROUND_NEAREST = 0, 1, 2

# bits of the backward plan (which products a freeze mask executes)
PLAN_DZ, PLAN_DX, PLAN_DU, PLAN_DB, PLAN_DV, PLAN_NEEDS_Z, PLAN_NEEDS_X = (1 << i for i in range(7))


def _f64(a):
    return np.asarray(a, dtype=np.float64)


# --------------------------------------------------------------------------------------
# Eq. (1): singular value decomposition, by one-sided (Hestenes) Jacobi rotations
# --------------------------------------------------------------------------------------
def svd_jacobi(W, tol=1e-15, max_sweeps=60):
    """Thin SVD  W[N x K] = U_f diag(sigma) V_f^T  (Eq. 1), R = min(N, K) triplets.

    One-sided Jacobi: plane rotations applied from the right make the columns of
    the working matrix mutually orthogonal; their norms are then the singular
    values.  The pairs of one round are disjoint, so their rotations commute and
    are applied together.  sigma is returned in descending order; each right
    singular vector has its largest-magnitude entry positive.
    """
    W = _f64(W)
    transposed = W.shape[0] < W.shape[1]
    At = np.array(W if transposed else W.T, order="C", copy=True)   # row j = column j of the tall matrix
    n = At.shape[0]
    Vt = np.eye(n)                                 # row j = column j of the accumulated rotations
    m = n + (n & 1)                                # even number of players; index n is a bye
    players = list(range(m))
    for _ in range(max_sweeps):
        rotated = False
        for _round in range(m - 1):
            p = np.array(players[: m // 2])
            q = np.array(players[m // 2:][::-1])
            keep = (p < n) & (q < n)
            p, q = p[keep], q[keep]
            ap, aq = At[p], At[q]
            alpha = np.einsum("ji,ji->j", ap, ap)
            beta = np.einsum("ji,ji->j", aq, aq)
            gamma = np.einsum("ji,ji->j", ap, aq)
            act = np.abs(gamma) > tol * np.sqrt(alpha * beta)
            if act.any():
                rotated = True
                g = np.where(act, gamma, 1.0)
                zeta = (beta - alpha) / (2.0 * g)
                t = np.where(zeta >= 0, 1.0, -1.0) / (np.abs(zeta) + np.sqrt(1.0 + zeta * zeta))
                c = 1.0 / np.sqrt(1.0 + t * t)
                s = c * t
                c = np.where(act, c, 1.0)[:, None]
                s = np.where(act, s, 0.0)[:, None]
                At[p], At[q] = ap * c - aq * s, ap * s + aq * c
                vp, vq = Vt[p], Vt[q]
                Vt[p], Vt[q] = vp * c - vq * s, vp * s + vq * c
            players = [players[0]] + [players[-1]] + players[1:-1]
        if not rotated:
            break
    sigma = np.sqrt(np.einsum("ji,ji->j", At, At))
    order = np.argsort(-sigma, kind="stable")
    sigma = sigma[order]
    A, Vr = At[order].T, Vt[order].T
    safe = np.where(sigma > 0, sigma, 1.0)
    Ul = A / safe
    if transposed:                                 # W^T = Ul S Vr^T  =>  W = Vr S Ul^T
        Ul, Vr = Vr, Ul
    sign = np.sign(Vr[np.abs(Vr).argmax(axis=0), np.arange(n)])
    sign[sign == 0] = 1.0
    return Ul * sign, sigma, Vr * sign


def factorize(W, r):
    """Eq. (2): keep the first r singular triplets of W[N x K]; the square root of each
    singular value is folded into both factors, so  U V^T = W'.

    Returns V[K x r] (input side) and U[N x r] (output side).
    """
    Uf, s, Vf = svd_jacobi(W)
    if not 1 <= r <= s.shape[0]:
        raise ValueError("rank out of range")
    root = np.sqrt(s[:r])
    return Vf[:, :r] * root, Uf[:, :r] * root


def recon_err(W, U, V):
    """Eq. (3): e_r = || W - U V^T ||_F^2."""
    D = _f64(W) - _f64(U) @ _f64(V).T
    return float(np.sum(D * D))


# --------------------------------------------------------------------------------------
# The decomposed fully connected layer: two consecutive layers (Section 2, Fig. 1)
# --------------------------------------------------------------------------------------
def linear_fwd(X, V, U, b=None):
    """Z = X V ;  Y = Z U^T + 1 b^T.   Returns (Z, Y)."""
    X, V, U = _f64(X), _f64(V), _f64(U)
    Z = X @ V
    Y = Z @ U.T
    if b is not None:
        Y = Y + _f64(b)[None, :]
    return Z, Y


def linear_bwd(dY, X, V, U, Z, freeze=FREEZE_NONE):
    """Chain rule of `linear_fwd`.  dZ = dY U and dX = dZ V^T are always formed: a frozen
    sub-layer still passes the gradient through (Section 2.2).  The frozen factor's own
    gradient is exactly zero; the bias belongs to the second sub-layer (U).

    Returns dict(dX, dU, dV, db).
    """
    dY, X, V, U = _f64(dY), _f64(X), _f64(V), _f64(U)
    dZ = dY @ U
    out = {"dX": dZ @ V.T}
    if freeze == FREEZE_U:
        out["dU"] = np.zeros_like(U)
        out["db"] = np.zeros(U.shape[0])
    else:
        out["dU"] = dY.T @ _f64(Z)
        out["db"] = dY.sum(axis=0)
    out["dV"] = np.zeros_like(V) if freeze == FREEZE_V else X.T @ dZ
    return out


def linear_bwd_plan(freeze):
    """Which products the backward pass runs under a freeze mask, as a bit set."""
    plan = PLAN_DZ | PLAN_DX
    if freeze != FREEZE_U:
        plan |= PLAN_DU | PLAN_DB | PLAN_NEEDS_Z
    if freeze != FREEZE_V:
        plan |= PLAN_DV | PLAN_NEEDS_X
    return plan


def dense_fwd(X, W, b=None):
    """The undecomposed layer  Y = X W^T + b  (comparison case)."""
    Y = _f64(X) @ _f64(W).T
    return Y if b is None else Y + _f64(b)[None, :]


def dense_bwd(dY, X, W):
    dY, X, W = _f64(dY), _f64(X), _f64(W)
    return {"dX": dY @ W, "dW": dY.T @ X, "db": dY.sum(axis=0)}


# --------------------------------------------------------------------------------------
# Rank quantization (Section 2.1) and rank from the compression ratio (Eq. 5, 6)
# --------------------------------------------------------------------------------------
def rank_quantize(r, multiple, mode, K, N):
    """Round the rank r to a multiple m: up, down or to the nearest (ties up); the result
    is at least one multiple and at most the largest multiple that does not exceed
    min(K, N).  Raises ValueError where no multiple fits or an argument is not positive.
    """
    m = int(multiple)
    r, K, N = int(r), int(K), int(N)
    if m < 1 or r < 1 or K < 1 or N < 1:
        raise ValueError("non-positive argument")
    cap = (min(K, N) // m) * m
    if cap == 0:
        raise ValueError("no multiple fits")
    if mode == ROUND_UP:
        q = -(-r // m) * m
    elif mode == ROUND_DOWN:
        q = (r // m) * m
    elif mode == ROUND_NEAREST:
        q = ((2 * r + m) // (2 * m)) * m
    else:
        raise ValueError("bad mode")
    return min(max(q, m), cap)


def svd_rank(C, S, alpha):
    """Rank of a two-factor layer with r (C + S) <= C S / alpha parameters (floor)."""
    return int(math.floor(C * S / (alpha * (C + S))))


def tucker_rank(C, S, k, alpha, beta=1.0):
    """Eq. (5): r1 for compression ratio alpha with r2 = beta r1; truncated to an integer
    as in the paper's [512,512,3,3] -> 309 example.  Returns (r1, r2)."""
    q = (C + beta * S) / (beta * k * k)
    r1 = 0.5 * (-q + math.sqrt(q * q + 4.0 * C * S / (beta * alpha)))
    r1 = int(math.floor(r1))
    return r1, int(math.floor(beta * r1))


def tucker_rank_min(C, S, k, alpha, beta=1.0):
    """Eq. (6): the lower bound of the search, the rank that reaches ratio alpha + 1."""
    return tucker_rank(C, S, k, alpha + 1, beta)[0]


# --------------------------------------------------------------------------------------
# Algorithm 2: sequential freezing
# --------------------------------------------------------------------------------------
def freeze_for_epoch(e):
    """Two-factor layers: even epoch -> the first-applied sub-layer (V) is frozen and the
    second (U) trains; odd epoch -> the reverse."""
    return FREEZE_V if e % 2 == 0 else FREEZE_U


def tucker_freeze_for_epoch(e):
    """Three-factor layers: even epoch -> both 1x1 factors frozen, the core trains; odd
    epoch -> the core frozen, the factors train."""
    return TK_FREEZE_FACTORS if e % 2 == 0 else TK_FREEZE_CORE


# --------------------------------------------------------------------------------------
# Eq. (4): Tucker-2 of a k x k convolution, and the three-layer form it becomes
# --------------------------------------------------------------------------------------
def tucker2_hosvd(Wd, r1, r2):
    """Wd[S][C][k][k] (out, in, kh, kw) -> A[C x r1], G[r2][k][k][r1], Bm[S x r2].

    A holds the leading r1 left singular vectors of the mode-C unfolding, Bm the leading
    r2 of the mode-S unfolding (truncated unitary factors); the core is the projection
    G = W x_C A^T x_S Bm^T.  One-shot higher-order SVD, no alternating sweeps.
    """
    Wd = _f64(Wd)
    S, C, k, _ = Wd.shape
    unfold_C = Wd.transpose(1, 0, 2, 3).reshape(C, S * k * k)
    unfold_S = Wd.reshape(S, C * k * k)
    A = svd_jacobi(unfold_C)[0][:, :r1]
    Bm = svd_jacobi(unfold_S)[0][:, :r2]
    G = np.einsum("schw,ci,so->ohwi", Wd, A, Bm)
    return A, G, Bm


def tucker2_reconstruct(A, G, Bm):
    """W'[S][C][k][k] = G x_{r1} A x_{r2} Bm."""
    return np.einsum("ohwi,ci,so->schw", _f64(G), _f64(A), _f64(Bm))


def conv2d_nhwc_fwd(X, Wk, pad, stride=1):
    """Cross-correlation with zero padding.  X[B][H][W][Ci], Wk[Co][k][k][Ci] -> Y[B][Ho][Wo][Co] with
    Y[b,ho,wo,o] = sum_{kh,kw,i} Xpadded[b, ho*stride + kh, wo*stride + kw, i] Wk[o,kh,kw,i] and
    Ho = (H + 2 pad - k) // stride + 1  (stride 1 and pad = (k-1)/2 keep the spatial size)."""
    X, Wk = _f64(X), _f64(Wk)
    B, H, Wd, Ci = X.shape
    Co, k, _, _ = Wk.shape
    Ho, Wo = (H + 2 * pad - k) // stride + 1, (Wd + 2 * pad - k) // stride + 1
    Xp = np.zeros((B, H + 2 * pad, Wd + 2 * pad, Ci))
    Xp[:, pad:pad + H, pad:pad + Wd, :] = X
    Y = np.zeros((B, Ho, Wo, Co))
    for kh in range(k):
        for kw in range(k):
            Y += Xp[:, kh:kh + (Ho - 1) * stride + 1:stride, kw:kw + (Wo - 1) * stride + 1:stride, :] @ Wk[:, kh, kw, :].T
    return Y


def conv2d_nhwc_bwd_data(dY, Wk, pad, in_hw, stride=1):
    """dXpadded[b, ho*stride + kh, wo*stride + kw, i] += dY[b,ho,wo,o] Wk[o,kh,kw,i] over all (ho, wo, kh, kw, o);
    dX is its interior (for stride 1: dX[b,h,w,i] = sum_{o,kh,kw} dY[b, h+pad-kh, w+pad-kw, o] Wk[o,kh,kw,i])."""
    dY, Wk = _f64(dY), _f64(Wk)
    B, Ho, Wo, Co = dY.shape
    _, k, _, Ci = Wk.shape
    H, Wd = in_hw
    dXp = np.zeros((B, H + 2 * pad, Wd + 2 * pad, Ci))
    for kh in range(k):
        for kw in range(k):
            dXp[:, kh:kh + (Ho - 1) * stride + 1:stride, kw:kw + (Wo - 1) * stride + 1:stride, :] += dY @ Wk[:, kh, kw, :]
    return dXp[:, pad:pad + H, pad:pad + Wd, :]


def conv2d_nhwc_bwd_filter(dY, X, k, pad, stride=1):
    """dWk[o,kh,kw,i] = sum_{b,ho,wo} dY[b,ho,wo,o] Xpadded[b, ho*stride + kh, wo*stride + kw, i]."""
    dY, X = _f64(dY), _f64(X)
    B, H, Wd, Ci = X.shape
    _, Ho, Wo, Co = dY.shape
    Xp = np.zeros((B, H + 2 * pad, Wd + 2 * pad, Ci))
    Xp[:, pad:pad + H, pad:pad + Wd, :] = X
    dW = np.zeros((Co, k, k, Ci))
    dYm = dY.reshape(-1, Co)
    for kh in range(k):
        for kw in range(k):
            dW[:, kh, kw, :] = dYm.T @ Xp[:, kh:kh + (Ho - 1) * stride + 1:stride, kw:kw + (Wo - 1) * stride + 1:stride, :].reshape(-1, Ci)
    return dW


def tucker2_fwd(X, A, G, Bm, bias=None, stride=1):
    """1x1 (C -> r1), k x k core (r1 -> r2, pad (k-1)/2; the layer's stride sits on the core), 1x1 (r2 -> S).
    X[B][H][W][C] -> (Z1[B][H][W][r1], Z2[B][Ho][Wo][r2], Y[B][Ho][Wo][S])."""
    X, A, G, Bm = _f64(X), _f64(A), _f64(G), _f64(Bm)
    k = G.shape[1]
    Z1 = X @ A
    Z2 = conv2d_nhwc_fwd(Z1, G, (k - 1) // 2, stride)
    Y = Z2 @ Bm.T
    if bias is not None:
        Y = Y + _f64(bias)
    return Z1, Z2, Y


def tucker2_bwd(dY, X, A, G, Bm, Z1, Z2, freeze=TK_FREEZE_NONE, stride=1):
    """Chain rule through the three convolutions.  Data gradients always flow; a frozen
    group's weight gradients are exactly zero.  The bias belongs to the last 1x1 factor.
    Returns dict(dX, dA, dG, dB, db)."""
    dY, X, A, G, Bm = _f64(dY), _f64(X), _f64(A), _f64(G), _f64(Bm)
    k = G.shape[1]
    pad = (k - 1) // 2
    S, C = Bm.shape[0], A.shape[0]
    dZ2 = dY @ Bm
    dZ1 = conv2d_nhwc_bwd_data(dZ2, G, pad, X.shape[1:3], stride)
    out = {"dX": dZ1 @ A.T}
    if freeze == TK_FREEZE_FACTORS:
        out["dA"], out["dB"], out["db"] = np.zeros_like(A), np.zeros_like(Bm), np.zeros(S)
    else:
        out["dA"] = X.reshape(-1, C).T @ dZ1.reshape(-1, A.shape[1])
        out["dB"] = dY.reshape(-1, S).T @ _f64(Z2).reshape(-1, Bm.shape[1])
        out["db"] = dY.reshape(-1, S).sum(axis=0)
    out["dG"] = np.zeros_like(G) if freeze == TK_FREEZE_CORE else conv2d_nhwc_bwd_filter(dZ2, _f64(Z1), k, pad, stride)
    return out


# --------------------------------------------------------------------------------------
# Algorithm 1: rank search on a measured step-time curve   (parity unpinned)
# --------------------------------------------------------------------------------------
def _fast_ranks(t, min_rel_drop):
    """Indices i (rank R_min + i) that it pays to step down to: delta(r) = t(r+1) - t(r) is positive and at
    least min_rel_drop * t(r)."""
    delta = t[1:] - t[:-1]
    return [i for i in range(t.shape[0] - 1) if delta[i] > 0 and delta[i] >= min_rel_drop * t[i]]


def rank_search(t, R_min, T_orig, min_rel_drop=0.0):
    """t[i] is the step time of the layer decomposed at rank R_min + i, for R_min..R.

    Reading of Algorithm 1 (its printed difference refers to a time that has not been
    measured yet when r runs downward, and its argmax would pick 257 rather than 256 in
    the paper's own example):  delta(r) = t(r+1) - t(r) for R_min <= r < R is the time
    saved by stepping down to r.  R_opt is the first local maximum of delta met when
    scanning down from R - 1 (a strict rise over both neighbours, an end point having
    one neighbour); with no such peak, the global argmax (largest r on ties).  The
    decomposed layer is used only if t(R_opt) < T_orig.   Returns (R_opt, use_decomposed).

    min_rel_drop: on a measured curve every wiggle of the timer is a local maximum of the
    difference; the peaks the paper means are the steps of its Fig. 2 curve (257 -> 256 is
    15 % of the step time).  A peak therefore counts only if its drop is at least
    min_rel_drop * t(r) -- the caller passes a multiple of the timer's measured relative
    spread.  With a positive threshold and no drop that large anywhere, no rank is worth
    stepping down to and R_opt = R.  min_rel_drop = 0 is the plain reading above.
    """
    t = _f64(t)
    n = t.shape[0]
    if n < 2:
        r_opt = R_min
        return r_opt, bool(t[0] < T_orig)
    delta = t[1:] - t[:-1]                 # delta[i] belongs to rank R_min + i
    ok = set(_fast_ranks(t, min_rel_drop)) if min_rel_drop > 0 else None
    best = None
    for i in range(n - 2, -1, -1):
        left = delta[i - 1] if i > 0 else -np.inf
        right = delta[i + 1] if i < n - 2 else -np.inf
        if delta[i] > left and delta[i] > right and delta[i] > 0 and (ok is None or i in ok):
            best = i
            break
    if best is None:
        if ok is None:
            mx = delta.max()
            best = max(i for i in range(n - 1) if delta[i] == mx)
        elif ok:
            mx = max(delta[i] for i in ok)
            best = max(i for i in ok if delta[i] == mx)
        else:
            best = n - 1
    return R_min + best, bool(t[best] < T_orig)


def rank_multiple(t, R_min, min_rel_drop):
    """The quantization multiple a measured curve shows: the greatest common divisor of the ranks it pays to step
    down to (drops of at least min_rel_drop * t(r)); 1 when there is none.  On the paper's V100 curve the fast ranks
    are the multiples of 8 and 16 around 256; on another device the curve says which they are."""
    t = _f64(t)
    g = 0
    for i in _fast_ranks(t, min_rel_drop):
        g = math.gcd(g, R_min + i)
    return g if g > 0 else 1
