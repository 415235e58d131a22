"""One-off layer preparation (not part of the per-step path): factor a dense weight into the two
low-rank factors, or a conv kernel into its Tucker-2 factors, with torch.linalg in float64.

The symmetric split puts the square root of each kept singular value into both factors, so
U @ V.T is the rank-r approximation of W (paper, Eq. 2).  Tucker-2 follows Eq. 4: truncated
unitary factors from the two channel-mode unfoldings and the projected core.
"""
from __future__ import annotations

import numpy as np
import torch


def _device():
    return "cuda" if torch.cuda.is_available() else "cpu"


def svd_factors_multi(W, ranks):
    """W[N x K] (numpy float64) -> {r: (V[K x r], U[N x r])} from one SVD."""
    Wt = torch.as_tensor(np.asarray(W), dtype=torch.float64, device=_device())
    Uf, s, Vh = torch.linalg.svd(Wt, full_matrices=False)
    out = {}
    for r in ranks:
        root = torch.sqrt(s[:r])
        out[r] = ((Vh[:r].T * root).cpu().numpy(), (Uf[:, :r] * root).cpu().numpy())
    return out


def svd_factors(W, r):
    return svd_factors_multi(W, [r])[r]


def tucker2_factors(Wd, r1, r2):
    """Wd[S][C][k][k] -> A[C x r1], G[r2][k][k][r1], Bm[S x r2]."""
    Wt = torch.as_tensor(np.asarray(Wd), dtype=torch.float64, device=_device())
    S, Cc, k, _ = Wt.shape
    A = torch.linalg.svd(Wt.permute(1, 0, 2, 3).reshape(Cc, -1), full_matrices=False)[0][:, :r1]
    Bm = torch.linalg.svd(Wt.reshape(S, -1), full_matrices=False)[0][:, :r2]
    G = torch.einsum("schw,ci,so->ohwi", Wt, A, Bm)
    return A.cpu().numpy(), G.contiguous().cpu().numpy(), Bm.cpu().numpy()
