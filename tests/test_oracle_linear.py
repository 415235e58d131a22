"""Pins for the oracle's decomposed linear layer: forward, backward and freeze masks."""
import numpy as np
import pytest

from oracle import lrd_oracle as o


def case(seed, M=6, K=5, N=7, r=3):
    g = np.random.default_rng(seed)
    return (g.standard_normal((M, K)), g.standard_normal((K, r)), g.standard_normal((N, r)),
            g.standard_normal(N), g.standard_normal((M, N)))


def test_forward_brute_force_tiny():
    X, V, U, b, _ = case(0, 3, 4, 5, 2)
    Z, Y = o.linear_fwd(X, V, U, b)
    for m in range(3):
        for j in range(2):
            assert abs(Z[m, j] - sum(X[m, k] * V[k, j] for k in range(4))) <= 1e-13
        for n in range(5):
            y = b[n] + sum(sum(X[m, k] * V[k, j] for k in range(4)) * U[n, j] for j in range(2))
            assert abs(Y[m, n] - y) <= 1e-13
    assert np.abs(o.linear_fwd(X, V, U, None)[1] - (Y - b)).max() <= 1e-14


def test_forward_equals_dense_layer_with_reconstructed_weight():
    X, V, U, b, _ = case(1, 17, 12, 9, 4)
    W = U @ V.T                                                   # [N x K]
    _, Y = o.linear_fwd(X, V, U, b)
    assert np.abs(Y - (X @ W.T + b)).max() <= 1e-12
    assert np.abs(Y - o.dense_fwd(X, W, b)).max() <= 1e-12


def test_backward_matches_central_finite_differences():
    X, V, U, b, dY = case(2)
    Z, _ = o.linear_fwd(X, V, U, b)
    g = o.linear_bwd(dY, X, V, U, Z, o.FREEZE_NONE)

    def loss(X_, V_, U_, b_):
        return float(np.sum(o.linear_fwd(X_, V_, U_, b_)[1] * dY))

    h = 1e-6
    for name, idx in (("dX", 0), ("dV", 1), ("dU", 2), ("db", 3)):
        args = [X, V, U, b]
        num = np.zeros_like(args[idx])
        it = np.nditer(args[idx], flags=["multi_index"])
        for _ in it:
            i = it.multi_index
            plus = [a.copy() for a in args]
            minus = [a.copy() for a in args]
            plus[idx][i] += h
            minus[idx][i] -= h
            num[i] = (loss(*plus) - loss(*minus)) / (2 * h)
        assert np.abs(num - g[name]).max() <= 1e-7 * max(1.0, np.abs(num).max()), name


def test_backward_dense_identities():
    X, V, U, b, dY = case(3, 11, 8, 10, 4)
    Z, _ = o.linear_fwd(X, V, U, b)
    g = o.linear_bwd(dY, X, V, U, Z)
    W = U @ V.T
    d = o.dense_bwd(dY, X, W)
    assert np.abs(g["dX"] - dY @ W).max() <= 1e-12
    assert np.abs(g["dX"] - d["dX"]).max() <= 1e-12
    assert np.abs(g["dU"] - d["dW"] @ V).max() <= 1e-11          # dU = (dY^T X) V
    assert np.abs(g["dV"] - d["dW"].T @ U).max() <= 1e-11        # dV = (X^T dY) U
    assert np.abs(g["db"] - dY.sum(0)).max() <= 1e-13
    assert g["dU"].shape == U.shape and g["dV"].shape == V.shape and g["dX"].shape == X.shape


def test_frozen_gradients_are_exactly_zero_and_others_unchanged():
    X, V, U, b, dY = case(4)
    Z, _ = o.linear_fwd(X, V, U, b)
    none = o.linear_bwd(dY, X, V, U, Z, o.FREEZE_NONE)
    fu = o.linear_bwd(dY, X, V, U, None, o.FREEZE_U)               # Z is not needed when U is frozen
    fv = o.linear_bwd(dY, None if False else X, V, U, Z, o.FREEZE_V)
    assert not fu["dU"].any() and not fu["db"].any() and not fv["dV"].any()
    assert np.array_equal(fu["dX"], none["dX"]) and np.array_equal(fu["dV"], none["dV"])
    assert np.array_equal(fv["dX"], none["dX"]) and np.array_equal(fv["dU"], none["dU"])
    assert np.array_equal(fv["db"], none["db"])
    assert none["dU"].any() and none["dV"].any() and none["db"].any()


def test_backward_plan_truth_table():
    DZ, DX, DU, DB, DV, NZ, NX = (o.PLAN_DZ, o.PLAN_DX, o.PLAN_DU, o.PLAN_DB, o.PLAN_DV,
                                  o.PLAN_NEEDS_Z, o.PLAN_NEEDS_X)
    assert o.linear_bwd_plan(o.FREEZE_NONE) == DZ | DX | DU | DB | DV | NZ | NX
    assert o.linear_bwd_plan(o.FREEZE_U) == DZ | DX | DV | NX
    assert o.linear_bwd_plan(o.FREEZE_V) == DZ | DX | DU | DB | NZ
    assert (DZ, DX, DU, DB, DV, NZ, NX) == (1, 2, 4, 8, 16, 32, 64)
