"""Pins for the oracle's SVD, truncation and reconstruction error (Eq. 1-3)."""
import numpy as np
import pytest

from oracle import lrd_oracle as o


def rng(seed):
    return np.random.default_rng(seed)


@pytest.mark.parametrize("shape", [(7, 5), (5, 7), (40, 64), (96, 33), (1, 6), (6, 1)])
def test_svd_against_library_and_invariants(shape):
    W = rng(1).standard_normal(shape)
    U, s, V = o.svd_jacobi(W)
    R = min(shape)
    assert U.shape == (shape[0], R) and V.shape == (shape[1], R) and s.shape == (R,)
    assert np.all(np.diff(s) <= 0) and np.all(s >= 0)
    assert np.abs(U.T @ U - np.eye(R)).max() <= 1e-12
    assert np.abs(V.T @ V - np.eye(R)).max() <= 1e-12
    assert abs(np.sum(s * s) - np.sum(W * W)) <= 1e-12 * np.sum(W * W)
    s_lib = np.linalg.svd(W, compute_uv=False)
    assert np.abs(s - s_lib).max() <= 1e-10 * s_lib.max()
    assert np.abs((U * s) @ V.T - W).max() <= 1e-10          # Eq. (1) is exact at R = min(C, S)
    # sign convention: largest-magnitude entry of each right singular vector is positive
    assert np.all(V[np.abs(V).argmax(axis=0), np.arange(R)] > 0)


def test_svd_known_singular_values():
    # W = Q1 diag(s) Q2^T with orthonormal Q1, Q2 has exactly the singular values s
    g = rng(2)
    Q1, _ = np.linalg.qr(g.standard_normal((12, 6)))
    Q2, _ = np.linalg.qr(g.standard_normal((9, 6)))
    s_true = np.array([9.0, 4.0, 2.5, 1.0, 0.25, 0.0625])
    W = (Q1 * s_true) @ Q2.T
    U, s, V = o.svd_jacobi(W)
    assert np.abs(s[:6] - s_true).max() <= 1e-12 and np.abs(s[6:]).max() <= 1e-12   # rank 6 of 9
    # the singular subspaces are those of Q1, Q2 (distinct values => vectors match up to sign)
    assert np.abs(np.abs(U[:, :6].T @ Q1) - np.eye(6)).max() <= 1e-10
    assert np.abs(np.abs(V[:, :6].T @ Q2) - np.eye(6)).max() <= 1e-10


def test_svd_diagonal_rank1_and_2x2_closed_forms():
    U, s, V = o.svd_jacobi(np.diag([3.0, -7.0, 0.5]))
    assert np.allclose(s, [7.0, 3.0, 0.5], atol=1e-14)
    a, b = np.array([1.0, 2.0, -2.0]), np.array([3.0, 0.0, 4.0, 0.0])
    _, s, _ = o.svd_jacobi(np.outer(a, b))                    # rank one: sigma_1 = |a||b|
    assert abs(s[0] - 15.0) <= 1e-12 and np.all(np.abs(s[1:]) <= 1e-12)
    M = np.array([[1.0, 2.0], [3.0, 4.0]])                    # 2x2: s^2 = (T +- sqrt(T^2 - 4 D^2)) / 2
    T, D = np.sum(M * M), abs(np.linalg.det(M))
    expect = np.sqrt([(T + np.sqrt(T * T - 4 * D * D)) / 2, (T - np.sqrt(T * T - 4 * D * D)) / 2])
    assert np.allclose(o.svd_jacobi(M)[1], expect, rtol=1e-13)


def test_svd_does_not_modify_its_input():
    W = rng(3).standard_normal((5, 9))
    W0 = W.copy()
    o.svd_jacobi(W)
    assert np.array_equal(W, W0)


@pytest.mark.parametrize("shape", [(48, 32), (32, 48)])
def test_factorize_full_rank_reproduces_w(shape):
    W = rng(4).standard_normal(shape)
    V, U = o.factorize(W, min(shape))
    assert V.shape == (shape[1], min(shape)) and U.shape == (shape[0], min(shape))
    assert np.abs(U @ V.T - W).max() <= 1e-10


def test_truncation_error_is_discarded_energy_and_monotone():
    N, K = 40, 56
    W = rng(5).standard_normal((N, K))
    s_lib = np.linalg.svd(W, compute_uv=False)
    prev = np.inf
    for r in [1, 2, 7, 20, 39, 40]:
        V, U = o.factorize(W, r)
        e = o.recon_err(W, U, V)                                  # Eq. (3), squared Frobenius norm
        tail = np.sum(s_lib[r:] ** 2)                              # Eckart-Young
        assert abs(np.sqrt(e) - np.sqrt(tail)) <= 1e-10 * s_lib[0]
        assert e <= prev + 1e-12
        prev = e
        if r < 40:                                                  # spectral norm of the residual = sigma_{r+1}
            assert abs(np.linalg.norm(W - U @ V.T, 2) - s_lib[r]) <= 1e-10 * s_lib[0]
    # recon_err against an element-by-element sum on a tiny case
    Wt, Ut, Vt = W[:3, :4], rng(6).standard_normal((3, 2)), rng(7).standard_normal((4, 2))
    brute = sum((Wt[i, j] - sum(Ut[i, k] * Vt[j, k] for k in range(2))) ** 2 for i in range(3) for j in range(4))
    assert abs(o.recon_err(Wt, Ut, Vt) - brute) <= 1e-12


def test_factor_split_is_symmetric_square_root():
    # Each factor carries sqrt(sigma_i): column norms squared equal sigma_i, columns are orthogonal,
    # V is K x r (input side) and U is N x r (output side).
    N, K, r = 24, 36, 10
    W = rng(8).standard_normal((N, K))
    s_lib = np.linalg.svd(W, compute_uv=False)
    V, U = o.factorize(W, r)
    assert V.shape == (K, r) and U.shape == (N, r)
    assert np.abs(V.T @ V - np.diag(s_lib[:r])).max() <= 1e-10
    assert np.abs(U.T @ U - np.diag(s_lib[:r])).max() <= 1e-10
    Ul, sl, Vlt = np.linalg.svd(W, full_matrices=False)
    assert np.abs(U @ V.T - (Ul[:, :r] * sl[:r]) @ Vlt[:r]).max() <= 1e-10
    with pytest.raises(ValueError):
        o.factorize(W, 25)
    with pytest.raises(ValueError):
        o.factorize(W, 0)
