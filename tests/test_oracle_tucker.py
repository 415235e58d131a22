"""Pins for the oracle's Tucker-2 decomposition (Eq. 4), its convolutions and their gradients."""
import numpy as np
import pytest

from oracle import lrd_oracle as o


def rng(seed):
    return np.random.default_rng(seed)


def conv_brute(X, Wk, pad):
    """Seven nested loops, straight from the definition of a zero-padded cross-correlation."""
    B, H, W, Ci = X.shape
    Co, k, _, _ = Wk.shape
    Y = np.zeros((B, H, W, Co))
    for b in range(B):
        for h in range(H):
            for w in range(W):
                for co in range(Co):
                    acc = 0.0
                    for kh in range(k):
                        for kw in range(k):
                            hh, ww = h + kh - pad, w + kw - pad
                            if 0 <= hh < H and 0 <= ww < W:
                                for ci in range(Ci):
                                    acc += X[b, hh, ww, ci] * Wk[co, kh, kw, ci]
                    Y[b, h, w, co] = acc
    return Y


def test_conv_forward_brute_force_and_delta_cases():
    g = rng(0)
    X, Wk = g.standard_normal((2, 4, 5, 3)), g.standard_normal((4, 3, 3, 3))
    assert np.abs(o.conv2d_nhwc_fwd(X, Wk, 1) - conv_brute(X, Wk, 1)).max() <= 1e-13
    # a single one at each corner and in the middle: the output is the flipped kernel around it, clipped
    for (h0, w0) in [(0, 0), (0, 4), (3, 0), (3, 4), (2, 2)]:
        D = np.zeros((1, 4, 5, 3))
        D[0, h0, w0, 1] = 1.0
        Y = o.conv2d_nhwc_fwd(D, Wk, 1)
        for h in range(4):
            for w in range(5):
                kh, kw = h0 - h + 1, w0 - w + 1
                want = Wk[:, kh, kw, 1] if 0 <= kh < 3 and 0 <= kw < 3 else np.zeros(4)
                assert np.allclose(Y[0, h, w], want, atol=1e-15)
    # a 1x1 convolution is the linear layer over M = B H W pixels
    A = g.standard_normal((3, 6))
    Y1 = o.conv2d_nhwc_fwd(X, A.T.reshape(6, 1, 1, 3), 0)
    assert np.abs(Y1.reshape(-1, 6) - X.reshape(-1, 3) @ A).max() <= 1e-13


def test_conv_gradients_are_adjoints_and_match_finite_differences():
    g = rng(1)
    X, Wk, dY = g.standard_normal((2, 4, 4, 3)), g.standard_normal((5, 3, 3, 3)), g.standard_normal((2, 4, 4, 5))
    dX = o.conv2d_nhwc_bwd_data(dY, Wk, 1, (4, 4))
    dW = o.conv2d_nhwc_bwd_filter(dY, X, 3, 1)
    assert dX.shape == X.shape and dW.shape == Wk.shape
    L = float(np.sum(o.conv2d_nhwc_fwd(X, Wk, 1) * dY))            # bilinear in (X, Wk)
    assert abs(np.sum(dX * X) - L) <= 1e-11 * abs(L) + 1e-12
    assert abs(np.sum(dW * Wk) - L) <= 1e-11 * abs(L) + 1e-12
    h = 1e-6
    for arr, grad, which in ((X, dX, 0), (Wk, dW, 1)):
        it = np.nditer(arr, flags=["multi_index"])
        for n, _ in enumerate(it):
            if n % 7:
                continue
            i = it.multi_index
            p, m = arr.copy(), arr.copy()
            p[i] += h
            m[i] -= h
            f = (lambda a: np.sum(o.conv2d_nhwc_fwd(a, Wk, 1) * dY)) if which == 0 else \
                (lambda a: np.sum(o.conv2d_nhwc_fwd(X, a, 1) * dY))
            assert abs((f(p) - f(m)) / (2 * h) - grad[i]) <= 1e-7 * max(1.0, abs(grad[i]))


def test_hosvd_factors_unitary_and_full_rank_exact():
    Wd = rng(2).standard_normal((10, 8, 3, 3))                     # [S][C][k][k]
    A, G, Bm = o.tucker2_hosvd(Wd, 8, 10)
    assert A.shape == (8, 8) and G.shape == (10, 3, 3, 8) and Bm.shape == (10, 10)
    assert np.abs(A.T @ A - np.eye(8)).max() <= 1e-12 and np.abs(Bm.T @ Bm - np.eye(10)).max() <= 1e-12
    assert np.abs(o.tucker2_reconstruct(A, G, Bm) - Wd).max() <= 1e-10
    A, G, Bm = o.tucker2_hosvd(Wd, 5, 6)
    assert A.shape == (8, 5) and G.shape == (6, 3, 3, 5) and Bm.shape == (10, 6)
    assert np.abs(A.T @ A - np.eye(5)).max() <= 1e-12 and np.abs(Bm.T @ Bm - np.eye(6)).max() <= 1e-12
    # truncation error lies between the larger discarded mode energy and their sum
    err = np.sum((o.tucker2_reconstruct(A, G, Bm) - Wd) ** 2)
    sC = np.linalg.svd(Wd.transpose(1, 0, 2, 3).reshape(8, -1), compute_uv=False)
    sS = np.linalg.svd(Wd.reshape(10, -1), compute_uv=False)
    tC, tS = np.sum(sC[5:] ** 2), np.sum(sS[6:] ** 2)
    assert max(tC, tS) - 1e-10 <= err <= tC + tS + 1e-10
    # the factors span the leading mode subspaces found by the library routine
    UC = np.linalg.svd(Wd.transpose(1, 0, 2, 3).reshape(8, -1))[0][:, :5]
    assert np.abs(A @ A.T - UC @ UC.T).max() <= 1e-10


def test_hosvd_k1_reduces_to_matrix_projection():
    W = rng(3).standard_normal((9, 7))                              # [S x C], k = 1
    A, G, Bm = o.tucker2_hosvd(W.reshape(9, 7, 1, 1), 7, 9)
    assert np.abs(o.tucker2_reconstruct(A, G, Bm)[:, :, 0, 0] - W).max() <= 1e-10
    r = 3
    A, G, Bm = o.tucker2_hosvd(W.reshape(9, 7, 1, 1), r, r)
    V, U = o.factorize(W, r)
    assert np.abs(o.tucker2_reconstruct(A, G, Bm)[:, :, 0, 0] - U @ V.T).max() <= 1e-10


def test_tucker_forward_equals_dense_conv_with_reconstructed_kernel():
    g = rng(4)
    C, S, r1, r2 = 6, 7, 4, 5
    A, G, Bm = g.standard_normal((C, r1)), g.standard_normal((r2, 3, 3, r1)), g.standard_normal((S, r2))
    X, bias = g.standard_normal((2, 5, 4, C)), g.standard_normal(S)
    Z1, Z2, Y = o.tucker2_fwd(X, A, G, Bm, bias)
    assert Z1.shape == (2, 5, 4, r1) and Z2.shape == (2, 5, 4, r2) and Y.shape == (2, 5, 4, S)
    Wd = o.tucker2_reconstruct(A, G, Bm)                            # [S][C][k][k]
    dense = conv_brute(X, Wd.transpose(0, 2, 3, 1), 1) + bias
    assert np.abs(Y - dense).max() <= 1e-11


def test_tucker_backward_finite_differences_and_masks():
    g = rng(5)
    C, S, r1, r2 = 3, 4, 2, 3
    A, G, Bm = g.standard_normal((C, r1)), g.standard_normal((r2, 3, 3, r1)), g.standard_normal((S, r2))
    X, bias, dY = g.standard_normal((1, 3, 4, C)), g.standard_normal(S), g.standard_normal((1, 3, 4, S))
    Z1, Z2, _ = o.tucker2_fwd(X, A, G, Bm, bias)
    gr = o.tucker2_bwd(dY, X, A, G, Bm, Z1, Z2, o.TK_FREEZE_NONE)
    args = {"dX": X, "dA": A, "dG": G, "dB": Bm, "db": bias}
    order = ["dX", "dA", "dG", "dB", "db"]

    def loss(vals):
        return float(np.sum(o.tucker2_fwd(*vals)[2] * dY))

    h = 1e-6
    for pos, name in enumerate(order):
        base = [args[n] for n in order]
        it = np.nditer(base[pos], flags=["multi_index"])
        for _ in it:
            i = it.multi_index
            p = [a.copy() for a in base]
            m = [a.copy() for a in base]
            p[pos][i] += h
            m[pos][i] -= h
            num = (loss(p) - loss(m)) / (2 * h)
            assert abs(num - gr[name][i]) <= 1e-6 * max(1.0, abs(num)), (name, i)
    ff = o.tucker2_bwd(dY, X, A, G, Bm, Z1, None, o.TK_FREEZE_FACTORS)
    fc = o.tucker2_bwd(dY, X, A, G, Bm, None, Z2, o.TK_FREEZE_CORE)
    assert not ff["dA"].any() and not ff["dB"].any() and not ff["db"].any() and not fc["dG"].any()
    assert np.array_equal(ff["dG"], gr["dG"]) and np.array_equal(ff["dX"], gr["dX"])
    for n in ("dA", "dB", "db", "dX"):
        assert np.array_equal(fc[n], gr[n])


def conv_brute_strided(X, Wk, pad, stride):
    """The definition again, with a stride: output pixel (ho, wo) looks at input rows ho * stride + kh - pad."""
    B, H, W, Ci = X.shape
    Co, k, _, _ = Wk.shape
    Ho, Wo = (H + 2 * pad - k) // stride + 1, (W + 2 * pad - k) // stride + 1
    Y = np.zeros((B, Ho, Wo, Co))
    for b in range(B):
        for ho in range(Ho):
            for wo in range(Wo):
                for co in range(Co):
                    acc = 0.0
                    for kh in range(k):
                        for kw in range(k):
                            hh, ww = ho * stride + kh - pad, wo * stride + kw - pad
                            if 0 <= hh < H and 0 <= ww < W:
                                for ci in range(Ci):
                                    acc += X[b, hh, ww, ci] * Wk[co, kh, kw, ci]
                    Y[b, ho, wo, co] = acc
    return Y


@pytest.mark.parametrize("k,stride,hw", [(3, 2, (5, 6)), (3, 2, (4, 4)), (5, 1, (5, 4)), (5, 2, (7, 5)), (1, 2, (5, 5)), (7, 1, (4, 6))])
def test_strided_and_wider_convolutions(k, stride, hw):
    """Forward against brute force and against the stride-1 result sampled every `stride` pixels; the gradients
    as adjoints of the forward map and against finite differences."""
    g = rng(40 + k + stride)
    H, W = hw
    pad = (k - 1) // 2
    X, Wk = g.standard_normal((2, H, W, 3)), g.standard_normal((4, k, k, 3))
    Y = o.conv2d_nhwc_fwd(X, Wk, pad, stride)
    assert Y.shape == (2, (H - 1) // stride + 1, (W - 1) // stride + 1, 4)
    assert np.abs(Y - conv_brute_strided(X, Wk, pad, stride)).max() <= 1e-13
    assert np.abs(Y - o.conv2d_nhwc_fwd(X, Wk, pad, 1)[:, ::stride, ::stride, :]).max() <= 1e-13
    dY = g.standard_normal(Y.shape)
    dX = o.conv2d_nhwc_bwd_data(dY, Wk, pad, (H, W), stride)
    dW = o.conv2d_nhwc_bwd_filter(dY, X, k, pad, stride)
    assert dX.shape == X.shape and dW.shape == Wk.shape
    L = float(np.sum(Y * dY))
    assert abs(np.sum(dX * X) - L) <= 1e-11 * abs(L) + 1e-12
    assert abs(np.sum(dW * Wk) - L) <= 1e-11 * abs(L) + 1e-12
    eps = 1e-6
    for which, (arr, grad) in enumerate(((X, dX), (Wk, dW))):
        for _ in range(6):
            idx = tuple(int(g.integers(0, n)) for n in arr.shape)
            hi, lo = arr.copy(), arr.copy()
            hi[idx] += eps
            lo[idx] -= eps
            f = (lambda a: np.sum(o.conv2d_nhwc_fwd(a, Wk, pad, stride) * dY)) if which == 0 else \
                (lambda a: np.sum(o.conv2d_nhwc_fwd(X, a, pad, stride) * dY))
            assert abs((f(hi) - f(lo)) / (2 * eps) - grad[idx]) <= 1e-7 * max(1.0, abs(grad[idx]))


@pytest.mark.parametrize("k,stride", [(3, 2), (5, 1), (1, 1)])
def test_tucker2_layer_with_stride_equals_the_dense_convolution_and_its_gradients(k, stride):
    """Forward = dense convolution with the reconstructed kernel at the same stride; every gradient against finite
    differences of the forward map."""
    g = rng(70 + k + stride)
    B, H, W, C, S, r1, r2 = 2, 5, 4, 4, 5, 3, 2
    X, A, G, Bm = g.standard_normal((B, H, W, C)), g.standard_normal((C, r1)), g.standard_normal((r2, k, k, r1)), g.standard_normal((S, r2))
    bias = g.standard_normal(S)
    Z1, Z2, Y = o.tucker2_fwd(X, A, G, Bm, bias, stride)
    Wd = o.tucker2_reconstruct(A, G, Bm)                      # [S][C][k][k]
    ref = o.conv2d_nhwc_fwd(X, np.transpose(Wd, (0, 2, 3, 1)), (k - 1) // 2, stride) + bias
    assert np.abs(Y - ref).max() <= 1e-12
    dY = g.standard_normal(Y.shape)
    gr = o.tucker2_bwd(dY, X, A, G, Bm, Z1, Z2, o.TK_FREEZE_NONE, stride)
    vals = [X, A, G, Bm, bias]
    eps = 1e-6
    for pos, name in ((0, "dX"), (1, "dA"), (2, "dG"), (3, "dB"), (4, "db")):
        for _ in range(4):
            idx = tuple(int(g.integers(0, n)) for n in vals[pos].shape)
            hi, lo = [v.copy() for v in vals], [v.copy() for v in vals]
            hi[pos][idx] += eps
            lo[pos][idx] -= eps
            fd = (np.sum(o.tucker2_fwd(*hi, stride)[2] * dY) - np.sum(o.tucker2_fwd(*lo, stride)[2] * dY)) / (2 * eps)
            assert abs(fd - gr[name][idx]) <= 1e-7 * max(1.0, abs(gr[name][idx])), name
