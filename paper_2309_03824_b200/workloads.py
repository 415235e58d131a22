"""Seeded synthetic inputs for low-rank decomposed layers.

Shapes, seeds, random draws and the single rounding to the working dtype live here and
nowhere else, so that the CUDA library and the CPU check see the same numbers.  This
module holds none of the method's arithmetic: the factorisation of a weight is done by a
callable that the caller passes in.

Recipe.  Every tensor is drawn with numpy's Generator(PCG64(seed)).standard_normal in
float64, scaled to its standard deviation, then rounded once (round to nearest even) to
the working dtype.  bf16 values are carried in float32 arrays that hold exactly
bf16-representable numbers.  seed = 1000 * config + tensor index, except that the weight
of config 0 uses seed 0.
"""
from __future__ import annotations

import numpy as np

# ---- layer shapes of the workloads (M tokens, K inputs, N outputs, r rank) -----------------
C0_LINEAR = dict(M=256, K=512, N=512, r=40, dtype="f32", w_std=(1.0 / 512.0) ** 0.5)
C1_BERT_LAYERS = [  # (name, K, N, r), M = 32 * 128 tokens
    ("attn_q", 768, 768, 192), ("attn_k", 768, 768, 192), ("attn_v", 768, 768, 192), ("attn_o", 768, 768, 192),
    ("ffn_1", 768, 3072, 384), ("ffn_2", 3072, 768, 384),
]
C1_M = 4096
C2_SWEEP = dict(M=8192, K=4096, N=4096, ranks=[100, 250, 500, 750, 1000], multiples=[8, 64, 128])
C3_TUCKER = dict(B=64, H=14, W=14, C=256, S=256, r1=96, r2=96, k=3, r_unquantized=88, multiple=32)
C4_GPT_LAYERS = [  # per block, M = 8 * 1024 tokens, 12 blocks
    ("attn_q", 1024, 1024, 256), ("attn_k", 1024, 1024, 256), ("attn_v", 1024, 1024, 256), ("attn_o", 1024, 1024, 256),
    ("ffn_1", 1024, 4096, 512), ("ffn_2", 4096, 1024, 512),
]
C4_M, C4_BLOCKS = 8192, 12
W_STD_TRANSFORMER = 0.02
BIAS_STD = 0.1          # bias ~ N(0, 0.01): 0.01 read as the variance


def round_to_bf16(a):
    """Round float values to bf16 (nearest even); returned as float32 holding those values."""
    f = np.ascontiguousarray(a, dtype=np.float32)
    u = f.view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).reshape(f.shape)


def round_to(a, dtype):
    if dtype == "bf16":
        return round_to_bf16(a)
    if dtype == "f32":
        return np.ascontiguousarray(a, dtype=np.float32)
    raise ValueError(dtype)


def normal(seed, shape, std=1.0):
    return np.random.Generator(np.random.PCG64(seed)).standard_normal(shape) * std


def weight(seed, N, K, std):
    """Dense weight W[N x K] in float64 (not rounded: it is the input of the factorisation)."""
    return normal(seed, (N, K), std)


def linear_case(M, K, N, r, dtype, seed_base, w_std, factorize, w_seed=None, with_bias=True, W=None):
    """One decomposed linear layer with its upstream gradient.

    factorize(W[N x K] float64, r) -> (V[K x r], U[N x r]) float64.
    Returns float32 arrays (values already rounded to `dtype`):  X[M x K], V, U, b[N], dY[M x N].
    """
    if W is None:
        W = weight(seed_base if w_seed is None else w_seed, N, K, w_std)
    V, U = factorize(W, r)
    case = {
        "X": round_to(normal(seed_base + 1, (M, K)), dtype),
        "V": round_to(V, dtype),
        "U": round_to(U, dtype),
        "dY": round_to(normal(seed_base + 3, (M, N)), dtype),
        "M": M, "K": K, "N": N, "r": r, "dtype": dtype,
    }
    case["b"] = round_to(normal(seed_base + 2, (N,), BIAS_STD), dtype) if with_bias else None
    return case


def random_factor_case(M, K, N, r, dtype, seed_base, with_bias=True):
    """A layer whose factors are drawn directly (no factorisation): N(0, 1/sqrt(K)) and
    N(0, 1/sqrt(r)) entries keep Z and Y at unit scale.  For shape sweeps and edge cases."""
    case = {
        "X": round_to(normal(seed_base + 1, (M, K)), dtype),
        "V": round_to(normal(seed_base + 4, (K, r), K ** -0.5), dtype),
        "U": round_to(normal(seed_base + 5, (N, r), r ** -0.5), dtype),
        "dY": round_to(normal(seed_base + 3, (M, N)), dtype),
        "M": M, "K": K, "N": N, "r": r, "dtype": dtype,
    }
    case["b"] = round_to(normal(seed_base + 2, (N,), BIAS_STD), dtype) if with_bias else None
    return case


def tucker_kernel(seed, S, C, k):
    """Dense conv kernel Wd[S][C][k][k] ~ N(0, 2 / fan_in), fan_in = C k k, float64."""
    return normal(seed, (S, C, k, k), (2.0 / (C * k * k)) ** 0.5)


def tucker_case(B, H, W, C, S, r1, r2, k, dtype, seed_base, decompose, with_bias=True):
    """One Tucker-2 decomposed k x k convolution, NHWC, with its upstream gradient.

    decompose(Wd[S][C][k][k] float64, r1, r2) -> (A[C x r1], G[r2][k][k][r1], Bm[S x r2]).
    """
    A, G, Bm = decompose(tucker_kernel(seed_base, S, C, k), r1, r2)
    case = {
        "X": round_to(normal(seed_base + 1, (B, H, W, C)), dtype),
        "A": round_to(A, dtype), "G": round_to(G, dtype), "Bm": round_to(Bm, dtype),
        "dY": round_to(normal(seed_base + 3, (B, H, W, S)), dtype),
        "B": B, "H": H, "W": W, "C": C, "S": S, "r1": r1, "r2": r2, "k": k, "dtype": dtype,
    }
    case["b"] = round_to(normal(seed_base + 2, (S,), BIAS_STD), dtype) if with_bias else None
    return case


def random_tucker_case(B, H, W, C, S, r1, r2, k, dtype, seed_base, with_bias=True, stride=1):
    """Tucker-2 layer with directly drawn factors (no decomposition), unit-scale activations.  The output (and dY)
    has (H - 1) // stride + 1 rows and (W - 1) // stride + 1 columns of pixels."""
    Ho, Wo = (H - 1) // stride + 1, (W - 1) // stride + 1
    case = {
        "X": round_to(normal(seed_base + 1, (B, H, W, C)), dtype),
        "A": round_to(normal(seed_base + 4, (C, r1), C ** -0.5), dtype),
        "G": round_to(normal(seed_base + 5, (r2, k, k, r1), (k * k * r1) ** -0.5), dtype),
        "Bm": round_to(normal(seed_base + 6, (S, r2), r2 ** -0.5), dtype),
        "dY": round_to(normal(seed_base + 3, (B, Ho, Wo, S)), dtype),
        "B": B, "H": H, "W": W, "C": C, "S": S, "r1": r1, "r2": r2, "k": k, "stride": stride, "dtype": dtype,
    }
    case["b"] = round_to(normal(seed_base + 2, (S,), BIAS_STD), dtype) if with_bias else None
    return case


def sample_rows(seed, n_rows, count):
    """`count` distinct row indices in [0, n_rows), sorted; always includes the first and last row."""
    count = min(count, n_rows)
    g = np.random.Generator(np.random.PCG64(seed))
    idx = set(g.choice(n_rows, size=count, replace=False).tolist()) | {0, n_rows - 1}
    return np.array(sorted(idx), dtype=np.int64)
