"""CPU tests of the library boundary: every declared symbol is exported, and the host-only entry
points agree bit for bit with the oracle.  No compute call is made here."""
import ctypes
import os
import re

import pytest

from oracle import lrd_oracle as o
from paper_2309_03824_b200 import binding as b

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "lrd.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(lrd_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib = ctypes.CDLL(b.LIB_PATH)
    names = declared_symbols()
    assert len(names) >= 16
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(b.EXPORTS) == names


def test_rank_quantize_bit_exact_against_oracle():
    for m in (1, 8, 16, 32, 64, 128):
        for r in range(1, 1300):
            for mode in (0, 1, 2):
                assert b.lrd_rank_quantize(r, m, mode, 1111, 2048) == o.rank_quantize(r, m, mode, 1111, 2048)
    # error mapping
    assert b.lrd_rank_quantize(0, 8, 0, 64, 64) == -b.LRD_ERR_INVALID_ARG
    assert b.lrd_rank_quantize(5, 0, 0, 64, 64) == -b.LRD_ERR_INVALID_ARG
    assert b.lrd_rank_quantize(5, 8, 9, 64, 64) == -b.LRD_ERR_INVALID_ARG
    assert b.lrd_rank_quantize(5, 128, 0, 64, 64) == -b.LRD_ERR_BAD_RANK
    assert b.lrd_rank_quantize(257, 64, b.LRD_ROUND_DOWN, 512, 512) == 256


def test_freeze_schedule_and_plan_bit_exact_against_oracle():
    for e in range(0, 50):
        assert b.lrd_freeze_for_epoch(e) == o.freeze_for_epoch(e)
        assert b.lrd_tucker_freeze_for_epoch(e) == o.tucker_freeze_for_epoch(e)
    for f in (0, 1, 2):
        assert b.lrd_linear_bwd_plan(f) == o.linear_bwd_plan(f)
    assert b.lrd_linear_bwd_plan(7) == 0
    assert (b.LRD_FREEZE_NONE, b.LRD_FREEZE_U, b.LRD_FREEZE_V) == (o.FREEZE_NONE, o.FREEZE_U, o.FREEZE_V)
    assert (b.LRD_TK_FREEZE_FACTORS, b.LRD_TK_FREEZE_CORE) == (o.TK_FREEZE_FACTORS, o.TK_FREEZE_CORE)


def test_status_strings_and_workspace_queries():
    for s in range(10):
        assert b.lrd_status_string(s) and b.lrd_status_string(s) != "unknown status"
    assert b.lrd_status_string(99) == "unknown status"
    d = b.linear_desc(4096, 768, 768, 192, b.LRD_BF16)
    fw, bw = b.lrd_linear_workspace_bytes(d, 0, 0), b.lrd_linear_workspace_bytes(d, 0, 1)
    assert fw >= 4096 * 192 * 2 and bw >= fw and fw % 256 == 0 and bw % 256 == 0
    assert b.lrd_linear_workspace_bytes(b.linear_desc(16, 8, 8, 9, b.LRD_BF16), 0, 0) == 0       # rank > min(K, N)
    assert b.lrd_linear_workspace_bytes(b.linear_desc(16, 8, 8, 4, 7), 0, 0) == 0                 # bad dtype
    t = b.tucker2_desc(64, 14, 14, 256, 256, 96, 96, b.LRD_BF16)
    assert b.lrd_tucker2_workspace_bytes(t, 0, 1) >= b.lrd_tucker2_workspace_bytes(t, 0, 0) > 0
    assert b.lrd_tucker2_workspace_bytes(b.tucker2_desc(1, 4, 4, 8, 8, 4, 4, b.LRD_F32, k=5), 0, 0) == 0


def test_argument_errors_are_reported_before_any_launch():
    # NULL pointers and inconsistent masks are rejected on the host; no device is touched.
    d = b.linear_desc(8, 16, 16, 4, b.LRD_F32)
    assert b._lib.lrd_linear_fwd(ctypes.byref(d), None, None, None, None, None, None, 0, None, 0, None) == b.LRD_ERR_INVALID_ARG
    bad = b.linear_desc(8, 16, 16, 17, b.LRD_F32)
    assert b._lib.lrd_linear_fwd(ctypes.byref(bad), None, None, None, None, None, None, 0, None, 0, None) == b.LRD_ERR_BAD_RANK
    assert b._lib.lrd_linear_bwd(ctypes.byref(d), None, None, None, None, None, None, None, None, None, 5, None, 0, None) == b.LRD_ERR_INVALID_ARG
    with pytest.raises(b.LrdError):
        b.lrd_set_path(17)
    b.lrd_set_path(b.LRD_PATH_AUTO)


def test_misaligned_pointers_are_rejected_before_any_launch():
    """Every entry point checks its base pointers against the element size on the host (odd addresses for bf16,
    addresses off a multiple of 4 for fp32) and returns LRD_ERR_ALIGNMENT without touching a device."""
    P = ctypes.c_void_p
    ok, odd, off2 = 0x7F0000001000, 0x7F0000001001, 0x7F0000001002
    for dt, bad in ((b.LRD_BF16, odd), (b.LRD_F32, off2), (b.LRD_F32, odd)):
        d = b.linear_desc(8, 16, 16, 4, dt)
        assert b._lib.lrd_linear_fwd(ctypes.byref(d), P(ok), P(bad), P(ok), None, P(ok), P(ok), 0, P(ok), 1 << 20, None) == b.LRD_ERR_ALIGNMENT
        assert b._lib.lrd_dense_fwd(ctypes.byref(d), P(bad), P(ok), None, P(ok), None, 0, None) == b.LRD_ERR_ALIGNMENT
        assert b._lib.lrd_dense_fwd(ctypes.byref(d), P(ok), P(ok), P(bad), P(ok), None, 0, None) == b.LRD_ERR_ALIGNMENT
        assert b._lib.lrd_dense_bwd(ctypes.byref(d), P(ok), P(ok), P(ok), P(ok), P(bad), None, P(ok), 1 << 20, None) == b.LRD_ERR_ALIGNMENT
        assert b._lib.lrd_dense_bwd(ctypes.byref(d), P(ok), P(ok), P(ok), None, P(ok), P(bad), P(ok), 1 << 20, None) == b.LRD_ERR_ALIGNMENT
        t = b.tucker2_desc(1, 4, 4, 8, 8, 4, 4, dt)
        assert b._lib.lrd_tucker2_fwd(ctypes.byref(t), P(ok), P(ok), P(bad), P(ok), None, P(ok), P(ok), P(ok), 0, P(ok), 1 << 20,
                                      None) == b.LRD_ERR_ALIGNMENT
        assert b._lib.lrd_tucker2_fwd(ctypes.byref(t), P(ok), P(ok), P(ok), P(ok), P(bad), P(ok), P(ok), P(ok), 0, P(ok), 1 << 20,
                                      None) == b.LRD_ERR_ALIGNMENT
        assert b._lib.lrd_tucker2_bwd(ctypes.byref(t), P(ok), P(ok), P(ok), P(ok), P(ok), P(ok), P(ok), P(ok), P(ok), P(ok), P(ok),
                                      P(bad), 0, P(ok), 1 << 20, None) == b.LRD_ERR_ALIGNMENT


def test_rank_search_bit_exact_against_oracle():
    """Algorithm 1 on synthetic step-time curves: the library's host routine and the oracle pick the same rank
    and take the same keep-the-original decision (staircases, ties, flat and monotone curves, one point)."""
    import numpy as np
    rng = np.random.default_rng(77)
    curves = [np.array([1.0 if r <= 256 else 1.15 for r in range(250, 263)]), np.array([1.0, 1.0, 1.3, 1.3, 1.3, 1.4, 1.4]),
              np.linspace(1.0, 2.0, 11), np.ones(9), np.array([3.0]), np.array([2.0, 1.0]), np.array([1.0, 2.0])]
    for _ in range(300):
        n = int(rng.integers(1, 40))
        kind = int(rng.integers(0, 3))
        if kind == 0:        # few distinct levels: many ties
            curves.append(rng.integers(1, 5, size=n).astype(np.float64))
        elif kind == 1:      # noisy rising curve with cliffs at multiples of 8
            r = np.arange(n)
            curves.append(1.0 + 0.01 * r + 0.2 * (r // 8) + 0.005 * rng.standard_normal(n))
        else:
            curves.append(rng.random(n))
    for t in curves:
        for T in (0.5, float(np.median(t)), 10.0):
            for floor in (0.0, 0.02, 0.1, 0.5):
                want = o.rank_search(t, 100, T, floor)
                got = b.lrd_rank_search(t, 100, T, floor)
                assert got == want, (t, T, floor, got, want)
        for floor in (0.0, 0.02, 0.1):
            assert b.lrd_rank_multiple(t, 100, floor) == o.rank_multiple(t, 100, floor)
    with pytest.raises(b.LrdError):
        b.lrd_rank_search([], 100, 1.0)
    with pytest.raises(b.LrdError):
        b.lrd_rank_search([1.0, 2.0], 0, 1.0)
    with pytest.raises(b.LrdError):
        b.lrd_rank_search([1.0, 2.0], 100, 1.0, -0.5)


def test_rank_search_with_a_noise_floor_picks_the_cliff_not_the_first_wiggle():
    """A staircase with the paper's 15 % step at 256 and at 248 under 1 % timer noise: the plain reading stops at the
    first wiggle below the starting rank, the reading with a noise floor picks 256, the multiple comes out as 8, and a
    flat noisy curve keeps the starting rank."""
    import numpy as np
    rng = np.random.default_rng(5)
    R_min, R = 240, 263
    ranks = np.arange(R_min, R + 1)
    clean = np.where(ranks <= 248, 0.85, np.where(ranks <= 256, 1.0, 1.15))
    hits = 0
    for trial in range(50):
        t = clean * (1.0 + 0.01 * rng.standard_normal(ranks.shape[0]))
        for fn in (lambda *a: o.rank_search(*a), lambda *a: b.lrd_rank_search(*a)):
            assert fn(t, R_min, 2.0, 0.05) == (256, True)
        hits += o.rank_search(t, R_min, 2.0)[0] == 256
        assert o.rank_multiple(t, R_min, 0.05) == 8 == b.lrd_rank_multiple(t, R_min, 0.05)
        flat = 1.0 + 0.01 * rng.standard_normal(ranks.shape[0])
        assert o.rank_search(flat, R_min, 2.0, 0.05)[0] == R == b.lrd_rank_search(flat, R_min, 2.0, 0.05)[0]
        assert o.rank_multiple(flat, R_min, 0.05) == 1
    assert hits < 25          # the plain reading mostly stops at timer noise: this is what the floor is for


def test_rank_formulas_of_the_search_driver_match_the_oracle():
    """The driver's own Eq. 5 / Eq. 6 and its fully-connected analogue against the oracle's, on a grid; and the
    paper's worked example."""
    from paper_2309_03824_b200 import rank_search as rs        # imports torch, makes no CUDA call at import
    assert rs.tucker_rank(512, 512, 3, 2) == 309 and rs.tucker_rank(512, 512, 3, 3) == o.tucker_rank_min(512, 512, 3, 2)
    assert b.lrd_tucker_rank(512, 512, 3, 2) == (309, 309) and b.lrd_tucker_rank_min(512, 512, 3, 2) == 244
    for C in (16, 64, 96, 256, 512, 2048):
        for S in (16, 48, 256, 512, 1024):
            for alpha in (2, 3, 4, 8, 2.5):
                for k in (1, 3, 5):
                    for beta in (1.0, 0.5, 2.0):
                        assert b.lrd_tucker_rank(C, S, k, alpha, beta) == o.tucker_rank(C, S, k, alpha, beta), (C, S, k, alpha, beta)
                        assert b.lrd_tucker_rank_min(C, S, k, alpha, beta) == o.tucker_rank_min(C, S, k, alpha, beta)
                assert b.lrd_svd_rank(C, S, alpha) == o.svd_rank(C, S, alpha)
                assert rs.tucker_rank(C, S, 3, alpha) == max(o.tucker_rank(C, S, 3, alpha)[0], 1), (C, S, alpha)
                assert rs.fc_rank(C, S, alpha) == max(o.svd_rank(C, S, alpha), 1), (C, S, alpha)
    assert b.lrd_svd_rank(0, 4, 2) < 0 and b.lrd_tucker_rank(4, 4, 3, 0.0)[0] < 0
