"""Pins for rank quantization, the rank formulas (Eq. 5, 6) and the freeze schedule (Algorithm 2)."""
import math
import os

import numpy as np
import pytest

from oracle import lrd_oracle as o

GOLDEN = {}
with open(os.path.join(os.path.dirname(__file__), "golden", "paper_values.txt")) as fh:
    for line in fh:
        line = line.split("#")[0].split()
        if len(line) == 2:
            GOLDEN[line[0]] = line[1]


def test_paper_worked_example_eq5():
    want = int(GOLDEN["tucker_rank_512_512_3_alpha2"])
    r1, r2 = o.tucker_rank(512, 512, 3, 2, 1.0)
    assert (r1, r2) == (want, want) == (309, 309)

    def ratio(r):
        return 512 * 512 * 9 / (512 * r + 9 * r * r + 512 * r)
    assert ratio(309) >= 2.0 > ratio(310)                          # truncation, not rounding
    # lower bound of the search (Eq. 6) sits where the paper's figure ends
    rmin = o.tucker_rank_min(512, 512, 3, 2, 1.0)
    assert rmin == 244
    assert int(GOLDEN["fig2_rank_low"]) <= rmin <= int(GOLDEN["fig2_rank_high"])


@pytest.mark.parametrize("C,S,k,alpha,beta", [(256, 256, 3, 2, 1.0), (64, 128, 3, 3, 1.0), (128, 64, 5, 2, 0.5),
                                                (512, 2048, 1, 4, 2.0)])
def test_tucker_rank_satisfies_parameter_budget(C, S, k, alpha, beta):
    r1, r2 = o.tucker_rank(C, S, k, alpha, beta)
    assert r2 == math.floor(beta * r1)
    params = lambda a: C * a + beta * k * k * a * a + beta * S * a     # with r2 = beta r1
    assert params(r1) <= C * S * k * k / alpha < params(r1 + 1)
    assert o.tucker_rank_min(C, S, k, alpha, beta) == o.tucker_rank(C, S, k, alpha + 1, beta)[0] <= r1


def test_svd_rank_formula():
    assert o.svd_rank(768, 768, 2) == 192 and o.svd_rank(1024, 1024, 2) == 256
    for C, S, a in [(768, 3072, 2), (100, 37, 3), (512, 512, 4)]:
        r = o.svd_rank(C, S, a)
        assert r * (C + S) <= C * S / a < (r + 1) * (C + S)


def test_quantize_paper_example_and_config_values():
    a, b = int(GOLDEN["efficient_rank_example_from"]), int(GOLDEN["efficient_rank_example_to"])
    for m in (8, 16, 32, 64, 128, 256):
        assert o.rank_quantize(a, m, o.ROUND_DOWN, 512, 512) == b
        assert o.rank_quantize(a, m, o.ROUND_NEAREST, 512, 512) == b
    assert o.rank_quantize(309, 32, o.ROUND_DOWN, 512, 512) == 288
    assert o.rank_quantize(309, 32, o.ROUND_UP, 512, 512) == 320
    ranks = [100, 250, 500, 750, 1000]
    assert [o.rank_quantize(r, 8, o.ROUND_UP, 4096, 4096) for r in ranks] == [104, 256, 504, 752, 1000]
    assert [o.rank_quantize(r, 64, o.ROUND_UP, 4096, 4096) for r in ranks] == [128, 256, 512, 768, 1024]
    assert [o.rank_quantize(r, 128, o.ROUND_UP, 4096, 4096) for r in ranks] == [128, 256, 512, 768, 1024]
    assert o.rank_quantize(88, 32, o.ROUND_UP, 256, 256) == 96
    for r in (192, 384, 256, 512):
        assert o.rank_quantize(r, 64, o.ROUND_UP, 768, 3072) == r


def test_quantize_exhaustive_against_one_line_definitions():
    K, N = 1500, 2048
    for m in (1, 8, 16, 32, 64, 128):
        cap = (min(K, N) // m) * m
        for r in range(1, 2049):
            up = o.rank_quantize(r, m, o.ROUND_UP, K, N)
            dn = o.rank_quantize(r, m, o.ROUND_DOWN, K, N)
            nr = o.rank_quantize(r, m, o.ROUND_NEAREST, K, N)
            assert up == min(max(math.ceil(r / m) * m, m), cap)
            assert dn == min(max(math.floor(r / m) * m, m), cap)
            assert nr == min(max(math.floor(r / m + 0.5) * m, m), cap)
            for q in (up, dn, nr):
                assert q % m == 0 and m <= q <= min(K, N)
                assert o.rank_quantize(q, m, o.ROUND_UP, K, N) == q      # idempotent
            assert up >= r or up == cap
            assert dn <= r or dn == m


def test_quantize_errors():
    for bad in [(0, 8, 0, 64, 64), (5, 0, 0, 64, 64), (5, 128, 0, 64, 64), (5, 8, 7, 64, 64), (5, 8, 0, 0, 64)]:
        with pytest.raises(ValueError):
            o.rank_quantize(*bad)


def test_sequential_freezing_truth_table():
    # L_r(0) is the first-applied sub-layer (V, or the first 1x1), L_r(1) the second (U, or the core).
    svd_frozen = {o.FREEZE_V: 0, o.FREEZE_U: 1}
    assert svd_frozen[o.freeze_for_epoch(0)] == int(GOLDEN["alg2_even_svd_frozen"])
    assert svd_frozen[o.freeze_for_epoch(1)] == int(GOLDEN["alg2_odd_svd_frozen"])
    tucker_frozen = {o.TK_FREEZE_FACTORS: "0,2", o.TK_FREEZE_CORE: "1"}
    assert tucker_frozen[o.tucker_freeze_for_epoch(0)] == GOLDEN["alg2_even_tucker_frozen"]
    assert tucker_frozen[o.tucker_freeze_for_epoch(1)] == GOLDEN["alg2_odd_tucker_frozen"]
    for e in range(0, 12):
        assert o.freeze_for_epoch(e) == o.freeze_for_epoch(e + 2) != o.freeze_for_epoch(e + 1)
        assert o.tucker_freeze_for_epoch(e) == o.tucker_freeze_for_epoch(e + 2) != o.tucker_freeze_for_epoch(e + 1)
        assert o.freeze_for_epoch(e) in (o.FREEZE_U, o.FREEZE_V)      # exactly one group frozen


def test_rank_search_reading_on_synthetic_curves():
    # staircase: ranks 250..256 cost 1.0, 257..262 cost 1.15 (the 257 -> 256 cliff of the paper's example)
    R_min, R = 250, 262
    t = np.array([1.0 if r <= 256 else 1.15 for r in range(R_min, R + 1)])
    assert o.rank_search(t, R_min, 2.0) == (256, True)
    assert o.rank_search(t, R_min, 0.9) == (256, False)            # the original layer is faster: keep it
    # two cliffs: the first one met when coming down from R wins
    t2 = np.array([1.0, 1.0, 1.3, 1.3, 1.3, 1.4, 1.4])
    assert o.rank_search(t2, 10, 5.0)[0] == 14
    # strictly linear curve has no interior peak: global argmax, largest rank on ties
    t3 = np.linspace(1.0, 2.0, 11)
    assert o.rank_search(t3, 100, 5.0)[0] in range(100, 110)
