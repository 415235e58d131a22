"""Algorithm 1 end to end on the GPU: the step-time curve is measured through the C ABI, the library's host
routine picks R_opt, and the oracle applied to the same measured curve must pick the same rank and take the
same keep-the-original decision (which ranks are fast is the hardware's business, not the test's)."""
import pytest

from oracle import lrd_oracle as o
from paper_2309_03824_b200 import binding as b
from paper_2309_03824_b200 import rank_search as rs

pytestmark = pytest.mark.gpu


def test_rank_search_on_measured_curve_matches_oracle():
    M, K, N = 512, 256, 320
    R, R_min = rs.fc_rank(K, N, 2), rs.fc_rank(K, N, 3)
    assert (R, R_min) == (71, 47) and R == o.svd_rank(K, N, 2) and R_min == o.svd_rank(K, N, 3)
    r_opt, use, curve, T, floor, mult = rs.search(M, K, N, R, R_min, iters=4)
    assert sorted(curve) == list(range(R_min, R + 1)) and all(v > 0 for v in curve.values()) and T > 0
    t = [curve[r] for r in range(R_min, R + 1)]
    assert floor >= rs.MIN_DROP
    assert (r_opt, use) == o.rank_search(t, R_min, T, floor)
    assert mult == o.rank_multiple(t, R_min, floor)
    assert R_min <= r_opt <= R
    assert b.lrd_check_device_status() == b.LRD_OK


def test_tucker_rank_search_on_measured_curve_matches_oracle():
    B, H, C, S = 2, 6, 48, 64
    R, R_min = rs.tucker_rank(C, S, 3, 2), rs.tucker_rank(C, S, 3, 3)
    assert (R, R_min) == (o.tucker_rank(C, S, 3, 2)[0], o.tucker_rank_min(C, S, 3, 2)) and R_min < R
    r_opt, use, curve, T, floor, mult = rs.search_tucker(B, H, H, C, S, R, R_min, iters=3)
    assert sorted(curve) == list(range(R_min, R + 1)) and all(v > 0 for v in curve.values()) and T > 0
    t = [curve[r] for r in range(R_min, R + 1)]
    assert (r_opt, use) == o.rank_search(t, R_min, T, floor) and R_min <= r_opt <= R
    assert mult == o.rank_multiple(t, R_min, floor)
    assert b.lrd_check_device_status() == b.LRD_OK
