"""Pins for the oracle's ideal-private-L2 remote-traffic count.  No GPU."""
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle as orc
from test_oracle_traffic import desc, A_, B_, C_, LOC, REM

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def test_hand_enumerated_case():
    rows = [l.split() for l in open(os.path.join(GOLD, "tiny_traffic_ideal_l2.txt")) if l.strip() and not l.startswith("#")]
    cases = {"row/rr": desc(8, 8, 4, 2, 16, BM=4, BN=4),
             "ccl/block": desc(8, 8, 4, 2, 16, ("row", "ccl", "ccl"), (orc.PLACE_RR, orc.PLACE_BLOCK, orc.PLACE_BLOCK), BM=4, BN=4)}
    res = {k: orc.traffic_ideal_l2(v) for k, v in cases.items()}
    for case, op, loc, rem in rows:
        assert tuple(res[case]["ABC".index(op)]) == (int(loc), int(rem)), (case, op)
    # without the L2 the B operand is counted once per tile: twice as much
    assert tuple(orc.traffic(cases["row/rr"])["totals"][B_]) == (64, 64)


@pytest.mark.parametrize("P", [1, 2, 4])
def test_bounds_and_special_cases(P):
    for lay in (("row", "row", "row"), ("row", "ccl", "ccl")):
        for place in ((0, 0, 0), (1, 1, 1)):
            d = desc(130, 96 * P, 40, P, 64, lay, place, BM=32, BN=32, align=64)
            ideal = orc.traffic_ideal_l2(d)
            full = orc.traffic(d)["totals"]
            assert (ideal <= full).all()                               # an L2 can only remove traffic
            np.testing.assert_array_equal(ideal[C_], full[C_])         # outputs are written once either way
            if P == 1:
                assert ideal[:, REM].sum() == 0
                # one chiplet reads every operand byte exactly once
                assert ideal[A_].sum() == 130 * 40 * 2 and ideal[B_].sum() == 40 * 96 * 2


def test_closed_forms_shared_and_private_operands():
    # N-partition, P = 4, 128x128 tiles.  A row-major under RR with K*e a multiple of S*P: every chiplet fetches all of A
    # once -> local |A|, remote (P-1)|A|.  B in CCL (whole pages per strip) + block placement: each strip fetched once by
    # its own chiplet -> local |B|, remote 0.
    M, N, K, P, S = 256, 1024, 2048, 4, 1024
    d = desc(M, N, K, P, S, ("row", "ccl", "ccl"), (orc.PLACE_RR, orc.PLACE_BLOCK, orc.PLACE_BLOCK))
    t = orc.traffic_ideal_l2(d)
    a_bytes, b_bytes = M * K * 2, K * N * 2
    assert tuple(t[A_]) == (a_bytes, (P - 1) * a_bytes)
    assert tuple(t[B_]) == (b_bytes, 0)
    # row-major B under RR, a row = 2 pages, strip = half a page: page owner = (2k + n/512) mod 4
    d2 = desc(M, N, K, P, S)
    t2 = orc.traffic_ideal_l2(d2)
    assert t2[B_].sum() == b_bytes                                     # still fetched once overall ...
    assert Fraction(int(t2[B_, REM]), b_bytes) == Fraction(3, 4)       # ... but three quarters of it from another chiplet


def test_explicit_assignment_and_best_is_rejected():
    d = desc(8, 8, 4, 2, 16, BM=4, BN=4, assign=orc.ASSIGN_EXPLICIT)
    t = orc.traffic_ideal_l2(d, explicit_q=np.array([0, 0, 0, 0], dtype=np.int32))
    assert t[:, REM].sum() > 0 and t[A_].sum() == 8 * 4 * 2 and t[B_].sum() == 4 * 8 * 2      # one chiplet: everything once
    with pytest.raises(ValueError):
        orc.traffic_ideal_l2(desc(8, 8, 4, 2, 16, place=(2, 2, 2), BM=4, BN=4))
