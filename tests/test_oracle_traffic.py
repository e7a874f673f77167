"""Pins for the oracle's remote-traffic count (Sec. 4.1 metric without the L2 filter).  No GPU."""
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle as orc

GOLD = os.path.join(os.path.dirname(__file__), "golden")
A_, B_, C_ = 0, 1, 2
LOC, REM = 0, 1


def desc(M, N, K, P, S, lay=("row", "row", "row"), place=(orc.PLACE_RR,) * 3, a_trans=0, b_trans=0, assign=orc.ASSIGN_N,
         BM=128, BN=128, strip_tiling=1, e=2, align=0, parts=None):
    """lay[X] in {"row", "ccl"}; the CCL split dimension follows the assignment unless parts is given."""
    d = orc.TrafficDesc()
    d.M, d.N, d.K, d.BM, d.BN = M, N, K, BM, BN
    shapes = [((K, M) if a_trans else (M, K)), ((N, K) if b_trans else (K, N)), (M, N)]
    if parts is None:
        if assign == orc.ASSIGN_M:
            parts = (orc.PART_COLS if a_trans else orc.PART_ROWS, orc.PART_NONE, orc.PART_ROWS)
        else:
            parts = (orc.PART_NONE, orc.PART_ROWS if b_trans else orc.PART_COLS, orc.PART_COLS)
    mats = []
    for X in range(3):
        ccl = lay[X] == "ccl" and parts[X] != orc.PART_NONE
        mats.append(orc.Mat(shapes[X][0], shapes[X][1], e, P, parts[X] if ccl else orc.PART_NONE,
                            orc.CCL if ccl else orc.ROWMAJOR, align if ccl else 0))
    d.A, d.B, d.C = mats
    d.a_trans, d.b_trans, d.P, d.page_bytes = a_trans, b_trans, P, S
    d.place[0], d.place[1], d.place[2] = place
    d.assign, d.strip_tiling = assign, strip_tiling
    return d


def test_hand_enumerated_tiny_case():
    rows = [l.split() for l in open(os.path.join(GOLD, "tiny_traffic.txt")) if l.strip() and not l.startswith("#")]
    cases = {
        "row/rr": desc(4, 8, 4, 2, 16, BM=4, BN=4),
        "ccl/block": desc(4, 8, 4, 2, 16, ("row", "ccl", "ccl"), (orc.PLACE_RR, orc.PLACE_BLOCK, orc.PLACE_BLOCK), BM=4, BN=4),
        "ccl/rr": desc(4, 8, 4, 2, 16, ("row", "ccl", "ccl"), BM=4, BN=4),
        "row/best": desc(4, 8, 4, 2, 16, place=(orc.PLACE_BEST,) * 3, BM=4, BN=4),
    }
    res = {k: orc.traffic(v, level="elem") for k, v in cases.items()}
    res_runs = {k: orc.traffic(v, level="runs") for k, v in cases.items()}
    for case, op, cta, loc, rem in rows:
        X = "ABC".index(op)
        for r in (res, res_runs):
            assert r[case]["per_cta"].shape == (2, 3, 2)
            assert tuple(r[case]["per_cta"][int(cta), X]) == (int(loc), int(rem)), (case, op, cta)
    # owners written out: CCL + block placement = the strip's chiplet
    np.testing.assert_array_equal(res["ccl/block"]["owner"][B_], [0, 0, 1, 1])
    np.testing.assert_array_equal(res["row/rr"]["owner"][B_], [0, 1, 0, 1])
    np.testing.assert_array_equal(res["row/best"]["owner"][B_], [0, 0, 0, 0])      # ties -> lowest chiplet
    np.testing.assert_array_equal(res["row/rr"]["per_page"][B_], np.full((4, 2), 8))


SHAPES = [
    dict(M=130, N=384, K=96, P=4, S=256),
    dict(M=130, N=384, K=96, P=2, S=4096),
    dict(M=64, N=200, K=40, P=2, S=16),                               # w = 100: not a multiple of 8
    dict(M=96, N=96, K=64, P=3, S=64, BM=32, BN=32),
    dict(M=256, N=768, K=128, P=4, S=4096, b_trans=1),
    dict(M=120, N=256, K=72, P=4, S=128, a_trans=1),
    dict(M=128, N=256, K=64, P=8, S=512, assign=orc.ASSIGN_M, BM=16, BN=64),
    dict(M=100, N=240, K=48, P=2, S=1 << 21),                         # one page holds everything
    dict(M=130, N=384, K=96, P=4, S=256, strip_tiling=0),
]
LAYS = [("row", "row", "row"), ("row", "ccl", "ccl"), ("ccl", "ccl", "ccl")]
PLACES = [(orc.PLACE_RR,) * 3, (orc.PLACE_BLOCK,) * 3, (orc.PLACE_BEST,) * 3, (orc.PLACE_RR, orc.PLACE_BLOCK, orc.PLACE_BEST)]


def touched_bytes(d, tiles):
    e = d.A.elem_bytes
    rows, cols = tiles[:, 1] - tiles[:, 0], tiles[:, 3] - tiles[:, 2]
    return np.stack([rows * d.K * e, d.K * cols * e, rows * cols * e], axis=1)


@pytest.mark.parametrize("shape", SHAPES)
@pytest.mark.parametrize("lay", LAYS)
@pytest.mark.parametrize("place", PLACES)
def test_invariants_and_run_level_equals_element_level(shape, lay, place):
    for align in (0, 1024):
        d = desc(lay=lay, place=place, align=align, **shape)
        el = orc.traffic(d, level="elem")
        ru = orc.traffic(d, level="runs")
        for k in ("per_cta", "totals"):
            np.testing.assert_array_equal(el[k], ru[k])
        for X in range(3):
            np.testing.assert_array_equal(el["per_page"][X], ru["per_page"][X])
            np.testing.assert_array_equal(el["owner"][X], ru["owner"][X])
        tiles = orc.traffic_tiles(d)
        # local + remote = bytes the CTA touches, per operand
        np.testing.assert_array_equal(el["per_cta"].sum(axis=2), touched_bytes(d, tiles).astype(np.uint64))
        # sum over CTAs = sum over pages and chiplets = totals
        for X in range(3):
            assert el["per_cta"][:, X].sum() == el["per_page"][X].sum() == el["totals"][X].sum()
        # the partition of C covers it once
        assert el["totals"][C_].sum() == d.M * d.N * 2
        # per-page demand never exceeds the page
        for X in range(3):
            assert el["per_page"][X].sum(axis=1).max() <= d.page_bytes * max(len(tiles), 1)


def test_p1_has_no_remote_and_single_page_rule():
    d = desc(130, 384, 96, 1, 256)
    assert orc.traffic(d)["totals"][:, REM].sum() == 0
    d = desc(100, 240, 48, 2, 1 << 21)                                # S >= buffer: one page, owner 0
    r = orc.traffic(d)
    tiles = orc.traffic_tiles(d)
    tb = touched_bytes(d, tiles)
    np.testing.assert_array_equal(r["per_cta"][:, :, REM], (tb * (tiles[:, 4:5] != 0)).astype(np.uint64))


@pytest.mark.parametrize("P,S", [(2, 4096), (4, 4096), (4, 256), (8, 64)])
def test_central_claim_ccl_block_has_no_remote_on_split_operands(P, S):
    # strips that are a whole number of pages: every page has one consumer chiplet  (Sec. 3.1, 3.2)
    M, N, K = 256, 2048, 64
    d = desc(M, N, K, P, S, ("row", "ccl", "ccl"), (orc.PLACE_RR, orc.PLACE_BLOCK, orc.PLACE_BLOCK))
    assert (K * (N // P) * 2) % S == 0 and (M * (N // P) * 2) % S == 0
    r = orc.traffic(d, level="runs")
    assert r["totals"][B_, REM] == 0 and r["totals"][C_, REM] == 0
    assert r["totals"][B_, LOC] == (M // 128) * K * N * 2
    # literal round-robin on the same CCL buffers spreads each strip over all chiplets: (P-1)/P remote
    d2 = desc(M, N, K, P, S, ("row", "ccl", "ccl"))
    r2 = orc.traffic(d2, level="runs")
    assert Fraction(int(r2["totals"][B_, REM]), int(r2["totals"][B_].sum())) == Fraction(P - 1, P)
    # unaligned packed strips + padding to the page size restore the claim
    d3 = desc(M, 2048 - 64 * P, K + 1, P, S, ("row", "ccl", "ccl"), (orc.PLACE_RR, orc.PLACE_BLOCK, orc.PLACE_BLOCK), align=S)
    r3 = orc.traffic(d3, level="runs")
    assert r3["totals"][B_, REM] == 0 and r3["totals"][C_, REM] == 0


def test_closed_form_llama_gateup_rowmajor_rr():
    # B [8192 x 57344] bf16 row-major, 4 KB round-robin, P = 4: a row is 28 pages, a strip 7 page-columns,
    # owner(page j of a row) = j mod 4, so exactly 2 of every strip's 7 page-columns are local: remote = 5/7.
    M, N, K = 256, 57344, 8192
    r = orc.traffic(desc(M, N, K, 4, 4096), level="runs")
    tot = (M // 128) * K * N * 2
    assert int(r["totals"][B_].sum()) == tot
    assert Fraction(int(r["totals"][B_, REM]), tot) == Fraction(5, 7)
    assert tot * 32 == 60_129_542_144 and tot * 32 * 5 // 7 == 42_949_672_960   # the M = 8192 figures (64 tile rows)
    # P = 2: remote exactly one half
    r = orc.traffic(desc(128, N, 1024, 2, 4096), level="runs")
    assert Fraction(int(r["totals"][B_, REM]), int(r["totals"][B_].sum())) == Fraction(1, 2)


def test_closed_form_llama_down_rowmajor_rr():
    # B [K x 8192]: a row is 4 pages.  P = 4: w = 2048 elements = one page, owner = g -> remote 0.
    for P, frac in [(4, Fraction(0)), (2, Fraction(1, 2)), (8, Fraction(7, 8))]:
        r = orc.traffic(desc(128, 8192, 512, P, 4096), level="runs")
        assert Fraction(int(r["totals"][B_, REM]), int(r["totals"][B_].sum())) == frac, P


@pytest.mark.parametrize("P", [2, 4, 8])
def test_closed_form_qwen_down_rowmajor_rr(P):
    # Wd [768 x 2048]: a row is exactly one 4 KB page, owner = k mod P -> remote (P-1)/P
    r = orc.traffic(desc(256, 2048, 768, P, 4096), level="runs")
    assert Fraction(int(r["totals"][B_, REM]), int(r["totals"][B_].sum())) == Fraction(P - 1, P)


def test_closed_form_fig3a_best_placement_cannot_fix_rowmajor():
    # Fig. 3(a): fused gate/up width 1536, bf16, 4 chiplets, 4 KB pages.  The ownership pattern repeats
    # every 3 pages (4 rows); the best owner keeps 768, 640, 768 of each page's 2048 elements.
    r = orc.traffic(desc(128, 1536, 64, 4, 4096, place=(orc.PLACE_BEST,) * 3), level="elem")
    assert Fraction(int(r["totals"][B_, REM]), int(r["totals"][B_].sum())) == Fraction(31, 48)
    np.testing.assert_array_equal(r["owner"][B_][:3], [0, 1, 3])


def test_shared_operand_and_ratio():
    # A row-major [M x K] under RR with K*e a multiple of S*P: every CTA sees (P-1)/P of A remote
    P = 4
    d = desc(256, 2048, 8192, P, 4096, ("row", "ccl", "ccl"), (orc.PLACE_RR, orc.PLACE_BLOCK, orc.PLACE_BLOCK))
    r = orc.traffic(d, level="runs")
    a = r["per_cta"][:, A_]
    assert (a[:, REM] * 1 == a.sum(axis=1) * (P - 1) // P).all()


def test_transposed_storage_of_b_is_coarse():
    # B stored [N x K] (column-major B): an N-split is a split along stored rows, already contiguous (Sec. 2.2),
    # so block placement on the plain row-major buffer is local whenever strips are whole pages.
    d = desc(128, 512, 256, 4, 4096, place=(orc.PLACE_BLOCK,) * 3, b_trans=1)
    r = orc.traffic(d, level="elem")
    assert r["totals"][B_, REM] == 0


def test_explicit_assignment_and_bad_descriptors():
    d = desc(8, 8, 4, 2, 16, BM=4, BN=4, assign=orc.ASSIGN_EXPLICIT)
    q = np.array([1, 0, 0, 1], dtype=np.int32)
    r = orc.traffic(d, explicit_q=q)
    tiles = orc.traffic_tiles(d, q)
    np.testing.assert_array_equal(tiles[:, 4], q)
    assert r["per_cta"].shape == (4, 3, 2)
    with pytest.raises(ValueError):
        orc.traffic(d, explicit_q=np.array([2, 0, 0, 1], dtype=np.int32))
    with pytest.raises(ValueError):
        orc.traffic(desc(8, 9, 4, 4, 16))          # strips of ceil(9/4) = 3 columns would leave the fourth chiplet none
    bad = desc(8, 8, 4, 2, 16)
    bad.A.rows = 9
    with pytest.raises(ValueError):
        orc.traffic(bad)


# ---------------------------------------------------------------- 2-D output partitions and ragged strips

def desc_2d(M, N, K, P, Pm, S, **kw):
    d = desc(M, N, K, P, S, assign=orc.ASSIGN_N, parts=(orc.PART_NONE,) * 3, **kw)
    d.assign, d.part_m = orc.ASSIGN_2D, Pm
    return d


def test_hand_enumerated_2d_partition():
    rows = [l.split() for l in open(os.path.join(GOLD, "tiny_traffic_2d.txt")) if l.strip() and not l.startswith("#")]
    cases = {"rr": desc_2d(4, 8, 4, 4, 2, 16, BM=2, BN=4), "best": desc_2d(4, 8, 4, 4, 2, 16, BM=2, BN=4, place=(orc.PLACE_BEST,) * 3)}
    for level in ("elem", "runs"):
        res = {k: orc.traffic(v, level=level) for k, v in cases.items()}
        for case, op, tile, loc, rem in rows:
            assert tuple(res[case]["per_cta"][int(tile), "ABC".index(op)]) == (int(loc), int(rem)), (case, op, tile)
    np.testing.assert_array_equal(orc.traffic_tiles(cases["rr"])[:, 4], [0, 1, 2, 3])
    np.testing.assert_array_equal(orc.traffic(cases["best"])["owner"][A_], [0, 2])
    np.testing.assert_array_equal(orc.traffic(cases["best"])["owner"][C_], [0, 0, 2, 2])


@pytest.mark.parametrize("M,N,K,P,S,BM,BN", [(128, 256, 64, 4, 256, 32, 32), (96, 384, 48, 8, 128, 16, 64), (130, 200, 40, 2, 64, 64, 64)])
def test_2d_partition_degenerates_to_strips(M, N, K, P, S, BM, BN):
    """part_m = 1 is the N-strip partition and part_m = P the M-strip partition, tile for tile."""
    for Pm, assign in ((1, orc.ASSIGN_N), (P, orc.ASSIGN_M)):
        if assign == orc.ASSIGN_M and (P - 1) * -(-M // P) >= M:
            continue
        a = orc.traffic(desc_2d(M, N, K, P, Pm, S, BM=BM, BN=BN), level="runs")
        b = orc.traffic(desc(M, N, K, P, S, assign=assign, parts=(orc.PART_NONE,) * 3, BM=BM, BN=BN), level="runs")
        for k in ("per_cta", "totals"):
            np.testing.assert_array_equal(a[k], b[k])


@pytest.mark.parametrize("kw", [dict(M=128, N=256, K=64, P=4, Pm=2, S=256, BM=32, BN=32), dict(M=120, N=200, K=40, P=6, Pm=3, S=64, BM=16, BN=32),
                                dict(M=130, N=384, K=96, P=8, Pm=2, S=512, BM=64, BN=64, strip_tiling=0),
                                dict(M=131, N=203, K=24, P=6, Pm=2, S=128, BM=32, BN=32)])
def test_2d_partition_invariants(kw):
    Pm = kw["Pm"]
    for place in PLACES:
        d = desc_2d(place=place, **kw)
        res, runs = orc.traffic(d, level="elem"), orc.traffic(d, level="runs")
        tiles = orc.traffic_tiles(d)
        np.testing.assert_array_equal(res["per_cta"], runs["per_cta"])
        np.testing.assert_array_equal(res["per_cta"].sum(axis=2), touched_bytes(d, tiles))
        Pn = d.P // Pm
        wM, wN = -(-d.M // Pm), -(-d.N // Pn)
        np.testing.assert_array_equal(tiles[:, 4], (tiles[:, 0] // wM) * Pn + tiles[:, 2] // wN)
        if d.strip_tiling:                               # no tile straddles a block
            assert ((tiles[:, 1] - 1) // wM == tiles[:, 0] // wM).all() and ((tiles[:, 3] - 1) // wN == tiles[:, 2] // wN).all()
        for X in range(3):
            assert res["per_page"][X].sum() == res["per_cta"][:, X].sum()
    with pytest.raises(ValueError):
        bad = desc_2d(**kw)
        bad.part_m = 5 if kw["P"] % 5 else 7
        orc.traffic(bad)


@pytest.mark.parametrize("N,P", [(200, 3), (1000, 7), (385, 4)])
def test_ragged_strips_in_the_counter(N, P):
    """N not a multiple of P: strips of ceil(N/P) columns and a narrower last one; element- and run-level counts agree, every
    byte is accounted for, tiles stay inside their strips, and CCL keeps each strip one contiguous block."""
    M, K, S = 96, 40, 256
    w = -(-N // P)
    for lay in LAYS:
        for place in PLACES[:3]:
            d = desc(M, N, K, P, S, lay, place, BM=32, BN=32)
            res, runs = orc.traffic(d, level="elem"), orc.traffic(d, level="runs")
            tiles = orc.traffic_tiles(d)
            np.testing.assert_array_equal(res["per_cta"], runs["per_cta"])
            np.testing.assert_array_equal(res["per_cta"].sum(axis=2), touched_bytes(d, tiles))
            np.testing.assert_array_equal(tiles[:, 4], tiles[:, 2] // w)
            assert ((tiles[:, 3] - 1) // w == tiles[:, 2] // w).all()
            assert sorted(set(tiles[:, 4])) == list(range(P))
    # CCL B: the bytes a strip's tiles read are exactly the strip's block [g K w, g K w + K w_g) of the buffer
    d = desc(M, N, K, P, S, ("row", "ccl", "row"), (orc.PLACE_RR,) * 3, BM=32, BN=32)
    pp = orc.traffic(d)["per_page"][B_]                  # [pages, P] bytes of each page demanded by each chiplet
    for g in range(P):
        lo, hi = g * K * w * 2, (g * K * w + K * min(w, N - g * w)) * 2
        touched = np.flatnonzero(pp[:, g])
        assert touched.min() == lo // S and touched.max() == (hi - 1) // S
        assert pp[:, g].sum() == (M // 32) * (hi - lo)
