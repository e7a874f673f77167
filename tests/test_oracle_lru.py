"""Pins of the oracle's finite-L2 traffic model (orc_traffic_lru): a hand-run access string, and the two limits in
which it must reduce to counts that are pinned elsewhere -- a one-line cache (nothing is ever reused: the uncached
count, in whole lines) and an unbounded cache (every chiplet fetches a line once: the ideal-L2 count).  No GPU."""
import os

import numpy as np
import pytest

import oracle as orc
from helpers import traffic_pair

HERE = os.path.dirname(os.path.abspath(__file__))


def test_hand_run():
    do, _ = traffic_pair(2, 2, 64, 1, 4096, BM=1, BN=1)
    for line in open(os.path.join(HERE, "golden", "lru_hand_run.txt")):
        if line.startswith("#") or not line.strip():
            continue
        sets, ways, a_bytes, b_bytes = (int(x) for x in line.split())
        t = orc.traffic_lru(do, orc.L2Model(sets * ways * 128, 128, ways, 0))
        assert (int(t[0].sum()), int(t[1].sum())) == (a_bytes, b_bytes), (sets, ways, t)
        assert int(t[2].sum()) == 2 * 2 * 2                         # C: every element written once


def test_wave_hand_run():
    do, _ = traffic_pair(2, 2, 64, 1, 4096, BM=1, BN=1)
    for line in open(os.path.join(HERE, "golden", "lru_wave_hand_run.txt")):
        if line.startswith("#") or not line.strip():
            continue
        sets, ways, wave, ks, a_bytes, b_bytes = (int(x) for x in line.split())
        t = orc.traffic_lru(do, orc.L2Model(sets * ways * 128, 128, ways, 0, 0, wave, ks))
        assert (int(t[0].sum()), int(t[1].sum())) == (a_bytes, b_bytes), (sets, ways, wave, ks, t)


def test_wave_shares_the_a_slice():
    """Closed form: a fully associative cache of 300 lines, one chiplet, tiles 128 x 128, K = 256 (bf16).  One CTA
    after the other, a tile's A rows (128 rows x 4 lines) and B columns (256 rows x 2 lines) are 512 lines each: no
    line survives to the next tile, so every tile fetches its whole A and B rectangle.  In waves of one tile row
    (4 CTAs) with k slices of 64, the 128 lines of an A slice come back after the 128 lines of one tile's B slice:
    they hit, and A is fetched once in all; B slices are private to a tile and return only a whole wave later."""
    M, N, K = 384, 512, 256
    do, _ = traffic_pair(M, N, K, 1, 4096, BM=128, BN=128)
    seq = orc.traffic_lru(do, orc.L2Model(300 * 128, 128, 300, 0))
    assert int(seq[0].sum()) == (N // 128) * M * K * 2 and int(seq[1].sum()) == (M // 128) * K * N * 2
    wav = orc.traffic_lru(do, orc.L2Model(300 * 128, 128, 300, 0, 0, 4, 64))
    assert int(wav[0].sum()) == M * K * 2 and int(wav[1].sum()) == (M // 128) * K * N * 2
    # a wave of two tile rows (8 CTAs): an A slice still returns after one B slice, while the B slice of a column
    # returns in the second tile row only after three other B slices and two A slices (640 lines): same counts
    w8 = orc.traffic_lru(do, orc.L2Model(300 * 128, 128, 300, 0, 0, 8, 64))
    np.testing.assert_array_equal(w8, wav)
    # ... and with room for all of that (4 B slices + 2 A slices = 768 lines) the second tile row of a wave finds
    # its B slices: B is fetched once per wave (rows 0-1, row 2) instead of once per tile row
    w8big = orc.traffic_lru(do, orc.L2Model(800 * 128, 128, 800, 0, 0, 8, 64))
    assert int(w8big[0].sum()) == M * K * 2 and int(w8big[1].sum()) == 2 * K * N * 2
    with pytest.raises(ValueError):
        orc.traffic_lru(do, orc.L2Model(300 * 128, 128, 300, 0, 0, 0, 64))     # a wave holds at least one CTA
    with pytest.raises(ValueError):
        orc.traffic_lru(do, orc.L2Model(300 * 128, 128, 300, 0, 0, 4, -1))


CASES = [
    # M, N, K, P, page, layouts, placement: every tile row segment is a whole number of 128-byte lines
    (256, 512, 128, 2, 4096, ("row", "row", "row"), (0, 0, 0)),
    (256, 512, 128, 2, 4096, ("row", "ccl", "ccl"), (0, 1, 1)),
    (384, 1024, 192, 4, 1024, ("row", "ccl", "ccl"), (0, 0, 0)),
    (256, 512, 128, 4, 4096, ("ccl", "row", "ccl"), (1, 0, 1)),
]


@pytest.mark.parametrize("M,N,K,P,S,lay,place", CASES)
@pytest.mark.parametrize("assign", [0, 1])
@pytest.mark.parametrize("traversal", [0, 1])
def test_limits(M, N, K, P, S, lay, place, assign, traversal):
    do, _ = traffic_pair(M, N, K, P, S, lay, place, assign=assign, BM=128, BN=64, align=S)
    plain = orc.traffic(do, level="runs")["totals"]
    ideal = orc.traffic_ideal_l2(do)
    one_line = orc.traffic_lru(do, orc.L2Model(128, 128, 1, traversal))
    np.testing.assert_array_equal(one_line, plain)                  # no reuse at all
    lines = sum(orc.buffer_bytes(m) for m in (do.A, do.B)) // 128
    unbounded = orc.traffic_lru(do, orc.L2Model(128 * 2 * lines, 128, 2 * lines, traversal))
    np.testing.assert_array_equal(unbounded, ideal)                 # each chiplet fetches a line once
    # more ways over the same sets never miss more (LRU stack inclusion), and the C row never changes
    prev = None
    for hashed in (0, 1):                                           # whatever the set index, as long as it is a function of the line
        prev = None
        for ways in (1, 2, 4, 16):
            t = orc.traffic_lru(do, orc.L2Model(8 * ways * 128, 128, ways, traversal, hashed))
            np.testing.assert_array_equal(t[2], plain[2])
            total = int(t[0].sum() + t[1].sum())
            assert int(ideal[0].sum() + ideal[1].sum()) <= total <= int(plain[0].sum() + plain[1].sum())
            if prev is not None:
                assert total <= prev
            prev = total
        np.testing.assert_array_equal(orc.traffic_lru(do, orc.L2Model(128, 128, 1, traversal, hashed)), plain)
    # both limits hold for waves in lockstep too (k slices of whole lines, so no line is shared by two slices)
    for wave, ks in ((3, 64), (1, 64), (5, 0)):
        np.testing.assert_array_equal(orc.traffic_lru(do, orc.L2Model(128, 128, 1, traversal, 0, wave, ks)), plain)
        np.testing.assert_array_equal(orc.traffic_lru(do, orc.L2Model(128 * 2 * lines, 128, 2 * lines, traversal, 1, wave, ks)), ideal)


def test_traversal_matters_and_rejections():
    # one chiplet, a cache that holds one tile row of A but not all of B: row-major order reuses A, column-major B
    do, _ = traffic_pair(512, 512, 256, 1, 4096, BM=128, BN=128)
    cap = 128 * 256 * 2 + 128 * 256 * 2 + 4096                     # one A tile row + one B tile column + a little
    cap -= cap % (128 * 16)
    row = orc.traffic_lru(do, orc.L2Model(cap, 128, 16, 0))
    col = orc.traffic_lru(do, orc.L2Model(cap, 128, 16, 1))
    assert row[0].sum() < col[0].sum() and row[1].sum() > col[1].sum()
    with pytest.raises(ValueError):
        orc.traffic_lru(do, orc.L2Model(1000, 128, 16, 0))         # capacity not a whole number of sets
    with pytest.raises(ValueError):
        orc.traffic_lru(do, orc.L2Model(8 << 20, 128, 16, 2))      # unknown traversal
    # a skewed index spreads a power-of-two stride over the sets: the column of lines 0, 64, 128, ... (pitch = sets)
    # all share set 0 under the plain index and thrash a 2-way set; skewed, they land in different sets
    ds, _ = traffic_pair(256, 128, 64, 1, 4096, BM=256, BN=128, b_trans=1)    # A [256 x 64]: one line per row, pitch one line
    one_set_plain = orc.traffic_lru(ds, orc.L2Model(2 * 128, 128, 2, 0, 0))     # 1 set: the index cannot matter
    one_set_hash = orc.traffic_lru(ds, orc.L2Model(2 * 128, 128, 2, 0, 1))
    np.testing.assert_array_equal(one_set_plain, one_set_hash)
    db, _ = traffic_pair(512, 512, 256, 2, 4096, place=(2, 2, 2))
    with pytest.raises(ValueError):
        orc.traffic_lru(db, orc.L2Model(8 << 20, 128, 16, 0))      # BEST placement is not modelled


# ---- the skewed set index (hash = 1), pinned by hand-worked cases -----------------------------------------------
def _skew_golden():
    H, cases, sets4 = {}, [], None
    for line in open(os.path.join(HERE, "golden", "lru_skew_index.txt")):
        f = line.split()
        if not f or f[0].startswith("#"):
            continue
        if f[0] == "H":
            H[int(f[1])] = (int(f[2], 16), int(f[3], 16), int(f[4]), int(f[5]))
        elif f[0] == "SETS4":
            sets4 = [int(x) for x in f[1:]]
        elif f[0] == "CASE":
            cases.append((f[1], *[int(x) for x in f[2:]]))
    return H, sets4, cases


def test_skew_golden_file_arithmetic_is_consistent():
    """The hand multiplication in the golden file, re-checked in exact integers (a check of the file, not of the oracle)."""
    H, sets4, _ = _skew_golden()
    for b, (prod, h, m4, m4096) in H.items():
        assert prod == (b * 0x9E3779B97F4A7C15) % (1 << 64) and h == prod >> 32 and m4 == h % 4 and m4096 == h % 4096
    assert sets4 == [(l % 4 + H[l // 4][2]) % 4 for l in range(16)]


@pytest.mark.parametrize("case", _skew_golden()[2], ids=lambda c: c[0])
def test_skewed_set_index_hand_cases(case):
    """Access strings whose hit / miss outcome depends on the set index: the totals worked out by hand in the golden file."""
    _, sets, hash_, M, N, K, BM, BN, bt, bstrips, balign, want_a, want_b = case
    d = orc.TrafficDesc()
    d.M, d.N, d.K, d.BM, d.BN = M, N, K, BM, BN
    d.A, d.C = orc.Mat(M, K, 2), orc.Mat(M, N, 2)
    if bstrips > 1:
        d.B = orc.Mat(N, K, 2, bstrips, orc.PART_ROWS, orc.CCL, balign) if bt else orc.Mat(K, N, 2, bstrips, orc.PART_COLS, orc.CCL, balign)
    else:
        d.B = orc.Mat(N, K, 2) if bt else orc.Mat(K, N, 2)
    d.a_trans, d.b_trans, d.P, d.page_bytes = 0, bt, 1, 16
    d.place[0] = d.place[1] = d.place[2] = orc.PLACE_RR
    d.assign, d.strip_tiling = orc.ASSIGN_N, 1
    t = orc.traffic_lru(d, orc.L2Model(sets * 16, 16, 1, 0, hash_, 1, 0))
    assert int(t[0, 0]) == want_a and int(t[0, 1]) == 0
    if want_b >= 0:
        assert int(t[1, 0]) == want_b
