"""Pins for the oracle's page-interleaved CCL layout (strip g's j-th chunk stored as chunk j*G + g).  No GPU."""
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle as orc
from test_oracle_traffic import desc, B_, C_, REM

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def inter(R, Cc, P, S, e=2, part=orc.PART_COLS):
    return orc.Mat(R, Cc, e, P, part, orc.CCL_INTERLEAVED, S)


def test_hand_example():
    rows = [l.split() for l in open(os.path.join(GOLD, "fig4a_interleaved_index.txt")) if l.strip() and not l.startswith("#")]
    hdr = {k: int(v) for k, v in rows[:4]}
    table = np.array(rows[4:], dtype=np.int64)
    m = inter(hdr["K"], hdr["N"], hdr["G"], hdr["CHUNK"] * 2)
    np.testing.assert_array_equal(orc.map_table(m), table)
    # chunk c of the buffer belongs to strip c mod G
    chip = np.repeat(np.arange(2), 4)[None, :].repeat(4, 0)
    owner_of_chunk = np.empty(4, dtype=np.int64)
    owner_of_chunk[table.reshape(-1) // 8] = chip.reshape(-1)
    np.testing.assert_array_equal(owner_of_chunk, [0, 1, 0, 1])


@pytest.mark.parametrize("R,Cc,P,S,e,part", [(4, 8, 2, 16, 2, 2), (7, 24, 3, 64, 2, 2), (33, 96, 4, 256, 1, 2), (12, 40, 4, 48, 4, 1),
                                             (130, 384, 4, 4096, 2, 2), (64, 200, 2, 64, 2, 2), (9, 40, 5, 16, 2, 2)])
def test_is_the_page_permutation_of_aligned_ccl(R, Cc, P, S, e, part):
    """Independent definition: take CCL with strips aligned to S (layout CCL), view the buffer as [G][chunks][S]
    and transpose the first two axes."""
    dt = {1: np.uint8, 2: np.uint16, 4: np.uint32}[e]
    x = np.random.default_rng(0).integers(1, 200, size=(R, Cc)).astype(dt)
    aligned = orc.repack(orc.Mat(R, Cc, e, P, part, orc.CCL, S), x, 0)
    got = orc.repack(orc.Mat(R, Cc, e, P, part, orc.CCL_INTERLEAVED, S), x, 0)
    per = S // e
    chunks = aligned.size // (P * per)
    want = aligned.reshape(P, chunks, per).transpose(1, 0, 2).reshape(-1)
    np.testing.assert_array_equal(got, want)
    assert orc.buffer_bytes(inter(R, Cc, P, S, e, part)) == aligned.size * e
    # round trip, injective map, inverse with padding holes
    m = inter(R, Cc, P, S, e, part)
    np.testing.assert_array_equal(orc.repack(m, got, 1).reshape(R, Cc), x)
    t = orc.map_table(m)
    assert len(np.unique(t)) == R * Cc
    hit = np.zeros(got.size, dtype=bool)
    hit[t.reshape(-1)] = True
    for off in range(got.size):
        rc, r, c = orc.map_inverse(m, off)
        assert (rc == 0 and t[r, c] == off) if hit[off] else rc == -2
    assert (got[~hit] == 0).all()                                       # padding is zero


def test_rejects_missing_chunk_size():
    with pytest.raises(ValueError):
        orc.map_table(inter(4, 8, 2, 0))
    with pytest.raises(ValueError):
        orc.strip_stride(inter(4, 8, 2, 16))


@pytest.mark.parametrize("P,S", [(2, 4096), (4, 4096), (4, 256), (8, 64), (3, 48)])
def test_literal_round_robin_is_local_on_interleaved_ccl(P, S):
    """The claim of Sec. 3.3 / 4.1: address-bit round-robin at the interleave granularity places every strip on its chiplet."""
    M, N, K = 256, 96 * P, 40                                            # strips are not a whole number of chunks
    d = desc(M, N, K, P, S, ("row", "ccl", "ccl"), (orc.PLACE_RR,) * 3, align=S)
    d.B.layout = d.C.layout = orc.CCL_INTERLEAVED
    for level in ("elem", "runs"):
        r = orc.traffic(d, level=level)
        assert r["totals"][B_, REM] == 0 and r["totals"][C_, REM] == 0
    np.testing.assert_array_equal(orc.traffic(d, level="elem")["per_cta"], orc.traffic(d, level="runs")["per_cta"])
    # the same buffers under a page size that differs from the chunk size are no longer fully local
    d.page_bytes = S * 2
    r2 = orc.traffic(d, level="runs")
    assert r2["totals"][B_, REM] > 0
    np.testing.assert_array_equal(orc.traffic(d, level="elem")["per_cta"], r2["per_cta"])
    # block placement on the interleaved buffer is what literal round-robin is on plain CCL: (P-1)/P remote
    d.page_bytes = S
    d.place[1] = orc.PLACE_BLOCK
    r3 = orc.traffic(d, level="runs")
    assert r3["totals"][B_, REM] > 0


@pytest.mark.parametrize("S,page", [(64, 64), (64, 16), (48, 96), (256, 4096)])
def test_run_level_equals_element_level(S, page):
    for lay in (("row", "ccl", "ccl"), ("ccl", "ccl", "ccl")):
        for kw in (dict(), dict(b_trans=1), dict(a_trans=1), dict(assign=orc.ASSIGN_M, BM=16, BN=64)):
            d = desc(128, 256, 72, 4, page, lay, (orc.PLACE_RR, orc.PLACE_BEST, orc.PLACE_BLOCK), align=S, **kw)
            for m in (d.A, d.B, d.C):
                if m.layout == orc.CCL:
                    m.layout = orc.CCL_INTERLEAVED
            el, ru = orc.traffic(d, level="elem"), orc.traffic(d, level="runs")
            np.testing.assert_array_equal(el["per_cta"], ru["per_cta"])
            for X in range(3):
                np.testing.assert_array_equal(el["per_page"][X], ru["per_page"][X])
                np.testing.assert_array_equal(el["owner"][X], ru["owner"][X])
