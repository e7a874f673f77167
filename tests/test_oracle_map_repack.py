"""Pins for the oracle's address map (Eq. 1-3) and repack.  No GPU."""
import os

import numpy as np
import pytest
import torch

import oracle as orc

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def ccl_cols(R, Cc, P, e=2, align=0):
    return orc.Mat(R, Cc, e, P, orc.PART_COLS, orc.CCL, align)


def ccl_rows(R, Cc, P, e=2, align=0):
    return orc.Mat(R, Cc, e, P, orc.PART_ROWS, orc.CCL, align)


def test_fig4a_worked_example():
    rows = [l.split() for l in open(os.path.join(GOLD, "fig4a_ccl_index.txt")) if l.strip() and not l.startswith("#")]
    hdr = {k: int(v) for k, v in rows[:3]}
    table = np.array(rows[3:], dtype=np.int64)
    assert table.shape == (hdr["K"], hdr["N"])
    m = ccl_cols(hdr["K"], hdr["N"], hdr["G"])
    np.testing.assert_array_equal(orc.map_table(m), table)
    assert orc.map_offset(m, 1, 5) == 21           # row-major would give 13
    # interleave granularity: 4 elements in row-major, 16 in CCL (contiguous run of one chiplet)
    inv = np.empty(32, dtype=np.int64)
    chip = np.repeat(np.arange(2), 4)[None, :].repeat(4, 0)           # chiplet of column n
    inv[table.reshape(-1)] = chip.reshape(-1)
    assert (inv[:16] == 0).all() and (inv[16:] == 1).all()
    rm = chip.reshape(-1)                                              # row-major memory order
    assert max(len(list(g)) for g in np.split(rm, np.flatnonzero(np.diff(rm)) + 1)) == 4


@pytest.mark.parametrize("R,Cc,P", [(4, 8, 2), (7, 12, 3), (5, 200, 2), (64, 1536, 4), (33, 768, 8), (2048, 1536, 4), (768, 2048, 2)])
def test_bijection_and_strips_packed(R, Cc, P):
    m = ccl_cols(R, Cc, P)
    t = orc.map_table(m)
    flat = np.sort(t.reshape(-1))
    np.testing.assert_array_equal(flat, np.arange(R * Cc))            # bijection onto [0, R*C)
    w = Cc // P
    for g in range(P):                                                # strip g is exactly [g*K*w, (g+1)*K*w)
        s = t[:, g * w:(g + 1) * w]
        assert s.min() == g * R * w and s.max() == (g + 1) * R * w - 1
    assert orc.buffer_bytes(m) == R * Cc * 2


@pytest.mark.parametrize("R,Cc,P", [(4, 8, 2), (7, 12, 3), (64, 1536, 4), (16, 768, 8)])
def test_stride_form(R, Cc, P):
    """Sec. 3.3: the view (K, G, N/G) with strides (w, K*w, 1)."""
    w = Cc // P
    k, g, n = np.meshgrid(np.arange(R), np.arange(P), np.arange(w), indexing="ij")
    stride_form = (k * w + g * (R * w) + n * 1).reshape(R, Cc)
    np.testing.assert_array_equal(orc.map_table(ccl_cols(R, Cc, P)), stride_form)


def test_identity_cases():
    R, Cc = 12, 40
    rm = np.arange(R * Cc).reshape(R, Cc)
    np.testing.assert_array_equal(orc.map_table(orc.Mat(R, Cc)), rm)                        # Eq. 2
    np.testing.assert_array_equal(orc.map_table(ccl_cols(R, Cc, 1)), rm)                   # G = 1
    np.testing.assert_array_equal(orc.map_table(ccl_rows(R, Cc, 4)), rm)                   # split along rows: already contiguous
    np.testing.assert_array_equal(orc.map_table(orc.Mat(R, Cc, 2, 4, orc.PART_COLS, orc.ROWMAJOR)), rm)


def test_slice_sizes_of_sec_2_2():
    # widths 768, 4096, 14336; bf16; four chiplets -> row slices of 384 B, 2 KB, 7168 B
    for width, nbytes in [(768, 384), (4096, 2048), (14336, 7168)]:
        m = ccl_cols(3, width, 4)
        run = orc.map_offset(m, 1, 0) - orc.map_offset(m, 0, 0)       # elements between consecutive rows of one strip
        assert run * 2 == nbytes
        assert orc.map_offset(m, 0, width // 4) == 3 * (width // 4)   # next chiplet's slice starts a new strip
    # fused gate/up width 1536 over 4 chiplets -> 384-element slices (Fig. 3(a))
    assert orc.map_offset(ccl_cols(2, 1536, 4), 1, 0) == 384


@pytest.mark.parametrize("part", ["cols", "rows"])
@pytest.mark.parametrize("align", [64, 4096])
def test_aligned_strips_injective_and_inverse(part, align):
    R, Cc, P = 6, 36, 3
    m = ccl_cols(R, Cc, P, 2, align) if part == "cols" else ccl_rows(R, Cc, P, 2, align)
    t = orc.map_table(m)
    assert len(np.unique(t)) == R * Cc
    st = orc.strip_stride(m)
    assert (st * 2) % align == 0 and st * 2 >= R * Cc * 2 // P
    assert orc.buffer_bytes(m) == P * st * 2
    hit = np.zeros(P * st, dtype=bool)
    hit[t.reshape(-1)] = True
    for off in range(P * st):
        rc, r, c = orc.map_inverse(m, off)
        if hit[off]:
            assert rc == 0 and t[r, c] == off
        else:
            assert rc == -2                                           # padding hole
    assert orc.map_inverse(m, P * st)[0] == -1


def test_inverse_packed_roundtrip():
    m = ccl_cols(9, 40, 5)
    t = orc.map_table(m)
    for off in range(9 * 40):
        rc, r, c = orc.map_inverse(m, off)
        assert rc == 0 and t[r, c] == off


def test_rejects_bad_descriptors():
    with pytest.raises(ValueError):
        orc.map_table(ccl_cols(4, 9, 4))           # w = ceil(9/4) = 3: the fourth strip would be empty
    with pytest.raises(ValueError):
        orc.map_table(ccl_rows(4, 8, 3))           # h = 2: the third strip would be empty
    with pytest.raises(ValueError):
        orc.map_offset(ccl_cols(4, 8, 2), 4, 0)    # out of range
    with pytest.raises(ValueError):
        orc.map_table(orc.Mat(4, 8, 3))            # element size


# ---------------------------------------------------------------- widths the chiplet count does not divide

def test_ragged_worked_example():
    rows = [l.split() for l in open(os.path.join(GOLD, "ragged_ccl_index.txt")) if l.strip() and not l.startswith("#")]
    hdr = {k: int(v) for k, v in rows[:3]}
    table = np.array(rows[3:], dtype=np.int64)
    m = ccl_cols(hdr["K"], hdr["N"], hdr["G"])
    np.testing.assert_array_equal(orc.map_table(m), table)
    assert orc.buffer_bytes(m) == hdr["K"] * hdr["N"] * 2 and orc.strip_stride(m) == 9
    np.testing.assert_array_equal(orc.map_table(ccl_rows(3, 7, 2)), np.arange(21).reshape(3, 7))


@pytest.mark.parametrize("R,Cc,P", [(3, 7, 3), (4, 10, 4), (5, 200, 3), (64, 1537, 4), (33, 770, 8), (17, 9, 2), (6, 1000, 7)])
def test_ragged_bijection_strips_and_slices(R, Cc, P):
    """Packed ragged CCL is a bijection onto [0, R*C); strip g is the contiguous block after the g strips before it and
    holds, row-major, the column slice [g w, min(C, (g+1) w)) -- written here with numpy slices, not with the map."""
    m = ccl_cols(R, Cc, P)
    t = orc.map_table(m)
    np.testing.assert_array_equal(np.sort(t.reshape(-1)), np.arange(R * Cc))
    w = -(-Cc // P)
    x = _rand_u16(R, Cc, seed=R + Cc)
    want = np.concatenate([x[:, g * w:min(Cc, (g + 1) * w)].reshape(-1) for g in range(P)])
    np.testing.assert_array_equal(orc.repack(m, x, 0), want)
    np.testing.assert_array_equal(orc.repack(m, orc.repack(m, x, 0), 1).reshape(R, Cc), x)
    for off in range(0, R * Cc, max(1, R * Cc // 97)):
        rc, r, c = orc.map_inverse(m, off)
        assert rc == 0 and t[r, c] == off
    # split along rows: strips of ceil(R/P) whole rows stay where they are
    if (P - 1) * -(-R // P) < R:
        np.testing.assert_array_equal(orc.map_table(ccl_rows(R, Cc, P)), np.arange(R * Cc).reshape(R, Cc))


@pytest.mark.parametrize("R,Cc,P,align", [(3, 7, 3, 64), (5, 200, 3, 4096), (9, 1537, 4, 256)])
def test_ragged_aligned_strips(R, Cc, P, align):
    """Aligned strips: every strip base is a multiple of the alignment, the map stays injective, padding holes invert to -2
    and the repack writes zeros there."""
    m = ccl_cols(R, Cc, P, align=align)
    t = orc.map_table(m)
    w = -(-Cc // P)
    st = orc.strip_stride(m)
    assert (st * 2) % align == 0 and st >= R * w
    assert len(np.unique(t)) == R * Cc
    for g in range(P):
        assert t[0, g * w] == g * st
    n = orc.buffer_bytes(m) // 2
    assert n == (P - 1) * st + -(-(R * (Cc - (P - 1) * w) * 2) // align) * align // 2
    x = np.random.default_rng(1).integers(1, 65536, size=(R, Cc), dtype=np.uint16)
    buf = orc.repack(m, x, 0)
    used = np.zeros(n, dtype=bool)
    used[t.reshape(-1)] = True
    assert (buf[~used] == 0).all() and (buf[used] != 0).all()
    holes = np.flatnonzero(~used)
    for off in holes[:: max(1, len(holes) // 50)]:
        assert orc.map_inverse(m, int(off))[0] == -2


def test_ragged_interleaved_is_a_chunk_permutation_of_aligned():
    """Page-interleaved ragged CCL: chunk j of strip g sits at chunk j*G + g; every strip gets the chunk count of the widest."""
    R, Cc, P, S = 5, 202, 3, 128
    mi = orc.Mat(R, Cc, 2, P, orc.PART_COLS, orc.CCL_INTERLEAVED, S)
    x = _rand_u16(R, Cc, seed=5)
    w = -(-Cc // P)
    chunks = -(-(R * w * 2) // S)
    buf = orc.repack(mi, x, 0).reshape(chunks, P, S // 2)
    for g in range(P):
        strip = x[:, g * w:min(Cc, (g + 1) * w)].reshape(-1)
        got = buf[:, g, :].reshape(-1)
        np.testing.assert_array_equal(got[:strip.size], strip)
        assert (got[strip.size:] == 0).all()
    np.testing.assert_array_equal(orc.repack(mi, buf.reshape(-1), 1).reshape(R, Cc), x)


# ---------------------------------------------------------------- repack

def _rand_u16(R, Cc, seed=0):
    return np.random.default_rng(seed).integers(0, 65536, size=(R, Cc), dtype=np.uint16)


@pytest.mark.parametrize("R,Cc,P", [(4, 8, 2), (130, 384, 4), (130, 384, 2), (5, 200, 2), (77, 96, 3), (256, 1536, 8)])
def test_repack_is_reshape_permute(R, Cc, P):
    x = _rand_u16(R, Cc, 1)
    got = orc.repack(ccl_cols(R, Cc, P), x, 0)
    want = torch.from_numpy(x.view(np.int16)).reshape(R, P, Cc // P).permute(1, 0, 2).contiguous().numpy().view(np.uint16)
    np.testing.assert_array_equal(got, want.reshape(-1))
    # equals P strided 2-D copies: strip g = columns [g*w, (g+1)*w) of every row
    w = Cc // P
    for g in range(P):
        np.testing.assert_array_equal(got[g * R * w:(g + 1) * R * w].reshape(R, w), x[:, g * w:(g + 1) * w])
    # a permutation: same multiset
    np.testing.assert_array_equal(np.sort(got), np.sort(x.reshape(-1)))
    # round trip
    np.testing.assert_array_equal(orc.repack(ccl_cols(R, Cc, P), got, 1).reshape(R, Cc), x)


def test_repack_p1_and_rows_are_memcpy():
    x = _rand_u16(33, 50, 2)
    np.testing.assert_array_equal(orc.repack(ccl_cols(33, 50, 1), x, 0), x.reshape(-1))
    np.testing.assert_array_equal(orc.repack(ccl_rows(33, 50, 3), x, 0), x.reshape(-1))


@pytest.mark.parametrize("e,dt", [(1, np.uint8), (2, np.uint16), (4, np.uint32)])
def test_repack_aligned_padding_is_zero(e, dt):
    R, Cc, P, align = 7, 24, 3, 256
    x = np.random.default_rng(3).integers(1, 200, size=(R, Cc)).astype(dt)    # no zeros in the payload
    m = ccl_cols(R, Cc, P, e, align)
    got = orc.repack(m, x, 0)
    st = orc.strip_stride(m)
    assert got.size == P * st
    w = Cc // P
    for g in range(P):
        np.testing.assert_array_equal(got[g * st:g * st + R * w].reshape(R, w), x[:, g * w:(g + 1) * w])
        assert (got[g * st + R * w:(g + 1) * st] == 0).all()
    np.testing.assert_array_equal(orc.repack(m, got, 1).reshape(R, Cc), x)
    mr = ccl_rows(6, Cc, P, e, align)
    xr = x[:6]
    gr = orc.repack(mr, xr, 0)
    sr = orc.strip_stride(mr)
    for g in range(P):
        np.testing.assert_array_equal(gr[g * sr:g * sr + 2 * Cc].reshape(2, Cc), xr[2 * g:2 * g + 2])
        assert (gr[g * sr + 2 * Cc:(g + 1) * sr] == 0).all()


def test_repack_transposed_hand_example_and_definition():
    # the Fig. 4(a) example with the operand stored as [N x K] = [8 x 4], src_t[n, k] = 4n + k: position index(k, n)
    # of the output holds 4n + k; by the table of the worked example the first strip (n < 4) is, row by row of k,
    # 0 4 8 12 | 1 5 9 13 | 2 6 10 14 | 3 7 11 15 and the second strip the same plus 16
    m = ccl_cols(4, 8, 2)
    got = orc.repack_transposed(m, np.arange(32, dtype=np.uint16).reshape(8, 4))
    first = np.array([0, 4, 8, 12, 1, 5, 9, 13, 2, 6, 10, 14, 3, 7, 11, 15], dtype=np.uint16)
    np.testing.assert_array_equal(got, np.concatenate([first, first + 16]))
    # in general it is the plain repack of the transposed array, padding included
    for R, Cc, P, e, dt, align, lay in ((130, 384, 4, 2, np.uint16, 0, orc.CCL), (7, 24, 3, 1, np.uint8, 256, orc.CCL),
                                        (33, 50, 5, 4, np.uint32, 0, orc.CCL), (64, 200, 2, 2, np.uint16, 40, orc.CCL_INTERLEAVED)):
        x = np.random.default_rng(5).integers(1, 200, size=(R, Cc)).astype(dt)
        for part in (orc.PART_COLS, orc.PART_ROWS):
            if part == orc.PART_ROWS and R % P:
                continue
            mm = orc.Mat(R, Cc, e, P, part, lay, align)
            np.testing.assert_array_equal(orc.repack_transposed(mm, np.ascontiguousarray(x.T)), orc.repack(mm, x, 0))
