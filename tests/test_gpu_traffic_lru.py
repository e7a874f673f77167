"""GPU parity, through the C ABI: ccl_traffic_lru (remote traffic behind a finite LRU L2 per chiplet) against the
oracle's run of the same model, bit for bit; and, at the benchmark's size, against what holds at any size."""
import os

import numpy as np
import pytest
import torch

import oracle as orc
from paper_2606_11718_b200 import binding as ccl
from helpers import traffic_pair

pytestmark = pytest.mark.gpu
HERE = os.path.dirname(os.path.abspath(__file__))


def run(dl, model):
    totals = torch.full((3, 2), -1, dtype=torch.int64, device="cuda")
    ccl.ccl_traffic_lru(dl, model, totals)
    return totals.cpu().numpy().astype(np.uint64)


def test_hand_run_on_the_gpu():
    do, dl = traffic_pair(2, 2, 64, 1, 4096, BM=1, BN=1)
    for line in open(os.path.join(HERE, "golden", "lru_hand_run.txt")):
        if line.startswith("#") or not line.strip():
            continue
        sets, ways, a_bytes, b_bytes = (int(x) for x in line.split())
        t = run(dl, ccl.L2Model(sets * ways * 128, 128, ways, 0))
        assert (int(t[0].sum()), int(t[1].sum()), int(t[2].sum())) == (a_bytes, b_bytes, 8)


def test_wave_hand_run_on_the_gpu():
    do, dl = traffic_pair(2, 2, 64, 1, 4096, BM=1, BN=1)
    for line in open(os.path.join(HERE, "golden", "lru_wave_hand_run.txt")):
        if line.startswith("#") or not line.strip():
            continue
        sets, ways, wave, ks, a_bytes, b_bytes = (int(x) for x in line.split())
        t = run(dl, ccl.L2Model(sets * ways * 128, 128, ways, 0, 0, wave, ks))
        assert (int(t[0].sum()), int(t[1].sum()), int(t[2].sum())) == (a_bytes, b_bytes, 8)


SHAPES = [
    # M, N, K, P, page, layouts, placement, BM, BN, a_trans, b_trans
    (256, 512, 128, 2, 4096, ("row", "row", "row"), (0, 0, 0), 128, 64, 0, 0),
    (256, 512, 128, 2, 4096, ("row", "ccl", "ccl"), (0, 1, 1), 128, 64, 0, 0),
    (384, 1024, 192, 4, 1024, ("row", "ccl", "ccl"), (0, 0, 0), 128, 128, 0, 0),
    (256, 512, 128, 4, 4096, ("ccl", "row", "ccl"), (1, 0, 1), 64, 128, 0, 0),
    (130, 384, 200, 4, 512, ("row", "ccl", "ccl"), (0, 1, 1), 128, 128, 0, 0),      # w = 96: 192-byte strip rows, ragged M and K
    (264, 768, 328, 3, 4096, ("row", "ccl", "ccl"), (0, 1, 1), 128, 128, 1, 0),     # A stored [K x M]
    (200, 512, 256, 2, 2048, ("row", "ccl", "ccl"), (0, 1, 1), 128, 128, 0, 1),     # B stored [N x K], split along rows
    (512, 2048, 1024, 4, 4096, ("row", "ccl", "ccl"), (0, 1, 1), 128, 128, 0, 0),   # many rows per B piece: the merged progressions
    (512, 2048, 1024, 4, 4096, ("row", "row", "row"), (0, 0, 0), 128, 128, 0, 0),
]
CACHES = [(128, 128, 1), (8 * 1024, 128, 4), (96 * 1024, 128, 16), (48 * 128 * 3, 128, 3), (64 * 1024, 64, 8), (1 << 20, 128, 16)]


@pytest.mark.parametrize("M,N,K,P,S,lay,place,BM,BN,at,bt", SHAPES)
@pytest.mark.parametrize("assign", [0, 1, 3])
def test_lru_bit_exact(M, N, K, P, S, lay, place, BM, BN, at, bt, assign):
    if assign == 3 and P < 4:
        pytest.skip("a 2-D partition needs at least 2 x 2 chiplets")
    do, dl = traffic_pair(M, N, K, P, S, lay, place, a_trans=at, b_trans=bt, assign=assign, BM=BM, BN=BN, align=S, part_m=2 if assign == 3 else 0)
    for cap, line, ways in CACHES:
        if S % line:
            continue
        for traversal, hashed in ((0, 0), (1, 0), (0, 1), (1, 1)):
            want = orc.traffic_lru(do, orc.L2Model(cap, line, ways, traversal, hashed))
            got = run(dl, ccl.L2Model(cap, line, ways, traversal, hashed))
            np.testing.assert_array_equal(got, want, err_msg=f"cache {cap}/{line}/{ways} traversal {traversal} hash {hashed}")
    # waves of CTAs in lockstep through K: whole-line and ragged k slices, waves that divide the tile count or not
    for cap, line, ways in ((8 * 1024, 128, 4), (96 * 1024, 128, 16), (1 << 20, 128, 16)):
        if S % line:
            continue
        for wave, ks, traversal, hashed in ((4, 64, 0, 1), (3, 96, 1, 0), (7, 40, 0, 0), (256, 64, 1, 1), (2, 0, 0, 1), (1, 32, 1, 1)):
            want = orc.traffic_lru(do, orc.L2Model(cap, line, ways, traversal, hashed, wave, ks))
            got = run(dl, ccl.L2Model(cap, line, ways, traversal, hashed, wave, ks))
            np.testing.assert_array_equal(got, want, err_msg=f"cache {cap}/{line}/{ways} traversal {traversal} hash {hashed} wave {wave} k_slice {ks}")


def test_lru_llama_gateup_full_size_properties():
    """The benchmark's gate+up GEMM (8192 x 57344 x 8192, P = 4, 4 KB pages, 8 MB / 16-way / 128 B per chiplet):
    the counts lie between the ideal-L2 and the uncached ones, C is untouched by the cache, CCL keeps B and C local,
    and under row-major traversal of N-strips a chiplet streams its strip of B once per tile row of A (an 8 MB cache
    never sees a second visit of B) while A is read about once per chiplet (skewed set index; with set = line mod sets
    the strided columns of B pile up in a few sets and push A's lines out of them: 3 to 8 times as much)."""
    M, N, K, P, S = 8192, 57344, 8192, 4, 4096
    model = ccl.L2Model(8 << 20, 128, 16, 0, 1)
    res = {}
    for tag, lay, place in (("rr", ("row", "row", "row"), (0, 0, 0)), ("ccl", ("row", "ccl", "ccl"), (0, 1, 1))):
        _, dl = traffic_pair(M, N, K, P, S, lay, place, align=S)
        t = run(dl, model)
        ideal = torch.zeros((3, 2), dtype=torch.int64, device="cuda")
        ccl.ccl_traffic_l2(dl, ideal)
        ideal = ideal.cpu().numpy().astype(np.uint64)
        nt, _ = ccl.ccl_traffic_sizes(dl)
        per_cta = torch.zeros((nt, 3, 2), dtype=torch.int64, device="cuda")
        plain = torch.zeros((3, 2), dtype=torch.int64, device="cuda")
        ccl.ccl_traffic(dl, per_cta, plain)
        plain = plain.cpu().numpy().astype(np.uint64)
        np.testing.assert_array_equal(t[2], plain[2])
        for X in (0, 1):
            assert ideal[X].sum() <= t[X].sum() <= plain[X].sum()
        res[tag] = t
        assert P * M * K * 2 <= int(t[0].sum()) <= 1.25 * P * M * K * 2
        assert int(t[1].sum()) == (M // 128) * K * N * 2
    assert res["ccl"][1][1] == 0 and res["ccl"][2][1] == 0            # CCL + page->strip placement: B and C local
    ratio = float(res["ccl"][:, 1].sum()) / float(res["rr"][:, 1].sum())
    assert ratio < 0.02                                               # A is what is left: ~1 % of the 4 KB round-robin traffic
    print("finite-L2 remote ratio CCL / rr4k on the Llama gate+up GEMM:", ratio)


def test_lru_rejections():
    import ctypes as C
    _, dl = traffic_pair(256, 512, 128, 2, 4096)
    l = ccl.lib()
    def rc(model, d=dl):
        return l.ccl_traffic_lru(C.byref(d), C.byref(model), C.c_void_p(256), None)
    assert rc(ccl.L2Model(1000, 128, 16, 0)) == ccl.ERR_INVALID_ARG
    assert rc(ccl.L2Model(8 << 20, 128, 64, 0)) == ccl.ERR_UNSUPPORTED
    assert rc(ccl.L2Model(8 << 20, 128, 16, 3)) == ccl.ERR_INVALID_ARG
    assert rc(ccl.L2Model(8 << 20, 8192, 16, 0)) == ccl.ERR_INVALID_ARG          # pages smaller than lines
    _, db = traffic_pair(256, 512, 128, 2, 4096, place=(2, 2, 2))
    assert rc(ccl.L2Model(), db) == ccl.ERR_UNSUPPORTED
    _, di = traffic_pair(256, 512, 128, 2, 1024, ("row", "ileave", "ileave"), align=1024)
    assert rc(ccl.L2Model(), di) == ccl.ERR_UNSUPPORTED
    _, de = traffic_pair(256, 512, 128, 2, 4096, assign=2)
    assert rc(ccl.L2Model(), de) == ccl.ERR_UNSUPPORTED


def _skew_cases():
    out = []
    for line in open(os.path.join(HERE, "golden", "lru_skew_index.txt")):
        f = line.split()
        if f and f[0] == "CASE":
            out.append((f[1], *[int(x) for x in f[2:]]))
    return out


@pytest.mark.parametrize("case", _skew_cases(), ids=lambda c: c[0])
def test_skewed_set_index_hand_cases_on_the_gpu(case):
    """The hand-worked access strings that pin the skewed set index (their hit / miss outcome depends on it)."""
    _, sets, hash_, M, N, K, BM, BN, bt, bstrips, balign, want_a, want_b = case
    d = ccl.TrafficDesc()
    d.M, d.N, d.K, d.BM, d.BN = M, N, K, BM, BN
    d.A, d.C = ccl.Mat(M, K, 2), ccl.Mat(M, N, 2)
    if bstrips > 1:
        d.B = ccl.Mat(N, K, 2, bstrips, ccl.PART_ROWS, ccl.CCL, balign) if bt else ccl.Mat(K, N, 2, bstrips, ccl.PART_COLS, ccl.CCL, balign)
    else:
        d.B = ccl.Mat(N, K, 2) if bt else ccl.Mat(K, N, 2)
    d.a_trans, d.b_trans, d.P, d.page_bytes = 0, bt, 1, 16
    d.place[0] = d.place[1] = d.place[2] = ccl.PLACE_RR
    d.assign, d.strip_tiling = ccl.ASSIGN_N_STRIPS, 1
    t = run(d, ccl.L2Model(sets * 16, 16, 1, 0, hash_, 1, 0))
    assert int(t[0, 0]) == want_a and int(t[0, 1]) == 0
    if want_b >= 0:
        assert int(t[1, 0]) == want_b
