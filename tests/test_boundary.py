"""C-ABI boundary on the CPU: the library loads, exports what include/ccl.h declares, its host-side
address map agrees with the oracle, and bad input is rejected before any launch.  No GPU."""
import ctypes as C
import os
import re

import numpy as np
import pytest

import oracle as orc
from paper_2606_11718_b200 import binding as ccl
from paper_2606_11718_b200 import build as ccl_build
from helpers import gemm_desc, mat_pair, traffic_pair

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def built():
    ccl_build.build()


def test_exports_match_header():
    hdr = open(os.path.join(ROOT, "include", "ccl.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    declared = sorted(set(re.findall(r"\b(ccl_[a-z0-9_]+)\s*\(", hdr)))
    assert declared == sorted(ccl.EXPORTS)
    l = ccl.lib()
    for name in declared:
        assert getattr(l, name) is not None
    assert ccl.ccl_version() == "0.1"


def test_struct_sizes_match_c_layout():
    # the ctypes mirrors follow the C rules; spot-check the sizes the header implies
    assert C.sizeof(ccl.Mat) == 40
    assert C.sizeof(ccl.GemmDesc) == 24 + 3 * 40 + 5 * 4 + 4
    assert C.sizeof(ccl.TrafficDesc) == 24 + 8 + 3 * 40 + 12 + 4 + 8 + 12 + 4 + 4 + 4


MAP_CASES = [
    dict(rows=4, cols=8, P=2, part=2, layout=1),
    dict(rows=7, cols=12, P=3, part=2, layout=1),
    dict(rows=33, cols=768, P=8, part=2, layout=1),
    dict(rows=64, cols=200, P=2, part=2, layout=1, e=4),
    dict(rows=12, cols=40, P=4, part=1, layout=1),
    dict(rows=12, cols=40, P=4, part=2, layout=0),
    dict(rows=12, cols=40, P=1, part=0, layout=0, e=1),
    dict(rows=6, cols=36, P=3, part=2, layout=1, align=256),
    dict(rows=6, cols=36, P=3, part=1, layout=1, align=4096),
    dict(rows=5, cols=30, P=5, part=2, layout=1, align=64, e=4),
    dict(rows=4, cols=8, P=2, part=2, layout=2, align=16),                 # page-interleaved CCL, the hand example
    dict(rows=7, cols=24, P=3, part=2, layout=2, align=64),
    dict(rows=12, cols=40, P=4, part=1, layout=2, align=48, e=4),
    dict(rows=33, cols=96, P=4, part=2, layout=2, align=256, e=1),
    dict(rows=3, cols=7, P=3, part=2, layout=1),                           # widths P does not divide: the hand example
    dict(rows=9, cols=1537, P=4, part=2, layout=1, align=256),
    dict(rows=13, cols=40, P=4, part=1, layout=1, align=64),
    dict(rows=5, cols=202, P=3, part=2, layout=2, align=128),
    dict(rows=11, cols=30, P=4, part=1, layout=2, align=48, e=4),
]


@pytest.mark.parametrize("case", MAP_CASES)
def test_host_map_equals_oracle(case):
    mo, ml = mat_pair(**case)
    table = orc.map_table(mo)
    for r in range(mo.rows):
        for c in range(mo.cols):
            assert ccl.ccl_map_offset(ml, r, c) == table[r, c]
    assert ccl.ccl_buffer_bytes(ml) == orc.buffer_bytes(mo)
    if case["layout"] == 1 and case["part"] != 0:
        assert ccl.ccl_strip_stride(ml) == orc.strip_stride(mo)
    if case["layout"] == 2:
        with pytest.raises(ccl.CclError):
            ccl.ccl_strip_stride(ml)
    n = orc.buffer_bytes(mo) // mo.elem_bytes
    for off in range(n):
        rc, r, c = orc.map_inverse(mo, off)
        if rc == 0:
            assert ccl.ccl_map_inverse(ml, off) == (r, c)
        else:
            with pytest.raises(ccl.CclError) as ei:
                ccl.ccl_map_inverse(ml, off)
            assert ei.value.status == ccl.ERR_PADDING


def test_large_offsets_use_64_bits():
    mo, ml = mat_pair(1 << 20, 1 << 16, 2, 4, 2, 1)                    # 2^36 elements
    for r, c in [(0, 0), (1 << 19, 40000), ((1 << 20) - 1, (1 << 16) - 1)]:
        assert ccl.ccl_map_offset(ml, r, c) == orc.map_offset(mo, r, c)


def expect(status, fn, *a, **k):
    with pytest.raises(ccl.CclError) as ei:
        fn(*a, **k)
    assert ei.value.status == status, ei.value
    assert ccl.lib().ccl_last_error() != b""


def test_map_error_codes():
    expect(ccl.ERR_SHAPE, ccl.ccl_map_offset, ccl.Mat(4, 9, 2, 4, 2, 1), 0, 0)       # 4 strips of ceil(9/4) = 3: the last would be empty
    expect(ccl.ERR_SHAPE, ccl.ccl_buffer_bytes, ccl.Mat(4, 8, 2, 3, 1, 1))
    expect(ccl.ERR_INVALID_ARG, ccl.ccl_map_offset, ccl.Mat(4, 8, 2, 2, 2, 1), 4, 0)
    expect(ccl.ERR_INVALID_ARG, ccl.ccl_map_offset, ccl.Mat(4, 8, 3, 2, 2, 1), 0, 0)
    expect(ccl.ERR_INVALID_ARG, ccl.ccl_map_offset, ccl.Mat(4, 8, 2, 0, 2, 1), 0, 0)
    expect(ccl.ERR_INVALID_ARG, ccl.ccl_map_offset, ccl.Mat(4, 8, 2, 2, 2, 1, 3), 0, 0)
    expect(ccl.ERR_INVALID_ARG, ccl.ccl_strip_stride, ccl.Mat(4, 8))
    expect(ccl.ERR_INVALID_ARG, ccl.ccl_map_offset, ccl.Mat(4, 8, 2, 2, 2, 2, 0), 0, 0)      # interleaved layout without a chunk size
    expect(ccl.ERR_INVALID_ARG, ccl.ccl_map_inverse, ccl.Mat(4, 8), 32)


def test_repack_rejects_bad_input_before_any_launch():
    l = ccl.lib()
    m = ccl.Mat(4, 8, 2, 2, 2, 1)
    assert l.ccl_repack(C.byref(m), None, None, 0, None) == ccl.ERR_INVALID_ARG
    assert l.ccl_repack(C.byref(m), C.c_void_p(256), C.c_void_p(512), 2, None) == ccl.ERR_INVALID_ARG
    assert l.ccl_repack(C.byref(m), C.c_void_p(256), C.c_void_p(256), 0, None) == ccl.ERR_INVALID_ARG
    assert l.ccl_repack(C.byref(m), C.c_void_p(257), C.c_void_p(512), 0, None) == ccl.ERR_ALIGN
    bad = ccl.Mat(4, 9, 2, 4, 2, 1)
    assert l.ccl_repack(C.byref(bad), C.c_void_p(256), C.c_void_p(512), 0, None) == ccl.ERR_SHAPE
    # a batch: count in range, outputs that do not overlap, strides in whole elements
    rb = lambda batch, ss, ds, d=0: l.ccl_repack_batched(C.byref(m), batch, C.c_void_p(256), ss, C.c_void_p(4096), ds, d, None)
    assert rb(0, 64, 64) == ccl.ERR_INVALID_ARG
    assert rb(70000, 64, 64) == ccl.ERR_INVALID_ARG
    assert rb(2, 64, 62) == ccl.ERR_INVALID_ARG                    # 4 x 8 x 2 = 64 bytes per output
    assert rb(2, -64, 64) == ccl.ERR_INVALID_ARG
    assert rb(2, 65, 66) == ccl.ERR_ALIGN
    padded = ccl.Mat(4, 8, 2, 2, 2, 1, 256)                        # strips padded to 256 bytes: 512 bytes per packed matrix
    assert l.ccl_repack_batched(C.byref(padded), 2, C.c_void_p(256), 64, C.c_void_p(4096), 64, 0, None) == ccl.ERR_INVALID_ARG


def test_gemm_grouped_rejects_bad_input_before_any_launch():
    l = ccl.lib()
    d = gemm_desc(1024, 768, 512, 4, ("row", "ccl", "ccl"), b_trans=1)
    call = lambda dd, groups=4, cap=256, offs=65536, b_stride=1 << 20: l.ccl_gemm_grouped(
        C.byref(dd), groups, cap, C.c_void_p(offs), C.c_void_p(4096), C.c_void_p(8192), b_stride, C.c_void_p(16384), None)
    assert call(d, offs=None) == ccl.ERR_INVALID_ARG                 # no row offsets
    assert call(d, offs=65538) == ccl.ERR_ALIGN
    assert call(d, cap=0) == ccl.ERR_INVALID_ARG and call(d, cap=1025) == ccl.ERR_INVALID_ARG
    assert call(d, b_stride=-16) == ccl.ERR_INVALID_ARG
    assert call(d, groups=0) == ccl.ERR_INVALID_ARG
    assert call(d, b_stride=1000) == ccl.ERR_INVALID_ARG             # smaller than one B
    assert call(gemm_desc(1024, 768, 512, 4, ("row", "ccl", "ccl"), a_trans=1)) == ccl.ERR_UNSUPPORTED
    assert call(gemm_desc(1024, 768, 512, 4, ("ccl", "row", "ccl"), out_part=1)) == ccl.ERR_UNSUPPORTED    # split along M


def test_gemm_grouped_k_rejects_bad_input_before_any_launch():
    l = ccl.lib()
    d = gemm_desc(768, 2048, 4096, 4, ("row", "ccl", "ccl"), a_trans=1)
    call = lambda dd, groups=4, offs=65536, c_stride=768 * 2048 * 2: l.ccl_gemm_grouped_k(
        C.byref(dd), groups, C.c_void_p(offs), C.c_void_p(4096), C.c_void_p(8192), C.c_void_p(16384), c_stride, None)
    assert call(d, offs=None) == ccl.ERR_INVALID_ARG
    assert call(d, offs=65537) == ccl.ERR_ALIGN
    assert call(d, c_stride=-2) == ccl.ERR_INVALID_ARG
    assert call(d, c_stride=1024) == ccl.ERR_INVALID_ARG                                        # smaller than one C
    assert call(gemm_desc(768, 2048, 4096, 4, ("row", "ccl", "ccl"))) == ccl.ERR_UNSUPPORTED   # A stored [M x K]
    assert call(gemm_desc(768, 2048, 4096, 4, ("row", "ccl", "ccl"), a_trans=1, b_trans=1)) == ccl.ERR_UNSUPPORTED


def gemm_rc(d, a=4096, b=8192, c=16384):
    return ccl.lib().ccl_gemm(C.byref(d), C.c_void_p(a), C.c_void_p(b), C.c_void_p(c), None, 0, None)


def test_gemm_rejects_bad_input_before_any_launch():
    ok = gemm_desc(256, 768, 2048, 4, ("row", "ccl", "ccl"), b_trans=1)
    assert ccl.ccl_gemm_workspace(ok) >= 0                                  # a short problem may be split along K
    assert ccl.ccl_gemm_workspace(gemm_desc(8192, 8192, 8192, 4, ("row", "ccl", "ccl"))) == 0
    small = gemm_desc(16, 8192, 28672, 4, ("row", "ccl", "ccl"))
    need = ccl.ccl_gemm_workspace(small)
    assert need >= 0 and need % (16 * 8192 * 4) == 0                        # a weight-streaming shape is split along K: in a
                                                                            # cluster (no workspace) or through fp32 partial sums
    assert ccl.lib().ccl_gemm(C.byref(ok), None, None, None, None, 0, None) == ccl.ERR_INVALID_ARG
    assert gemm_rc(gemm_desc(128, 200, 64, 2, ("row", "ccl", "ccl"))) == ccl.ERR_UNSUPPORTED        # w = 100
    assert gemm_rc(gemm_desc(128, 256, 100)) == ccl.ERR_UNSUPPORTED                                  # K % 8 for A rows
    assert gemm_rc(ok, a=4100) == ccl.ERR_ALIGN
    d = gemm_desc(128, 256, 64)
    d.A.rows = 100
    assert gemm_rc(d) == ccl.ERR_SHAPE
    d = gemm_desc(128, 256, 64)
    d.C.elem_bytes = 4
    assert gemm_rc(d) == ccl.ERR_UNSUPPORTED
    d = gemm_desc(128, 256, 64, 4, ("row", "ccl", "ccl"))
    d.C.P = 2                                                                                        # B and C strips differ
    assert gemm_rc(d) == ccl.ERR_UNSUPPORTED
    d = gemm_desc(128, 256, 64, 3, ("row", "row", "row"))
    assert gemm_rc(d) == ccl.ERR_SHAPE                                                               # N % P with a grouped raster
    assert gemm_rc(gemm_desc(128, 264, 64, 4, ("row", "ccl", "row"), grouped=0)) == ccl.ERR_UNSUPPORTED   # strips of 66 columns
    assert gemm_rc(gemm_desc(128, 1000, 64, 4, ("row", "row", "row"), out_part=2, grouped=1)) == ccl.ERR_UNSUPPORTED   # tiles would start at multiples of 250 columns
    assert gemm_rc(gemm_desc(264, 1000, 64, 3, ("row", "ccl", "row"), b_trans=1)) == ccl.ERR_UNSUPPORTED   # B [N x K] in strips of 334 rows: C's tiles would start there
    d = gemm_desc(256, 512, 64, 4, ("row", "row", "row"), out_part=3)
    d.part_m = 3
    assert gemm_rc(d) == ccl.ERR_INVALID_ARG                                                         # part_m must divide P
    d.part_m = 2
    d.M = 255; d.A.rows = 255; d.C.rows = 255
    assert gemm_rc(d) == ccl.ERR_SHAPE                                                               # M not divisible by part_m
    # page-interleaved operands: chunks must line up with the strip rows (w = 96 elements = 192 bytes here)
    assert gemm_rc(gemm_desc(128, 192, 64, 2, ("row", "ileave", "ccl"), align=256)) == ccl.ERR_UNSUPPORTED    # neither divides
    assert gemm_rc(gemm_desc(128, 192, 64, 2, ("row", "ileave", "ccl"), align=576)) == ccl.ERR_UNSUPPORTED    # 3 rows per chunk
    assert gemm_rc(gemm_desc(128, 192, 64, 2, ("row", "ccl", "ileave"), align=64)) == ccl.ERR_UNSUPPORTED     # 3 chunks of 32 elements
    assert gemm_rc(gemm_desc(128, 512, 72, 2, ("row", "ileave", "ccl"), align=8192)) == ccl.ERR_UNSUPPORTED   # K tail ends inside a chunk
    d = gemm_desc(128, 256, 64)
    d.out_part = 7
    assert gemm_rc(d) == ccl.ERR_INVALID_ARG
    d = gemm_desc(128, 512, 96, 2, ("row", "ccl", "row"), parts=(0, 1, 0))                            # B split along K, 48-row strips
    assert gemm_rc(d) == ccl.ERR_UNSUPPORTED
    d = gemm_desc(128, 512, 64, 2, ("row", "ccl", "ccl"), align=8)
    d.B.rows = 63; d.K = 63; d.A.cols = 63                                                           # strip stride 63*256*2 is fine; K=63 breaks A
    assert gemm_rc(d) == ccl.ERR_UNSUPPORTED


def test_traffic_sizes_and_rejections():
    do, dl = traffic_pair(130, 384, 96, 4, 256, ("row", "ccl", "ccl"), (0, 1, 1))
    assert ccl.ccl_traffic_sizes(dl) == tuple(orc.traffic_sizes(do))
    do, dl = traffic_pair(130, 384, 96, 4, 256, strip_tiling=0)
    assert ccl.ccl_traffic_sizes(dl) == tuple(orc.traffic_sizes(do))
    do, dl = traffic_pair(128, 256, 64, 8, 512, assign=1, BM=16, BN=64, lay=("ccl", "row", "ccl"), align=1024)
    assert ccl.ccl_traffic_sizes(dl) == tuple(orc.traffic_sizes(do))
    l = ccl.lib()
    _, bad = traffic_pair(8, 9, 4, 4, 16)
    assert l.ccl_traffic(C.byref(bad), None, C.c_void_p(256), None, None, C.c_void_p(512), None) == ccl.ERR_SHAPE
    do, dl = traffic_pair(8, 9, 4, 2, 16)                                                            # strips of 5 and 4 columns
    assert ccl.ccl_traffic_sizes(dl) == tuple(orc.traffic_sizes(do))
    do, dl = traffic_pair(131, 203, 24, 6, 128, assign=3, part_m=2, BM=32, BN=32)                    # 2 x 3 blocks, ragged both ways
    assert ccl.ccl_traffic_sizes(dl) == tuple(orc.traffic_sizes(do))
    _, d = traffic_pair(128, 256, 24, 6, 128, assign=3, part_m=4)
    assert l.ccl_traffic(C.byref(d), None, C.c_void_p(256), None, None, C.c_void_p(512), None) == ccl.ERR_INVALID_ARG
    _, d = traffic_pair(8, 8, 4, 2, 16)
    assert l.ccl_traffic(C.byref(d), None, None, None, None, C.c_void_p(512), None) == ccl.ERR_INVALID_ARG
    _, d = traffic_pair(8, 8, 4, 2, 16, place=(2, 2, 2))
    assert l.ccl_traffic(C.byref(d), None, C.c_void_p(256), None, None, C.c_void_p(512), None) == ccl.ERR_WORKSPACE
    _, d = traffic_pair(8, 8, 4, 2, 16, assign=2)
    assert l.ccl_traffic(C.byref(d), None, C.c_void_p(256), None, None, C.c_void_p(512), None) == ccl.ERR_INVALID_ARG
    _, d = traffic_pair(8, 8, 4, 2, 16, assign=4)
    assert l.ccl_traffic(C.byref(d), None, C.c_void_p(256), None, None, C.c_void_p(512), None) == ccl.ERR_INVALID_ARG
    _, d = traffic_pair(8, 8, 4, 2, 3)
    assert l.ccl_traffic(C.byref(d), None, C.c_void_p(256), None, None, C.c_void_p(512), None) == ccl.ERR_INVALID_ARG
    _, d = traffic_pair(8, 8, 4, 2, 16)
    d.A.rows = 9
    assert l.ccl_traffic(C.byref(d), None, C.c_void_p(256), None, None, C.c_void_p(512), None) == ccl.ERR_SHAPE
