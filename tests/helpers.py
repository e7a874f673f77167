"""Builds matching descriptors for the oracle and for the CUDA library from one plain spec.

The two descriptor types are separate ctypes structures (the oracle and the library share no
definitions); this file only copies numbers into both.
"""
import oracle as orc
from paper_2606_11718_b200 import binding as ccl


def mat_pair(rows, cols, e=2, P=1, part=0, layout=0, align=0):
    return orc.Mat(rows, cols, e, P, part, layout, align), ccl.Mat(rows, cols, e, P, part, layout, align)


def operand_shapes(M, N, K, a_trans, b_trans):
    return [((K, M) if a_trans else (M, K)), ((N, K) if b_trans else (K, N)), (M, N)]


def n_split_parts(a_trans, b_trans):
    """Stored dimension that an N-partition of C splits: nothing for A, N for B and C."""
    return (0, 1 if b_trans else 2, 2)


def m_split_parts(a_trans, b_trans):
    return (2 if a_trans else 1, 0, 1)


def traffic_pair(M, N, K, P, S, lay=("row", "row", "row"), place=(0, 0, 0), a_trans=0, b_trans=0, assign=0, BM=128, BN=128,
                 strip_tiling=1, e=2, align=0, parts=None, part_m=0, mat_P=None):
    """assign = 3: a 2-D output partition of part_m x (P / part_m) blocks; mat_P: strips of the CCL operands (default P)."""
    if parts is None:
        parts = m_split_parts(a_trans, b_trans) if assign == 1 else n_split_parts(a_trans, b_trans)
    mat_P = mat_P if mat_P is not None else (P, P, P)
    shapes = operand_shapes(M, N, K, a_trans, b_trans)
    out = []
    for mod, cls in ((orc, orc.TrafficDesc), (ccl, ccl.TrafficDesc)):
        d = cls()
        d.M, d.N, d.K, d.BM, d.BN = M, N, K, BM, BN
        mats = []
        for X in range(3):
            is_ccl = lay[X] in ("ccl", "ileave") and parts[X] != 0      # "ileave": page-interleaved CCL, align = chunk size
            mats.append(mod.Mat(shapes[X][0], shapes[X][1], e, mat_P[X], parts[X] if is_ccl else 0,
                                (2 if lay[X] == "ileave" else 1) if is_ccl else 0, align if is_ccl else 0))
        d.A, d.B, d.C = mats
        d.a_trans, d.b_trans, d.P, d.page_bytes = a_trans, b_trans, P, S
        d.place[0], d.place[1], d.place[2] = place
        d.assign, d.strip_tiling, d.part_m = assign, strip_tiling, part_m
        out.append(d)
    return out


def gemm_desc(M, N, K, P=1, lay=("row", "row", "row"), a_trans=0, b_trans=0, out_part=2, grouped=1, align=0, parts=None, part_m=0, mat_P=None):
    """Library GEMM descriptor; lay[X] == "ccl" ("ileave": page-interleaved CCL with chunks of `align` bytes) stores
    operand X in CCL split as `parts` says
    (default: the split an N- or M-partition of C implies)."""
    if parts is None:
        parts = m_split_parts(a_trans, b_trans) if out_part == 1 else n_split_parts(a_trans, b_trans)
    mat_P = mat_P if mat_P is not None else (P, P, P)
    shapes = operand_shapes(M, N, K, a_trans, b_trans)
    d = ccl.GemmDesc()
    d.M, d.N, d.K = M, N, K
    mats = []
    for X in range(3):
        is_ccl = lay[X] in ("ccl", "ileave") and parts[X] != 0
        layout = (2 if lay[X] == "ileave" else 1) if is_ccl else 0
        mats.append(ccl.Mat(shapes[X][0], shapes[X][1], 2, mat_P[X], parts[X] if is_ccl else 0, layout, align if is_ccl else 0))
    d.A, d.B, d.C = mats
    d.a_trans, d.b_trans, d.out_part, d.P, d.grouped_raster, d.part_m = a_trans, b_trans, out_part, P, grouped, part_m
    return d
