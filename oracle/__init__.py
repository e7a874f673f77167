"""ctypes front end of the CPU oracle (oracle/ccl_oracle.cpp).

TEST INFRASTRUCTURE ONLY: imported by tests/, the smoke check and the
benchmark's CPU-baseline leg.  It shares nothing with the CUDA package and
must never be imported by it.
"""
import ctypes as C
import os

import numpy as np

from . import build as _build

ROWMAJOR, CCL, CCL_INTERLEAVED = 0, 1, 2
PART_NONE, PART_ROWS, PART_COLS = 0, 1, 2
PLACE_RR, PLACE_BLOCK, PLACE_BEST = 0, 1, 2
ASSIGN_N, ASSIGN_M, ASSIGN_EXPLICIT, ASSIGN_2D = 0, 1, 2, 3


class Mat(C.Structure):
    _fields_ = [("rows", C.c_int64), ("cols", C.c_int64), ("elem_bytes", C.c_int32), ("P", C.c_int32),
                ("part", C.c_int32), ("layout", C.c_int32), ("strip_align_bytes", C.c_int64)]

    def __init__(self, rows, cols, elem_bytes=2, P=1, part=PART_NONE, layout=ROWMAJOR, strip_align_bytes=0):
        super().__init__(rows, cols, elem_bytes, P, part, layout, strip_align_bytes)


class TrafficDesc(C.Structure):
    _fields_ = [("M", C.c_int64), ("N", C.c_int64), ("K", C.c_int64), ("BM", C.c_int32), ("BN", C.c_int32),
                ("A", Mat), ("B", Mat), ("C", Mat), ("a_trans", C.c_int32), ("b_trans", C.c_int32),
                ("P", C.c_int32), ("page_bytes", C.c_int64), ("place", C.c_int32 * 3), ("assign", C.c_int32),
                ("strip_tiling", C.c_int32), ("part_m", C.c_int32)]


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(_build.build())
        _lib.orc_f32_to_bf16.restype = C.c_uint16
        _lib.orc_f32_to_bf16.argtypes = [C.c_float]
    return _lib


def _p(a):
    return a.ctypes.data_as(C.c_void_p)


def map_offset(m, r, c):
    off = C.c_int64()
    rc = lib().orc_map_offset(C.byref(m), C.c_int64(r), C.c_int64(c), C.byref(off))
    if rc:
        raise ValueError("orc_map_offset rejected the arguments")
    return off.value


def map_inverse(m, off):
    r, c = C.c_int64(), C.c_int64()
    rc = lib().orc_map_inverse(C.byref(m), C.c_int64(off), C.byref(r), C.byref(c))
    return rc, r.value, c.value


def map_table(m):
    out = np.empty((m.rows, m.cols), dtype=np.int64)
    if lib().orc_map_table(C.byref(m), _p(out)):
        raise ValueError("bad descriptor")
    return out


def buffer_bytes(m):
    b = C.c_int64()
    if lib().orc_buffer_bytes(C.byref(m), C.byref(b)):
        raise ValueError("bad descriptor")
    return b.value


def strip_stride(m):
    b = C.c_int64()
    if lib().orc_strip_stride(C.byref(m), C.byref(b)):
        raise ValueError("bad descriptor")
    return b.value


def repack(m, src, direction=0):
    """src: contiguous numpy array whose itemsize is m.elem_bytes (flat or 2-D). Returns a flat array."""
    src = np.ascontiguousarray(src)
    assert src.itemsize == m.elem_bytes
    n_out = buffer_bytes(m) // m.elem_bytes if direction == 0 else m.rows * m.cols
    n_in = m.rows * m.cols if direction == 0 else buffer_bytes(m) // m.elem_bytes
    assert src.size == n_in, (src.size, n_in)
    dst = np.empty(n_out, dtype=src.dtype)
    if lib().orc_repack(C.byref(m), _p(src), _p(dst), C.c_int(direction)):
        raise ValueError("bad descriptor")
    return dst


def repack_transposed(m, src_t):
    """Transposing repack (Sec. 3.3: an operand stored the other way round is repacked into CCL): src_t is the
    row-major transpose [cols x rows] of the matrix `m` describes; element (r, c) of that matrix, src_t[c, r], goes to
    offset index(r, c) of Eq. 1-3 (map_table); padding is zero.  Written from the map alone, one element at a time."""
    src_t = np.ascontiguousarray(src_t).reshape(m.cols, m.rows)
    assert src_t.itemsize == m.elem_bytes
    table = map_table(m)
    out = np.zeros(buffer_bytes(m) // m.elem_bytes, dtype=src_t.dtype)
    for r in range(m.rows):
        out[table[r]] = src_t[:, r]
    return out


def gemm(A, B, M, N, K, a_trans=0, b_trans=0, block=None, want64=False, threads=None):
    """A, B: uint16 (bf16 bit patterns), stored row-major as the flags say.
    Returns (ref32, ref64 or None, out_bf16_bits) for block = (m0, m1, n0, n1) or the whole C."""
    A = np.ascontiguousarray(A, dtype=np.uint16).reshape(-1)
    B = np.ascontiguousarray(B, dtype=np.uint16).reshape(-1)
    assert A.size == M * K and B.size == K * N
    m0, m1, n0, n1 = block if block is not None else (0, M, 0, N)
    ref32 = np.empty((m1 - m0, n1 - n0), dtype=np.float32)
    ref64 = np.empty((m1 - m0, n1 - n0), dtype=np.float64) if want64 else None
    out = np.empty((m1 - m0, n1 - n0), dtype=np.uint16)
    if threads is None:
        threads = os.cpu_count() or 1
    rc = lib().orc_gemm(C.c_int64(M), C.c_int64(N), C.c_int64(K), _p(A), C.c_int(a_trans), _p(B), C.c_int(b_trans),
                        C.c_int64(m0), C.c_int64(m1), C.c_int64(n0), C.c_int64(n1), _p(ref32),
                        _p(ref64) if want64 else None, _p(out), C.c_int(threads))
    if rc:
        raise ValueError("orc_gemm rejected the arguments")
    return ref32, ref64, out


def gemm_axpby(A, B, Cin, M, N, K, alpha, beta, a_trans=0, b_trans=0, threads=None):
    """alpha * A*B + beta * Cin (Cin: logical [M x N] bf16 bits).  Returns (ref32, out_bf16_bits)."""
    A = np.ascontiguousarray(A, dtype=np.uint16).reshape(-1)
    B = np.ascontiguousarray(B, dtype=np.uint16).reshape(-1)
    Cin = np.ascontiguousarray(Cin, dtype=np.uint16).reshape(-1)
    assert A.size == M * K and B.size == K * N and Cin.size == M * N
    ref32 = np.empty((M, N), dtype=np.float32)
    out = np.empty((M, N), dtype=np.uint16)
    if threads is None:
        threads = os.cpu_count() or 1
    rc = lib().orc_gemm_axpby(C.c_int64(M), C.c_int64(N), C.c_int64(K), _p(A), C.c_int(a_trans), _p(B), C.c_int(b_trans),
                              C.c_double(alpha), C.c_double(beta), _p(Cin), _p(ref32), _p(out), C.c_int(threads))
    if rc:
        raise ValueError("orc_gemm_axpby rejected the arguments")
    return ref32, out


def gemm_swiglu(A, B, M, N, K, P=1, a_trans=0, b_trans=0, threads=None):
    """silu(gate) * up on the product of a fused gate/up operand whose column strips (P of them) hold gate | up halves.
    Returns (ref32 [M x N/2], out_bf16_bits)."""
    A = np.ascontiguousarray(A, dtype=np.uint16).reshape(-1)
    B = np.ascontiguousarray(B, dtype=np.uint16).reshape(-1)
    assert A.size == M * K and B.size == K * N
    ref32 = np.empty((M, N // 2), dtype=np.float32)
    out = np.empty((M, N // 2), dtype=np.uint16)
    if threads is None:
        threads = os.cpu_count() or 1
    rc = lib().orc_gemm_swiglu(C.c_int64(M), C.c_int64(N), C.c_int64(K), C.c_int64(P), _p(A), C.c_int(a_trans), _p(B), C.c_int(b_trans),
                               _p(ref32), _p(out), C.c_int(threads))
    if rc:
        raise ValueError("orc_gemm_swiglu rejected the arguments")
    return ref32, out


class L2Model(C.Structure):
    """orc_l2_model"""
    _fields_ = [("capacity_bytes", C.c_int64), ("line_bytes", C.c_int32), ("ways", C.c_int32), ("traversal", C.c_int32),
                ("hash", C.c_int32), ("wave_ctas", C.c_int32), ("k_slice", C.c_int32)]

    def __init__(self, capacity_bytes=8 << 20, line_bytes=128, ways=16, traversal=0, hash=0, wave_ctas=1, k_slice=0):
        super().__init__(capacity_bytes, line_bytes, ways, traversal, hash, wave_ctas, k_slice)


def traffic_lru(d, l2):
    """Local / remote bytes [3,2] behind a finite LRU L2 per chiplet (the model stated in ccl_oracle.cpp)."""
    totals = np.zeros((3, 2), dtype=np.uint64)
    if lib().orc_traffic_lru(C.byref(d), C.byref(l2), _p(totals)):
        raise ValueError("orc_traffic_lru rejected the arguments")
    return totals


def traffic_sizes(d):
    nt = C.c_int64()
    pages = (C.c_int64 * 3)()
    if lib().orc_traffic_sizes(C.byref(d), C.byref(nt), pages):
        raise ValueError("bad traffic descriptor")
    return nt.value, list(pages)


def traffic_tiles(d, explicit_q=None):
    nt, _ = traffic_sizes(d)
    out = np.empty((nt, 5), dtype=np.int64)
    q = None if explicit_q is None else _p(np.ascontiguousarray(explicit_q, dtype=np.int32))
    if lib().orc_traffic_tiles(C.byref(d), q, _p(out)):
        raise ValueError("bad traffic descriptor")
    return out


def traffic(d, explicit_q=None, level="elem"):
    """Returns dict(per_cta [ntiles,3,2], per_page [3 x (pages,P)], owner [3 x (pages,)], totals [3,2])."""
    nt, pages = traffic_sizes(d)
    per_cta = np.zeros((nt, 3, 2), dtype=np.uint64)
    per_page = [np.zeros((pages[x], d.P), dtype=np.uint64) for x in range(3)]
    owner = [np.zeros(pages[x], dtype=np.uint8) for x in range(3)]
    totals = np.zeros((3, 2), dtype=np.uint64)
    pp = (C.c_void_p * 3)(*[a.ctypes.data for a in per_page])
    ow = (C.c_void_p * 3)(*[a.ctypes.data for a in owner])
    qarr = None if explicit_q is None else np.ascontiguousarray(explicit_q, dtype=np.int32)
    fn = lib().orc_traffic_elem if level == "elem" else lib().orc_traffic_runs
    rc = fn(C.byref(d), None if qarr is None else _p(qarr), _p(per_cta), pp, ow, _p(totals))
    if rc:
        raise ValueError("bad traffic descriptor")
    return dict(per_cta=per_cta, per_page=per_page, owner=owner, totals=totals)


def traffic_ideal_l2(d, explicit_q=None):
    """Local / remote bytes [3,2] when every chiplet fetches each byte at most once (ideal private L2)."""
    totals = np.zeros((3, 2), dtype=np.uint64)
    qarr = None if explicit_q is None else np.ascontiguousarray(explicit_q, dtype=np.int32)
    if lib().orc_traffic_ideal_l2(C.byref(d), None if qarr is None else _p(qarr), _p(totals)):
        raise ValueError("bad traffic descriptor (or a BEST placement)")
    return totals


def f32_to_bf16(x):
    return lib().orc_f32_to_bf16(C.c_float(x))
