"""Thin ctypes binding of the C-ABI library declared in include/ccl.h.

Argument marshalling only: every step runs in the CUDA kernels of libccl.so.  Tensors are
torch CUDA tensors used as plain device buffers; the stream is torch's current stream.
There is no CPU fallback: if libccl.so is missing the import of this module's functions
raises, and device entry points fail without a CUDA device.
"""
import ctypes as C
import os

import torch

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libccl.so")

OK, ERR_INVALID_ARG, ERR_SHAPE, ERR_ALIGN, ERR_UNSUPPORTED, ERR_CUDA, ERR_WORKSPACE, ERR_TIMEOUT, ERR_PADDING = range(9)
ROWMAJOR, CCL, CCL_INTERLEAVED = 0, 1, 2
PART_NONE, PART_ROWS, PART_COLS, PART_2D = 0, 1, 2, 3
PLACE_RR, PLACE_BLOCK, PLACE_BEST = 0, 1, 2
ASSIGN_N_STRIPS, ASSIGN_M_STRIPS, ASSIGN_EXPLICIT, ASSIGN_2D = 0, 1, 2, 3

EXPORTS = ["ccl_map_offset", "ccl_map_inverse", "ccl_buffer_bytes", "ccl_strip_stride", "ccl_repack", "ccl_repack_batched", "ccl_repack_transpose", "ccl_gemm_workspace",
           "ccl_gemm", "ccl_gemm_batched_workspace", "ccl_gemm_batched", "ccl_gemm_grouped", "ccl_gemm_grouped_swiglu", "ccl_gemm_grouped_k", "ccl_gemm_axpby", "ccl_gemm_swiglu", "ccl_gemm_static_ws", "ccl_gemm_status", "ccl_selftest_wait_timeout", "ccl_traffic_sizes", "ccl_traffic", "ccl_traffic_l2", "ccl_traffic_lru", "ccl_probe_l2_latency", "ccl_last_error", "ccl_launch_count", "ccl_version"]


class CclError(RuntimeError):
    def __init__(self, status, message):
        super().__init__(f"ccl status {status}: {message}")
        self.status = status


class Mat(C.Structure):
    """ccl_mat"""
    _fields_ = [("rows", C.c_int64), ("cols", C.c_int64), ("elem_bytes", C.c_int32), ("P", C.c_int32),
                ("part", C.c_int32), ("layout", C.c_int32), ("strip_align_bytes", C.c_int64)]

    def __init__(self, rows=0, cols=0, elem_bytes=2, P=1, part=PART_NONE, layout=ROWMAJOR, strip_align_bytes=0):
        super().__init__(rows, cols, elem_bytes, P, part, layout, strip_align_bytes)


class GemmDesc(C.Structure):
    """ccl_gemm_desc"""
    _fields_ = [("M", C.c_int64), ("N", C.c_int64), ("K", C.c_int64), ("A", Mat), ("B", Mat), ("C", Mat),
                ("a_trans", C.c_int32), ("b_trans", C.c_int32), ("out_part", C.c_int32), ("P", C.c_int32),
                ("grouped_raster", C.c_int32), ("part_m", C.c_int32)]


class TrafficDesc(C.Structure):
    """ccl_traffic_desc"""
    _fields_ = [("M", C.c_int64), ("N", C.c_int64), ("K", C.c_int64), ("BM", C.c_int32), ("BN", C.c_int32),
                ("A", Mat), ("B", Mat), ("C", Mat), ("a_trans", C.c_int32), ("b_trans", C.c_int32), ("P", C.c_int32),
                ("page_bytes", C.c_int64), ("place", C.c_int32 * 3), ("assign", C.c_int32), ("strip_tiling", C.c_int32),
                ("part_m", C.c_int32)]


class L2Model(C.Structure):
    """ccl_l2_model"""
    _fields_ = [("capacity_bytes", C.c_int64), ("line_bytes", C.c_int32), ("ways", C.c_int32), ("traversal", C.c_int32),
                ("hash", C.c_int32), ("wave_ctas", C.c_int32), ("k_slice", C.c_int32)]

    def __init__(self, capacity_bytes=8 << 20, line_bytes=128, ways=16, traversal=0, hash=0, wave_ctas=1, k_slice=0):
        super().__init__(capacity_bytes, line_bytes, ways, traversal, hash, wave_ctas, k_slice)


_lib = None


def lib():
    """Loads libccl.so (built by paper_2606_11718_b200.build); raises if it is missing."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} not found: build it with `python -m paper_2606_11718_b200.build` "
                              "(there is no fallback path)")
        l = C.CDLL(LIB_PATH)
        l.ccl_last_error.restype = C.c_char_p
        l.ccl_version.restype = C.c_char_p
        l.ccl_launch_count.restype = C.c_uint64
        l.ccl_map_offset.argtypes = [C.POINTER(Mat), C.c_int64, C.c_int64, C.POINTER(C.c_int64)]
        l.ccl_map_inverse.argtypes = [C.POINTER(Mat), C.c_int64, C.POINTER(C.c_int64), C.POINTER(C.c_int64)]
        l.ccl_buffer_bytes.argtypes = [C.POINTER(Mat), C.POINTER(C.c_int64)]
        l.ccl_strip_stride.argtypes = [C.POINTER(Mat), C.POINTER(C.c_int64)]
        l.ccl_repack.argtypes = [C.POINTER(Mat), C.c_void_p, C.c_void_p, C.c_int, C.c_void_p]
        l.ccl_repack_transpose.argtypes = [C.POINTER(Mat), C.c_void_p, C.c_void_p, C.c_void_p]
        l.ccl_repack_batched.argtypes = [C.POINTER(Mat), C.c_int32, C.c_void_p, C.c_int64, C.c_void_p, C.c_int64, C.c_int, C.c_void_p]
        l.ccl_gemm_workspace.argtypes = [C.POINTER(GemmDesc), C.POINTER(C.c_size_t)]
        l.ccl_gemm.argtypes = [C.POINTER(GemmDesc), C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
        l.ccl_gemm_grouped.argtypes = [C.POINTER(GemmDesc), C.c_int32, C.c_int64, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p, C.c_void_p]
        l.ccl_gemm_grouped_swiglu.argtypes = l.ccl_gemm_grouped.argtypes
        l.ccl_probe_l2_latency.argtypes = [C.c_void_p, C.c_int32, C.c_int64, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p]
        l.ccl_gemm_grouped_k.argtypes = [C.POINTER(GemmDesc), C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p]
        l.ccl_gemm_batched_workspace.argtypes = [C.POINTER(GemmDesc), C.c_int32, C.POINTER(C.c_size_t)]
        l.ccl_gemm_batched.argtypes = [C.POINTER(GemmDesc), C.c_int32, C.c_void_p, C.c_int64, C.c_void_p, C.c_int64, C.c_void_p, C.c_int64,
                                       C.c_void_p, C.c_size_t, C.c_void_p]
        l.ccl_gemm_axpby.argtypes = [C.POINTER(GemmDesc), C.c_float, C.c_float, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
        l.ccl_gemm_swiglu.argtypes = [C.POINTER(GemmDesc), C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        l.ccl_gemm_static_ws.argtypes = [C.POINTER(GemmDesc), C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        l.ccl_gemm_status.argtypes = [C.c_void_p, C.POINTER(C.c_int32)]
        l.ccl_selftest_wait_timeout.argtypes = [C.c_int32, C.c_uint32, C.c_void_p, C.c_void_p]
        l.ccl_traffic_sizes.argtypes = [C.POINTER(TrafficDesc), C.POINTER(C.c_int64), C.POINTER(C.c_int64)]
        l.ccl_traffic.argtypes = [C.POINTER(TrafficDesc), C.c_void_p, C.c_void_p, C.POINTER(C.c_void_p), C.POINTER(C.c_void_p),
                                  C.c_void_p, C.c_void_p]
        l.ccl_traffic_l2.argtypes = [C.POINTER(TrafficDesc), C.c_void_p, C.c_void_p, C.c_void_p]
        l.ccl_traffic_lru.argtypes = [C.POINTER(TrafficDesc), C.POINTER(L2Model), C.c_void_p, C.c_void_p]
        _lib = l
    return _lib


def _check(status):
    if status != OK:
        raise CclError(status, lib().ccl_last_error().decode())


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _ptr(t):
    return C.c_void_p(t.data_ptr()) if t is not None else None


def ccl_version():
    return lib().ccl_version().decode()


def ccl_launch_count():
    return int(lib().ccl_launch_count())


def ccl_map_offset(m, r, c):
    off = C.c_int64()
    _check(lib().ccl_map_offset(C.byref(m), r, c, C.byref(off)))
    return off.value


def ccl_map_inverse(m, elem_off):
    r, c = C.c_int64(), C.c_int64()
    _check(lib().ccl_map_inverse(C.byref(m), elem_off, C.byref(r), C.byref(c)))
    return r.value, c.value


_bytes_cache = {}


def ccl_buffer_bytes(m):
    key = (m.rows, m.cols, m.elem_bytes, m.P, m.part, m.layout, m.strip_align_bytes)
    v = _bytes_cache.get(key)
    if v is None:
        b = C.c_int64()
        _check(lib().ccl_buffer_bytes(C.byref(m), C.byref(b)))
        v = _bytes_cache[key] = b.value
    return v


def ccl_strip_stride(m):
    b = C.c_int64()
    _check(lib().ccl_strip_stride(C.byref(m), C.byref(b)))
    return b.value


def ccl_repack(m, src, dst, direction=0):
    """src, dst: CUDA tensors (any dtype; only their bytes matter)."""
    need_src = m.rows * m.cols * m.elem_bytes if direction == 0 else ccl_buffer_bytes(m)
    need_dst = ccl_buffer_bytes(m) if direction == 0 else m.rows * m.cols * m.elem_bytes
    if src.numel() * src.element_size() < need_src or dst.numel() * dst.element_size() < need_dst:
        raise ValueError("ccl_repack: buffer too small")
    _check(lib().ccl_repack(C.byref(m), _ptr(src), _ptr(dst), direction, _stream()))


def ccl_repack_transpose(m, src, dst):
    """src: the row-major transpose [cols x rows] of the matrix `m` describes; dst: the layout `m` describes."""
    if src.numel() * src.element_size() < m.rows * m.cols * m.elem_bytes or dst.numel() * dst.element_size() < ccl_buffer_bytes(m):
        raise ValueError("ccl_repack_transpose: buffer too small")
    _check(lib().ccl_repack_transpose(C.byref(m), _ptr(src), _ptr(dst), _stream()))


def ccl_repack_batched(m, batch, src, src_stride_bytes, dst, dst_stride_bytes, direction=0):
    """`batch` matrices of one descriptor in one launch; matrix i at src + i * src_stride_bytes -> dst + i * dst_stride_bytes."""
    need_src = m.rows * m.cols * m.elem_bytes if direction == 0 else ccl_buffer_bytes(m)
    need_dst = ccl_buffer_bytes(m) if direction == 0 else m.rows * m.cols * m.elem_bytes
    if batch >= 1 and (src.numel() * src.element_size() < (batch - 1) * src_stride_bytes + need_src
                       or dst.numel() * dst.element_size() < (batch - 1) * dst_stride_bytes + need_dst):
        raise ValueError("ccl_repack_batched: buffer too small")
    _check(lib().ccl_repack_batched(C.byref(m), batch, _ptr(src), src_stride_bytes, _ptr(dst), dst_stride_bytes, direction, _stream()))


def ccl_gemm_workspace(d):
    n = C.c_size_t()
    _check(lib().ccl_gemm_workspace(C.byref(d), C.byref(n)))
    return n.value


def ccl_gemm(d, A, B, Cout, ws=None):
    for t, m in ((A, d.A), (B, d.B), (Cout, d.C)):
        if t.numel() * t.element_size() < ccl_buffer_bytes(m):
            raise ValueError("ccl_gemm: operand buffer too small")
    ws_bytes = ws.numel() * ws.element_size() if ws is not None else 0
    _check(lib().ccl_gemm(C.byref(d), _ptr(A), _ptr(B), _ptr(Cout), _ptr(ws), ws_bytes, _stream()))


def ccl_gemm_batched_workspace(d, batch):
    n = C.c_size_t()
    _check(lib().ccl_gemm_batched_workspace(C.byref(d), batch, C.byref(n)))
    return n.value


def ccl_gemm_batched(d, batch, A, a_stride, B, b_stride, Cout, c_stride, ws=None):
    """`batch` GEMMs of one shape in one launch; X_stride: bytes between consecutive problems' buffers (0: shared A / B)."""
    for t, m, st in ((A, d.A, a_stride), (B, d.B, b_stride), (Cout, d.C, c_stride)):
        if t.numel() * t.element_size() < (batch - 1) * st + ccl_buffer_bytes(m):
            raise ValueError("ccl_gemm_batched: operand buffer too small")
    ws_bytes = ws.numel() * ws.element_size() if ws is not None else 0
    _check(lib().ccl_gemm_batched(C.byref(d), batch, _ptr(A), a_stride, _ptr(B), b_stride, _ptr(Cout), c_stride, _ptr(ws), ws_bytes, _stream()))


def ccl_probe_l2_latency(zero_buf, nlines, stride_bytes, nctas):
    """Returns (lat [nctas x nlines] float32 CUDA tensor of cycles per load, smid [nctas] int32 CUDA tensor)."""
    if zero_buf.numel() * zero_buf.element_size() < (nlines - 1) * stride_bytes + 8:
        raise ValueError("ccl_probe_l2_latency: buffer too small")
    lat = torch.zeros((nctas, nlines), dtype=torch.float32, device=zero_buf.device)
    smid = torch.zeros(nctas, dtype=torch.int32, device=zero_buf.device)
    _check(lib().ccl_probe_l2_latency(_ptr(zero_buf), nlines, stride_bytes, nctas, _ptr(lat), _ptr(smid), _stream()))
    return lat, smid


def ccl_gemm_grouped_k(d, groups, k_offsets, A, B, Cbuf, c_stride_bytes):
    """Ragged K: problem e contracts rows [k_offsets[e], k_offsets[e + 1]) of A [K x M] and B [K x N] into its own C."""
    if k_offsets.dtype != torch.int32 or not k_offsets.is_cuda or k_offsets.numel() < groups + 1:
        raise ValueError("ccl_gemm_grouped_k: k_offsets must be an int32 CUDA tensor with groups + 1 entries")
    _check(lib().ccl_gemm_grouped_k(C.byref(d), groups, _ptr(k_offsets), _ptr(A), _ptr(B), _ptr(Cbuf), c_stride_bytes, _stream()))


def ccl_gemm_grouped_swiglu(d, groups, max_rows, row_offsets, A, B, b_stride_bytes, Cbuf):
    """ccl_gemm_grouped with silu(gate) * up in the epilogue (d.N = gate + up columns, C [M x N/2])."""
    if row_offsets.dtype != torch.int32 or not row_offsets.is_cuda or row_offsets.numel() < groups + 1:
        raise ValueError("ccl_gemm_grouped_swiglu: row_offsets must be an int32 CUDA tensor with groups + 1 entries")
    _check(lib().ccl_gemm_grouped_swiglu(C.byref(d), groups, max_rows, _ptr(row_offsets), _ptr(A), _ptr(B), b_stride_bytes, _ptr(Cbuf), _stream()))


def ccl_gemm_grouped(d, groups, max_rows, row_offsets, A, B, b_stride_bytes, Cbuf):
    """Ragged batch: problem e owns rows [row_offsets[e], row_offsets[e + 1]) of A [M x K] and C [M x N] and has its own B
    (b_stride_bytes apart).  row_offsets: int32 CUDA tensor with groups + 1 entries."""
    if row_offsets.dtype != torch.int32 or not row_offsets.is_cuda or row_offsets.numel() < groups + 1:
        raise ValueError("ccl_gemm_grouped: row_offsets must be an int32 CUDA tensor with groups + 1 entries")
    _check(lib().ccl_gemm_grouped(C.byref(d), groups, max_rows, _ptr(row_offsets), _ptr(A), _ptr(B), b_stride_bytes, _ptr(Cbuf), _stream()))


def ccl_gemm_axpby(d, alpha, beta, A, B, Cinout, ws=None):
    """C <- alpha * A*B + beta * C."""
    for t, m in ((A, d.A), (B, d.B), (Cinout, d.C)):
        if t.numel() * t.element_size() < ccl_buffer_bytes(m):
            raise ValueError("ccl_gemm_axpby: operand buffer too small")
    ws_bytes = ws.numel() * ws.element_size() if ws is not None else 0
    _check(lib().ccl_gemm_axpby(C.byref(d), alpha, beta, _ptr(A), _ptr(B), _ptr(Cinout), _ptr(ws), ws_bytes, _stream()))


def ccl_gemm_swiglu(d, A, B, Cout):
    """C[M x N/2] = silu(gate) * up of the product with a fused gate/up weight (d.C describes the output)."""
    for t, m in ((A, d.A), (B, d.B), (Cout, d.C)):
        if t.numel() * t.element_size() < ccl_buffer_bytes(m):
            raise ValueError("ccl_gemm_swiglu: operand buffer too small")
    _check(lib().ccl_gemm_swiglu(C.byref(d), _ptr(A), _ptr(B), _ptr(Cout), _stream()))


GEMM_STATIC_WS_BYTES = 8 * 1024 * 1024


def ccl_gemm_static_ws(d, A, B, Cout):
    """ccl_gemm without a workspace argument: split-K partial sums go to the scratch array built into the library
    (for callers that cannot allocate device memory).  Raises CclError(ERR_WORKSPACE) if the problem needs more
    than GEMM_STATIC_WS_BYTES."""
    for t, m in ((A, d.A), (B, d.B), (Cout, d.C)):
        if t.numel() * t.element_size() < ccl_buffer_bytes(m):
            raise ValueError("ccl_gemm_static_ws: operand buffer too small")
    _check(lib().ccl_gemm_static_ws(C.byref(d), _ptr(A), _ptr(B), _ptr(Cout), _stream()))


def ccl_gemm_status():
    detail = C.c_int32()
    st = lib().ccl_gemm_status(_stream(), C.byref(detail))
    return st, detail.value


def ccl_selftest_wait_timeout(which, limit_us, src=None):
    """Test support: launches a CTA whose bounded wait runs out after limit_us (0: the GEMM's path, 1: the repack ring)."""
    _check(lib().ccl_selftest_wait_timeout(which, limit_us, _ptr(src), _stream()))


def ccl_traffic_sizes(d):
    nt = C.c_int64()
    pages = (C.c_int64 * 3)()
    _check(lib().ccl_traffic_sizes(C.byref(d), C.byref(nt), pages))
    return nt.value, list(pages)


def ccl_traffic(d, per_cta, totals, per_page=None, owner=None, cta_chiplet=None):
    """per_cta: uint64-sized CUDA tensor [ntiles,3,2]; totals [3,2]; per_page / owner: lists of 3 tensors or None."""
    pp = (C.c_void_p * 3)(*[(t.data_ptr() if t is not None else None) for t in per_page]) if per_page is not None else None
    ow = (C.c_void_p * 3)(*[(t.data_ptr() if t is not None else None) for t in owner]) if owner is not None else None
    _check(lib().ccl_traffic(C.byref(d), _ptr(cta_chiplet), _ptr(per_cta), pp, ow, _ptr(totals), _stream()))


def ccl_traffic_lru(d, model, totals):
    """Local / remote bytes [3,2] behind a finite LRU L2 per chiplet (tile-level model, see include/ccl.h)."""
    _check(lib().ccl_traffic_lru(C.byref(d), C.byref(model), _ptr(totals), _stream()))


def ccl_traffic_l2(d, totals_l2, cta_chiplet=None):
    """Local / remote bytes [3,2] behind an ideal private L2 per chiplet (each chiplet fetches a byte at most once)."""
    _check(lib().ccl_traffic_l2(C.byref(d), _ptr(cta_chiplet), _ptr(totals_l2), _stream()))
