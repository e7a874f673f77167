"""GPU parity, through the C ABI: ccl_gemm_swiglu against the oracle's gated-activation GEMM.

Tolerance: the GEMM's own (1e-2 * sqrt(K/1024) relative to max(1, |ref|)) applied to the activation output, plus the
rounding of that output to bf16, half an ulp = 2^-8 relative at most (for short K the GEMM term alone, 2.5e-3 at
K = 64, is smaller than that rounding); the device's fast exp (2 ulp of fp32) is far inside either."""
import ctypes as C

import numpy as np
import pytest
import torch

import oracle as orc
from paper_2606_11718_b200 import binding as ccl
from paper_2606_11718_b200 import synth
from helpers import gemm_desc
from test_gpu_gemm import GUARD, from_layout, to_layout, tol

pytestmark = pytest.mark.gpu


def swiglu_desc(M, N, K, P, lay, at, bt, out_part=2, grouped=1, align=0):
    d = gemm_desc(M, N, K, P, lay, at, bt, out_part, grouped, align=align)
    c = d.C
    d.C = ccl.Mat(M, N // 2, 2, c.P, c.part, c.layout, c.strip_align_bytes)          # the output is half as wide
    return d


def run(d, A, B):
    a_dev, b_dev = to_layout(synth.bits(A), d.A), to_layout(synth.bits(B), d.B)
    nc = ccl.ccl_buffer_bytes(d.C) // 2
    c_dev = torch.full((nc + GUARD,), 0x7FC0, dtype=torch.int16, device="cuda")   # NaN poison, and a guard zone behind C
    ccl.ccl_gemm_swiglu(d, a_dev, b_dev, c_dev)
    st, detail = ccl.ccl_gemm_status()
    assert st == ccl.OK, detail
    assert (c_dev[nc:] == 0x7FC0).all(), "the kernel wrote past the end of C"
    return from_layout(c_dev[:nc], d.C)


CASES = [
    # M, N (gate + up), K, P, layouts(A, B, C), a_trans, b_trans, out_part
    (256, 512, 64, 1, ("row", "row", "row"), 0, 0, 0),          # one tile: gate = columns 0..255, up = 256..511
    (256, 512, 256, 1, ("row", "row", "row"), 0, 1, 0),         # B stored [N x K]
    (130, 1536, 200, 4, ("row", "ccl", "ccl"), 0, 0, 2),        # strips of 384 = 192 gate | 192 up, ragged M and K
    (296, 1024, 328, 2, ("row", "ccl", "ccl"), 1, 0, 2),        # A stored [K x M]
    (520, 2048, 192, 4, ("row", "ccl", "row"), 0, 1, 2),        # CCL weight, row-major activation out
    (512, 4096, 512, 4, ("row", "row", "ccl"), 0, 0, 2),        # plain weight with per-strip halves, CCL out
    (640, 4096, 256, 2, ("row", "ccl", "ccl"), 0, 0, 2),        # several tiles per CTA pair
    (16, 1536, 512, 1, ("row", "row", "row"), 0, 0, 0),         # few rows
    (264, 1552, 128, 1, ("row", "row", "row"), 0, 0, 0),        # halves of 776 columns: ragged last tile
]


@pytest.mark.parametrize("M,N,K,P,lay,at,bt,op", CASES)
def test_swiglu_matches_oracle(M, N, K, P, lay, at, bt, op):
    A, B = synth.gemm_operands(M, N, K, at, bt, seed=21, tag="swiglu", b_std=0.05)
    for grouped, align in ((1, 0), (0, 4096)):
        d = swiglu_desc(M, N, K, P, lay, at, bt, op, grouped, align if "ccl" in lay else 0)
        got = run(d, A, B)
        S = P if (op == 2 and P > 1) else 1
        ref32, ref_bits = orc.gemm_swiglu(synth.bits(A), synth.bits(B), M, N, K, P=S, a_trans=at, b_trans=bt)
        g = synth.from_bits(got).to(torch.float32).numpy()
        assert np.isfinite(g).all(), "unwritten (poisoned) output elements"
        err = np.abs(g - ref32) / np.maximum(1.0, np.abs(ref32))
        assert err.max() <= tol(K) + 2.0 ** -8, (err.max(), tol(K))
        # most outputs round to the very same bf16 value as the oracle's
        assert (got == ref_bits).mean() > 0.97


def test_swiglu_equals_gemm_then_activation():
    """The fused call against the unfused path of this library: plain ccl_gemm, then the activation on the host."""
    M, N, K, P = 384, 2048, 512, 4
    A, B = synth.gemm_operands(M, N, K, 0, 0, seed=3, tag="swiglu2", b_std=0.05)
    d = swiglu_desc(M, N, K, P, ("row", "ccl", "ccl"), 0, 0)
    fused = synth.from_bits(run(d, A, B)).to(torch.float32)
    d0 = gemm_desc(M, N, K, P, ("row", "ccl", "ccl"), 0, 0, 2, 1)
    a_dev, b_dev = to_layout(synth.bits(A), d0.A), to_layout(synth.bits(B), d0.B)
    c_dev = torch.zeros(ccl.ccl_buffer_bytes(d0.C) // 2, dtype=torch.int16, device="cuda")
    ccl.ccl_gemm(d0, a_dev, b_dev, c_dev)
    H = synth.from_bits(from_layout(c_dev, d0.C)).to(torch.float32)              # bf16-rounded H
    Wp = N // P
    Hs = H.view(M, P, 2, Wp // 2)
    unfused = (torch.nn.functional.silu(Hs[:, :, 0]) * Hs[:, :, 1]).reshape(M, N // 2)
    # the unfused path rounds H to bf16 first: agreement to a few bf16 ulps of the operands' scale
    assert ((fused - unfused).abs() / unfused.abs().clamp(min=1.0)).max() < 2e-2


def test_swiglu_rejections():
    l = ccl.lib()
    def rc(d):
        return l.ccl_gemm_swiglu(C.byref(d), C.c_void_p(4096), C.c_void_p(1 << 20), C.c_void_p(1 << 21), None)
    assert rc(gemm_desc(128, 512, 64)) == ccl.ERR_SHAPE                                     # C described with N columns
    assert rc(swiglu_desc(128, 510, 64, 1, ("row", "row", "row"), 0, 0, 0)) == ccl.ERR_UNSUPPORTED   # halves of 255 columns
    d = swiglu_desc(128, 1024, 64, 4, ("row", "ccl", "ccl"), 0, 0)
    d.C.P = 2                                                                               # C strips are not the halves' strips
    assert rc(d) == ccl.ERR_UNSUPPORTED
    d = swiglu_desc(128, 1024, 64, 2, ("row", "ileave", "row"), 0, 0, align=1024)
    assert rc(d) == ccl.ERR_UNSUPPORTED
