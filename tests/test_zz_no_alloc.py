"""ccl_gemm_static_ws: the GEMM entry point for callers that cannot allocate device memory.

Collected last on purpose (the file name sorts after every other test file), so a run that stops at
the first failure has already exercised everything else.  The new entry point must give exactly what
ccl_gemm gives with a caller-provided workspace -- same kernels, same plan -- on two calls in a row
that share the built-in scratch array, the second one a different problem that finds the first one's
partial sums still lying there.
"""
import contextlib
import ctypes as C
import os

import numpy as np
import pytest
import torch

from paper_2606_11718_b200 import binding as ccl
from paper_2606_11718_b200 import synth
from helpers import gemm_desc

pytestmark = pytest.mark.gpu


@contextlib.contextmanager
def forced_split(n):
    """Pins the plan to n K-splits of the 1-CTA kernel, so that the test does not depend on the planner's taste."""
    keys = {"CCL_GEMM_SPLITK": str(n), "CCL_GEMM_CTAS": "1"}
    old = {k: os.environ.get(k) for k in keys}
    os.environ.update(keys)
    try:
        yield
    finally:
        for k, v in old.items():
            if v is None:
                os.environ.pop(k, None)
            else:
                os.environ[k] = v


def via_existing_entry(d, a, b):
    need = ccl.ccl_gemm_workspace(d)
    assert 0 < need <= ccl.GEMM_STATIC_WS_BYTES, "pick a problem that is split along K and fits the built-in scratch"
    ws = torch.full((need // 4,), float("nan"), dtype=torch.float32, device="cuda")
    c = torch.full((d.M * d.N,), 0x7FC0, dtype=torch.int16, device="cuda")
    ccl.ccl_gemm(d, a, b, c, ws)
    assert ccl.ccl_gemm_status()[0] == ccl.OK
    return c.cpu().numpy()


def via_no_alloc_entry(d, a, b):
    c = torch.full((d.M * d.N,), 0x7FC0, dtype=torch.int16, device="cuda")     # the caller still owns inputs and output
    rc = ccl.lib().ccl_gemm_static_ws(C.byref(d), C.c_void_p(a.data_ptr()), C.c_void_p(b.data_ptr()), C.c_void_p(c.data_ptr()),
                                      C.c_void_p(torch.cuda.current_stream().cuda_stream))
    assert rc == ccl.OK, ccl.lib().ccl_last_error()
    assert ccl.ccl_gemm_status()[0] == ccl.OK
    return c.cpu().numpy()


def test_static_workspace_entry_matches_ccl_gemm_on_two_calls_in_a_row():
    with forced_split(4):
        check_two_calls_in_a_row()


def check_two_calls_in_a_row():
    problems = [(256, 768, 2048, 4, 1), (16, 1024, 4096, 2, 0)]          # M, N, K, P, b_trans: both get split along K
    expected, operands = [], []
    for M, N, K, P, bt in problems:
        A, B = synth.gemm_operands(M, N, K, 0, bt, seed=7, tag="noalloc")
        d = gemm_desc(M, N, K, P, ("row", "row", "row"), 0, bt, 2, 1)
        a, b = A.cuda(), B.cuda()
        operands.append((d, a, b, A, B))
        expected.append(via_existing_entry(d, a, b))
    got = [via_no_alloc_entry(d, a, b) for d, a, b, _, _ in operands]    # back to back, sharing the built-in scratch
    for (d, a, b, A, B), want, have in zip(operands, expected, got):
        w = synth.from_bits(want.view(np.uint16)).to(torch.float32).numpy()
        h = synth.from_bits(have.view(np.uint16)).to(torch.float32).numpy()
        assert np.isfinite(h).all()
        err = np.abs(h - w) / np.maximum(1.0, np.abs(w))
        assert err.max() <= 1e-2 * (d.K / 1024.0) ** 0.5                # the GEMM tests' tolerance ...
        np.testing.assert_array_equal(have, want)                        # ... and in fact the same bits: same kernels, same plan
        ref = (A.float() @ (B.float().T if d.b_trans else B.float())).numpy().reshape(-1)
        assert (np.abs(h - ref) / np.maximum(1.0, np.abs(ref))).max() <= 1e-2 * (d.K / 1024.0) ** 0.5
    # and once more in the opposite order
    np.testing.assert_array_equal(via_no_alloc_entry(*operands[0][:3]), expected[0])


def test_static_workspace_entry_rejects_what_does_not_fit():
    d = gemm_desc(128, 8192, 28672, 4, ("row", "row", "row"), 0, 0, 2, 1)      # weight streaming, long K: 16 MB of partial sums
    with forced_split(4):
        assert ccl.ccl_gemm_workspace(d) > ccl.GEMM_STATIC_WS_BYTES
        rc = ccl.lib().ccl_gemm_static_ws(C.byref(d), C.c_void_p(256), C.c_void_p(512), C.c_void_p(1024), None)
        assert rc == ccl.ERR_WORKSPACE
        assert b"built-in scratch" in ccl.lib().ccl_last_error()
    big = gemm_desc(1024, 1024, 1024, 1, ("row", "row", "row"), 0, 0, 0, 0)    # needs no workspace at all: runs as usual
    assert ccl.ccl_gemm_workspace(big) == 0
    A, B = synth.gemm_operands(1024, 1024, 1024, 0, 0, seed=8, tag="noalloc2")
    a, b = A.cuda(), B.cuda()
    c1 = torch.zeros(1024 * 1024, dtype=torch.int16, device="cuda")
    ccl.ccl_gemm(big, a, b, c1)
    np.testing.assert_array_equal(via_no_alloc_entry(big, a, b), c1.cpu().numpy())
