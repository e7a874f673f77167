"""The expiry path of the bounded device-side waits, exercised without hanging anything: a test entry point launches
one small CTA whose wait cannot be satisfied, with a limit of a millisecond; the wait gives up by itself, the kernel
records its code and leaves the way the real kernels do (TMEM released / outstanding ring loads drained), the host
reads CCL_ERR_TIMEOUT exactly once, and the library goes on working."""
import numpy as np
import pytest
import torch

import oracle as orc
from paper_2606_11718_b200 import binding as ccl
from paper_2606_11718_b200 import synth
from helpers import gemm_desc
from test_gpu_gemm import check

pytestmark = pytest.mark.gpu


def small_gemm_passes():
    M, N, K, P = 264, 768, 328, 4
    A, B = synth.gemm_operands(M, N, K, 0, 0, seed=3, tag="after-timeout")
    check(gemm_desc(M, N, K, P, ("row", "ccl", "ccl"), 0, 0, 2, 1), A, B)


@pytest.mark.parametrize("which,code", [(0, 6), (1, 101)])
def test_bounded_wait_runs_out_and_is_reported_once(which, code):
    st, _ = ccl.ccl_gemm_status()                      # start from a clean status word
    src = torch.arange(2048, dtype=torch.uint8, device="cuda")
    ccl.ccl_selftest_wait_timeout(which, 1000, src)    # 1 ms limit
    st, detail = ccl.ccl_gemm_status()
    assert st == ccl.ERR_TIMEOUT and detail == code, (st, detail)
    assert "wait expired" in ccl.lib().ccl_last_error().decode()
    st, detail = ccl.ccl_gemm_status()                 # reported once, then cleared
    assert st == ccl.OK and detail == 0
    small_gemm_passes()                                # the context is intact: a GEMM right after passes parity
    if which == 1:                                     # ... and so does a repack through the TMA ring
        mo = orc.Mat(512, 1024, 2, 4, orc.PART_COLS, orc.CCL, 4096)
        ml = ccl.Mat(512, 1024, 2, 4, ccl.PART_COLS, ccl.CCL, 4096)
        x = np.random.default_rng(0).integers(1, 65535, size=(512, 1024), dtype=np.uint16)
        dst = torch.zeros(ccl.ccl_buffer_bytes(ml) // 2, dtype=torch.int16, device="cuda")
        ccl.ccl_repack(ml, torch.from_numpy(x.view(np.int16)).cuda(), dst, 0)
        np.testing.assert_array_equal(dst.cpu().numpy().view(np.uint16), orc.repack(mo, x, 0))
    st, _ = ccl.ccl_gemm_status()
    assert st == ccl.OK


def test_selftest_rejects_bad_arguments():
    for which, limit in ((2, 1000), (0, 0), (0, 10 ** 6)):
        with pytest.raises(ccl.CclError) as ei:
            ccl.ccl_selftest_wait_timeout(which, limit, None)
        assert ei.value.status == ccl.ERR_INVALID_ARG
    with pytest.raises(ccl.CclError) as ei:
        ccl.ccl_selftest_wait_timeout(1, 1000, None)
    assert ei.value.status == ccl.ERR_ALIGN
