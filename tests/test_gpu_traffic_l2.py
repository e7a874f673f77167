"""GPU parity, through the C ABI: ccl_traffic_l2 (ideal private L2 per chiplet) against the oracle's bitmap count, bit for bit."""
import numpy as np
import pytest
import torch

import oracle as orc
from paper_2606_11718_b200 import binding as ccl
from helpers import traffic_pair

pytestmark = pytest.mark.gpu


def run(do, dl, explicit_q=None):
    want = orc.traffic_ideal_l2(do, explicit_q=explicit_q)
    out = torch.full((3, 2), -1, dtype=torch.int64, device="cuda")
    q = None if explicit_q is None else torch.from_numpy(np.asarray(explicit_q, dtype=np.int32)).cuda()
    ccl.ccl_traffic_l2(dl, out, q)
    np.testing.assert_array_equal(out.cpu().numpy().view(np.uint64), want)
    return want


SHAPES = [
    dict(M=8, N=8, K=4, P=2, S=16, BM=4, BN=4),                       # the hand-enumerated case
    dict(M=130, N=384, K=96, P=4, S=256),
    dict(M=130, N=384, K=96, P=2, S=4096),
    dict(M=96, N=96, K=64, P=3, S=48, BM=32, BN=32),
    dict(M=256, N=768, K=128, P=4, S=4096, b_trans=1),
    dict(M=120, N=256, K=72, P=4, S=128, a_trans=1),
    dict(M=128, N=256, K=64, P=8, S=512, assign=1, BM=16, BN=64),
    dict(M=130, N=384, K=96, P=4, S=256, strip_tiling=0),
    dict(M=1, N=512, K=256, P=4, S=4096),
]
LAYS = [("row", "row", "row"), ("row", "ccl", "ccl"), ("ccl", "ccl", "ccl"), ("row", "ileave", "ileave")]


@pytest.mark.parametrize("shape", SHAPES)
@pytest.mark.parametrize("lay", LAYS)
@pytest.mark.parametrize("place", [(0, 0, 0), (1, 1, 1), (0, 1, 1)])
def test_ideal_l2_bit_exact(shape, lay, place):
    run(*traffic_pair(lay=lay, place=place, align=1024 if "ileave" in lay else 0, **shape))
    run(*traffic_pair(lay=lay, place=place, align=256, **shape))


def test_ideal_l2_explicit_assignment_and_rejections():
    do, dl = traffic_pair(64, 96, 32, 3, 64, BM=16, BN=32, assign=2, lay=("row", "ccl", "ccl"), place=(0, 1, 1), parts=(0, 2, 2))
    nt, _ = ccl.ccl_traffic_sizes(dl)
    run(do, dl, explicit_q=np.random.default_rng(0).integers(0, 3, size=nt).astype(np.int32))
    _, best = traffic_pair(64, 96, 32, 3, 64, place=(2, 2, 2))
    with pytest.raises(ccl.CclError) as ei:
        ccl.ccl_traffic_l2(best, torch.zeros((3, 2), dtype=torch.int64, device="cuda"))
    assert ei.value.status == ccl.ERR_UNSUPPORTED


def test_ideal_l2_qwen_config_closed_forms():
    """A Qwen-size GEMM (bitmaps still small enough for the oracle) and the closed forms that hold behind an ideal L2:
    every chiplet fetches the shared operand A once (local |A|, remote (P-1)|A| under round-robin), and with CCL + whole-page
    strips B and C never leave their chiplet."""
    from paper_2606_11718_b200 import synth
    g = synth.qwen_ffn_gemms()[0]
    M, N, K, P = 1024, g["N"], g["K"], 4
    base = dict(M=M, N=N, K=K, P=P, S=4096)
    rr = run(*traffic_pair(**base))
    cc = run(*traffic_pair(lay=("row", "ccl", "ccl"), place=(0, 1, 1), align=4096, **base))
    a_bytes = M * K * 2
    assert tuple(cc[0]) == (a_bytes, (P - 1) * a_bytes) and tuple(rr[0]) == tuple(cc[0])
    assert tuple(cc[1]) == (K * N * 2, 0) and tuple(cc[2]) == (M * N * 2, 0)
    assert rr[1].sum() == K * N * 2 and rr[1, 1] > 0                  # row-major B: fetched once, but partly from other chiplets
