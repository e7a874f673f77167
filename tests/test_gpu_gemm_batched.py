"""GPU parity, through the C ABI: ccl_gemm_batched against the fp32 oracle, problem by problem, and against
`batch` separate ccl_gemm calls (bit for bit)."""
import math
import os

import numpy as np
import pytest
import torch

import oracle as orc
from paper_2606_11718_b200 import binding as ccl
from paper_2606_11718_b200 import synth
from helpers import gemm_desc
from test_gpu_gemm import from_layout, to_layout, tol

pytestmark = pytest.mark.gpu


def pad16(n):
    return (n + 15) // 16 * 16


def run_batched(d, batch, As, Bs, share_a=False, share_b=False, gap=0):
    """As / Bs: per-problem bf16 CPU tensors as stored.  Returns the list of C matrices (uint16 bits, logical order)."""
    sa, sb, sc = (pad16(ccl.ccl_buffer_bytes(m)) + gap for m in (d.A, d.B, d.C))
    def pack(mats, m, stride, shared):
        n = 1 if shared else batch
        buf = torch.zeros(n * stride // 2, dtype=torch.int16, device="cuda")
        for e in range(n):
            x = to_layout(synth.bits(mats[e]), m)
            buf[e * stride // 2: e * stride // 2 + x.numel()] = x
        return buf
    a_dev, b_dev = pack(As, d.A, sa, share_a), pack(Bs, d.B, sb, share_b)
    c_dev = torch.full((batch * sc // 2,), 0x7FC0, dtype=torch.int16, device="cuda")               # NaN poison
    need = ccl.ccl_gemm_batched_workspace(d, batch)
    ws = torch.full((need // 4,), float("nan"), dtype=torch.float32, device="cuda") if need else None
    ccl.ccl_gemm_batched(d, batch, a_dev, 0 if share_a else sa, b_dev, 0 if share_b else sb, c_dev, sc, ws)
    st, detail = ccl.ccl_gemm_status()
    assert st == ccl.OK, detail
    nc = ccl.ccl_buffer_bytes(d.C) // 2
    if gap:                                                       # bytes between the problems' buffers stay untouched
        tail = c_dev.view(batch, sc // 2)[:, nc:]
        assert (tail == 0x7FC0).all()
    return [from_layout(c_dev[e * sc // 2: e * sc // 2 + nc], d.C) for e in range(batch)]


def single(d, A, B):
    a_dev, b_dev = to_layout(synth.bits(A), d.A), to_layout(synth.bits(B), d.B)
    c_dev = torch.full((ccl.ccl_buffer_bytes(d.C) // 2,), 0x7FC0, dtype=torch.int16, device="cuda")
    need = ccl.ccl_gemm_workspace(d)
    ws = torch.full((need // 4,), float("nan"), dtype=torch.float32, device="cuda") if need else None
    ccl.ccl_gemm(d, a_dev, b_dev, c_dev, ws)
    assert ccl.ccl_gemm_status()[0] == ccl.OK
    return from_layout(c_dev, d.C)


CASES = [
    # M, N, K, P, layouts, a_trans, b_trans, out_part, batch
    (256, 768, 512, 4, ("row", "ccl", "ccl"), 0, 1, 2, 5),       # the expert up-projection shape, shortened K
    (130, 384, 200, 2, ("row", "ccl", "ccl"), 0, 0, 2, 3),       # ragged tiles in M and K
    (64, 512, 256, 1, ("row", "row", "row"), 1, 0, 0, 7),        # plain row-major, A stored [K x M]
    (512, 512, 192, 2, ("ccl", "row", "ccl"), 0, 0, 1, 2),       # M-partition
    (16, 1024, 2048, 2, ("row", "ccl", "ccl"), 0, 0, 2, 4),      # weight streaming, split along K in every problem
    (300, 1024, 256, 4, ("row", "ileave", "ileave"), 0, 0, 2, 3),  # page-interleaved CCL, 2 rows per chunk
]


@pytest.mark.parametrize("M,N,K,P,lay,at,bt,op,batch", CASES)
@pytest.mark.parametrize("ctas", ["auto", "1", "2", "2/384", "2/192"])
def test_batched_equals_oracle_and_single_calls(M, N, K, P, lay, at, bt, op, batch, ctas, monkeypatch):
    """ctas: CTAs per tile, optionally with the tile width forced too (the 256 + 128 pair tile; 256 x 192 pairs, whose CTAs
    stage a box and a half of an N-contiguous B)."""
    old = os.environ.pop("CCL_GEMM_CTAS", None)
    if ctas != "auto":
        os.environ["CCL_GEMM_CTAS"] = ctas.split("/")[0]
        if "/" in ctas:
            monkeypatch.setenv("CCL_GEMM_BN", ctas.split("/")[1])
    try:
        ops = [synth.gemm_operands(M, N, K, at, bt, seed=11 + e, tag="batched") for e in range(batch)]
        As, Bs = [o[0] for o in ops], [o[1] for o in ops]
        align = 1024 if "ileave" in lay else 0
        d = gemm_desc(M, N, K, P, lay, at, bt, op, 1, align=align)
        try:
            ccl.ccl_gemm_batched_workspace(d, batch)
        except ccl.CclError as e:                      # a forced variant that this operand layout does not take
            assert "/" in ctas and e.status == ccl.ERR_UNSUPPORTED
            pytest.skip("variant not available for this operand layout")
        got = run_batched(d, batch, As, Bs, gap=64)
        for e in range(batch):
            ref32, _, _ = orc.gemm(synth.bits(As[e]), synth.bits(Bs[e]), M, N, K, at, bt)
            g = synth.from_bits(got[e]).to(torch.float32).numpy()
            assert np.isfinite(g).all(), f"problem {e}: unwritten output"
            err = np.abs(g - ref32) / np.maximum(1.0, np.abs(ref32))
            assert err.max() <= tol(K), (e, err.max())
        # the same plan per problem as a single call only when the planner picks the same tile for one problem
        # as for the batch; the values agree to rounding either way, and bit for bit when it does
        one = single(d, As[-1], Bs[-1])
        diff = np.abs(synth.from_bits(one).to(torch.float32).numpy() - synth.from_bits(got[-1]).to(torch.float32).numpy())
        assert diff.max() <= 2.0 * tol(K)
    finally:
        os.environ.pop("CCL_GEMM_CTAS", None)
        if old is not None:
            os.environ["CCL_GEMM_CTAS"] = old


def test_batched_shared_operands_and_batch_of_one():
    M, N, K, P, batch = 200, 768, 320, 4, 4
    ops = [synth.gemm_operands(M, N, K, 0, 0, seed=20 + e, tag="shared") for e in range(batch)]
    d = gemm_desc(M, N, K, P, ("row", "ccl", "ccl"), 0, 0, 2, 1)
    # every problem multiplies the same A by its own B
    got = run_batched(d, batch, [ops[0][0]] * batch, [o[1] for o in ops], share_a=True)
    for e in range(batch):
        np.testing.assert_array_equal(got[e], single(d, ops[0][0], ops[e][1]))
    # ... and its own A by the same B
    got = run_batched(d, batch, [o[0] for o in ops], [ops[1][1]] * batch, share_b=True)
    for e in range(batch):
        np.testing.assert_array_equal(got[e], single(d, ops[e][0], ops[1][1]))
    # a batch of one is ccl_gemm
    np.testing.assert_array_equal(run_batched(d, 1, [ops[2][0]], [ops[2][1]])[0], single(d, ops[2][0], ops[2][1]))


def test_batched_qwen_experts_sampled():
    """The paper's MoE shape: 32 experts' up-projections (256 tokens each) in one launch; four experts checked in full."""
    g = synth.config1_gemm()
    M, N, K, at, bt, batch = g["M"], g["N"], g["K"], g["a_trans"], g["b_trans"], 32
    ops = [synth.gemm_operands(M, N, K, at, bt, seed=100 + e, tag="experts") for e in range(batch)]
    d = gemm_desc(M, N, K, 4, ("row", "ccl", "ccl"), at, bt, 2, 1)
    got = run_batched(d, batch, [o[0] for o in ops], [o[1] for o in ops])
    for e in (0, 13, 30, 31):
        ref32, _, _ = orc.gemm(synth.bits(ops[e][0]), synth.bits(ops[e][1]), M, N, K, at, bt)
        gq = synth.from_bits(got[e]).to(torch.float32).numpy()
        err = np.abs(gq - ref32) / np.maximum(1.0, np.abs(ref32))
        assert err.max() <= tol(K), (e, err.max())


def test_batched_rejections():
    import ctypes as C
    d = gemm_desc(128, 256, 64, 2, ("row", "ccl", "ccl"))
    l = ccl.lib()
    def rc(batch, sa, sb, sc):
        return l.ccl_gemm_batched(C.byref(d), batch, C.c_void_p(4096), sa, C.c_void_p(1 << 20), sb, C.c_void_p(1 << 21), sc, None, 0, None)
    na, nb, nc = (ccl.ccl_buffer_bytes(m) for m in (d.A, d.B, d.C))
    assert rc(0, na, nb, nc) == ccl.ERR_INVALID_ARG
    assert rc(70000, na, nb, nc) == ccl.ERR_INVALID_ARG
    assert rc(2, na - 16, nb, nc) == ccl.ERR_INVALID_ARG            # overlapping A buffers
    assert rc(2, na, nb, 0) == ccl.ERR_INVALID_ARG                   # C cannot be shared
    assert rc(2, na + 8, nb, nc) == ccl.ERR_ALIGN
    assert rc(2, -16, nb, nc) == ccl.ERR_INVALID_ARG
