"""GPU parity, through the C ABI: ccl_gemm_grouped (a ragged batch: every problem its own row count and its own B)
against the fp32 oracle problem by problem; rows no problem owns stay untouched."""
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
POISON = 0x7FC0


def pad16(n):
    return (n + 15) // 16 * 16


def run_grouped(N, K, P, lay, bt, counts, first=0, slack=0, max_rows=None, expect=ccl.OK, share_b=False):
    """counts[e] rows for problem e, the first problem starts at row `first`, `slack` unowned rows at the end.
    Returns (C bits [M x N], offsets, As, Bs)."""
    E = len(counts)
    offs = np.concatenate([[first], first + np.cumsum(counts)]).astype(np.int32)
    M = int(offs[-1]) + slack
    d = gemm_desc(M, N, K, P, lay, 0, bt, 2, 1)
    A = synth.gemm_operands(M, N, K, 0, bt, seed=5, tag="grouped")[0]
    Bs = [synth.gemm_operands(8, N, K, 0, bt, seed=40 + e, tag="grouped")[1] for e in range(E)]
    sb = pad16(ccl.ccl_buffer_bytes(d.B)) + 64
    b_dev = torch.zeros((1 if share_b else E) * sb // 2, dtype=torch.int16, device="cuda")
    for e in range(1 if share_b else E):
        x = to_layout(synth.bits(Bs[e]), d.B)
        b_dev[e * sb // 2: e * sb // 2 + x.numel()] = x
    a_dev = to_layout(synth.bits(A), d.A)
    nc = ccl.ccl_buffer_bytes(d.C) // 2
    c_dev = torch.full((nc + 4096,), POISON, dtype=torch.int16, device="cuda")
    ccl.ccl_gemm_grouped(d, E, max_rows if max_rows is not None else max(1, int(max(counts))), torch.from_numpy(offs).cuda(),
                         a_dev, b_dev, 0 if share_b else sb, c_dev)
    st, detail = ccl.ccl_gemm_status()
    assert st == expect, (st, detail)
    assert (c_dev[nc:] == POISON).all(), "wrote past the end of C"
    return from_layout(c_dev[:nc], d.C), offs, A, Bs


def check(Cbits, offs, A, Bs, N, K, bt, skip=()):
    g = synth.from_bits(Cbits).to(torch.float32).numpy()
    a_bits = synth.bits(A)
    M = Cbits.shape[0]
    owned = np.zeros(M, dtype=bool)
    for e in range(len(Bs)):
        o0, o1 = int(offs[e]), int(offs[e + 1])
        if o1 <= o0 or e in skip:
            continue
        owned[o0:o1] = True
        ref32, _, _ = orc.gemm(a_bits[o0:o1], synth.bits(Bs[e]), o1 - o0, N, K, 0, bt)
        assert np.isfinite(g[o0:o1]).all(), f"problem {e}: unwritten output"
        err = np.abs(g[o0:o1] - ref32) / np.maximum(1.0, np.abs(ref32))
        assert err.max() <= tol(K), (e, err.max())
    assert (Cbits[~owned] == POISON).all(), "rows no problem owns were written"


CASES = [
    # N, K, P, layouts, b_trans, counts, first, slack
    (768, 512, 4, ("row", "ccl", "ccl"), 1, [256, 0, 37, 300, 1, 128, 513], 0, 0),     # expert up-projections, ragged token counts
    (384, 200, 2, ("row", "ccl", "ccl"), 0, [130, 5, 260], 3, 9),                       # unowned rows before and after, ragged K
    (512, 256, 1, ("row", "row", "row"), 0, [64, 64, 64, 64], 0, 0),                    # equal counts: a plain batch
    (1024, 256, 4, ("row", "ccl", "row"), 0, [700, 20], 0, 0),                          # C row-major
    (512, 1088, 2, ("row", "ccl", "ccl"), 1, [1, 2, 3, 250, 4], 8, 0),
]


@pytest.mark.parametrize("N,K,P,lay,bt,counts,first,slack", CASES)
@pytest.mark.parametrize("tile", ["auto", "1,128", "1,256", "2,256", "2,512"])
@pytest.mark.parametrize("walk", ["dense", "skip"])
def test_grouped_equals_oracle(N, K, P, lay, bt, counts, first, slack, tile, walk):
    """Both tile walks: the dense one (a prefix of the problems' tile counts) and the fixed grid of max_rows per problem
    with empty tiles skipped, which batches of more than 4096 problems use."""
    saved = {k: os.environ.pop(k, None) for k in ("CCL_GEMM_CTAS", "CCL_GEMM_BN", "CCL_GEMM_RAGGED_DENSE")}
    if tile != "auto":
        os.environ["CCL_GEMM_CTAS"], os.environ["CCL_GEMM_BN"] = tile.split(",")
    if walk == "skip":
        os.environ["CCL_GEMM_RAGGED_DENSE"] = "0"
    try:
        Cb, offs, A, Bs = run_grouped(N, K, P, lay, bt, counts, first, slack)
        check(Cb, offs, A, Bs, N, K, bt)
        # a looser bound on the rows per problem gives the same bits (more empty tiles, same tiles computed)
        Cb2, _, _, _ = run_grouped(N, K, P, lay, bt, counts, first, slack, max_rows=min(int(offs[-1]) + slack, max(counts) + 300))
        np.testing.assert_array_equal(Cb, Cb2)
    finally:
        for k, v in saved.items():
            os.environ.pop(k, None)
            if v is not None:
                os.environ[k] = v


def test_grouped_shared_b_is_one_gemm():
    """With one shared B the ragged batch is a plain GEMM on the owned rows."""
    N, K, P = 768, 320, 4
    Cb, offs, A, Bs = run_grouped(N, K, P, ("row", "ccl", "ccl"), 0, [100, 28, 200], share_b=True)
    check(Cb, offs, A, [Bs[0]] * 3, N, K, 0)


def test_grouped_reports_a_problem_that_exceeds_the_bound():
    """A problem with more rows than max_rows is left out and reported; the others are computed."""
    N, K, P = 512, 256, 2
    counts = [40, 300, 64]
    Cb, offs, A, Bs = run_grouped(N, K, P, ("row", "ccl", "ccl"), 0, counts, max_rows=128, expect=ccl.ERR_SHAPE)
    check(Cb, offs, A, Bs, N, K, 0, skip=(1,))
    assert ccl.ccl_gemm_status()[0] == ccl.OK                      # the flag is cleared by the read


def test_grouped_qwen_experts_full_size():
    """128 experts of the Qwen-style layer with 32768 routed tokens (uneven counts): sampled problems in full."""
    rng = np.random.default_rng(9)
    w = rng.dirichlet(np.full(128, 2.0))
    counts = np.floor(w * 32768).astype(np.int64)
    counts[0] += 32768 - counts.sum()
    Cb, offs, A, Bs = run_grouped(768, 2048, 4, ("row", "ccl", "ccl"), 1, [int(c) for c in counts], max_rows=int(counts.max()))
    g = synth.from_bits(Cb).to(torch.float32).numpy()
    assert np.isfinite(g).all()
    a_bits = synth.bits(A)
    for e in (0, 17, 64, 127):
        o0, o1 = int(offs[e]), int(offs[e + 1])
        ref32, _, _ = orc.gemm(a_bits[o0:o1], synth.bits(Bs[e]), o1 - o0, 768, 2048, 0, 1)
        err = np.abs(g[o0:o1] - ref32) / np.maximum(1.0, np.abs(ref32))
        assert err.max() <= tol(2048), (e, err.max())


SWIGLU_CASES = [
    # N (gate + up), K, P, layouts, b_trans, counts
    (1536, 512, 4, ("row", "ccl", "ccl"), 1, [256, 0, 37, 300, 1, 130]),      # Qwen expert gate/up, strips of 192 | 192
    (1024, 200, 2, ("row", "ccl", "ccl"), 0, [130, 5, 260]),
    (512, 256, 1, ("row", "row", "row"), 0, [64, 200]),
]


@pytest.mark.parametrize("N,K,P,lay,bt,counts", SWIGLU_CASES)
@pytest.mark.parametrize("walk", ["dense", "skip"])
def test_grouped_swiglu_equals_oracle(N, K, P, lay, bt, counts, walk):
    """The first half of an MoE expert FFN in one launch: per problem silu(gate) * up of its rows times its own B."""
    saved = os.environ.pop("CCL_GEMM_RAGGED_DENSE", None)
    if walk == "skip":
        os.environ["CCL_GEMM_RAGGED_DENSE"] = "0"
    try:
        E = len(counts)
        offs = np.concatenate([[0], np.cumsum(counts)]).astype(np.int32)
        M = int(offs[-1]) + 5                                         # five rows nobody owns
        d = gemm_desc(M, N, K, P, lay, 0, bt, 2, 1)
        c = d.C
        d.C = ccl.Mat(M, N // 2, 2, c.P, c.part, c.layout, c.strip_align_bytes)
        A = synth.gemm_operands(M, N, K, 0, bt, seed=6, tag="grouped_swiglu")[0]
        Bs = [synth.gemm_operands(8, N, K, 0, bt, seed=60 + e, tag="grouped_swiglu", b_std=0.05)[1] for e in range(E)]
        sb = pad16(ccl.ccl_buffer_bytes(d.B))
        b_dev = torch.zeros(E * sb // 2, dtype=torch.int16, device="cuda")
        for e in range(E):
            x = to_layout(synth.bits(Bs[e]), d.B)
            b_dev[e * sb // 2: e * sb // 2 + x.numel()] = x
        nc = ccl.ccl_buffer_bytes(d.C) // 2
        c_dev = torch.full((nc + 4096,), POISON, dtype=torch.int16, device="cuda")
        ccl.ccl_gemm_grouped_swiglu(d, E, max(counts), torch.from_numpy(offs).cuda(), to_layout(synth.bits(A), d.A), b_dev, sb, c_dev)
        assert ccl.ccl_gemm_status()[0] == ccl.OK
        assert (c_dev[nc:] == POISON).all()
        got = from_layout(c_dev[:nc], d.C)
        g = synth.from_bits(got).to(torch.float32).numpy()
        a_bits = synth.bits(A)
        S = P if P > 1 else 1
        for e in range(E):
            o0, o1 = int(offs[e]), int(offs[e + 1])
            if o1 == o0:
                continue
            ref32, _ = orc.gemm_swiglu(a_bits[o0:o1], synth.bits(Bs[e]), o1 - o0, N, K, P=S, a_trans=0, b_trans=bt)
            assert np.isfinite(g[o0:o1]).all()
            err = np.abs(g[o0:o1] - ref32) / np.maximum(1.0, np.abs(ref32))
            assert err.max() <= tol(K) + 2.0 ** -8, (e, err.max())
        assert (got[int(offs[-1]):] == POISON).all(), "rows no problem owns were written"
    finally:
        os.environ.pop("CCL_GEMM_RAGGED_DENSE", None)
        if saved is not None:
            os.environ["CCL_GEMM_RAGGED_DENSE"] = saved


RAGGED_K = [
    # M, N, P, layouts, counts (rows of K per problem)
    (768, 512, 4, ("row", "ccl", "ccl"), [256, 0, 37, 300, 1, 128, 64, 17]),      # expert weight gradients, ragged token counts
    (256, 384, 2, ("row", "ccl", "ccl"), [130, 5, 260, 16, 15, 49]),
    (128, 256, 1, ("row", "row", "row"), [64, 64, 128]),                          # whole blocks only
    (256, 1024, 4, ("ccl", "ccl", "row"), [1000, 3]),                             # A split along M, C row-major
]


@pytest.mark.parametrize("M,N,P,lay,counts", RAGGED_K)
@pytest.mark.parametrize("bn", ["auto", "128", "192", "256"])
def test_grouped_k_equals_oracle(M, N, P, lay, counts, bn):
    """Ragged K (the weight gradients of the experts): problem e contracts its own rows of A [K x M] and B [K x N]."""
    saved = os.environ.pop("CCL_GEMM_BN", None)
    if bn != "auto":
        os.environ["CCL_GEMM_BN"] = bn
    try:
        E = len(counts)
        offs = np.concatenate([[0], np.cumsum(counts)]).astype(np.int32)
        K = int(offs[-1]) + 11                                          # eleven rows no problem owns
        parts = (2 if lay[0] == "ccl" else 0, 2, 2)                      # A [K x M] split along M, B [K x N] and C along N
        d = gemm_desc(M, N, K, P, lay, 1, 0, 2, 1, parts=parts)
        d.C = ccl.Mat(M, N, 2, d.C.P, d.C.part, d.C.layout, d.C.strip_align_bytes)
        A, B = synth.gemm_operands(M, N, K, 1, 0, seed=7, tag="grouped_k")
        a_bits, b_bits = synth.bits(A), synth.bits(B)
        try:
            sc = pad16(ccl.ccl_buffer_bytes(d.C)) + 64
            c_dev = torch.full((E * sc // 2 + 4096,), POISON, dtype=torch.int16, device="cuda")
            ccl.ccl_gemm_grouped_k(d, E, torch.from_numpy(offs).cuda(), to_layout(a_bits, d.A), to_layout(b_bits, d.B), c_dev, sc)
        except ccl.CclError as e:
            assert e.status == ccl.ERR_UNSUPPORTED
            pytest.skip("tile width not available for this operand layout")
        assert ccl.ccl_gemm_status()[0] == ccl.OK
        nc = ccl.ccl_buffer_bytes(d.C) // 2
        buf = c_dev[:E * sc // 2].view(E, sc // 2)
        assert (buf[:, nc:] == POISON).all() and (c_dev[E * sc // 2:] == POISON).all(), "wrote between or past the outputs"
        for e in range(E):
            o0, o1 = int(offs[e]), int(offs[e + 1])
            got = synth.from_bits(from_layout(buf[e, :nc], d.C)).to(torch.float32).numpy()
            if o1 == o0:
                assert (got == 0).all(), f"problem {e} has no rows: its output is zero"
                continue
            ref32, _, _ = orc.gemm(a_bits[o0:o1], b_bits[o0:o1], M, N, o1 - o0, 1, 0)
            assert np.isfinite(got).all()
            err = np.abs(got - ref32) / np.maximum(1.0, np.abs(ref32))
            assert err.max() <= tol(max(o1 - o0, 64)), (e, o1 - o0, err.max())
    finally:
        os.environ.pop("CCL_GEMM_BN", None)
        if saved is not None:
            os.environ["CCL_GEMM_BN"] = saved


def test_grouped_k_neighbours_do_not_leak():
    """The rows after a problem's last row belong to its neighbour: huge values there must not reach the result."""
    M, N, counts = 128, 256, [37, 90]
    offs = np.array([0, 37, 127], dtype=np.int32)
    K = 127
    d = gemm_desc(M, N, K, 1, ("row", "row", "row"), 1, 0, 0, 0)
    A, B = synth.gemm_operands(M, N, K, 1, 0, seed=8, tag="grouped_k_leak")
    a_bits, b_bits = synth.bits(A).copy(), synth.bits(B).copy()
    a_bits[37:40] = 0x7F00                                              # ~1.7e38 in the first rows of the second problem
    b_bits[37:40] = 0x7F80                                              # +inf
    nc = M * N
    c_dev = torch.full((2 * nc,), POISON, dtype=torch.int16, device="cuda")
    ccl.ccl_gemm_grouped_k(d, 2, torch.from_numpy(offs).cuda(), to_layout(a_bits, d.A), to_layout(b_bits, d.B), c_dev, nc * 2)
    assert ccl.ccl_gemm_status()[0] == ccl.OK
    got = synth.from_bits(c_dev[:nc].cpu().numpy().view(np.uint16).reshape(M, N)).to(torch.float32).numpy()
    ref32, _, _ = orc.gemm(a_bits[:37], b_bits[:37], M, N, 37, 1, 0)
    assert np.isfinite(got).all()
    assert (np.abs(got - ref32) / np.maximum(1.0, np.abs(ref32))).max() <= tol(64)
