"""The device entry points are plain stream work: after one eager call (which fills the library's host-side plan cache
and configures the kernels) a whole step -- repack, GEMM, split-K GEMM, batched GEMM, gated-activation GEMM, traffic
count -- can be captured into a CUDA graph and replayed, with the same bits as the eager calls."""
import numpy as np
import pytest
import torch

import oracle as orc
from paper_2606_11718_b200 import binding as ccl
from paper_2606_11718_b200 import synth
from helpers import gemm_desc, traffic_pair
from test_gpu_gemm_swiglu import swiglu_desc

pytestmark = pytest.mark.gpu


def test_step_replays_from_a_cuda_graph():
    M, N, K, P, E = 384, 1536, 512, 4, 3
    A, B = synth.gemm_operands(M, N, K, 0, 0, seed=31, tag="graph", b_std=0.05)
    a, b = A.cuda(), B.cuda()
    d = gemm_desc(M, N, K, P, ("row", "ccl", "ccl"), 0, 0, 2, 1, align=4096)
    ds = swiglu_desc(M, N, K, P, ("row", "ccl", "ccl"), 0, 0, 2, 1, align=4096)
    dk = gemm_desc(16, N, 2048, P, ("row", "ccl", "ccl"), 0, 0, 2, 1)                    # split along K
    Ak, Bk = synth.gemm_operands(16, N, 2048, 0, 0, seed=32, tag="graphk")
    ak, bk_row = Ak.cuda(), Bk.cuda()
    nb, nc = ccl.ccl_buffer_bytes(d.B) // 2, ccl.ccl_buffer_bytes(d.C) // 2
    b_ccl = torch.empty(nb, dtype=torch.bfloat16, device="cuda")
    bk_ccl = torch.empty(ccl.ccl_buffer_bytes(dk.B) // 2, dtype=torch.bfloat16, device="cuda")
    c1 = torch.zeros(nc, dtype=torch.bfloat16, device="cuda")
    c2 = torch.zeros(ccl.ccl_buffer_bytes(ds.C) // 2, dtype=torch.bfloat16, device="cuda")
    ck = torch.zeros(ccl.ccl_buffer_bytes(dk.C) // 2, dtype=torch.bfloat16, device="cuda")
    need = ccl.ccl_gemm_workspace(dk)                      # (a short problem: split along K in one way or another)
    ws = torch.empty(max(need, 16) // 4, dtype=torch.float32, device="cuda")
    ab = a.repeat(E, 1).contiguous()
    cb = torch.zeros(E * nc, dtype=torch.bfloat16, device="cuda")
    needb = ccl.ccl_gemm_batched_workspace(d, E)
    wsb = torch.empty(max(needb, 4) // 4, dtype=torch.float32, device="cuda")
    _, td = traffic_pair(M, N, K, P, 4096, ("row", "ccl", "ccl"), (0, 1, 1), align=4096)
    nt, _ = ccl.ccl_traffic_sizes(td)
    per_cta = torch.zeros((nt, 3, 2), dtype=torch.int64, device="cuda")
    totals = torch.zeros((3, 2), dtype=torch.int64, device="cuda")

    # a GEMM whose last round is cut into equal shares (partial sums and their flags in the workspace)
    db = gemm_desc(4096, 2048, 1536, P, ("row", "ccl", "ccl"), 0, 1, 2, 1)
    Ab, Bb = synth.gemm_operands(4096, 2048, 1536, 0, 1, seed=33, tag="graphb")
    import os
    os.environ["CCL_GEMM_BALANCED"] = "1"
    needbal = ccl.ccl_gemm_workspace(db)
    abal, bbal = Ab.cuda(), torch.from_numpy(orc.repack(orc.Mat(2048, 1536, 2, P, orc.PART_ROWS, orc.CCL, 0), synth.bits(Bb), 0).view(np.int16)).cuda()
    cbal = torch.zeros(ccl.ccl_buffer_bytes(db.C) // 2, dtype=torch.bfloat16, device="cuda")
    wsbal = torch.empty(needbal // 4, dtype=torch.float32, device="cuda")
    assert needbal > 0

    def step():
        ccl.ccl_gemm(db, abal, bbal, cbal, wsbal)
        ccl.ccl_repack(d.B, b, b_ccl, 0)
        ccl.ccl_repack(dk.B, bk_row, bk_ccl, 0)
        ccl.ccl_gemm(d, a, b_ccl, c1)
        ccl.ccl_gemm_swiglu(ds, a, b_ccl, c2)
        ccl.ccl_gemm(dk, ak, bk_ccl, ck, ws)
        ccl.ccl_gemm_batched(d, E, ab, M * K * 2, b_ccl, 0, cb, nc * 2, wsb if needb else None)
        ccl.ccl_traffic(td, per_cta, totals)

    outs = (c1, c2, ck, cb, per_cta, totals, cbal)
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        step()                                                   # eager: plans cached, kernels configured
        side.synchronize()
        assert ccl.ccl_gemm_status()[0] == ccl.OK
        want = [o.clone() for o in outs]
        for o in outs:
            o.zero_()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            step()
    for _ in range(3):
        for o in outs:
            o.zero_()
        graph.replay()
        torch.cuda.synchronize()
        for o, w in zip(outs, want):
            assert torch.equal(o, w)
    assert ccl.ccl_gemm_status()[0] == ccl.OK
    os.environ.pop("CCL_GEMM_BALANCED", None)
    ref32, _, _ = orc.gemm(synth.bits(Ab), synth.bits(Bb), 4096, 2048, 1536, 0, 1, block=(0, 256, 0, 2048))
    got = orc.repack(orc.Mat(4096, 2048, 2, P, orc.PART_COLS, orc.CCL, 0), cbal.view(torch.int16).cpu().numpy().view(np.uint16), 1).reshape(4096, 2048)
    g = synth.from_bits(got[:256]).to(torch.float32).numpy()
    assert (np.abs(g - ref32) / np.maximum(1.0, np.abs(ref32))).max() <= 1e-2 * (1536 / 1024.0) ** 0.5


def test_ragged_batch_in_a_graph_follows_the_offsets_on_the_device():
    """ccl_gemm_grouped reads the row offsets on the device: one captured launch serves whatever routing the offsets
    hold at replay time (as long as no problem exceeds the bound the graph was captured with)."""
    N, K, P, E, M = 768, 256, 4, 6, 1024
    A, _ = synth.gemm_operands(M, N, K, 0, 1, seed=41, tag="graph_ragged")
    Bs = [synth.gemm_operands(8, N, K, 0, 1, seed=50 + e, tag="graph_ragged")[1] for e in range(E)]
    d = gemm_desc(M, N, K, P, ("row", "row", "row"), 0, 1, 2, 1)
    a = A.cuda()
    b = torch.stack(Bs).cuda().contiguous()                              # [E, N, K] row-major
    c = torch.zeros(M * N, dtype=torch.bfloat16, device="cuda")
    offs = torch.zeros(E + 1, dtype=torch.int32, device="cuda")
    routings = [[100, 200, 0, 300, 24, 400], [400, 0, 0, 1, 223, 400], [170, 170, 170, 170, 170, 174]]

    def set_offsets(counts):
        offs.copy_(torch.tensor([0] + list(np.cumsum(counts)), dtype=torch.int32), non_blocking=False)

    def expect(counts):                                                  # the oracle's GEMM, problem by problem
        out = torch.zeros(M, N, dtype=torch.float32)
        o = 0
        for e, n in enumerate(counts):
            if n:
                out[o:o + n] = torch.from_numpy(orc.gemm(synth.bits(A)[o:o + n], synth.bits(Bs[e]), n, N, K, 0, 1)[0])
            o += n
        return out

    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        set_offsets(routings[0])
        ccl.ccl_gemm_grouped(d, E, 400, offs, a, b, N * K * 2, c)       # eager: plan cached, kernel configured
        side.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            ccl.ccl_gemm_grouped(d, E, 400, offs, a, b, N * K * 2, c)
    for counts in routings:
        set_offsets(counts)
        c.zero_()
        graph.replay()
        torch.cuda.synchronize()
        got = c.view(M, N).float().cpu()
        want = expect(counts)
        owned = sum(counts)
        err = (got[:owned] - want[:owned]).abs() / want[:owned].abs().clamp(min=1.0)
        assert err.max() <= 1e-2 * (K / 1024.0) ** 0.5 + 2.0 ** -8
        assert (got[owned:] == 0).all()
    assert ccl.ccl_gemm_status()[0] == ccl.OK


def test_large_gemm_with_its_wave_barrier_replays_from_a_graph():
    """A problem of several rounds of tiles zeroes its meeting-point counter with a memset node in front of the launch:
    captured and replayed, it gives the bits of the eager call every time."""
    M, N, K, P = 4096, 8192, 512, 4
    A, B = synth.gemm_operands(M, N, K, 0, 0, seed=61, tag="graph_big")
    d = gemm_desc(M, N, K, P, ("row", "ccl", "ccl"), 0, 0, 2, 1)
    assert ccl.ccl_gemm_workspace(d) == 0
    a = A.cuda()
    b_ccl = torch.empty(ccl.ccl_buffer_bytes(d.B) // 2, dtype=torch.bfloat16, device="cuda")
    ccl.ccl_repack(d.B, B.cuda(), b_ccl, 0)
    c = torch.zeros(ccl.ccl_buffer_bytes(d.C) // 2, dtype=torch.bfloat16, device="cuda")
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        ccl.ccl_gemm(d, a, b_ccl, c)
        side.synchronize()
        want = c.clone()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            ccl.ccl_gemm(d, a, b_ccl, c)
            ccl.ccl_gemm(d, a, b_ccl, c)                               # twice in a row: each launch has its own counter
    for _ in range(3):
        c.zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert torch.equal(c, want)
    assert ccl.ccl_gemm_status()[0] == ccl.OK
    # sampled against the oracle
    rows = [0, 1, 777, 4095]
    ref32, _, _ = orc.gemm(synth.bits(A)[rows], synth.bits(B), len(rows), N, K, 0, 0)
    from test_gpu_gemm import from_layout, tol
    got = synth.from_bits(from_layout(c.view(torch.int16), d.C)).to(torch.float32).numpy()[rows]
    assert (np.abs(got - ref32) / np.maximum(1.0, np.abs(ref32))).max() <= tol(K)
