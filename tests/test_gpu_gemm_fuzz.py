"""Seeded random descriptors through ccl_gemm / ccl_gemm_axpby against the oracle: shapes, strip counts (equal and
unequal strips), layouts, operand majors, output partitions, rasters and forced kernel variants drawn at random; what the
library rejects before any launch (CCL_ERR_UNSUPPORTED / CCL_ERR_SHAPE / CCL_ERR_ALIGN) is counted, everything it accepts
must match the oracle within the GEMM tolerance and leave the guard zone behind C untouched."""
import os
import random

import numpy as np
import pytest
import torch

import oracle as orc
from paper_2606_11718_b200 import binding as ccl
from paper_2606_11718_b200 import synth
from helpers import gemm_desc
from test_gpu_gemm import GUARD, from_layout, to_layout, tol

pytestmark = pytest.mark.gpu

KNOBS = ("CCL_GEMM_CTAS", "CCL_GEMM_BN", "CCL_GEMM_SPLITK", "CCL_GEMM_CLUSTERK")


def draw(rng):
    P = rng.choice([1, 2, 3, 4, 4, 8, 16])
    at, bt = rng.choice([0, 0, 1]), rng.choice([0, 1])
    op = rng.choice([2, 2, 2, 1, 0])
    M = rng.choice([1, 3, 8, 16, 100, 128, 130, 256, 264, 330, 520])
    N, K = 8 * rng.randint(1, 128), 8 * rng.randint(32, 96)    # (K >= 256: the tolerance 1e-2 sqrt(K / 1024) must leave room for the bf16
                                                               #  rounding of the output, up to 2^-8 relative to max(1, |C|))
    if at:
        M = (M + 7) // 8 * 8
    if op == 1:
        lay = (rng.choice(["ccl", "row"]), "row", rng.choice(["ccl", "row"]))
    elif op == 2:
        lay = ("row", rng.choice(["ccl", "row", "ileave"]), rng.choice(["ccl", "row", "ileave"]))
    else:
        lay = ("row", "row", "row")
    align = rng.choice([256, 1024, 2048, 4096]) if "ileave" in lay else rng.choice([0, 0, 256, 1024, 4096])
    env = {}
    if rng.random() < 0.5:
        env["CCL_GEMM_CTAS"] = rng.choice(["1", "2"])
    if rng.random() < 0.5:
        env["CCL_GEMM_BN"] = rng.choice(["128", "192", "256", "384", "512"])
    if rng.random() < 0.2:
        env["CCL_GEMM_SPLITK"] = rng.choice(["2", "3", "4"])
    if rng.random() < 0.2:
        env["CCL_GEMM_CLUSTERK"] = rng.choice(["0", "2", "4", "8"])
    scal = (1.0, 0.0) if rng.random() < 0.7 else (rng.choice([0.5, -2.0]), rng.choice([0.0, 1.0, 0.5]))
    return dict(M=M, N=N, K=K, P=P, lay=lay, at=at, bt=bt, op=op, grouped=rng.choice([0, 1]), align=align, env=env, scal=scal)


@pytest.mark.parametrize("seed", [1, 2, 3])
def test_random_descriptors_match_the_oracle(seed):
    rng = random.Random(seed)
    saved = {k: os.environ.pop(k, None) for k in KNOBS}
    accepted = rejected = 0
    try:
        while accepted < 120:
            c = draw(rng)
            for k in KNOBS:
                os.environ.pop(k, None)
            os.environ.update(c["env"])
            M, N, K, at, bt = c["M"], c["N"], c["K"], c["at"], c["bt"]
            alpha, beta = c["scal"]
            try:
                d = gemm_desc(M, N, K, c["P"], c["lay"], at, bt, c["op"], c["grouped"], align=c["align"])
                need = ccl.ccl_gemm_workspace(d)
            except ccl.CclError as e:
                assert e.status in (ccl.ERR_UNSUPPORTED, ccl.ERR_SHAPE, ccl.ERR_ALIGN, ccl.ERR_INVALID_ARG), (c, e.status)
                rejected += 1
                continue
            A, B = synth.gemm_operands(M, N, K, at, bt, seed=rng.randint(0, 1 << 30), tag="fuzz")
            Cin = synth.randn_bf16(M, N, 1.0, seed, "fuzz/C")
            a_dev, b_dev = to_layout(synth.bits(A), d.A), to_layout(synth.bits(B), d.B)
            nc = ccl.ccl_buffer_bytes(d.C) // 2
            c_dev = torch.full((nc + GUARD,), 0x7FC0, dtype=torch.int16, device="cuda")
            if beta != 0.0:
                c_dev[:nc] = to_layout(synth.bits(Cin), d.C)
            ws = torch.full((need // 4,), float("nan"), dtype=torch.float32, device="cuda") if need else None
            try:
                if (alpha, beta) == (1.0, 0.0):
                    ccl.ccl_gemm(d, a_dev, b_dev, c_dev, ws)
                else:
                    ccl.ccl_gemm_axpby(d, alpha, beta, a_dev, b_dev, c_dev, ws)
            except ccl.CclError as e:                      # (the alpha / beta form plans on its own)
                assert e.status in (ccl.ERR_UNSUPPORTED, ccl.ERR_WORKSPACE), (c, e.status)
                rejected += 1
                continue
            st, detail = ccl.ccl_gemm_status()
            assert st == ccl.OK, (c, st, detail)
            assert (c_dev[nc:] == 0x7FC0).all(), ("the kernel wrote past the end of C", c)
            got = synth.from_bits(from_layout(c_dev[:nc], d.C)).to(torch.float32).numpy()
            assert np.isfinite(got).all(), ("unwritten (poisoned) output elements", c)
            if (alpha, beta) == (1.0, 0.0):
                ref32, _, _ = orc.gemm(synth.bits(A), synth.bits(B), M, N, K, at, bt)
                lim = tol(K)
            else:
                ref32, _ = orc.gemm_axpby(synth.bits(A), synth.bits(B), synth.bits(Cin), M, N, K, alpha, beta, at, bt)
                lim = abs(alpha) * tol(K) + 2.0 ** -8
            err = np.abs(got - ref32) / np.maximum(1.0, np.abs(ref32))
            assert err.max() <= lim, (c, err.max(), lim)
            accepted += 1
    finally:
        for k in KNOBS:
            os.environ.pop(k, None)
            if saved[k] is not None:
                os.environ[k] = saved[k]
    assert rejected < 20 * accepted        # (most draws must be runnable, or the test checks little)
