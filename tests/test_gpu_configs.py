"""GPU parity on the benchmark configurations' own shapes: the token-count / chiplet-count / page-size sweep
(M in {1,16,128,1024}, P in {2,4,8}, pages of 4 KB / 64 KB / 2 MB) and the backward GEMMs, through the C ABI,
against the oracle.  Counts and repacks bit for bit, GEMMs within the stated tolerance."""
import numpy as np
import pytest
import torch

import oracle as orc
from paper_2606_11718_b200 import binding as ccl
from paper_2606_11718_b200 import synth
from helpers import gemm_desc, mat_pair, traffic_pair
from test_gpu_gemm import check
from test_gpu_repack_traffic import run_repack, run_traffic

pytestmark = pytest.mark.gpu

LLAMA = {g["name"]: g for g in synth.llama_fwd_gemms() + synth.llama_bwd_gemms()}
QWEN = {g["name"]: g for g in synth.qwen_ffn_gemms()}
POLICIES = [("row_rr", ("row", "row", "row"), (0, 0, 0)), ("row_block", ("row", "row", "row"), (1, 1, 1)),
            ("ccl_block", ("row", "ccl", "ccl"), (0, 1, 1)), ("ccl_rr", ("row", "ccl", "ccl"), (0, 0, 0))]


@pytest.mark.parametrize("name", ["llama_fwd_gateup", "llama_fwd_down"])
@pytest.mark.parametrize("M", [1, 16, 128, 1024])
def test_traffic_sweep_llama(name, M):
    g = LLAMA[name]
    combos = [(4, 4096)] if M != 1024 else [(2, 4096), (4, 65536), (8, 2 << 20), (8, 4096), (2, 2 << 20)]
    for P, S in combos:
        for _, lay, place in POLICIES:
            run_traffic(*traffic_pair(M, g["N"], g["K"], P, S, lay=lay, place=place, align=S), level="runs")
        if M % P == 0 and M >= P:                                       # the M-partition of C, where it applies
            run_traffic(*traffic_pair(M, g["N"], g["K"], P, S, lay=("ccl", "row", "ccl"), place=(1, 0, 1), assign=1, align=S), level="runs")


@pytest.mark.parametrize("name", ["qwen_fwd_gateup", "qwen_fwd_down", "qwen_wgrad_gateup", "qwen_dgrad_down"])
def test_traffic_sweep_qwen(name):
    g = QWEN[name]
    for M in (1, 16, 128, 1024):
        Mx = M if name.startswith("qwen_fwd") or name.startswith("qwen_dgrad") else g["M"]
        K = g["K"] if name.startswith("qwen_fwd") or name.startswith("qwen_dgrad") else M * 4    # wgrad: K = tokens
        for P, S in [(2, 4096), (4, 65536), (8, 2 << 20), (8, 4096)]:
            for _, lay, place in POLICIES[:3]:
                run_traffic(*traffic_pair(Mx, g["N"], K, P, S, lay=lay, place=place, a_trans=g["a_trans"], b_trans=g["b_trans"], align=S),
                            level="runs")
        run_traffic(*traffic_pair(Mx, g["N"], K, 4, 4096, place=(2, 2, 2), a_trans=g["a_trans"], b_trans=g["b_trans"]), level="runs")


@pytest.mark.parametrize("name,P", [("llama_wgrad", 2), ("llama_wgrad", 4), ("llama_dgrad", 4)])
def test_traffic_llama_backward_full_size(name, P):
    g = LLAMA[name]
    for _, lay, place in (POLICIES[0], POLICIES[2]):
        run_traffic(*traffic_pair(g["M"], g["N"], g["K"], P, 4096, lay=lay, place=place, a_trans=g["a_trans"], b_trans=g["b_trans"], align=4096),
                    level="runs")


@pytest.mark.parametrize("P", [2, 4, 8])
@pytest.mark.parametrize("align", [0, 4096, 65536, 2 << 20])
def test_repack_sweep_qwen_weights(P, align):
    run_repack(dict(rows=2048, cols=1536, P=P, part=2, layout=1, align=align))      # gate+up weight: 384 / 192 / 96-element... slices
    run_repack(dict(rows=768, cols=2048, P=P, part=2, layout=1, align=align))       # down weight
    run_repack(dict(rows=1536, cols=2048, P=P, part=1, layout=1, align=align))      # stored weight [N x K] split along N = along rows


@pytest.mark.parametrize("P", [2, 8])
def test_gemm_qwen_forward_other_chiplet_counts(P):
    for name in ("qwen_fwd_gateup", "qwen_fwd_down"):
        g = QWEN[name]
        for M in (16, 1024):
            A, B = synth.gemm_operands(M, g["N"], g["K"], 0, 0, seed=0, tag=f"{name}/{M}")
            check(gemm_desc(M, g["N"], g["K"], P, ("row", "ccl", "ccl"), 0, 0, 2, 1, align=65536), A, B)


def test_gemm_m_partition_qwen():
    """C split along M (CTA groups own row strips): A and C in CCL along rows, B shared."""
    g = QWEN["qwen_fwd_gateup"]
    A, B = synth.gemm_operands(g["M"], g["N"], g["K"], 0, 0, seed=0, tag="mpart")
    check(gemm_desc(g["M"], g["N"], g["K"], 4, ("ccl", "row", "ccl"), 0, 0, 1, 1, align=4096), A, B)
