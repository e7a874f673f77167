"""Seeded synthetic inputs and the workload shapes.

This module serves both the CUDA path's tests/benchmark and the CPU oracle's
tests.  It holds none of the method's arithmetic (no address map, no GEMM, no
counting): only random bf16 matrices and the list of GEMM shapes, which stand
in for the Qwen 3 30B / Llama 3.1 70B FFN GEMMs of the paper's Sec. 4.1
"Workloads" (shapes only: no model weights or datasets are involved).

Value recipe: activations and gradients ~ N(0, 1), weights ~ N(0, 0.02)
(0.02 is the standard deviation), drawn in fp32 from torch's CPU generator
seeded with ``seed`` and a per-operand stream id, then rounded to bf16.
"""
import zlib

import numpy as np
import torch

ACT_STD = 1.0
WEIGHT_STD = 0.02


def _gen(seed, stream):
    g = torch.Generator(device="cpu")
    g.manual_seed((int(seed) * 1000003 + zlib.crc32(str(stream).encode())) % (2 ** 63 - 1))
    return g


def randn_bf16(rows, cols, std, seed=0, stream="x"):
    """[rows x cols] bf16 CPU tensor ~ N(0, std)."""
    g = _gen(seed, stream)
    x = torch.randn(rows, cols, generator=g, dtype=torch.float32)
    if std != 1.0:
        x.mul_(std)
    return x.to(torch.bfloat16)


def bits(t):
    """bf16 CPU tensor -> numpy uint16 view of the same bits."""
    return t.contiguous().view(torch.int16).numpy().view(np.uint16)


def from_bits(a):
    """numpy uint16 bit patterns -> bf16 CPU tensor."""
    return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).view(torch.bfloat16)


def gemm_operands(M, N, K, a_trans=0, b_trans=0, seed=0, tag="", a_std=ACT_STD, b_std=WEIGHT_STD):
    """Stored operands of one GEMM: A is [M x K] (or [K x M] if a_trans), B is [K x N] (or [N x K])."""
    a_shape = (K, M) if a_trans else (M, K)
    b_shape = (N, K) if b_trans else (K, N)
    A = randn_bf16(a_shape[0], a_shape[1], a_std, seed, f"{tag}/A/{M}x{N}x{K}/{a_trans}")
    B = randn_bf16(b_shape[0], b_shape[1], b_std, seed, f"{tag}/B/{M}x{N}x{K}/{b_trans}")
    return A, B


# ---------------------------------------------------------------------------------------------
# Workload shapes.  Each GEMM: name, M, N, K, a_trans, b_trans, a_std, b_std.
# ---------------------------------------------------------------------------------------------

def qwen_ffn_gemms(T=4096, H=2048, I=768):
    """Qwen3-30B-style MoE expert FFN, forward + backward (gate and up fused, width 2*I)."""
    return [
        dict(name="qwen_fwd_gateup", M=T, N=2 * I, K=H, a_trans=0, b_trans=0, a_std=ACT_STD, b_std=WEIGHT_STD),
        dict(name="qwen_fwd_down", M=T, N=H, K=I, a_trans=0, b_trans=0, a_std=ACT_STD, b_std=WEIGHT_STD),
        dict(name="qwen_dgrad_gateup", M=T, N=H, K=2 * I, a_trans=0, b_trans=1, a_std=ACT_STD, b_std=WEIGHT_STD),
        dict(name="qwen_wgrad_gateup", M=H, N=2 * I, K=T, a_trans=1, b_trans=0, a_std=ACT_STD, b_std=ACT_STD),
        dict(name="qwen_dgrad_down", M=T, N=I, K=H, a_trans=0, b_trans=1, a_std=ACT_STD, b_std=WEIGHT_STD),
        dict(name="qwen_wgrad_down", M=I, N=H, K=T, a_trans=1, b_trans=0, a_std=ACT_STD, b_std=ACT_STD),
    ]


def llama_fwd_gemms(T=8192, H=8192, I=28672):
    """Llama-3.1-70B-style dense FFN forward."""
    return [
        dict(name="llama_fwd_gateup", M=T, N=2 * I, K=H, a_trans=0, b_trans=0, a_std=ACT_STD, b_std=WEIGHT_STD),
        dict(name="llama_fwd_down", M=T, N=H, K=I, a_trans=0, b_trans=0, a_std=ACT_STD, b_std=WEIGHT_STD),
    ]


def llama_bwd_gemms(T=8192, H=8192, I=28672):
    """Llama-3.1-70B-style FFN backward of the down projection: dgrad and wgrad (K = tokens)."""
    return [
        dict(name="llama_dgrad", M=T, N=H, K=I, a_trans=0, b_trans=0, a_std=ACT_STD, b_std=WEIGHT_STD),
        dict(name="llama_wgrad", M=I, N=H, K=T, a_trans=1, b_trans=0, a_std=ACT_STD, b_std=ACT_STD),
    ]


def config1_gemm():
    """Single Qwen3-30B-style expert up-projection: X[256x2048] times W[768x2048]^T."""
    return dict(name="qwen_expert_up", M=256, N=768, K=2048, a_trans=0, b_trans=1, a_std=ACT_STD, b_std=WEIGHT_STD)
