"""Pins for the oracle's GEMM (Sec. 2.2: C = A*B; bf16 in, fp32 accumulate, bf16 out).  No GPU."""
import numpy as np
import pytest
import torch

import oracle as orc
from paper_2606_11718_b200 import synth


def to_bits(x):
    return synth.bits(torch.as_tensor(np.asarray(x, dtype=np.float32)).to(torch.bfloat16))


def to_f64(bits_arr):
    return synth.from_bits(bits_arr).to(torch.float64).numpy()


def test_brute_force_small_integers():
    """Pure-Python triple loop on small integers (exact in every precision), all four storage combos."""
    rng = np.random.default_rng(0)
    M, N, K = 5, 7, 6
    A = rng.integers(-4, 5, size=(M, K))
    B = rng.integers(-4, 5, size=(K, N))
    want = [[sum(int(A[m, k]) * int(B[k, n]) for k in range(K)) for n in range(N)] for m in range(M)]
    for at in (0, 1):
        for bt in (0, 1):
            As = to_bits(A.T if at else A)
            Bs = to_bits(B.T if bt else B)
            r32, r64, out = orc.gemm(As, Bs, M, N, K, at, bt, want64=True)
            np.testing.assert_array_equal(r32, np.array(want, dtype=np.float32))
            np.testing.assert_array_equal(r64, np.array(want, dtype=np.float64))
            np.testing.assert_array_equal(to_f64(out), np.array(want, dtype=np.float64))


def test_asymmetric_hand_case():
    # A = [[1,2,3],[4,5,6]], B = [[1,0],[0,1],[2,-1]]  ->  C = [[7,-1],[16,-1]]  (worked by hand)
    A = [[1, 2, 3], [4, 5, 6]]
    B = [[1, 0], [0, 1], [2, -1]]
    r32, _, _ = orc.gemm(to_bits(A), to_bits(B), 2, 2, 3)
    np.testing.assert_array_equal(r32, [[7, -1], [16, -1]])


def test_identity_and_ones():
    A = synth.randn_bf16(33, 64, 1.0, 0, "id")
    I = to_bits(np.eye(64))
    _, _, out = orc.gemm(synth.bits(A), I, 33, 64, 64)
    np.testing.assert_array_equal(out, synth.bits(A))                  # B = I  =>  C = A bit for bit
    ones_a, ones_b = to_bits(np.ones((8, 256))), to_bits(np.ones((256, 16)))
    r32, _, out = orc.gemm(ones_a, ones_b, 8, 16, 256)
    assert (r32 == 256.0).all() and (to_f64(out) == 256.0).all()


@pytest.mark.parametrize("M,N,K,at,bt", [(130, 200, 512, 0, 0), (64, 96, 2048, 0, 1), (96, 64, 1024, 1, 0), (40, 72, 300, 1, 1)])
def test_against_library_matmul_and_fp64_bound(M, N, K, at, bt):
    A, B = synth.gemm_operands(M, N, K, at, bt, seed=1, tag="orc")
    r32, r64, out = orc.gemm(synth.bits(A), synth.bits(B), M, N, K, at, bt, want64=True)
    Al = A.to(torch.float64).T if at else A.to(torch.float64)
    Bl = B.to(torch.float64).T if bt else B.to(torch.float64)
    lib = (Al @ Bl).numpy()                                            # library routine, exact products, fp64 sums
    np.testing.assert_allclose(r64, lib, rtol=0, atol=1e-9)
    # fp32 sequential accumulation: |ref32 - exact| <= K * 2^-24 * sum_k |a*b| (first-order bound, 2x slack)
    bound = 2 * K * 2.0 ** -24 * (Al.abs() @ Bl.abs()).numpy()
    assert (np.abs(r32.astype(np.float64) - lib) <= bound + 1e-30).all()
    # bf16 output = round-to-nearest-even of the fp32 sums (torch's own rounding as the second opinion)
    want = synth.bits(torch.from_numpy(r32).to(torch.bfloat16))
    np.testing.assert_array_equal(out, want)


def test_rne_ties():
    # 1 + 2^-8 lies exactly between bf16(1.0) and the next value: ties go to even (1.0);
    # 1 + 3*2^-8 lies between 1+2^-7 (odd mantissa) and 1+2^-6 (even): goes up.
    assert orc.f32_to_bf16(1.0 + 2.0 ** -8) == 0x3F80
    assert orc.f32_to_bf16(1.0 + 3 * 2.0 ** -8) == 0x3F82
    assert orc.f32_to_bf16(1.0 + 2.0 ** -8 + 2.0 ** -20) == 0x3F81
    assert orc.f32_to_bf16(-2.5) == 0xC020


def test_block_equals_slice_of_full():
    M, N, K = 70, 90, 128
    A, B = synth.gemm_operands(M, N, K, 0, 0, seed=2, tag="blk")
    full, _, _ = orc.gemm(synth.bits(A), synth.bits(B), M, N, K)
    blk, _, _ = orc.gemm(synth.bits(A), synth.bits(B), M, N, K, block=(10, 50, 33, 80))
    np.testing.assert_array_equal(blk, full[10:50, 33:80])
    one, _, _ = orc.gemm(synth.bits(A), synth.bits(B), M, N, K, threads=1)
    np.testing.assert_array_equal(one, full)


def test_axpby_special_cases_and_exact_integers():
    """alpha * A*B + beta * C (Sec. 2.2): reduces to the pinned GEMM, to C itself, and is exact on small integers."""
    rng = np.random.default_rng(11)
    M, N, K = 7, 10, 33

    def bf(x):
        u = np.asarray(x, dtype=np.float32).view(np.uint32)
        return ((u + 0x7FFF + ((u >> 16) & 1)) >> 16).astype(np.uint16)

    def f32(b):
        return (np.asarray(b, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32)

    A = bf(rng.standard_normal((M, K)).astype(np.float32))
    B = bf(rng.standard_normal((K, N)).astype(np.float32))
    Cin = bf(rng.standard_normal((M, N)).astype(np.float32))
    H32, _, Hb = orc.gemm(A, B, M, N, K)
    r, o = orc.gemm_axpby(A, B, Cin, M, N, K, 1.0, 0.0)
    np.testing.assert_array_equal(r, H32)
    np.testing.assert_array_equal(o, Hb)
    r, o = orc.gemm_axpby(A, B, Cin, M, N, K, 0.0, 1.0)
    np.testing.assert_array_equal(o, Cin.reshape(M, N))                      # C comes back bit for bit
    r2, _ = orc.gemm_axpby(A, B, Cin, M, N, K, 2.0, 0.0)
    np.testing.assert_array_equal(r2, 2.0 * H32)                             # scaling by a power of two is exact
    r3, _ = orc.gemm_axpby(A, B, Cin, M, N, K, -0.5, 3.0)
    want = -0.5 * H32.astype(np.float64) + 3.0 * f32(Cin).reshape(M, N).astype(np.float64)
    np.testing.assert_allclose(r3, want, rtol=1e-7, atol=0)
    # small integers: everything exact
    Ai = bf(rng.integers(-3, 4, size=(M, K)).astype(np.float32))
    Bi = bf(rng.integers(-3, 4, size=(K, N)).astype(np.float32))
    Ci = bf(rng.integers(-8, 9, size=(M, N)).astype(np.float32))
    ri, _ = orc.gemm_axpby(Ai, Bi, Ci, M, N, K, 2.0, -3.0)
    wi = 2.0 * (f32(Ai).reshape(M, K).astype(np.int64) @ f32(Bi).reshape(K, N).astype(np.int64)) - 3.0 * f32(Ci).reshape(M, N)
    np.testing.assert_array_equal(ri, wi.astype(np.float32))
    # transposed storage of A and B changes nothing
    rT, _ = orc.gemm_axpby(np.ascontiguousarray(A.reshape(M, K).T), np.ascontiguousarray(B.reshape(K, N).T), Cin, M, N, K, -0.5, 3.0,
                           a_trans=1, b_trans=1)
    np.testing.assert_array_equal(rT, r3)
