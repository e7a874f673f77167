"""Pins of the oracle's gated-activation GEMM (orc_gemm_swiglu): the pairing of gate and up columns inside the
column strips of a fused gate/up operand (Fig. 3) and the activation itself, against hand-enumerated cases, closed
forms and numpy evaluated independently in float64.  No GPU."""
import math
import os

import numpy as np
import pytest

import oracle as orc

HERE = os.path.dirname(os.path.abspath(__file__))


def bf16(x):
    """float -> nearest bf16 bit pattern (numbers used here are exactly representable, or rounding is checked apart)."""
    u = np.asarray(x, dtype=np.float32).view(np.uint32)
    r = ((u >> 16) & 1) + 0x7FFF
    return ((u + r) >> 16).astype(np.uint16)


def f32(bits):
    return (np.asarray(bits, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32)


def silu64(x):
    return x / (1.0 + np.exp(-x))


def test_pairing_hand_example_two_strips():
    # K = 1, A = [1]: H is the row of B.  N = 8, P = 2: strips (H0 H1 | H2 H3) and (H4 H5 | H6 H7), gate | up.
    # golden file: the eight inputs and the four expected outputs, written out by hand with silu(0) = 0,
    # silu(x) - silu(-x) = x and up = 1 or 2 (exact in binary)
    rows = [l.split() for l in open(os.path.join(HERE, "golden", "swiglu_pairing.txt")) if l.strip() and not l.startswith("#")]
    H = np.array([float(v) for v in rows[0]], dtype=np.float32)
    pairs = [(int(a), int(b)) for a, b in (p.split(",") for p in rows[1])]
    assert pairs == [(0, 2), (1, 3), (4, 6), (5, 7)]                       # (gate column, up column) of outputs 0..3
    ref32, out = orc.gemm_swiglu(bf16([1.0]), bf16(H), 1, 8, 1, P=2)
    want = np.array([silu64(float(H[g])) * float(H[u]) for g, u in pairs])
    np.testing.assert_allclose(ref32[0], want, rtol=1e-6)
    assert ref32[0][0] == 0.0                                               # silu(0) * anything
    # one strip: plain halves
    ref1, _ = orc.gemm_swiglu(bf16([1.0]), bf16(H), 1, 8, 1, P=1)
    want1 = np.array([silu64(float(H[j])) * float(H[4 + j]) for j in range(4)])
    np.testing.assert_allclose(ref1[0], want1, rtol=1e-6)


def test_activation_closed_forms():
    # silu(ln 3) = (3/4) ln 3;  silu(x) - silu(-x) = x;  silu(x) -> x for large x, -> 0 for very negative x
    x = np.float32(math.log(3.0))
    xb = f32(bf16([x]))[0]                                                  # what the operand really holds
    r, _ = orc.gemm_swiglu(bf16([1.0]), bf16([xb, 1.0]), 1, 2, 1)
    assert abs(r[0, 0] - xb / (1.0 + math.exp(-float(xb)))) < 1e-6
    assert abs(r[0, 0] - 0.75 * math.log(3.0)) < 3e-3                       # bf16 input rounding only
    for v in (0.5, 2.0, 7.0):
        a, _ = orc.gemm_swiglu(bf16([1.0]), bf16([v, 1.0]), 1, 2, 1)
        b, _ = orc.gemm_swiglu(bf16([1.0]), bf16([-v, 1.0]), 1, 2, 1)
        assert abs(float(a[0, 0]) - float(b[0, 0]) - v) < 1e-6
    big, _ = orc.gemm_swiglu(bf16([1.0]), bf16([64.0, 3.0, -64.0, 3.0]), 1, 4, 1, P=2)
    assert big[0, 0] == 192.0 and abs(big[0, 1]) < 1e-20


def test_against_numpy_float64_and_plain_gemm():
    rng = np.random.default_rng(5)
    M, N, K, P = 9, 24, 40, 3
    A = bf16(rng.standard_normal((M, K)).astype(np.float32))
    B = bf16((rng.standard_normal((K, N)) * 0.2).astype(np.float32))
    H32, _, _ = orc.gemm(A, B, M, N, K)                                     # the pinned fp32 GEMM
    Wp = N // P
    want = np.empty((M, N // 2))
    for g in range(P):
        gate = H32[:, g * Wp: g * Wp + Wp // 2].astype(np.float64)
        up = H32[:, g * Wp + Wp // 2: (g + 1) * Wp].astype(np.float64)
        want[:, g * Wp // 2: (g + 1) * Wp // 2] = silu64(gate) * up
    ref32, out = orc.gemm_swiglu(A, B, M, N, K, P=P)
    np.testing.assert_allclose(ref32, want, rtol=2e-7, atol=1e-30)
    np.testing.assert_array_equal(out, bf16(ref32))                         # one rounding to bf16, nearest-even
    # stored transposed operands give the same numbers
    refT, _ = orc.gemm_swiglu(np.ascontiguousarray(A.reshape(M, K).T), np.ascontiguousarray(B.reshape(K, N).T), M, N, K, P=P, a_trans=1, b_trans=1)
    np.testing.assert_array_equal(refT, ref32)
    # zero gate columns give zero output whatever the up columns hold
    B0 = B.reshape(K, N).copy()
    B0[:, 0:Wp // 2] = 0
    z, _ = orc.gemm_swiglu(A, B0, M, N, K, P=P)
    assert (z[:, 0:Wp // 2] == 0).all() and (z[:, Wp // 2:] == ref32[:, Wp // 2:]).all()


def test_rejections():
    one = bf16([1.0])
    with pytest.raises(ValueError):
        orc.gemm_swiglu(one, bf16([1.0, 2.0, 3.0]), 1, 3, 1)               # odd N
    with pytest.raises(ValueError):
        orc.gemm_swiglu(one, bf16(np.ones(6)), 1, 6, 1, P=2)               # strips of odd width
