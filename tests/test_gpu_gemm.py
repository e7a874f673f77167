"""GPU parity, through the C ABI: ccl_gemm against the fp32 oracle.

Tolerance (stated by the benchmark spec): err = |C_gpu - ref32| / max(1, |ref32|) <= 1e-2 * sqrt(K / 1024),
where ref32 is the oracle's fp32-accumulate sum from the logical (row-major) operands.
"""
import math
import os

import numpy as np
import pytest
import torch

import oracle as orc
from paper_2606_11718_b200 import binding as ccl
from paper_2606_11718_b200 import synth
from helpers import gemm_desc

pytestmark = pytest.mark.gpu


GUARD = 8192        # elements of untouched memory that must stay untouched behind every output buffer


def tol(K):
    return 1e-2 * math.sqrt(K / 1024.0)


def to_layout(x_bits, m):
    """Host bits of a stored row-major operand -> device buffer in the layout `m` (library descriptor) describes.
    Uses the oracle's repack on the host, so a wrong device-side map cannot cancel out."""
    mo = orc.Mat(m.rows, m.cols, m.elem_bytes, m.P, m.part, m.layout, m.strip_align_bytes)
    buf = orc.repack(mo, x_bits, 0)
    return torch.from_numpy(buf.view(np.int16)).cuda()


def from_layout(buf, m):
    mo = orc.Mat(m.rows, m.cols, m.elem_bytes, m.P, m.part, m.layout, m.strip_align_bytes)
    return orc.repack(mo, buf.cpu().numpy().view(np.uint16), 1).reshape(m.rows, m.cols)


def run_gemm(d, A, B):
    """A, B: bf16 CPU tensors as stored (row-major).  Returns C as uint16 bits [M x N] (logical order)."""
    a_dev, b_dev = to_layout(synth.bits(A), d.A), to_layout(synth.bits(B), d.B)
    nc = ccl.ccl_buffer_bytes(d.C) // 2
    c_dev = torch.full((nc + GUARD,), 0x7FC0, dtype=torch.int16, device="cuda")   # NaN poison, and a guard zone behind C
    need = ccl.ccl_gemm_workspace(d)
    ws = torch.full((need // 4,), float("nan"), dtype=torch.float32, device="cuda") if need else None
    ccl.ccl_gemm(d, a_dev, b_dev, c_dev, ws)
    st, detail = ccl.ccl_gemm_status()
    assert st == ccl.OK, detail
    assert (c_dev[nc:] == 0x7FC0).all(), "the kernel wrote past the end of C"
    return from_layout(c_dev[:nc], d.C)


def check(d, A, B, block=None):
    got = run_gemm(d, A, B)
    M, N, K = d.M, d.N, d.K
    ref32, _, ref_bits = orc.gemm(synth.bits(A), synth.bits(B), M, N, K, d.a_trans, d.b_trans, block=block)
    if block is not None:
        got = got[block[0]:block[1], block[2]:block[3]]
    g = synth.from_bits(got).to(torch.float32).numpy()
    assert np.isfinite(g).all(), "unwritten (poisoned) output elements"
    err = np.abs(g - ref32) / np.maximum(1.0, np.abs(ref32))
    assert err.max() <= tol(K), (err.max(), tol(K))
    return got, ref_bits


SMALL = [
    # M, N, K, P, layouts(A,B,C), a_trans, b_trans, out_part
    (128, 256, 64, 1, ("row", "row", "row"), 0, 1, 0),     # one tile, both operands K-major
    (128, 256, 64, 1, ("row", "row", "row"), 0, 0, 0),     # B N-contiguous (MN-major)
    (128, 256, 64, 1, ("row", "row", "row"), 1, 0, 0),     # A M-contiguous
    (128, 256, 64, 1, ("row", "row", "row"), 1, 1, 0),
    (130, 384, 96, 2, ("row", "row", "row"), 0, 0, 2),     # partial tiles in M, K not a multiple of 64
    (130, 384, 96, 2, ("row", "ccl", "ccl"), 0, 0, 2),     # w = 192
    (130, 384, 96, 4, ("row", "ccl", "ccl"), 0, 0, 2),     # w = 96: partial 128-wide tiles inside every strip
    (130, 384, 200, 4, ("row", "ccl", "ccl"), 0, 1, 2),    # B stored [N x K], N-split = row split
    (264, 768, 328, 4, ("row", "ccl", "ccl"), 1, 0, 2),
    (264, 768, 328, 3, ("row", "ccl", "ccl"), 1, 1, 2),    # P = 3, w = 256
    (512, 1024, 256, 8, ("row", "ccl", "ccl"), 0, 0, 2),
    (512, 512, 256, 4, ("ccl", "row", "ccl"), 0, 0, 1),    # M-partition: A and C split along rows
    (512, 512, 256, 2, ("ccl", "row", "ccl"), 1, 0, 1),    # M-partition with A stored [K x M]: a column split of A
    (1, 512, 256, 4, ("row", "ccl", "ccl"), 0, 0, 2),      # M = 1
    (16, 512, 256, 2, ("row", "ccl", "ccl"), 0, 0, 2),
    (640, 2560, 512, 2, ("row", "ccl", "ccl"), 0, 0, 2),   # several tiles per CTA group, 5 stages wrap
    (256, 512, 128, 2, ("ccl", "ccl", "row"), 0, 0, 0),    # A and B split along K (parts below), plain raster
]


PART_2D = [
    # M, N, K, P, part_m, layouts(A,B,C), strips of (A, B, C), splits of (A, B, C), a_trans, b_trans
    (512, 1024, 256, 4, 2, ("row", "row", "row"), (1, 1, 1), (0, 0, 0), 0, 0),       # 2 x 2 blocks of a row-major C
    (512, 1024, 256, 4, 2, ("ccl", "ccl", "ccl"), (2, 2, 2), (1, 2, 1), 0, 0),       # A, C in 2 row strips, B in 2 column strips
    (768, 1536, 200, 8, 2, ("ccl", "ccl", "ccl"), (2, 4, 4), (1, 2, 2), 0, 0),       # 2 x 4 blocks, C split along N into 4
    (768, 1536, 328, 8, 4, ("ccl", "ccl", "row"), (4, 2, 1), (2, 1, 0), 1, 1),       # A [K x M] split along cols, B [N x K] along rows
    (1536, 768, 192, 6, 3, ("row", "ccl", "ccl"), (1, 2, 3), (0, 2, 1), 0, 0),       # 3 x 2 blocks
    (2048, 4096, 512, 4, 2, ("row", "ccl", "ccl"), (1, 2, 2), (0, 2, 2), 0, 0),      # several tiles per group
]


@pytest.mark.parametrize("M,N,K,P,pm,lay,mp,parts,at,bt", PART_2D)
def test_gemm_2d_output_partition(M, N, K, P, pm, lay, mp, parts, at, bt):
    """Sec. 4.1 (output-partition choices): CTA group (qm, qn) computes block (qm, qn) of C; the result is the plain product,
    bit for bit the one of the plain raster."""
    A, B = synth.gemm_operands(M, N, K, at, bt, seed=0, tag="2d")
    d = gemm_desc(M, N, K, P, lay, at, bt, out_part=3, grouped=1, parts=parts, part_m=pm, mat_P=mp)
    got, _ = check(d, A, B)
    d0 = gemm_desc(M, N, K, P, lay, at, bt, out_part=3, grouped=0, parts=parts, part_m=pm, mat_P=mp)
    np.testing.assert_array_equal(got, run_gemm(d0, A, B))


@pytest.fixture(params=["auto", "1", "2"])
def cta_mode(request):
    """Forces the 1-CTA or the 2-CTA (cta_group::2 pair) kernel, or leaves the library's own choice."""
    old = os.environ.pop("CCL_GEMM_CTAS", None)
    if request.param != "auto":
        os.environ["CCL_GEMM_CTAS"] = request.param
    yield request.param
    os.environ.pop("CCL_GEMM_CTAS", None)
    if old is not None:
        os.environ["CCL_GEMM_CTAS"] = old


@pytest.mark.parametrize("M,N,K,P,lay,at,bt,op", SMALL)
def test_gemm_small_shapes(M, N, K, P, lay, at, bt, op, cta_mode):
    parts = None
    if lay == ("ccl", "ccl", "row") and op == 0:
        parts = (1 if at else 2, 2 if bt else 1, 0)                    # both operands split along K
    A, B = synth.gemm_operands(M, N, K, at, bt, seed=0, tag="small")
    for grouped in (1, 0):
        d = gemm_desc(M, N, K, P, lay, at, bt, op, grouped, parts=parts)
        check(d, A, B)
    if any(l == "ccl" for l in lay) and parts is None:
        d = gemm_desc(M, N, K, P, lay, at, bt, op, 1, align=4096)      # page-aligned strips
        check(d, A, B)


INTERLEAVED = [
    # M, N, K, P, layouts(A,B,C), a_trans, b_trans, out_part, chunk bytes
    (130, 384, 96, 2, ("row", "ileave", "ileave"), 0, 0, 2, 1536),      # w = 192: 4 strip rows per chunk
    (130, 384, 96, 4, ("row", "ileave", "ileave"), 0, 0, 2, 768),       # w = 96: ragged tiles inside every strip, 4 rows per chunk
    (264, 1024, 328, 4, ("row", "ileave", "ileave"), 0, 0, 2, 256),     # w = 256: a strip row is 2 chunks
    (264, 1024, 328, 4, ("row", "ileave", "ileave"), 1, 0, 2, 128),     # ... 4 chunks of 64 elements
    (264, 1024, 328, 4, ("row", "ileave", "ileave"), 0, 0, 2, 512),     # a chunk is exactly one strip row
    (200, 512, 256, 4, ("row", "ileave", "ileave"), 0, 1, 2, 4096),     # B stored [N x K]: 8 of its rows per chunk; 16 rows of C
    (520, 1024, 256, 2, ("row", "ileave", "ileave"), 0, 1, 2, 65536),   # 128 B rows per chunk for B, 64 for C
    (512, 512, 256, 4, ("ileave", "row", "ileave"), 0, 0, 1, 2048),     # M-partition: A and C split along rows
    (512, 512, 256, 2, ("ileave", "row", "ileave"), 1, 0, 1, 256),      # A stored [K x M], split along its columns (w = 256)
    (512, 512, 192, 2, ("ileave", "row", "ileave"), 1, 0, 1, 2048),     # ... 4 rows of A per chunk, 2 rows of C
    (16, 1024, 2048, 2, ("row", "ileave", "ileave"), 0, 0, 2, 4096),    # split along K: the reduction writes interleaved C
    (640, 2560, 512, 2, ("row", "ileave", "ileave"), 0, 0, 2, 10240),   # several tiles per CTA group, 4 rows per chunk
    (256, 4096, 512, 4, ("row", "ileave", "ileave"), 0, 0, 2, 4096),    # the common case: 4 KB pages, 2 KB strip rows
    # chunks and strip rows that do not line up (no affine box: the operand ring is filled row by row)
    (264, 3584, 512, 4, ("row", "ileave", "ileave"), 0, 0, 2, 4096),    # w = 896: a strip row is 1792 B = 0.4375 chunks
    (264, 3584, 328, 4, ("row", "ileave", "row"), 0, 0, 2, 4096),       # ... K not a multiple of 64 (K runs along B's rows)
    (1024, 7168, 256, 8, ("row", "ileave", "ileave"), 0, 0, 2, 1024),   # w = 896 against 512-element chunks, P = 8
    (300, 1792, 512, 2, ("row", "ileave", "ileave"), 0, 1, 2, 768),     # B stored [N x K]: rows of 512 elements, chunks of 384
    (768, 512, 320, 2, ("ileave", "row", "ileave"), 1, 0, 1, 640),      # A stored [K x M] split along its columns (w = 384), chunks of 320
    (1792, 512, 256, 2, ("ileave", "row", "ileave"), 0, 0, 1, 768),     # A [M x K] split along rows: rows of 256, chunks of 384 elements
]


@pytest.mark.parametrize("M,N,K,P,lay,at,bt,op,chunk", INTERLEAVED)
def test_gemm_page_interleaved_operands(M, N, K, P, lay, at, bt, op, chunk, cta_mode, monkeypatch):
    """The page-interleaved form of CCL changes the address map only: same bits as from packed CCL operands (under the
    same plan: the cluster split, which page-interleaved operands do not take, sums K in another order)."""
    monkeypatch.setenv("CCL_GEMM_CLUSTERK", "0")
    A, B = synth.gemm_operands(M, N, K, at, bt, seed=5, tag="ileave")
    plain = tuple("ccl" if l == "ileave" else l for l in lay)
    want = run_gemm(gemm_desc(M, N, K, P, plain, at, bt, op, 1), A, B)
    for grouped in (1, 0):
        d = gemm_desc(M, N, K, P, lay, at, bt, op, grouped, align=chunk)
        got, _ = check(d, A, B)
        np.testing.assert_array_equal(got, want)


def test_gemm_exact_cases():
    eye = synth.from_bits(synth.bits(torch.eye(256).to(torch.bfloat16)))
    A = synth.randn_bf16(200, 256, 1.0, 0, "eye")
    d = gemm_desc(200, 256, 256, 2, ("row", "ccl", "ccl"))
    np.testing.assert_array_equal(run_gemm(d, A, eye), synth.bits(A))                  # B = I  =>  C = A, bit for bit
    ones_a, ones_b = torch.ones(128, 256).to(torch.bfloat16), torch.ones(256, 512).to(torch.bfloat16)
    d = gemm_desc(128, 512, 256, 4, ("row", "ccl", "ccl"))
    got = synth.from_bits(run_gemm(d, ones_a, ones_b)).to(torch.float32)
    assert (got == 256.0).all()                                                        # all ones => K, exactly


@pytest.mark.parametrize("at,bt", [(0, 0), (0, 1), (1, 0)])
def test_layout_invariance_and_strip_independence(at, bt):
    """Sec. 3.3: the GEMM computation is unchanged, only the address map: same bits from CCL and row-major operands."""
    M, N, K, P = 384, 1536, 512, 4
    A, B = synth.gemm_operands(M, N, K, at, bt, seed=3, tag="inv")
    c_row = run_gemm(gemm_desc(M, N, K, P, ("row", "row", "row"), at, bt, 2, 1), A, B)
    c_ccl = run_gemm(gemm_desc(M, N, K, P, ("row", "ccl", "ccl"), at, bt, 2, 1), A, B)
    c_pad = run_gemm(gemm_desc(M, N, K, P, ("row", "ccl", "ccl"), at, bt, 2, 0, align=65536), A, B)
    np.testing.assert_array_equal(c_row, c_ccl)
    np.testing.assert_array_equal(c_row, c_pad)
    # zeroing strip 2 of B changes strip 2 of C only
    w = N // P
    B2 = B.clone()
    if bt:
        B2[2 * w:3 * w, :] = 0
    else:
        B2[:, 2 * w:3 * w] = 0
    c2 = run_gemm(gemm_desc(M, N, K, P, ("row", "ccl", "ccl"), at, bt, 2, 1), A, B2)
    keep = np.ones(N, dtype=bool)
    keep[2 * w:3 * w] = False
    np.testing.assert_array_equal(c2[:, keep], c_ccl[:, keep])
    assert (c2[:, ~keep] == 0).all()


def test_gemm_config1_expert_up_projection():
    g = synth.config1_gemm()
    A, B = synth.gemm_operands(g["M"], g["N"], g["K"], g["a_trans"], g["b_trans"], seed=0, tag=g["name"])
    d = gemm_desc(g["M"], g["N"], g["K"], 4, ("row", "ccl", "ccl"), g["a_trans"], g["b_trans"], 2, 1)
    got, ref_bits = check(d, A, B)
    ulp = np.abs(got.astype(np.int32) - ref_bits.astype(np.int32))
    big = np.abs(synth.from_bits(ref_bits).to(torch.float32).numpy()) > 1e-2
    assert ulp[big].max() <= 2
    # 1b: W^T materialised [K x N], w = 192 (384-byte slices)
    Bt = B.T.contiguous()
    check(gemm_desc(g["M"], g["N"], g["K"], 4, ("row", "ccl", "ccl"), 0, 0, 2, 1), A, Bt)


@pytest.mark.parametrize("P", [2, 4])
def test_gemm_qwen_config(P):
    for g in synth.qwen_ffn_gemms():
        A, B = synth.gemm_operands(g["M"], g["N"], g["K"], g["a_trans"], g["b_trans"], seed=0, tag=g["name"],
                                   a_std=g["a_std"], b_std=g["b_std"])
        d = gemm_desc(g["M"], g["N"], g["K"], P, ("row", "ccl", "ccl"), g["a_trans"], g["b_trans"], 2, 1, align=4096)
        check(d, A, B)


def sample_blocks(M, N, P, rng, n_random=8, bm=128, bn=128):
    w = N // P
    blocks = {(0, 0), (0, N - bn), (M - bm, 0), (M - bm, N - bn)}
    for g in range(P):                                                 # first and last tile of every strip, and across its edges
        blocks.add((0, g * w)); blocks.add((M - bm, (g + 1) * w - bn))
        if g:
            blocks.add((bm, g * w - bn // 2))
    for _ in range(n_random):
        blocks.add((int(rng.integers(0, M - bm + 1)), int(rng.integers(0, N - bn + 1))))
    return [(m, m + bm, n, n + bn) for m, n in sorted(blocks)]


def check_sampled(d, A, B, g, P, rng, n_random=8):
    """Sampled 128x128 blocks element by element against the oracle, plus the +-1 projection over every output."""
    M, N, K = d.M, d.N, d.K
    got = run_gemm(d, A, B)
    gf = synth.from_bits(got).to(torch.float32)
    assert torch.isfinite(gf).all()
    worst = 0.0
    for blk in sample_blocks(M, N, P, rng, n_random):
        ref32, _, _ = orc.gemm(synth.bits(A), synth.bits(B), M, N, K, g["a_trans"], g["b_trans"], block=blk)
        sub = gf[blk[0]:blk[1], blk[2]:blk[3]].numpy()
        err = np.abs(sub - ref32) / np.maximum(1.0, np.abs(ref32))
        assert err.max() <= tol(K), (blk, err.max())
        worst = max(worst, float(err.max()))
    # property over every output element: C v = A (B v) for random +-1 vectors (exact arithmetic up to rounding)
    Al = (A.T if g["a_trans"] else A).to(torch.float32)
    Bl = (B.T if g["b_trans"] else B).to(torch.float32)
    sigma_c = g["a_std"] * g["b_std"] * math.sqrt(K)
    for s in range(2):
        v = torch.from_numpy(rng.choice([-1.0, 1.0], size=N).astype(np.float32))
        lhs = gf.to(torch.float64) @ v.to(torch.float64)
        rhs = Al.to(torch.float64) @ (Bl.to(torch.float64) @ v.to(torch.float64)) if K * N < 3e8 else \
            (Al @ (Bl @ v)).to(torch.float64)
        # bf16 rounding of C: each element off by <= 2^-9 relative; random signs -> sqrt(N) growth, 8 sigma margin
        bound = 8 * math.sqrt(N) * sigma_c * 2.0 ** -8
        assert (lhs - rhs).abs().max().item() <= bound
    return worst


# name, P, strip alignment: the benchmark's own launch is the first (B and C in CCL, P = 4, strips aligned to 4 KB pages)
LLAMA_FULL = [("llama_fwd_gateup", 4, 4096), ("llama_fwd_gateup", 2, 4096), ("llama_fwd_down", 4, 0), ("llama_fwd_down", 2, 4096),
              ("llama_dgrad", 4, 4096), ("llama_wgrad", 2, 0), ("llama_wgrad", 4, 4096)]


@pytest.mark.parametrize("name,P,align", LLAMA_FULL)
def test_gemm_llama_full_size_sampled(name, P, align):
    """Full Llama-70B-size GEMMs in the benchmark's launch configuration (CCL B and C, grouped raster): sampled
    128x128 blocks against the oracle, plus a randomised projection check over the whole output."""
    g = {x["name"]: x for x in synth.llama_fwd_gemms() + synth.llama_bwd_gemms()}[name]
    M, N, K = g["M"], g["N"], g["K"]
    A, B = synth.gemm_operands(M, N, K, g["a_trans"], g["b_trans"], seed=0, tag=name, a_std=g["a_std"], b_std=g["b_std"])
    d = gemm_desc(M, N, K, P, ("row", "ccl", "ccl"), g["a_trans"], g["b_trans"], 2, 1, align=align)
    check_sampled(d, A, B, g, P, np.random.default_rng(0))


@pytest.mark.parametrize("name,P", [("llama_fwd_gateup", 4), ("llama_fwd_gateup", 8), ("llama_fwd_down", 2), ("llama_fwd_down", 4)])
def test_gemm_m1024_llama_weights(name, P):
    """The 1024-token row of the token-count sweep on the full Llama weights (CCL B and C, 4 KB-aligned strips)."""
    g = dict({x["name"]: x for x in synth.llama_fwd_gemms()}[name])
    M, N, K = 1024, g["N"], g["K"]
    A, B = synth.gemm_operands(M, N, K, 0, 0, seed=0, tag=name + "/m1024")
    d = gemm_desc(M, N, K, P, ("row", "ccl", "ccl"), 0, 0, 2, 1, align=4096)
    check_sampled(d, A, B, g, P, np.random.default_rng(1), n_random=6)


@pytest.fixture(params=[(1, 128), (1, 192), (1, 256), (2, 128), (2, 192), (2, 256), (2, 384), (2, 512)], ids=lambda v: f"c{v[0]}b{v[1]}")
def tile_mode(request):
    """Forces one kernel variant: CTAs per tile (1, or a cta_group::2 pair) and tile width."""
    keys = ("CCL_GEMM_CTAS", "CCL_GEMM_BN")
    old = {k: os.environ.pop(k, None) for k in keys}
    os.environ["CCL_GEMM_CTAS"], os.environ["CCL_GEMM_BN"] = str(request.param[0]), str(request.param[1])
    yield request.param
    for k in keys:
        os.environ.pop(k, None)
        if old[k] is not None:
            os.environ[k] = old[k]


@pytest.mark.parametrize("M,N,K,P,at,bt", [(520, 1536, 328, 4, 0, 0), (300, 2304, 512, 2, 0, 1), (512, 768, 192, 1, 1, 0),
                                           (256, 3072, 1024, 4, 1, 1)])
def test_gemm_every_tile_shape(M, N, K, P, at, bt, tile_mode):
    """Each kernel variant on shapes with ragged tiles in M and N, several tiles per CTA and both operand majors."""
    A, B = synth.gemm_operands(M, N, K, at, bt, seed=7, tag="tiles")
    d = gemm_desc(M, N, K, P, ("row", "ccl", "ccl"), at, bt, 2, 1)
    try:
        ccl.ccl_gemm_workspace(d)
    except ccl.CclError as e:                      # e.g. 192-wide pair tiles need a K-contiguous B
        assert e.status == ccl.ERR_UNSUPPORTED
        pytest.skip("variant not available for this operand layout")
    check(d, A, B)


RAGGED_STRIPS = [
    # M, N, K, P, layouts, a_trans, b_trans, out_part -- the split dimension is not a multiple of P: strips of ceil(./P), the last one shorter
    (330, 512, 256, 4, ("ccl", "row", "ccl"), 0, 0, 1),        # M-partition: A and C in strips of 83 rows, the last of 81
    (1301, 256, 200, 3, ("ccl", "row", "ccl"), 0, 0, 1),       # ... strips of 434 rows (several tiles each), the last of 433; ragged K
    (264, 1016, 328, 16, ("row", "ccl", "row"), 0, 1, 2),      # B stored [N x K] in strips of 64 rows, the last of 56; C row-major
    (130, 1016, 192, 16, ("row", "ccl", "ccl"), 0, 0, 2),      # column strips of 64, the last of 56 (P = 16)
    (1016, 256, 128, 16, ("ccl", "row", "row"), 1, 0, 1),      # A stored [K x M] in column strips of 64, the last of 56
    (700, 2040, 512, 16, ("row", "ccl", "ccl"), 0, 0, 2),      # column strips of 128, the last of 120; several tiles per CTA
]


@pytest.mark.parametrize("M,N,K,P,lay,at,bt,op", RAGGED_STRIPS)
def test_gemm_strips_of_unequal_size(M, N, K, P, lay, at, bt, op, cta_mode):
    """Operands whose last strip is narrower / lower than the others (reading: w = ceil(N / P)): the last strip has a tensor
    map of its own.  Parity with the oracle, grouped and plain raster; the guard zone behind C stays untouched."""
    A, B = synth.gemm_operands(M, N, K, at, bt, seed=13, tag="ragstrips")
    for grouped in (1, 0):
        check(gemm_desc(M, N, K, P, lay, at, bt, op, grouped), A, B)
    if "ccl" in lay:
        check(gemm_desc(M, N, K, P, lay, at, bt, op, 1, align=4096), A, B)   # page-aligned strips


def test_gemm_strips_of_unequal_size_axpby():
    M, N, K, P = 330, 512, 256, 4
    A, B = synth.gemm_operands(M, N, K, 0, 0, seed=14, tag="ragstrips/axpby")
    Cin = synth.randn_bf16(M, N, 1.0, 14, "ragstrips/C")
    d = gemm_desc(M, N, K, P, ("ccl", "row", "ccl"), 0, 0, 1, 1)
    a_dev, b_dev, c_dev = to_layout(synth.bits(A), d.A), to_layout(synth.bits(B), d.B), to_layout(synth.bits(Cin), d.C)
    ccl.ccl_gemm_axpby(d, 0.5, 2.0, a_dev, b_dev, c_dev)
    assert ccl.ccl_gemm_status()[0] == ccl.OK
    got = synth.from_bits(from_layout(c_dev, d.C)).to(torch.float32).numpy()
    ref32, _ = orc.gemm_axpby(synth.bits(A), synth.bits(B), synth.bits(Cin), M, N, K, 0.5, 2.0, 0, 0)
    err = np.abs(got - ref32) / np.maximum(1.0, np.abs(ref32))
    assert err.max() <= 0.5 * tol(K) + 2.0 ** -8, err.max()


WIDE384 = [
    # M, N, K, P, layouts, a_trans, b_trans, out_part, chunk bytes (page-interleaved operands), alpha, beta
    (4096, 1536, 256, 4, ("row", "ccl", "ccl"), 0, 0, 2, 0, 1.0, 0.0),          # strips of exactly one tile width (the Qwen gate+up shape, short K)
    (520, 1536, 328, 2, ("row", "ccl", "ccl"), 0, 1, 2, 0, 1.0, 0.0),           # B stored [N x K]: three 64-row boxes per CTA; two tiles per strip
    (304, 1000, 512, 1, ("row", "row", "row"), 1, 1, 0, 0, 1.0, 0.0),           # ragged in M and N: a last tile that ends inside its first sub-tile ... (1000 = 2 * 384 + 232)
    (300, 1096, 512, 1, ("row", "row", "row"), 0, 0, 0, 0, 1.0, 0.0),           # ... and one that ends inside its second (1096 = 2 * 384 + 256 + 72)
    (264, 1536, 328, 4, ("row", "ileave", "ileave"), 0, 0, 2, 256, 1.0, 0.0),   # a strip row of 3 chunks
    (200, 768, 256, 2, ("row", "ileave", "ileave"), 0, 1, 2, 4096, 1.0, 0.0),   # B stored [N x K] in chunks of 8 rows
    (264, 3584, 512, 4, ("row", "ileave", "ileave"), 0, 0, 2, 4096, 1.0, 0.0),  # chunks and strip rows that do not line up: row-by-row fetch
    (512, 768, 256, 4, ("ileave", "row", "ileave"), 0, 0, 1, 2048, 1.0, 0.0),   # M-partition
    (520, 1536, 328, 4, ("row", "ccl", "ccl"), 0, 0, 2, 0, 0.5, 2.0),           # alpha / beta
]


@pytest.mark.parametrize("M,N,K,P,lay,at,bt,op,chunk,alpha,beta", WIDE384)
def test_gemm_384_wide_pair_tile(M, N, K, P, lay, at, bt, op, chunk, alpha, beta, monkeypatch):
    """The 256 x 384 pair tile (a 256-wide and a 128-wide MMA per k step) forced on: parity with the oracle; with K split too."""
    monkeypatch.setenv("CCL_GEMM_CTAS", "2")
    monkeypatch.setenv("CCL_GEMM_BN", "384")
    monkeypatch.setenv("CCL_GEMM_CLUSTERK", "0")
    A, B = synth.gemm_operands(M, N, K, at, bt, seed=11, tag="w384")
    d = gemm_desc(M, N, K, P, lay, at, bt, op, 1, align=chunk)
    if alpha == 1.0 and beta == 0.0:
        check(d, A, B)
        monkeypatch.setenv("CCL_GEMM_SPLITK", "2")
        check(d, A, B)
        return
    Cin = synth.randn_bf16(M, N, 1.0, 11, "w384/C")
    a_dev, b_dev, c_dev = to_layout(synth.bits(A), d.A), to_layout(synth.bits(B), d.B), to_layout(synth.bits(Cin), d.C)
    ccl.ccl_gemm_axpby(d, alpha, beta, a_dev, b_dev, c_dev)
    assert ccl.ccl_gemm_status()[0] == ccl.OK
    got = synth.from_bits(from_layout(c_dev, d.C)).to(torch.float32).numpy()
    ref32, _ = orc.gemm_axpby(synth.bits(A), synth.bits(B), synth.bits(Cin), M, N, K, alpha, beta, at, bt)
    err = np.abs(got - ref32) / np.maximum(1.0, np.abs(ref32))
    assert err.max() <= abs(alpha) * tol(K) + 2.0 ** -8, err.max()


@pytest.fixture(params=["auto", "1", "2", "4", "8", "2p", "4p"])
def split_mode(request):
    """Forces the number of K splits (partial sums in the workspace, fixed-order reduction); "2p", "4p": with CTA pairs."""
    keys = ("CCL_GEMM_SPLITK", "CCL_GEMM_CTAS")
    old = {k: os.environ.pop(k, None) for k in keys}
    if request.param != "auto":
        os.environ["CCL_GEMM_SPLITK"] = request.param.rstrip("p")
        os.environ["CCL_GEMM_CTAS"] = "2" if request.param.endswith("p") else "1"
    yield request.param
    for k in keys:
        os.environ.pop(k, None)
        if old[k] is not None:
            os.environ[k] = old[k]


@pytest.mark.parametrize("M,N,K,P,at,bt", [(130, 384, 1000, 2, 0, 0), (16, 512, 2048, 4, 0, 1), (1, 768, 1536, 4, 0, 0),
                                           (264, 768, 1088, 3, 1, 0)])
def test_gemm_split_k(M, N, K, P, at, bt, split_mode):
    A, B = synth.gemm_operands(M, N, K, at, bt, seed=5, tag="splitk")
    d = gemm_desc(M, N, K, P, ("row", "ccl", "ccl"), at, bt, 2, 1)
    try:
        need = ccl.ccl_gemm_workspace(d)
    except ccl.CclError as e:                                          # e.g. 8 splits of 17 k blocks: some split would be empty
        assert e.status == ccl.ERR_UNSUPPORTED
        pytest.skip("forced split count does not divide this K")
    if split_mode not in ("auto", "1"):
        assert need == int(split_mode.rstrip("p")) * M * N * 4
    got1, _ = check(d, A, B)
    got2, _ = check(d, A, B)
    np.testing.assert_array_equal(got1, got2)                          # fixed-order reduction: run-to-run identical
    if need:                                                           # too small a workspace is refused, nothing runs
        a_dev, b_dev = to_layout(synth.bits(A), d.A), to_layout(synth.bits(B), d.B)
        c_dev = torch.zeros(M * N, dtype=torch.int16, device="cuda")
        with pytest.raises(ccl.CclError) as ei:
            ccl.ccl_gemm(d, a_dev, b_dev, c_dev, torch.empty(need // 4 - 4, dtype=torch.float32, device="cuda"))
        assert ei.value.status == ccl.ERR_WORKSPACE
        with pytest.raises(ccl.CclError):
            ccl.ccl_gemm(d, a_dev, b_dev, c_dev, None)


@pytest.mark.parametrize("name", ["llama_fwd_down", "llama_fwd_gateup"])
def test_gemm_small_m_sweep_llama_shapes(name):
    """The token-count sweep at weight-streaming sizes: M in {1, 16, 128} on the full Llama weight matrices."""
    g = {x["name"]: x for x in synth.llama_fwd_gemms()}[name]
    N, K = g["N"], g["K"]
    Bfull = synth.randn_bf16(K, N, synth.WEIGHT_STD, 0, name + "/B")
    for M, Ps in ((1, (4,)), (16, (2, 8)), (128, (4,))):
        A = synth.randn_bf16(M, K, synth.ACT_STD, 0, f"{name}/A{M}")
        for P in Ps:
            d = gemm_desc(M, N, K, P, ("row", "ccl", "ccl"), 0, 0, 2, 1)
            got = run_gemm(d, A, Bfull)
            gf = synth.from_bits(got).to(torch.float32).numpy()
            assert np.isfinite(gf).all()
            rng = np.random.default_rng(M * 10 + P)
            cols = sorted({0, N - 256, *(int(c) for c in rng.integers(0, N // 256, size=6) * 256)})
            for n0 in cols:                                            # sampled 256-column blocks, all rows
                ref32, _, _ = orc.gemm(synth.bits(A), synth.bits(Bfull), M, N, K, 0, 0, block=(0, M, n0, n0 + 256))
                err = np.abs(gf[:, n0:n0 + 256] - ref32) / np.maximum(1.0, np.abs(ref32))
                assert err.max() <= tol(K), (M, P, n0, err.max())
            # every column: projection on a random +-1 vector over rows is cheap here (M is small): full check in fp64
            full = (A.to(torch.float64) @ Bfull.to(torch.float64)).numpy() if M <= 16 else None
            if full is not None:
                err = np.abs(gf - full) / np.maximum(1.0, np.abs(full))
                assert err.max() <= tol(K)


AXPBY = [
    # M, N, K, P, layouts, a_trans, b_trans, out_part, alpha, beta
    (130, 384, 96, 2, ("row", "ccl", "ccl"), 0, 0, 2, 0.5, 2.0),          # ragged tiles, CCL output read and written
    (264, 768, 328, 4, ("row", "ccl", "row"), 1, 0, 2, -1.25, 0.75),
    (512, 1024, 256, 4, ("row", "ccl", "ccl"), 0, 1, 2, 1.0, 1.0),         # accumulation into C (e.g. weight gradients)
    (16, 1024, 2048, 2, ("row", "ccl", "ccl"), 0, 0, 2, 2.0, -0.5),        # split along K: the reduction applies the scalars
    (300, 1024, 256, 4, ("row", "ileave", "ileave"), 0, 0, 2, 0.25, 3.0),  # page-interleaved C
    (640, 2560, 512, 2, ("row", "ccl", "ccl"), 0, 0, 2, 3.0, 0.0),         # beta = 0: C is not read
    (256, 768, 2048, 4, ("row", "ccl", "ccl"), 0, 1, 2, 0.5, 2.0),         # few tiles: split inside clusters, the owners of the sums apply the scalars
    (130, 400, 4096, 2, ("row", "ccl", "ccl"), 0, 0, 2, -2.0, 1.0),        # ... with ragged rows and columns
]


@pytest.mark.parametrize("M,N,K,P,lay,at,bt,op,alpha,beta", AXPBY)
def test_gemm_axpby(M, N, K, P, lay, at, bt, op, alpha, beta, cta_mode):
    """C <- alpha * A*B + beta * C (Sec. 2.2) against the oracle; tolerance: the GEMM's, scaled by |alpha|, plus the bf16
    rounding of the result (2^-8 relative)."""
    A, B = synth.gemm_operands(M, N, K, at, bt, seed=9, tag="axpby")
    Cin = synth.randn_bf16(M, N, 1.0, 9, "axpby/C")
    d = gemm_desc(M, N, K, P, lay, at, bt, op, 1, align=1024 if "ileave" in lay else 0)
    a_dev, b_dev = to_layout(synth.bits(A), d.A), to_layout(synth.bits(B), d.B)
    nc = ccl.ccl_buffer_bytes(d.C) // 2
    c_dev = torch.full((nc + GUARD,), 0x7FC0, dtype=torch.int16, device="cuda")
    if beta != 0.0:
        c_dev[:nc] = to_layout(synth.bits(Cin), d.C)
    need = ccl.ccl_gemm_workspace(d)
    ws = torch.full((need // 4,), float("nan"), dtype=torch.float32, device="cuda") if need else None
    ccl.ccl_gemm_axpby(d, alpha, beta, a_dev, b_dev, c_dev, ws)
    assert ccl.ccl_gemm_status()[0] == ccl.OK
    assert (c_dev[nc:] == 0x7FC0).all(), "the kernel wrote past the end of C"
    got = synth.from_bits(from_layout(c_dev[:nc], d.C)).to(torch.float32).numpy()
    ref32, _ = orc.gemm_axpby(synth.bits(A), synth.bits(B), synth.bits(Cin), M, N, K, alpha, beta, at, bt)
    assert np.isfinite(got).all()
    err = np.abs(got - ref32) / np.maximum(1.0, np.abs(ref32))
    assert err.max() <= abs(alpha) * tol(K) + 2.0 ** -8, err.max()


def test_gemm_axpby_identity_scalars_equal_plain_gemm():
    M, N, K, P = 384, 1536, 512, 4
    A, B = synth.gemm_operands(M, N, K, 0, 0, seed=10, tag="axpby1")
    d = gemm_desc(M, N, K, P, ("row", "ccl", "ccl"), 0, 0, 2, 1)
    want = run_gemm(d, A, B)
    a_dev, b_dev = to_layout(synth.bits(A), d.A), to_layout(synth.bits(B), d.B)
    c_dev = torch.full((ccl.ccl_buffer_bytes(d.C) // 2,), 0x7FC0, dtype=torch.int16, device="cuda")
    ccl.ccl_gemm_axpby(d, 1.0, 0.0, a_dev, b_dev, c_dev)
    np.testing.assert_array_equal(from_layout(c_dev, d.C), want)
    # alpha = 0, beta = 1 leaves C as it was
    Cin = synth.randn_bf16(M, N, 1.0, 10, "axpby1/C")
    c_dev = to_layout(synth.bits(Cin), d.C)
    ccl.ccl_gemm_axpby(d, 0.0, 1.0, a_dev, b_dev, c_dev)
    np.testing.assert_array_equal(from_layout(c_dev, d.C), synth.bits(Cin))
    with pytest.raises(ccl.CclError) as ei:
        ccl.ccl_gemm_axpby(d, float("nan"), 0.0, a_dev, b_dev, c_dev)
    assert ei.value.status == ccl.ERR_INVALID_ARG


# ---------------------------------------------------------------------------------------------
# balanced split: every unit gets the same number of k blocks; tiles cut between units are summed in the order of k
# ---------------------------------------------------------------------------------------------
@pytest.fixture
def balanced():
    keys = ("CCL_GEMM_BALANCED", "CCL_GEMM_CTAS", "CCL_GEMM_BN")
    old = {k: os.environ.pop(k, None) for k in keys}
    os.environ["CCL_GEMM_BALANCED"] = "1"
    yield
    for k in keys:
        os.environ.pop(k, None)
        if old[k] is not None:
            os.environ[k] = old[k]


BALANCED = [
    # M, N, K, P, layouts, a_trans, b_trans, out_part
    (768, 2048, 4096, 4, ("row", "ccl", "ccl"), 1, 0, 2),      # fewer tiles than units: the shares of a tile run side by side
    (256, 768, 2048, 4, ("row", "ccl", "ccl"), 0, 1, 2),       # the single-expert GEMM: many shares per tile
    (4096, 1536, 2048, 4, ("row", "ccl", "ccl"), 0, 0, 2),     # 1.3 rounds of tiles: a unit finishes the tile its neighbour began
    (4096, 768, 2048, 2, ("row", "ccl", "ccl"), 0, 1, 2),
    (520, 1536, 328, 4, ("row", "ccl", "ccl"), 0, 0, 2),       # ragged tiles in M, K not a multiple of 64
    (300, 2304, 512, 2, ("row", "ccl", "row"), 0, 1, 2),
    (1032, 1024, 1096, 1, ("row", "row", "row"), 1, 1, 0),     # plain raster
    (2048, 2048, 2048, 4, ("ccl", "row", "ccl"), 0, 0, 1),     # M strips
    (130, 384, 4096, 4, ("row", "ccl", "ccl"), 0, 0, 2),       # strips of 96 columns: every tile partial in N
    (1024, 1024, 1024, 4, ("row", "ileave", "ileave"), 0, 0, 2),   # page-interleaved operands
]


@pytest.mark.parametrize("M,N,K,P,lay,at,bt,op", BALANCED)
@pytest.mark.parametrize("variant", [None, (1, 128), (1, 256), (2, 256), (2, 512)], ids=lambda v: "auto" if v is None else f"c{v[0]}b{v[1]}")
def test_gemm_balanced_split(balanced, M, N, K, P, lay, at, bt, op, variant):
    """The balanced split forced on: parity with the oracle, the same bits on every run, flags left clear."""
    if variant is not None:
        os.environ["CCL_GEMM_CTAS"], os.environ["CCL_GEMM_BN"] = str(variant[0]), str(variant[1])
    A, B = synth.gemm_operands(M, N, K, at, bt, seed=5, tag="balanced")
    d = gemm_desc(M, N, K, P, lay, at, bt, op, 1, align=4096 if "ileave" in lay else 0)
    got1, _ = check(d, A, B)
    got2, _ = check(d, A, B)
    np.testing.assert_array_equal(got1, got2)


def test_gemm_balanced_split_needs_its_workspace_or_steps_aside(balanced):
    """Without a workspace the call runs whole tiles (the balanced split is optional); with one that is too small for the
    partial sums but not empty, likewise; results agree within the tolerance either way."""
    M, N, K, P = 768, 2048, 4096, 4
    A, B = synth.gemm_operands(M, N, K, 1, 0, seed=6, tag="balanced-ws")
    d = gemm_desc(M, N, K, P, ("row", "ccl", "ccl"), 1, 0, 2, 1)
    need = ccl.ccl_gemm_workspace(d)
    a_dev, b_dev = to_layout(synth.bits(A), d.A), to_layout(synth.bits(B), d.B)
    ref32, _, _ = orc.gemm(synth.bits(A), synth.bits(B), M, N, K, 1, 0)
    os.environ.pop("CCL_GEMM_BALANCED")                      # the planner's own choice from here on
    for ws in (None, torch.empty(1024, dtype=torch.float32, device="cuda"), torch.empty(need // 4, dtype=torch.float32, device="cuda")):
        c_dev = torch.zeros(M * N, dtype=torch.int16, device="cuda")
        if ws is not None and ws.numel() * 4 < ccl.ccl_gemm_workspace(d):
            try:
                ccl.ccl_gemm(d, a_dev, b_dev, c_dev, ws)
            except ccl.CclError as e:                         # a plan split along K in the old way insists on its workspace
                assert e.status == ccl.ERR_WORKSPACE
                continue
        else:
            try:
                ccl.ccl_gemm(d, a_dev, b_dev, c_dev, ws)
            except ccl.CclError as e:
                assert ws is None and e.status == ccl.ERR_WORKSPACE
                continue
        assert ccl.ccl_gemm_status()[0] == ccl.OK
        g = synth.from_bits(from_layout(c_dev, d.C)).to(torch.float32).numpy()
        err = np.abs(g - ref32) / np.maximum(1.0, np.abs(ref32))
        assert err.max() <= tol(K)


# ---------------------------------------------------------------------------------------------
# cluster split: the CTAs of a cluster share one tile along K, partial sums meet in distributed shared memory
# ---------------------------------------------------------------------------------------------
CLUSTERK = [
    # M, N, K, P, layouts, a_trans, b_trans, out_part
    (256, 768, 2048, 4, ("row", "ccl", "ccl"), 0, 1, 2),       # the single-expert GEMM (configuration 1)
    (256, 768, 2048, 4, ("row", "ccl", "ccl"), 0, 0, 2),       # ... with the weight materialised [K x N]: strips of 192 columns
    (768, 2048, 4096, 4, ("row", "ccl", "ccl"), 1, 0, 2),      # the Qwen down-projection weight gradient
    (130, 384, 1096, 2, ("row", "ccl", "ccl"), 0, 0, 2),       # ragged rows, K not a multiple of 64
    (304, 520, 512, 1, ("row", "row", "row"), 1, 1, 0),        # ragged columns, plain raster, both operands transposed
    (512, 512, 8192, 4, ("ccl", "row", "ccl"), 0, 0, 1),       # M strips
    (1, 1024, 4096, 4, ("row", "ccl", "ccl"), 0, 0, 2),        # one row
]


@pytest.mark.parametrize("M,N,K,P,lay,at,bt,op", CLUSTERK)
@pytest.mark.parametrize("ks", [2, 4, 8])
@pytest.mark.parametrize("bn", [None, 128, 192, 256])
def test_gemm_cluster_split(M, N, K, P, lay, at, bt, op, ks, bn):
    """The cluster split forced on (cluster size and tile width): parity with the oracle, the same bits on every run."""
    keys = ("CCL_GEMM_CLUSTERK", "CCL_GEMM_BN")
    old = {k: os.environ.pop(k, None) for k in keys}
    os.environ["CCL_GEMM_CLUSTERK"] = str(ks)
    if bn is not None:
        os.environ["CCL_GEMM_BN"] = str(bn)
    try:
        A, B = synth.gemm_operands(M, N, K, at, bt, seed=9, tag="clusterk")
        d = gemm_desc(M, N, K, P, lay, at, bt, op, 1)
        got1, _ = check(d, A, B)
        got2, _ = check(d, A, B)
        np.testing.assert_array_equal(got1, got2)
    finally:
        for k in keys:
            os.environ.pop(k, None)
            if old[k] is not None:
                os.environ[k] = old[k]
