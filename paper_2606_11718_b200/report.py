"""Per-GEMM report over the five workload configurations (single GPU).

    python -m paper_2606_11718_b200.report [--config 1..5 | all] [--out DIR] [--quick]

For every GEMM of a configuration it measures, with CUDA events on the launching stream:
  * ccl_repack of the B operand (row-major -> CCL), GB/s of read+write bytes;
  * ccl_gemm with B and C in CCL under the chiplet-grouped raster, and with row-major operands
    under the plain raster (Sec. 3.3: the layout should not change the speed);
  * ccl_traffic under the policies of Sec. 4.1 -- row-major + round-robin at 4 KB (the baseline),
    64 KB and 2 MB, row-major + coarse block placement, row-major + best page-granular placement,
    CCL + page->strip placement, CCL + literal round-robin, page-interleaved CCL + literal round-robin
    -- for the N- and the M-partition of C,
    and prints remote bytes relative to the 4 KB round-robin baseline (no L2 filter: every byte a CTA
    touches is counted, so the ratios are not the paper's simulated ones).
Roofline per GEMM: min(tensor peak, HBM peak * arithmetic intensity), against the measured peaks in
MEASURED_PEAKS.json when present.  One JSON object per GEMM is written to DIR/report_config<N>.json
and a table is printed.  Nothing here calls the CPU oracle.
"""
import argparse
import json
import math
import os

import torch

from . import binding as ccl
from . import synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        j = json.load(open(p))
        return dict(hbm=j["hbm_gbs"], tf=j["bf16_tflops"], src="measured")
    return dict(hbm=6650.0, tf=1590.0, src="fallback")


def configs(which, quick):
    out = {}
    g1 = synth.config1_gemm()
    out[1] = [dict(g1, P=4, S=4096), dict(g1, name="qwen_expert_up_wT", b_trans=0, P=4, S=4096)]
    out[2] = [dict(g, P=P, S=S) for g in synth.qwen_ffn_gemms() for P in (2, 4) for S in (4096, 65536)]
    out[3] = [dict(g, P=P, S=4096) for g in synth.llama_fwd_gemms() for P in (2, 4)]
    out[4] = [dict(g, P=P, S=4096) for g in synth.llama_bwd_gemms() for P in (2, 4)]
    sweep = []
    for g in synth.llama_fwd_gemms() + synth.qwen_ffn_gemms()[:2]:
        for M in (1, 16, 128, 1024, 8192):
            for P in ((4,) if quick else (2, 4, 8)):
                sweep.append(dict(g, name=f"{g['name']}_M{M}", M=M, P=P, S=4096))
    out[5] = sweep
    want = [w.strip() for w in str(which).split(",")]
    return {k: v for k, v in out.items() if "all" in want or str(k) in want}


def mats(g, layout_bc, align=0):
    M, N, K, at, bt, P = g["M"], g["N"], g["K"], g["a_trans"], g["b_trans"], g["P"]
    a_shape = (K, M) if at else (M, K)
    b_shape = (N, K) if bt else (K, N)
    b_part = ccl.PART_ROWS if bt else ccl.PART_COLS
    mA = ccl.Mat(a_shape[0], a_shape[1], 2)
    mB = ccl.Mat(b_shape[0], b_shape[1], 2, P, b_part, layout_bc, align if layout_bc == ccl.CCL else 0)
    mC = ccl.Mat(M, N, 2, P, ccl.PART_COLS, layout_bc, align if layout_bc == ccl.CCL else 0)
    return mA, mB, mC


_NVML = {}
LAST_CLOCK = dict(sm_mhz=None, sm_max_mhz=None)


def sm_clock():
    """SM clock of the current device in MHz (read through NVML; None where that is not possible).  Reading only."""
    try:
        import pynvml
        if "h" not in _NVML:
            pynvml.nvmlInit()
            uuid = str(torch.cuda.get_device_properties(torch.cuda.current_device()).uuid)
            _NVML["h"] = pynvml.nvmlDeviceGetHandleByUUID(("GPU-" + uuid if not uuid.startswith("GPU-") else uuid).encode())
            _NVML["max"] = pynvml.nvmlDeviceGetMaxClockInfo(_NVML["h"], pynvml.NVML_CLOCK_SM)
        return dict(sm_mhz=pynvml.nvmlDeviceGetClockInfo(_NVML["h"], pynvml.NVML_CLOCK_SM), sm_max_mhz=_NVML["max"])
    except Exception:
        return dict(sm_mhz=None, sm_max_mhz=None)


def timed(fn, reps, warm=2):
    """Mean device time of `fn` in ms over `reps` back-to-back launches (CUDA events on the current stream).
    The launches are queued behind a short device-side spin, so that a kernel of a few microseconds is not
    timed at the rate the host can issue it."""
    for _ in range(warm):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda._sleep(min(200_000_000, 1_000_000 + 40_000 * reps))      # cycles; ~20 us of head start per launch
    e0.record()
    for _ in range(reps):
        fn()
    e1.record()
    LAST_CLOCK.update(sm_clock())            # sampled while the queued launches run
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / reps


def partitions(g):
    """Output partitions swept per GEMM (Sec. 4.1 sweeps them and reports the best): N strips, M strips where M divides,
    and the 2-D cuts pm x pn of P with both factors above 1.  Entries: (label, assign, part_m)."""
    M, N, P = g["M"], g["N"], g["P"]
    out = [("N", ccl.ASSIGN_N_STRIPS, 0)]
    if M % P == 0 and M >= P:
        out.append(("M", ccl.ASSIGN_M_STRIPS, 0))
    for pm in range(2, P):
        if P % pm == 0 and M % pm == 0 and N % (P // pm) == 0:
            out.append((f"{pm}x{P // pm}", ccl.ASSIGN_2D, pm))
    return out


def operand_mats(g, layout_bc, assign, part_m, align, e=2):
    """Descriptors of A, B, C under one output partition: the operands whose rows / columns the partition cuts follow it in
    the given layout (strips = the blocks along that dimension), the others stay row-major.  Returns (mats, parts)."""
    M, N, K, P = g["M"], g["N"], g["K"], g["P"]
    at, bt = g["a_trans"], g["b_trans"]
    pm = P if assign == ccl.ASSIGN_M_STRIPS else (part_m if assign == ccl.ASSIGN_2D else 1)
    pn = P if assign == ccl.ASSIGN_N_STRIPS else (P // part_m if assign == ccl.ASSIGN_2D else 1)
    a_part = (ccl.PART_COLS if at else ccl.PART_ROWS) if pm > 1 else ccl.PART_NONE
    b_part = (ccl.PART_ROWS if bt else ccl.PART_COLS) if pn > 1 else ccl.PART_NONE
    c_part = ccl.PART_COLS if pn > 1 and pm == 1 else (ccl.PART_ROWS if pm > 1 else ccl.PART_NONE)   # 2-D: C's rows follow A
    parts = (a_part, b_part, c_part)
    strips = (pm, pn, pn if c_part == ccl.PART_COLS else pm)
    shapes = ((K, M) if at else (M, K), (N, K) if bt else (K, N), (M, N))
    ms = []
    for X in range(3):
        is_ccl = layout_bc != ccl.ROWMAJOR and parts[X] != ccl.PART_NONE
        ms.append(ccl.Mat(shapes[X][0], shapes[X][1], e, strips[X] if is_ccl else 1, parts[X] if is_ccl else ccl.PART_NONE,
                          layout_bc if is_ccl else ccl.ROWMAJOR, align if is_ccl else 0))
    return ms, parts


def traffic_remote(g, layout_bc, place_bc, S, assign, align=0, part_m=0):
    """Remote bytes (A, B, C) of one policy under one output partition."""
    M, N, K, P = g["M"], g["N"], g["K"], g["P"]
    at, bt = g["a_trans"], g["b_trans"]
    td = ccl.TrafficDesc()
    td.M, td.N, td.K, td.BM, td.BN = M, N, K, 128, 128
    ms, parts = operand_mats(g, layout_bc, assign, part_m, align)
    td.A, td.B, td.C = ms
    td.a_trans, td.b_trans, td.P, td.page_bytes = at, bt, P, S
    for X in range(3):
        split = parts[X] != ccl.PART_NONE
        td.place[X] = place_bc if split else (ccl.PLACE_RR if place_bc != ccl.PLACE_BEST else ccl.PLACE_BEST)
    td.assign, td.strip_tiling, td.part_m = assign, 1, part_m
    nt, pages = ccl.ccl_traffic_sizes(td)
    per_cta = torch.empty((nt, 3, 2), dtype=torch.int64, device="cuda")
    totals = torch.empty((3, 2), dtype=torch.int64, device="cuda")
    pp = ow = None
    if place_bc == ccl.PLACE_BEST:
        pp = [torch.empty((pages[x], P), dtype=torch.int64, device="cuda") for x in range(3)]
        ow = [torch.empty((pages[x],), dtype=torch.uint8, device="cuda") for x in range(3)]
    ms_t = timed(lambda: ccl.ccl_traffic(td, per_cta, totals, pp, ow), 3, 1)
    t = totals.cpu()
    out = dict(remote=[int(x) for x in t[:, 1]], total=int(t.sum()), ms=ms_t)
    if place_bc != ccl.PLACE_BEST:            # the same policy behind an ideal private L2 per chiplet
        l2 = torch.empty((3, 2), dtype=torch.int64, device="cuda")
        ccl.ccl_traffic_l2(td, l2)
        out["remote_ideal_l2"] = [int(x) for x in l2.cpu()[:, 1]]
    return out


def traffic_desc(g, layout_bc, place_bc, S, assign, align=0, e=2, part_m=0):
    """Library descriptor of one placement policy under one output partition."""
    M, N, K, P = g["M"], g["N"], g["K"], g["P"]
    td = ccl.TrafficDesc()
    td.M, td.N, td.K, td.BM, td.BN = M, N, K, 128, 128
    ms, parts = operand_mats(g, layout_bc, assign, part_m, align, e)
    td.A, td.B, td.C = ms
    td.a_trans, td.b_trans, td.P, td.page_bytes = g["a_trans"], g["b_trans"], P, S
    for X in range(3):
        td.place[X] = place_bc if parts[X] != ccl.PART_NONE else ccl.PLACE_RR
    td.assign, td.strip_tiling, td.part_m = assign, 1, part_m
    return td


LRU_EXEC = dict(wave_ctas=1, k_slice=0)       # how a chiplet's CTAs run in the finite-L2 model (--lru-wave, --lru-kslice)


def traffic_lru_best(g, layout_bc, place_bc, S, model_kw, e=2):
    """Remote bytes (A, B, C) behind a finite LRU L2 per chiplet: the best of the output partitions (N strips, M strips, 2-D cuts) and both CTA
    traversals, as the paper reports (Sec. 4.1 sweeps the CTA traversal and the output partition and keeps the best)."""
    best = None
    for label, assign, pm in partitions(g):
        td = traffic_desc(g, layout_bc, place_bc, S, assign, align=S, e=e, part_m=pm)
        for traversal in (0, 1):
            t = torch.empty((3, 2), dtype=torch.int64, device="cuda")
            ccl.ccl_traffic_lru(td, ccl.L2Model(traversal=traversal, **model_kw, **LRU_EXEC), t)
            r = [int(x) for x in t.cpu()[:, 1]]
            if best is None or sum(r) < sum(best["remote"]):
                best = dict(remote=r, partition=label, traversal=traversal)
    return best


def run_gemm(g, pk, reps, lru=False):
    M, N, K, at, bt, P, S = g["M"], g["N"], g["K"], g["a_trans"], g["b_trans"], g["P"], g["S"]
    dev = "cuda"
    A = torch.empty((K, M) if at else (M, K), dtype=torch.bfloat16, device=dev).normal_(0, g["a_std"])
    B = torch.empty((N, K) if bt else (K, N), dtype=torch.bfloat16, device=dev).normal_(0, g["b_std"])
    res = dict(name=g["name"], M=M, N=N, K=K, P=P, page=S, a_trans=at, b_trans=bt)
    flop = 2.0 * M * N * K
    bytes_alg = 2.0 * (M * K + K * N + M * N)
    roof_tf = min(pk["tf"], pk["hbm"] * flop / bytes_alg / 1e3)
    res.update(flop=flop, algorithmic_bytes=bytes_alg, roofline_tflops=roof_tf, roofline_bound="tensor" if roof_tf >= pk["tf"] else "hbm")
    outs = {}
    for tag, lay, grouped in (("ccl_grouped", ccl.CCL, 1), ("row_plain", ccl.ROWMAJOR, 0)):
        mA, mB, mC = mats(g, lay, S)
        d = ccl.GemmDesc()
        d.M, d.N, d.K, d.A, d.B, d.C = M, N, K, mA, mB, mC
        d.a_trans, d.b_trans, d.out_part, d.P, d.grouped_raster = at, bt, ccl.PART_COLS, P, grouped
        try:
            need = ccl.ccl_gemm_workspace(d)
        except ccl.CclError as e:
            res[tag] = dict(error=str(e))
            continue
        ws = torch.empty(max(need, 16) // 4, dtype=torch.float32, device=dev)
        Bl = B
        if lay == ccl.CCL:
            Bl = torch.empty(ccl.ccl_buffer_bytes(mB) // 2, dtype=torch.bfloat16, device=dev)
            rp_ms = timed(lambda: ccl.ccl_repack(mB, B, Bl, 0), reps)
            rp_bytes = 2.0 * K * N * 2
            res["repack"] = dict(ms=rp_ms, gbs=rp_bytes / rp_ms / 1e6, frac_of_hbm=rp_bytes / rp_ms / 1e6 / pk["hbm"])
        Cb = torch.empty(ccl.ccl_buffer_bytes(mC) // 2, dtype=torch.bfloat16, device=dev)
        ms_g = timed(lambda: ccl.ccl_gemm(d, A, Bl, Cb, ws), reps)
        st, detail = ccl.ccl_gemm_status()
        tf = flop / ms_g / 1e9
        res[tag] = dict(ms=ms_g, tflops=tf, frac_of_roofline=tf / roof_tf, split_k_workspace=need, status=st, **LAST_CLOCK)
        if lay == ccl.CCL:
            Cr = torch.empty(M * N, dtype=torch.bfloat16, device=dev)
            ccl.ccl_repack(mC, Cb, Cr, 1)
            outs[tag] = Cr
        else:
            outs[tag] = Cb
    if len(outs) == 2:
        res["ccl_equals_rowmajor_bits"] = bool(torch.equal(outs["ccl_grouped"], outs["row_plain"]))
    # library matmul on the same operands: context only
    Al = A.t() if at else A
    Bm = B.t() if bt else B
    ms_t = timed(lambda: torch.matmul(Al, Bm), reps)
    res["torch_matmul_tflops"] = flop / ms_t / 1e9
    # remote traffic under the placement policies
    base = None
    pol = {}
    for tag, lay, place, Sp in (("row_rr4k", ccl.ROWMAJOR, ccl.PLACE_RR, 4096), ("row_rr64k", ccl.ROWMAJOR, ccl.PLACE_RR, 65536),
                                ("row_rr2m", ccl.ROWMAJOR, ccl.PLACE_RR, 2 << 20), ("row_block", ccl.ROWMAJOR, ccl.PLACE_BLOCK, S),
                                ("row_best", ccl.ROWMAJOR, ccl.PLACE_BEST, S), ("ccl_block", ccl.CCL, ccl.PLACE_BLOCK, S),
                                ("ccl_rr", ccl.CCL, ccl.PLACE_RR, S), ("ileave_rr", ccl.CCL_INTERLEAVED, ccl.PLACE_RR, S)):
        best = None
        for label, assign, pm in partitions(g):
            r = traffic_remote(g, lay, place, Sp, assign, align=Sp, part_m=pm)
            r["partition"] = label
            if best is None or sum(r["remote"]) < sum(best["remote"]):
                best = r
        pol[tag] = best
        if tag == "row_rr4k":
            base = sum(best["remote"])
    base_l2 = sum(pol["row_rr4k"]["remote_ideal_l2"])
    for tag, r in pol.items():
        r["ratio_vs_rr4k"] = (sum(r["remote"]) / base) if base else None
        if "remote_ideal_l2" in r:
            r["ratio_vs_rr4k_ideal_l2"] = (sum(r["remote_ideal_l2"]) / base_l2) if base_l2 else None
    res["traffic"] = pol
    if lru:                                       # the paper's metric: behind an 8 MB, 16-way, 128-byte-line L2 per chiplet
        kw = dict(capacity_bytes=8 << 20, line_bytes=128, ways=16, hash=1)
        fin = {tag: traffic_lru_best(g, lay, place, Sp, kw) for tag, lay, place, Sp in
               (("row_rr4k", ccl.ROWMAJOR, ccl.PLACE_RR, 4096), ("row_block", ccl.ROWMAJOR, ccl.PLACE_BLOCK, S), ("ccl_block", ccl.CCL, ccl.PLACE_BLOCK, S))}
        b = sum(fin["row_rr4k"]["remote"])
        for r in fin.values():
            r["ratio_vs_rr4k"] = sum(r["remote"]) / b if b else None
        res["traffic_finite_l2"] = fin
    return res


def capacity_and_dtype_sweep(out_dir, quick):
    """The two sweeps of the paper's last figure (Sec. 4.2: remote traffic against the per-chiplet L2 capacity with bf16
    fixed, and against the data type with 8 MB fixed; average absolute traffic over the GEMMs at 4K tokens), under this
    library's finite-L2 model: P = 4, 4 KB pages, best output partition and traversal per GEMM."""
    T = 4096
    gemms = [dict(g, P=4) for g in synth.qwen_ffn_gemms(T=T) + synth.llama_fwd_gemms(T=T) + synth.llama_bwd_gemms(T=T)]
    if quick:
        gemms = gemms[:6]
    policies = (("rr4k", ccl.ROWMAJOR, ccl.PLACE_RR), ("coarse", ccl.ROWMAJOR, ccl.PLACE_BLOCK), ("ccl", ccl.CCL, ccl.PLACE_BLOCK))
    settings = [("capacity", mb, 2) for mb in ((4, 8, 16) if quick else (2, 4, 8, 16, 32))] + [("dtype", 8, e) for e in (1, 4)]
    table = []
    for kind, mb, e in settings:
        kw = dict(capacity_bytes=mb << 20, line_bytes=128, ways=16, hash=1)
        avg = {}
        for tag, lay, place in policies:
            tot = 0
            for g in gemms:
                tot += sum(traffic_lru_best(g, lay, place, 4096, kw, e=e)["remote"])
            avg[tag] = tot / len(gemms)
        table.append(dict(sweep=kind, l2_mb=mb, elem_bytes=e, avg_remote_bytes=avg))
        print(f"sweep {kind:8s} L2 {mb:2d} MB, {e}-byte elements: average remote bytes over {len(gemms)} GEMMs at {T} tokens: "
              + "  ".join(f"{k} {v / 1e9:8.3f} GB" for k, v in avg.items()) + f"  | CCL / coarse = {avg['ccl'] / avg['coarse']:.3f}", flush=True)
    json.dump(table, open(os.path.join(out_dir, "report_l2_sweep.json"), "w"), indent=1)


def paper_sweep(out_dir, quick):
    """The paper's headline experiment (Sec. 4.2) under this library's finite-L2 model: the six FFN GEMMs (gate/up and
    down; forward, data gradient, weight gradient) of the Qwen-3-30B-style expert and the Llama-3.1-70B-style layer at
    4K / 8K / 16K tokens (18 GEMMs per model), P = 4, 4 KB pages, 8 MB / 16-way / 128-byte L2 per chiplet, best output
    partition and traversal per GEMM; remote traffic of coarse locality-aware placement and of CCL against 4 KB
    round-robin, as geometric means; run for both execution models (one CTA after the other; waves in lockstep)."""
    kw = dict(capacity_bytes=8 << 20, line_bytes=128, ways=16, hash=1)
    policies = (("rr4k", ccl.ROWMAJOR, ccl.PLACE_RR), ("coarse", ccl.ROWMAJOR, ccl.PLACE_BLOCK), ("ccl", ccl.CCL, ccl.PLACE_BLOCK))
    tokens = (4096,) if quick else (4096, 8192, 16384)
    gm = lambda xs: math.exp(sum(math.log(x) for x in xs) / len(xs)) if xs else float("nan")
    out = []
    for exec_name, exec_kw in (("one CTA after the other", dict(wave_ctas=1, k_slice=0)), ("waves of 76 CTAs, 256 elements of K per step", dict(wave_ctas=76, k_slice=256))):
        LRU_EXEC.update(exec_kw)
        for model, H, I in (("qwen", 2048, 768), ("llama", 8192, 28672)):
            rows = []
            for T in tokens:
                for g in synth.qwen_ffn_gemms(T=T, H=H, I=I):
                    g = dict(g, P=4, name=g["name"].replace("qwen", model) + f"_T{T}")
                    rem = {tag: sum(traffic_lru_best(g, lay, place, 4096, kw)["remote"]) for tag, lay, place in policies}
                    rows.append(dict(name=g["name"], M=g["M"], N=g["N"], K=g["K"], remote_bytes=rem))
                    print(f"  {g['name']:28s} M {g['M']:6d} N {g['N']:6d} K {g['K']:6d}: remote GB rr4k {rem['rr4k'] / 1e9:8.3f} coarse {rem['coarse'] / 1e9:8.3f} "
                          f"CCL {rem['ccl'] / 1e9:8.3f}", flush=True)
            pos = [r["remote_bytes"] for r in rows if min(r["remote_bytes"].values()) > 0]
            fine = [r for r in pos if r["ccl"] < r["coarse"]]
            summary = dict(exec=exec_name, model=model, gemms=len(rows), ccl_over_rr4k=gm([r["ccl"] / r["rr4k"] for r in pos]),
                           coarse_over_rr4k=gm([r["coarse"] / r["rr4k"] for r in pos]), coarse_over_ccl=gm([r["coarse"] / r["ccl"] for r in pos]),
                           fine_optimal=len(fine), max_coarse_over_ccl=max([r["coarse"] / r["ccl"] for r in pos], default=float("nan")))
            out.append(dict(summary=summary, gemms=rows))
            print(f"sweep [{exec_name}] {model}: {len(rows)} GEMMs ({len(rows) - len(pos)} with a zero count left out of the means): geometric mean CCL / rr4k "
                  f"{summary['ccl_over_rr4k']:.3f}, coarse / rr4k {summary['coarse_over_rr4k']:.3f}, coarse / CCL {summary['coarse_over_ccl']:.2f}x "
                  f"(max {summary['max_coarse_over_ccl']:.1f}x); CCL strictly below coarse on {len(fine)} GEMMs", flush=True)
    json.dump(out, open(os.path.join(out_dir, "report_paper_sweep.json"), "w"), indent=1)


def topology(out_dir):
    """Which SMs share a die with which part of the L2 (an experiment, not part of the benchmark): every SM times
    dependent L1-bypassing loads to 512 cache lines; after removing each line's and each SM's mean, the first singular
    vector of the SM x line latency matrix splits the SMs and the lines into two sides."""
    import numpy as np
    nsm = torch.cuda.get_device_properties(0).multi_processor_count
    nl = 512
    buf = torch.zeros(8 << 20, dtype=torch.uint8, device="cuda")
    sides = []
    for rep in range(2):
        lat, smid = ccl.ccl_probe_l2_latency(buf, nl, 4096 + 128 * rep, nsm)
        torch.cuda.synchronize()
        L, sm = lat.cpu().numpy().astype(np.float64), smid.cpu().numpy()
        order = np.argsort(sm)
        L, sm = L[order], sm[order]
        X = L - L.mean(0, keepdims=True)
        X = X - X.mean(1, keepdims=True)
        U, S, Vt = np.linalg.svd(X, full_matrices=False)
        side = U[:, 0] > 0
        if not side[0]:
            side = ~side
        lines = X[side].mean(0) < 0                          # the lines this side of SMs reaches faster
        near = (L[np.ix_(side, lines)].mean() + L[np.ix_(~side, ~lines)].mean()) / 2
        far = (L[np.ix_(side, ~lines)].mean() + L[np.ix_(~side, lines)].mean()) / 2
        sides.append(side)
        print(f"topology run {rep}: {len(set(sm.tolist()))} SMs probed; singular values {S[0]:.0f}, {S[1]:.0f}, {S[2]:.0f}; sides of {int(side.sum())} and "
              f"{int((~side).sum())} SMs; {int(lines.sum())} of {nl} lines nearer to the first side; mean load latency {near:.0f} cycles to the near "
              f"half of the L2, {far:.0f} to the far half", flush=True)
    agree = int((sides[0] == sides[1]).sum())
    print(f"topology: the two runs put {agree} of {nsm} SMs on the same side; first side (by %smid): {sm[sides[0]].tolist()}", flush=True)
    json.dump(dict(sm_count=nsm, side_of_sm={int(a): int(b) for a, b in zip(sm, sides[0])}, agree=agree),
              open(os.path.join(out_dir, "report_topology.json"), "w"), indent=1)


def extras(out_dir, quick, only=None):
    """The entry points around the plain GEMM, timed on the shapes they are meant for: the batch of expert GEMMs in one
    launch, the gated activation fused into the gate/up GEMM, and alpha/beta accumulation."""
    dev, rows = "cuda", []
    want = lambda section: only is None or only in section       # --only batched | swiglu | axpby | transpose | experts

    def desc(M, N, K, P, bt=0, c_cols=None):
        d = ccl.GemmDesc()
        d.M, d.N, d.K = M, N, K
        d.A = ccl.Mat(M, K, 2)
        d.B = ccl.Mat(N, K, 2, P, ccl.PART_ROWS, ccl.CCL, 4096) if bt else ccl.Mat(K, N, 2, P, ccl.PART_COLS, ccl.CCL, 4096)
        d.C = ccl.Mat(M, c_cols or N, 2, P, ccl.PART_COLS, ccl.CCL, 4096)
        d.a_trans, d.b_trans, d.out_part, d.P, d.grouped_raster = 0, bt, ccl.PART_COLS, P, 1
        return d

    def buf(m, n=1):
        return torch.empty(n * ccl.ccl_buffer_bytes(m) // 2, dtype=torch.bfloat16, device=dev).normal_(0, 0.05)

    # 1. the experts of an MoE layer: one launch against one launch per expert and against torch.bmm
    for E, M, N, K, bt in (((128, 256, 768, 2048, 1), (128, 256, 2048, 768, 0)) if not quick else ((32, 256, 768, 2048, 1),)) if want("batched_gemm") else ():
        d = desc(M, N, K, 4, bt)
        A, B, Cb = buf(d.A, E), buf(d.B, E), buf(d.C, E)
        sa, sb, sc = (ccl.ccl_buffer_bytes(m) for m in (d.A, d.B, d.C))
        need = ccl.ccl_gemm_batched_workspace(d, E)
        ws = torch.empty(max(need, 16) // 4, dtype=torch.float32, device=dev)
        t_b = timed(lambda: ccl.ccl_gemm_batched(d, E, A, sa, B, sb, Cb, sc, ws if need else None), 20)
        need1 = ccl.ccl_gemm_workspace(d)
        ws1 = torch.empty(max(need1, 16) // 4, dtype=torch.float32, device=dev)
        views = [(A[e * sa // 2:(e + 1) * sa // 2], B[e * sb // 2:(e + 1) * sb // 2], Cb[e * sc // 2:(e + 1) * sc // 2]) for e in range(E)]

        def one_by_one():
            for a, b, c in views:
                ccl.ccl_gemm(d, a, b, c, ws1 if need1 else None)
        t_l = timed(one_by_one, 3)
        Al = A.view(E, M, K)
        Bl = B.view(E, N, K).transpose(1, 2) if bt else B.view(E, K, N)        # same bytes read as plain matrices: timing only
        t_t = timed(lambda: torch.bmm(Al, Bl), 20)
        fl = 2.0 * E * M * N * K
        rows.append(dict(what="batched", E=E, M=M, N=N, K=K, batched_ms=t_b, launches_ms=t_l, torch_bmm_ms=t_t,
                         batched_tflops=fl / t_b / 1e9, torch_bmm_tflops=fl / t_t / 1e9))
        print(f"extras batched {E} x {M}x{N}x{K}: one launch {t_b * 1e3:8.1f} us ({fl / t_b / 1e9:6.0f} TFLOP/s) | {E} launches {t_l * 1e3:8.1f} us | "
              f"torch.bmm {t_t * 1e3:8.1f} us", flush=True)
    # 1b. the same experts with uneven (routed) token counts: the ragged batch in one launch
    for E, T, N, K, bt in (((128, 32768, 768, 2048, 1), (128, 32768, 2048, 768, 0)) if not quick else ((32, 8192, 768, 2048, 1),)) if want("grouped_gemm") else ():
        import numpy as np
        for conc, label in ((1e6, "equal counts"), (2.0, "Dirichlet(2) counts"), (0.5, "Dirichlet(0.5) counts")):
            wts = np.random.default_rng(3).dirichlet(np.full(E, conc))
            counts = np.floor(wts * T).astype(np.int64)
            counts[0] += T - counts.sum()
            offs = torch.from_numpy(np.concatenate([[0], np.cumsum(counts)]).astype(np.int32)).to(dev)
            d = desc(T, N, K, 4, bt)
            A, B, Cb = buf(d.A), buf(d.B, E), buf(d.C)
            sb = ccl.ccl_buffer_bytes(d.B)
            cap = int(counts.max())
            t_g = timed(lambda: ccl.ccl_gemm_grouped(d, E, cap, offs, A, B, sb, Cb), 20)
            Av, Bv = A.view(T, K), (B.view(E, N, K) if bt else B.view(E, K, N))
            bounds = [int(x) for x in offs.cpu()]

            def torch_loop():
                for e in range(E):
                    if bounds[e + 1] > bounds[e]:
                        torch.matmul(Av[bounds[e]:bounds[e + 1]], Bv[e].t() if bt else Bv[e])
            t_t = timed(torch_loop, 3)
            t_lib = None                                           # the library's own grouped GEMM, where this torch has one
            try:
                Bk = Bv.transpose(1, 2) if bt else Bv              # [E, K, N] view
                ends = offs[1:].contiguous()
                t_lib = timed(lambda: torch._grouped_mm(Av, Bk, offs=ends), 20)
            except Exception as err:                               # noqa: BLE001 (absent or unsupported: report and go on)
                print(f"extras grouped: torch._grouped_mm not usable here ({type(err).__name__})", flush=True)
            tf = 2.0 * T * N * K / (t_g * 1e-3) / 1e12
            rows.append(dict(what="grouped", experts=E, tokens=T, N=N, K=K, counts=label, max_count=cap, grouped_ms=t_g, torch_loop_ms=t_t,
                             torch_grouped_mm_ms=t_lib, tflops=tf))
            print(f"extras grouped {E} experts, {T} tokens x {N} x {K}, {label} (max {cap}): one launch {t_g * 1e3:8.1f} us ({tf:6.0f} TFLOP/s) | "
                  f"torch.matmul per expert {t_t * 1e3:8.1f} us" + (f" | torch._grouped_mm {t_lib * 1e3:8.1f} us" if t_lib else ""), flush=True)
    # 1c. a whole MoE expert FFN forward on routed tokens: gate/up with the activation fused, then down -- two launches
    for E, T, H, I in (((128, 32768, 2048, 768),) if not quick else ((32, 8192, 2048, 768),)) if want("moe_ffn") else ():
        import numpy as np
        wts = np.random.default_rng(3).dirichlet(np.full(E, 2.0))
        counts = np.floor(wts * T).astype(np.int64)
        counts[0] += T - counts.sum()
        offs = torch.from_numpy(np.concatenate([[0], np.cumsum(counts)]).astype(np.int32)).to(dev)
        cap = int(counts.max())
        d1 = desc(T, 2 * I, H, 4, 0, c_cols=I)                       # X [T x H] * Wgu [H x 2I] -> silu(gate) * up [T x I]
        d2 = desc(T, H, I, 4, 0)                                     # ... * Wd [I x H] -> [T x H]
        d2.A = d1.C                                                  # the down GEMM reads the activation where the first wrote it
        X, Wgu, Act, Wd, Y = buf(d1.A), buf(d1.B, E), buf(d1.C), buf(d2.B, E), buf(d2.C)
        s1, s2 = ccl.ccl_buffer_bytes(d1.B), ccl.ccl_buffer_bytes(d2.B)
        try:
            def ffn():
                ccl.ccl_gemm_grouped_swiglu(d1, E, cap, offs, X, Wgu, s1, Act)
                ccl.ccl_gemm_grouped(d2, E, cap, offs, Act, Wd, s2, Y)
            t_f = timed(ffn, 20)
            t_1 = timed(lambda: ccl.ccl_gemm_grouped_swiglu(d1, E, cap, offs, X, Wgu, s1, Act), 20)
            fl = 2.0 * T * (2 * I * H + H * I)
            rows.append(dict(what="moe_ffn", experts=E, tokens=T, H=H, I=I, ffn_ms=t_f, gateup_ms=t_1, tflops=fl / (t_f * 1e-3) / 1e12))
            print(f"extras MoE FFN forward, {E} experts, {T} routed tokens (Dirichlet(2), max {cap}), H {H} I {I}: gate/up + activation {t_1 * 1e3:7.1f} us, "
                  f"with down {t_f * 1e3:7.1f} us ({fl / (t_f * 1e-3) / 1e12:6.0f} TFLOP/s)", flush=True)
        except ccl.CclError as err:
            print(f"extras MoE FFN forward: not supported in this form ({err})", flush=True)
    # 1d. the weight gradients of the experts: ragged K in one launch
    for E, T, H, I in (((128, 32768, 2048, 768),) if not quick else ((32, 8192, 2048, 768),)) if want("moe_wgrad") else ():
        import numpy as np
        wts = np.random.default_rng(3).dirichlet(np.full(E, 2.0))
        counts = np.floor(wts * T).astype(np.int64)
        counts[0] += T - counts.sum()
        offs = torch.from_numpy(np.concatenate([[0], np.cumsum(counts)]).astype(np.int32)).to(dev)
        bounds = [int(x) for x in offs.cpu()]
        for name, M, N in (("down: act^T x dY", I, H), ("gate/up: X^T x dAct", H, 2 * I)):
            d = ccl.GemmDesc()
            d.M, d.N, d.K = M, N, T
            d.A = ccl.Mat(T, M, 2)                                    # stored [K x M]
            d.B = ccl.Mat(T, N, 2)
            d.C = ccl.Mat(M, N, 2, 4, ccl.PART_COLS, ccl.CCL, 4096)   # the gradient in the layout of the weight
            d.a_trans, d.b_trans, d.out_part, d.P, d.grouped_raster = 1, 0, ccl.PART_COLS, 4, 1
            A, B, Cb = buf(d.A), buf(d.B), buf(d.C, E)
            sc = ccl.ccl_buffer_bytes(d.C)
            t_g = timed(lambda: ccl.ccl_gemm_grouped_k(d, E, offs, A, B, Cb, sc), 20)
            Av, Bv = A.view(T, M), B.view(T, N)

            def torch_loop():
                for e in range(E):
                    if bounds[e + 1] > bounds[e]:
                        torch.matmul(Av[bounds[e]:bounds[e + 1]].t(), Bv[bounds[e]:bounds[e + 1]])
            t_t = timed(torch_loop, 3)
            t_lib = None
            try:
                ends = offs[1:].contiguous()
                t_lib = timed(lambda: torch._grouped_mm(Av.t(), Bv, offs=ends), 20)
            except Exception as err:                               # noqa: BLE001
                print(f"extras MoE weight gradient: torch._grouped_mm not usable here ({type(err).__name__})", flush=True)
            tf = 2.0 * T * M * N / (t_g * 1e-3) / 1e12
            rows.append(dict(what="moe_wgrad", name=name, experts=E, tokens=T, M=M, N=N, grouped_k_ms=t_g, torch_loop_ms=t_t, torch_grouped_mm_ms=t_lib, tflops=tf))
            print(f"extras MoE weight gradient ({name}), {E} experts, {T} routed tokens, {M} x {N} each: one launch {t_g * 1e3:8.1f} us ({tf:6.0f} TFLOP/s) | "
                  f"torch.matmul per expert {t_t * 1e3:8.1f} us" + (f" | torch._grouped_mm {t_lib * 1e3:8.1f} us" if t_lib else ""), flush=True)
    # 2. gate/up GEMM with the gated activation in the epilogue against GEMM + elementwise kernel
    for M, N, K in (((8192, 57344, 8192), (16384, 1536, 2048)) if not quick else ((1024, 57344, 8192),)) if want("swiglu") else ():
        d0, d1 = desc(M, N, K, 4), desc(M, N, K, 4, c_cols=N // 2)
        A, B, C0, C1 = buf(d0.A), buf(d0.B), buf(d0.C), buf(d1.C)
        reps = 5 if M * N * K > 1e11 else 50
        t_g = timed(lambda: ccl.ccl_gemm(d0, A, B, C0), reps)
        H = C0.view(M, N)
        out = torch.empty(M, N // 2, dtype=torch.bfloat16, device=dev)
        t_a = timed(lambda: torch.mul(torch.nn.functional.silu(H[:, :N // 2]), H[:, N // 2:], out=out), reps)
        t_f = timed(lambda: ccl.ccl_gemm_swiglu(d1, A, B, C1), reps)
        rows.append(dict(what="swiglu", M=M, N=N, K=K, gemm_ms=t_g, elementwise_ms=t_a, fused_ms=t_f))
        print(f"extras gate/up {M}x{N}x{K}: GEMM {t_g * 1e3:8.1f} us + silu*mul kernel {t_a * 1e3:8.1f} us = {(t_g + t_a) * 1e3:8.1f} us | "
              f"fused {t_f * 1e3:8.1f} us ({2.0 * M * N * K / t_f / 1e9:6.0f} TFLOP/s)", flush=True)
    # 3. alpha / beta: what reading C in the epilogue costs
    for M, N, K in (((8192, 8192, 8192),) if not quick else ((2048, 8192, 2048),)) if want("axpby") else ():
        d = desc(M, N, K, 4)
        A, B, Cc = buf(d.A), buf(d.B), buf(d.C)
        t_p = timed(lambda: ccl.ccl_gemm(d, A, B, Cc), 10)
        t_x = timed(lambda: ccl.ccl_gemm_axpby(d, 1.0, 1.0, A, B, Cc), 10)
        rows.append(dict(what="axpby", M=M, N=N, K=K, gemm_ms=t_p, axpby_ms=t_x))
        print(f"extras accumulate {M}x{N}x{K}: C = A*B {t_p * 1e3:8.1f} us | C += A*B {t_x * 1e3:8.1f} us", flush=True)
    # 4. transposing repack: a weight kept as [N x K] becomes CCL [K x N]; against the plain repack and a strided copy
    for name, R, Cc in ((("llama_down", 28672, 8192), ("llama_gateup", 8192, 57344)) if not quick else (("qwen_x16", 4096, 16 * 1536),)) if want("transpose") else ():
        for layout, S in ((ccl.CCL, 0), (ccl.CCL_INTERLEAVED, 4096)):
            m = ccl.Mat(R, Cc, 2, 4, ccl.PART_COLS, layout, S)
            src = torch.empty(R * Cc, dtype=torch.int16, device=dev).random_()
            dst = torch.empty(ccl.ccl_buffer_bytes(m) // 2, dtype=torch.int16, device=dev)
            xt, y = src.view(Cc, R), torch.empty(R, Cc, dtype=torch.int16, device=dev)
            t_t = timed(lambda: ccl.ccl_repack_transpose(m, src, dst), 10)
            t_r = timed(lambda: ccl.ccl_repack(m, src, dst, 0), 10)
            t_c = timed(lambda: y.copy_(xt.t()), 5)
            gbs = lambda ms: 2 * R * Cc * 2 / (ms * 1e-3) / 1e9
            rows.append(dict(what="repack_transpose", name=name, rows=R, cols=Cc, layout=layout, transpose_gbs=gbs(t_t), repack_gbs=gbs(t_r), torch_t_copy_gbs=gbs(t_c)))
            print(f"extras transposing repack {name} [{Cc}x{R}] -> CCL [{R}x{Cc}] P 4 layout {layout}: {gbs(t_t):7.0f} GB/s | plain repack {gbs(t_r):7.0f} GB/s | "
                  f"torch copy_(x.t()) {gbs(t_c):7.0f} GB/s", flush=True)
    # 5. the weights of all experts in one launch
    for R, Cc in (((2048, 1536), (768, 2048))) if want("experts_repack") else ():
        E = 128 if not quick else 16
        m = ccl.Mat(R, Cc, 2, 4, ccl.PART_COLS, ccl.CCL, 4096)
        nb = ccl.ccl_buffer_bytes(m)
        src = torch.empty(E * R * Cc, dtype=torch.int16, device=dev).random_()
        dst = torch.empty(E * nb // 2, dtype=torch.int16, device=dev)
        t_b = timed(lambda: ccl.ccl_repack_batched(m, E, src, R * Cc * 2, dst, nb, 0), 10)

        def loop():
            for i in range(E):
                ccl.ccl_repack(m, src[i * R * Cc:(i + 1) * R * Cc], dst[i * nb // 2:(i + 1) * nb // 2], 0)
        t_l = timed(loop, 5)
        gbs = lambda ms: 2 * E * R * Cc * 2 / (ms * 1e-3) / 1e9
        rows.append(dict(what="repack_batched", experts=E, rows=R, cols=Cc, batched_gbs=gbs(t_b), looped_gbs=gbs(t_l)))
        print(f"extras repack of {E} expert weights [{R}x{Cc}]: one launch {gbs(t_b):7.0f} GB/s ({t_b * 1e3:7.1f} us) | {E} launches {gbs(t_l):7.0f} GB/s ({t_l * 1e3:7.1f} us)", flush=True)
    json.dump(rows, open(os.path.join(out_dir, "report_extras.json"), "w"), indent=1)


def one_gemm(args):
    f = [int(x) for x in args.gemm.split(",")]
    M, N, K = f[:3]
    at, bt = (f[3], f[4]) if len(f) >= 5 else (0, 0)
    P, page = 4, 4096
    mB = ccl.Mat(N, K, 2, P, ccl.PART_ROWS, ccl.CCL, page) if bt else ccl.Mat(K, N, 2, P, ccl.PART_COLS, ccl.CCL, page)
    mC = ccl.Mat(M, N, 2, P, ccl.PART_COLS, ccl.CCL, page)
    d = ccl.GemmDesc()
    d.M, d.N, d.K, d.A, d.B, d.C = M, N, K, (ccl.Mat(K, M, 2) if at else ccl.Mat(M, K, 2)), mB, mC
    d.a_trans, d.b_trans, d.out_part, d.P, d.grouped_raster = at, bt, ccl.PART_COLS, P, 1
    a = torch.empty((K, M) if at else (M, K), dtype=torch.bfloat16, device="cuda").normal_(0, 1)
    b = torch.empty(ccl.ccl_buffer_bytes(mB) // 2, dtype=torch.bfloat16, device="cuda").normal_(0, 0.02)
    c = torch.empty(ccl.ccl_buffer_bytes(mC) // 2, dtype=torch.bfloat16, device="cuda")
    need = ccl.ccl_gemm_workspace(d)
    ws = torch.empty(max(need, 16) // 4, dtype=torch.float32, device="cuda")
    ms = timed(lambda: ccl.ccl_gemm(d, a, b, c, ws), args.reps, 1)
    st, detail = ccl.ccl_gemm_status()
    print(f"gemm {M}x{N}x{K} a_trans {at} b_trans {bt}: {ms * 1e3:.1f} us, {2.0 * M * N * K / ms / 1e9:.1f} TFLOP/s, "
          f"algorithmic bytes {2 * (M * K + K * N + M * N)}, status {st}", flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--config", default="all", help="all, one configuration (1-5) or a comma-separated list (e.g. 1,2)")
    ap.add_argument("--out", default=os.path.join(ROOT, "report_out"))
    ap.add_argument("--quick", action="store_true", help="fewer repetitions and P = 4 only in the sweep")
    ap.add_argument("--lru", action="store_true", help="also score the placements behind a finite LRU L2 per chiplet (slow at Llama sizes)")
    ap.add_argument("--lru-wave", type=int, default=1, help="finite-L2 model: CTAs of a chiplet in flight together (1: one after the other)")
    ap.add_argument("--lru-kslice", type=int, default=0, help="finite-L2 model: elements of K a wave consumes per lockstep step (0: all of K)")
    ap.add_argument("--l2-sweep", action="store_true", help="remote traffic against L2 capacity and data type under the finite-L2 model (then exit)")
    ap.add_argument("--paper-sweep", action="store_true", help="the 2 x 18-GEMM sweep of Sec. 4.2 under the finite-L2 model, both execution models (then exit)")
    ap.add_argument("--topology", action="store_true", help="experiment: split the SMs into the two dies by their latency to the L2 (then exit)")
    ap.add_argument("--extras", action="store_true", help="time the batched, gated-activation, alpha/beta, transposing- and batched-repack entry points (then exit)")
    ap.add_argument("--gemm", default=None, help="M,N,K[,a_trans,b_trans]: run just this GEMM (B and C in CCL, P = 4, strips aligned to 4 KB, "
                                                   "grouped raster) --reps times and print its time (e.g. for a profiler capture), then exit")
    ap.add_argument("--reps", type=int, default=3)
    ap.add_argument("--only", default=None, help="run only the GEMMs whose name contains this text (e.g. for a profiler capture)")
    args = ap.parse_args()
    assert torch.cuda.is_available(), "report needs a CUDA device"
    pk = peaks()
    os.makedirs(args.out, exist_ok=True)
    LRU_EXEC.update(wave_ctas=args.lru_wave, k_slice=args.lru_kslice)
    if args.paper_sweep:
        paper_sweep(args.out, args.quick)
        return
    if args.gemm:
        one_gemm(args)
        return
    if args.topology:
        topology(args.out)
        return
    if args.extras:
        extras(args.out, args.quick, args.only)
        return
    if args.l2_sweep:
        capacity_and_dtype_sweep(args.out, args.quick)
        return
    for cfg, gemms in configs(args.config, args.quick).items():
        rows = []
        for g in gemms:
            if args.only and args.only not in g["name"]:
                continue
            big = g["M"] * g["N"] * g["K"] > 1e11
            r = run_gemm(g, pk, 3 if (big or args.quick) else 100, lru=args.lru)
            rows.append(r)
            c, rw = r.get("ccl_grouped", {}), r.get("row_plain", {})
            t = r["traffic"]
            print(f"cfg{cfg} {r['name']:24s} M{r['M']:5d} N{r['N']:5d} K{r['K']:5d} P{r['P']} S{r['page']:7d} | "
                  f"gemm ccl {c.get('tflops', float('nan')):7.1f} row {rw.get('tflops', float('nan')):7.1f} torch {r['torch_matmul_tflops']:7.1f} TF "
                  f"(roof {r['roofline_tflops']:6.1f} {r['roofline_bound']}, {100 * c.get('frac_of_roofline', float('nan')):5.1f}%, {c.get('ms', float('nan')) * 1e3:.1f} us at {c.get('sm_mhz')} MHz) "
                  f"bits_equal={r.get('ccl_equals_rowmajor_bits')} | repack {r.get('repack', {}).get('gbs', float('nan')):7.1f} GB/s | "
                  f"remote/rr4k: rr64k {t['row_rr64k']['ratio_vs_rr4k']:.3f} rr2m {t['row_rr2m']['ratio_vs_rr4k']:.3f} "
                  f"block {t['row_block']['ratio_vs_rr4k']:.3f} best {t['row_best']['ratio_vs_rr4k']:.3f} "
                  f"CCL {t['ccl_block']['ratio_vs_rr4k']:.3f} ({t['ccl_block']['partition']}) ccl+rr {t['ccl_rr']['ratio_vs_rr4k']:.3f} "
                  f"interleaved-CCL+rr {t['ileave_rr']['ratio_vs_rr4k']:.3f} | behind an ideal L2: block {t['row_block']['ratio_vs_rr4k_ideal_l2']:.3f} "
                  f"CCL {t['ccl_block']['ratio_vs_rr4k_ideal_l2']:.3f} interleaved-CCL+rr {t['ileave_rr']['ratio_vs_rr4k_ideal_l2']:.3f}"
                  + (f" | behind an 8 MB LRU L2 (best partition / traversal): block {r['traffic_finite_l2']['row_block']['ratio_vs_rr4k']:.3f} "
                     f"CCL {r['traffic_finite_l2']['ccl_block']['ratio_vs_rr4k']:.3f}" if args.lru else ""), flush=True)
        json.dump(dict(config=cfg, peaks=pk, gemms=rows), open(os.path.join(args.out, f"report_config{cfg}.json"), "w"), indent=1)
        nz = [r["traffic"]["ccl_block"]["ratio_vs_rr4k"] for r in rows if r["traffic"]["ccl_block"]["ratio_vs_rr4k"]]
        if nz:
            print(f"cfg{cfg}: geometric mean of CCL/rr4k remote-traffic ratios over {len(nz)} GEMMs with non-zero ratio "
                  f"({len(rows) - len(nz)} zero): {math.exp(sum(math.log(x) for x in nz) / len(nz)):.3f}", flush=True)
        if args.lru and rows:
            for tag in ("row_block", "ccl_block"):
                rs = [r["traffic_finite_l2"][tag]["ratio_vs_rr4k"] for r in rows if r["traffic_finite_l2"][tag]["ratio_vs_rr4k"]]
                if rs:
                    print(f"cfg{cfg}: behind an 8 MB LRU L2, geometric mean of {tag}/rr4k over {len(rs)} GEMMs: "
                          f"{math.exp(sum(math.log(x) for x in rs) / len(rs)):.3f}", flush=True)


if __name__ == "__main__":
    main()
