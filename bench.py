#!/usr/bin/env python
"""Benchmark of the CCL hot path on B200: repack -> GEMM on CCL operands -> remote-traffic count.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--P 4] [--page 4096]

Workload (N = 1): the Llama-3.1-70B-style dense FFN forward at 8192 tokens,
    gate+up  [8192 x 8192] x [8192 x 57344]   and   down  [8192 x 28672] x [28672 x 8192],
bf16, activations ~N(0,1), weights ~N(0,0.02), synthetic and seeded.  One step is one pass of the
whole hot path over that batch: both weights are repacked row-major -> CCL, both GEMMs run with
B and C in CCL under the chiplet-grouped raster, and the remote-traffic counter scores
CCL + page->strip placement for both GEMMs.  Every operand is far larger than the 126 MB L2.

The metric is GEMM TFLOP/s: 2*M*N*K of both GEMMs divided by the time of the WHOLE step
(repack and counting included).  Kernel-only figures are reported next to it.

With --gpus N > 1 (torchrun, one rank per GPU) every rank processes its own batch with no
data-path collective (weak scaling); the value is the aggregate over ranks, the time the max.

--impl reference times the CPU oracle (test infrastructure, deliberately plain) on a bounded
sample of the same workload; it is the only other place that executes oracle/.
"""
import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "CCL bf16 GEMM TFLOP/s"
UNIT = "TFLOP/s"
T, H, I = 8192, 8192, 28672                         # tokens, hidden, intermediate (Llama-3.1-70B FFN)
GEMMS = [dict(name="gateup", M=T, N=2 * I, K=H), dict(name="down", M=T, N=H, K=I)]
FLOP_PER_STEP = sum(2 * g["M"] * g["N"] * g["K"] for g in GEMMS)


# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) of the two GEMM launches of one step, from the
# single-pass ncu capture of this very workload (profiles/ccl_gemm_kernel_llama_gateup_1024tok.md, second
# table): gate+up 6.40 + 0.93 GB, down 3.03 + 0.12 GB (19.05 GB before the CTAs were kept in step between rounds
# of tiles).  Only valid for the default configuration.
GEMM_DRAM_BYTES_PER_STEP = {(8192, 4, 4096): 10.48e9}


def set_tokens(t):
    """--tokens: a smaller batch of the same FFN (for profiler captures); the default is the 8192-token workload."""
    global T, GEMMS, FLOP_PER_STEP
    T = t
    GEMMS = [dict(name="gateup", M=T, N=2 * I, K=H), dict(name="down", M=T, N=H, K=I)]
    FLOP_PER_STEP = sum(2 * g["M"] * g["N"] * g["K"] for g in GEMMS)


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm_gbs=p["hbm_gbs"], tf_burst=p["bf16_tflops"], tf_sustained=p["bf16_tflops_sustained"], source="measured")
    return dict(hbm_gbs=6650.0, tf_burst=1590.0, tf_sustained=1400.0, source="fallback")


# ---------------------------------------------------------------------------------------------
# clocks: nvidia-smi sampled during the timed region
# ---------------------------------------------------------------------------------------------
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, uuid):
        self.uuid, self.proc, self.path = uuid, None, None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(["nvidia-smi", "-i", self.uuid, f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                                          "-lms", "20"], stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
            time.sleep(0.4)                                            # nvidia-smi needs a moment before its first sample
        except Exception:
            self.proc = None

    def stop(self):
        out = dict(sm_mhz=None, sm_max_mhz=None, reasons=[], samples=0)
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, pw, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in open(self.path):
            f = [x.strip() for x in line.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1])); pw.append(float(f[2]))
            except ValueError:
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        os.unlink(self.path)
        if sm:
            busy = [c for c, w in zip(sm, pw) if w > 0.6 * max(pw)] or sm     # samples taken under load (by power draw)
            out.update(sm_mhz=statistics.median(busy), sm_max_mhz=max(mx), reasons=sorted(reasons), samples=len(sm))
        return out


# ---------------------------------------------------------------------------------------------
# the CUDA arm
# ---------------------------------------------------------------------------------------------
def make_descs(ccl, P, page):
    out = []
    for g in GEMMS:
        M, N, K = g["M"], g["N"], g["K"]
        mA = ccl.Mat(M, K, 2)
        mB = ccl.Mat(K, N, 2, P, ccl.PART_COLS, ccl.CCL, page)          # strips aligned to the page size (Sec. 3.2)
        mC = ccl.Mat(M, N, 2, P, ccl.PART_COLS, ccl.CCL, page)
        gd = ccl.GemmDesc()
        gd.M, gd.N, gd.K, gd.A, gd.B, gd.C = M, N, K, mA, mB, mC
        gd.a_trans, gd.b_trans, gd.out_part, gd.P, gd.grouped_raster = 0, 0, ccl.PART_COLS, P, 1
        tds = {}
        for name, lay, place in (("ccl", ccl.CCL, ccl.PLACE_BLOCK), ("rr4k", ccl.ROWMAJOR, ccl.PLACE_RR)):
            td = ccl.TrafficDesc()
            td.M, td.N, td.K, td.BM, td.BN = M, N, K, 128, 128
            td.A = mA
            td.B = ccl.Mat(K, N, 2, P, ccl.PART_COLS, lay, page if lay == ccl.CCL else 0)
            td.C = ccl.Mat(M, N, 2, P, ccl.PART_COLS, lay, page if lay == ccl.CCL else 0)
            td.a_trans, td.b_trans, td.P = 0, 0, P
            td.page_bytes = page if name == "ccl" else 4096              # the baseline is 4 KB round-robin
            td.place[0], td.place[1], td.place[2] = ccl.PLACE_RR, place, place
            td.assign, td.strip_tiling = ccl.ASSIGN_N_STRIPS, 1
            tds[name] = td
        out.append(dict(g=g, mB=mB, mC=mC, gd=gd, td=tds))
    return out


def run_cuda(args):
    import torch
    from paper_2606_11718_b200 import binding as ccl
    from paper_2606_11718_b200 import synth
    from paper_2606_11718_b200 import dist as ccl_dist

    rank, world, local = ccl_dist.env_world()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device (there is no CPU fallback; use --impl reference for the oracle)")
    torch.cuda.set_device(local)
    group = ccl_dist.Group("nccl", torch.device("cuda", local))
    ccl.lib()
    P, page = args.P, args.page
    descs = make_descs(ccl, P, page)

    # seeded synthetic inputs (each rank its own batch and weights)
    host = {}
    host["X"] = synth.randn_bf16(T, H, synth.ACT_STD, rank, "bench/X").pin_memory()
    host["Wgu"] = synth.randn_bf16(H, 2 * I, synth.WEIGHT_STD, rank, "bench/Wgu").pin_memory()
    host["Z"] = synth.randn_bf16(T, I, synth.ACT_STD, rank, "bench/Z").pin_memory()
    host["Wd"] = synth.randn_bf16(I, H, synth.WEIGHT_STD, rank, "bench/Wd").pin_memory()
    devb = {k: torch.empty_like(v, device="cuda") for k, v in host.items()}
    for k in host:
        devb[k].copy_(host[k], non_blocking=True)
    for d, a, w in zip(descs, ("X", "Z"), ("Wgu", "Wd")):
        d["a"], d["w"] = a, w
        d["w_ccl"] = torch.empty(ccl.ccl_buffer_bytes(d["mB"]) // 2, dtype=torch.bfloat16, device="cuda")
        d["c_ccl"] = torch.empty(ccl.ccl_buffer_bytes(d["mC"]) // 2, dtype=torch.bfloat16, device="cuda")
        nt, _ = ccl.ccl_traffic_sizes(d["td"]["ccl"])
        d["per_cta"] = torch.empty((nt, 3, 2), dtype=torch.int64, device="cuda")
        d["totals"] = torch.empty((3, 2), dtype=torch.int64, device="cuda")
        d["host_c"] = torch.empty(d["c_ccl"].shape, dtype=torch.bfloat16).pin_memory()
        d["host_tot"] = torch.empty((3, 2), dtype=torch.int64).pin_memory()
    torch.cuda.synchronize()

    ev = lambda: torch.cuda.Event(enable_timing=True)
    kernel_events = {"repack": [], "gemm": [], "traffic": []}

    def step(record):
        for d in descs:
            e = [ev() for _ in range(4)] if record else None
            if record: e[0].record()
            ccl.ccl_repack(d["mB"], devb[d["w"]], d["w_ccl"], 0)
            if record: e[1].record()
            ccl.ccl_gemm(d["gd"], devb[d["a"]], d["w_ccl"], d["c_ccl"])
            if record: e[2].record()
            ccl.ccl_traffic(d["td"]["ccl"], d["per_cta"], d["totals"])
            if record:
                e[3].record()
                kernel_events["repack"].append((e[0], e[1])); kernel_events["gemm"].append((e[1], e[2]))
                kernel_events["traffic"].append((e[2], e[3]))

    barrier, max_over_ranks = group.barrier, group.max_over_ranks

    # ---- device-resident timing (the clock sampler runs from the warm-up on; idle samples are dropped by power draw)
    uuid = "GPU-" + str(torch.cuda.get_device_properties(local).uuid).replace("GPU-", "")
    sampler = ClockSampler(uuid)
    sampler.start()
    for _ in range(args.warmup):
        step(False)
    st, detail = ccl.ccl_gemm_status()
    if st != ccl.OK:
        raise SystemExit(f"bench.py: device-side wait expired during warm-up (code {detail})")
    barrier()
    launches0 = ccl.ccl_launch_count()
    t0, t1 = ev(), ev()
    t0.record()
    for _ in range(args.steps):
        step(True)
    t1.record()
    barrier()
    launches = ccl.ccl_launch_count() - launches0
    clocks = sampler.stop()
    ms_total = max_over_ranks(t0.elapsed_time(t1))
    ms_step = ms_total / args.steps
    st, detail = ccl.ccl_gemm_status()
    if st != ccl.OK:
        raise SystemExit(f"bench.py: device-side wait expired (code {detail})")
    kms = {k: sum(a.elapsed_time(b) for a, b in v) / args.steps for k, v in kernel_events.items()}   # per step
    value = world * FLOP_PER_STEP / (ms_step * 1e-3) / 1e12

    # ---- remote-traffic ratio (CCL vs row-major under 4 KB round-robin), outside the timed region
    remote = {"ccl": 0, "rr4k": 0}
    for d in descs:
        for name in remote:
            ccl.ccl_traffic(d["td"][name], d["per_cta"], d["totals"])
            remote[name] += int(d["totals"].cpu()[:, 1].sum())
    ratio = remote["ccl"] / max(1, remote["rr4k"])

    # ---- end to end: host buffers in, result out, every step
    h2d = sum(v.numel() * 2 for v in host.values())
    d2h = sum(d["host_c"].numel() * 2 + 48 for d in descs)

    # Three streams, two buffer slots: the host->device copy of step i+1 and the device->host copy of step i-1
    # overlap the kernels of step i.  Every step still moves all of its inputs in and all of its results out.
    s_in, s_out, s_cmp = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.current_stream()
    slots = []
    for sl in range(2):
        dv = devb if sl == 0 else {k: torch.empty_like(v) for k, v in devb.items()}
        outs = [dict(c_ccl=d["c_ccl"] if sl == 0 else torch.empty_like(d["c_ccl"]),
                     totals=d["totals"] if sl == 0 else torch.empty_like(d["totals"]),
                     per_cta=d["per_cta"] if sl == 0 else torch.empty_like(d["per_cta"])) for d in descs]
        slots.append(dict(dev=dv, outs=outs, ev_in=torch.cuda.Event(), ev_cmp=torch.cuda.Event(), ev_out=torch.cuda.Event()))
    for sl in slots:
        sl["ev_cmp"].record(s_cmp); sl["ev_out"].record(s_cmp)

    def e2e_step(i):
        sl = slots[i % 2]
        with torch.cuda.stream(s_in):
            s_in.wait_event(sl["ev_cmp"])                      # the kernels that last read this slot's inputs are done
            for k in host:
                sl["dev"][k].copy_(host[k], non_blocking=True)
            sl["ev_in"].record(s_in)
        s_cmp.wait_event(sl["ev_in"])
        s_cmp.wait_event(sl["ev_out"])                         # this slot's previous results have left the device
        for d, o in zip(descs, sl["outs"]):
            ccl.ccl_repack(d["mB"], sl["dev"][d["w"]], d["w_ccl"], 0)
            ccl.ccl_gemm(d["gd"], sl["dev"][d["a"]], d["w_ccl"], o["c_ccl"])
            ccl.ccl_traffic(d["td"]["ccl"], o["per_cta"], o["totals"])
        sl["ev_cmp"].record(s_cmp)
        with torch.cuda.stream(s_out):
            s_out.wait_event(sl["ev_cmp"])
            for d, o in zip(descs, sl["outs"]):
                d["host_c"].copy_(o["c_ccl"], non_blocking=True)
                d["host_tot"].copy_(o["totals"], non_blocking=True)
            sl["ev_out"].record(s_out)

    e2e_steps = max(4, min(args.steps, 8))
    e2e_step(0); e2e_step(1)
    barrier()
    t0.record()
    for i in range(e2e_steps):
        e2e_step(i)
    for sl in slots:
        s_cmp.wait_event(sl["ev_out"])
    t1.record()
    barrier()
    e2e_ms = max_over_ranks(t0.elapsed_time(t1)) / e2e_steps
    e2e_value = world * FLOP_PER_STEP / (e2e_ms * 1e-3) / 1e12

    peaks = measured_peaks()
    gemm_tf = FLOP_PER_STEP / (kms["gemm"] * 1e-3) / 1e12
    repack_bytes = sum(2 * g["K"] * g["N"] * 2 for g in GEMMS)
    repack_gbs = repack_bytes / (kms["repack"] * 1e-3) / 1e9
    line = {
        "metric": METRIC, "value": round(value, 2), "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": round(ms_step, 4), "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic",
        "config": {"workload": f"llama31_70b_ffn_fwd_{T}tok: gateup {T}x57344x8192 + down {T}x8192x28672, B and C in CCL",
                   "P": P, "page_bytes": page, "tokens_per_gpu": T, "l2": "inputs larger than L2 (no flush needed)",
                   "step": "2 repack + 2 gemm + 2 traffic"},
        "clocks": clocks,
        "e2e": {"value": round(e2e_value, 2), "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "ms_per_step": round(e2e_ms, 3)},
        "gpu_launches": int(launches),
        "roofline": {"kernel": "ccl_gemm_kernel", "bound": "tensor", "achieved": round(gemm_tf, 1), "peak": peaks["tf_sustained"],
                     "unit": "TFLOP/s", "frac": round(gemm_tf / peaks["tf_sustained"], 4), "traffic": GEMM_DRAM_BYTES_PER_STEP.get((T, P, page)),
                     "traffic_unit": "bytes per step (2 launches), ncu", "algorithmic_bytes_per_step": sum(2 * (g["M"] * g["K"] + g["K"] * g["N"] + g["M"] * g["N"]) for g in GEMMS),
                     "peak_source": f"bf16 sustained, {peaks['source']}", "frac_of_burst": round(gemm_tf / peaks["tf_burst"], 4),
                     "frac_of_nominal_2250": round(gemm_tf / 2250.0, 4), "ms_per_step": round(kms["gemm"], 4)},
        "kernels": {"gemm_tflops": round(gemm_tf, 1), "repack_gbs": round(repack_gbs, 1),
                    "repack_frac_of_hbm": round(repack_gbs / peaks["hbm_gbs"], 4), "repack_ms": round(kms["repack"], 4),
                    "traffic_ms": round(kms["traffic"], 4),
                    "remote_traffic_ratio_ccl_vs_rr4k": round(ratio, 4), "remote_bytes": remote},
    }
    if rank == 0:
        if world == 1 and not args.no_cpu_baseline:
            line["cpu_baseline"] = oracle_sample(P, page, synth, host)
        print(json.dumps(line), flush=True)
    group.close()


# ---------------------------------------------------------------------------------------------
# the oracle on a bounded sample (cpu_baseline and --impl reference)
# ---------------------------------------------------------------------------------------------
SAMPLE_ROWS = 128          # GEMM slab: output rows [0, 128) of the gate+up GEMM, all 57344 columns
SAMPLE_REPACK_ROWS = 1024  # repack slab: the first 1024 rows of the gate+up weight
REFERENCE_COLS = 16384     # --impl reference: each step covers this many output columns of the slab


def oracle_sample(P, page, synth, host=None, ncols=None):
    """Times the oracle, as it stands, on a slab of the workload.  Returns the cpu_baseline object."""
    import oracle as orc
    g = GEMMS[0]
    M, N, K = g["M"], g["N"], g["K"]
    ncols = N if ncols is None else ncols
    if host is None:
        X = synth.randn_bf16(SAMPLE_ROWS, K, synth.ACT_STD, 0, "bench/X")
        W = synth.randn_bf16(K, N, synth.WEIGHT_STD, 0, "bench/Wgu")
    else:
        X, W = host["X"][:SAMPLE_ROWS], host["Wgu"]
    xb, wb = synth.bits(X), synth.bits(W)
    cores = os.cpu_count() or 1
    t0 = time.perf_counter()
    orc.repack(orc.Mat(SAMPLE_REPACK_ROWS, N, 2, P, orc.PART_COLS, orc.CCL, page), wb[:SAMPLE_REPACK_ROWS], 0)
    t1 = time.perf_counter()
    orc.gemm(xb, wb, SAMPLE_ROWS, N, K, 0, 0, block=(0, SAMPLE_ROWS, 0, ncols), threads=cores)
    t2 = time.perf_counter()
    td = orc.TrafficDesc()
    td.M, td.N, td.K, td.BM, td.BN = SAMPLE_ROWS, N, K, 128, 128
    td.A = orc.Mat(SAMPLE_ROWS, K, 2)
    td.B = orc.Mat(K, N, 2, P, orc.PART_COLS, orc.CCL, page)
    td.C = orc.Mat(SAMPLE_ROWS, N, 2, P, orc.PART_COLS, orc.CCL, page)
    td.a_trans, td.b_trans, td.P, td.page_bytes = 0, 0, P, page
    td.place[0], td.place[1], td.place[2] = orc.PLACE_RR, orc.PLACE_BLOCK, orc.PLACE_BLOCK
    td.assign, td.strip_tiling = orc.ASSIGN_N, 1
    orc.traffic(td, level="runs")
    t3 = time.perf_counter()
    flop = 2.0 * SAMPLE_ROWS * ncols * K
    total = t3 - t0
    return {"value": round(flop / total / 1e12, 6), "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"gate+up GEMM rows [0,{SAMPLE_ROWS}) x columns [0,{ncols}) of {N} (fp32 oracle, {cores} threads), repack of the first "
                      f"{SAMPLE_REPACK_ROWS} weight rows and the traffic count of one tile row (both single-threaded)",
            "seconds": {"repack": round(t1 - t0, 3), "gemm": round(t2 - t1, 3), "traffic": round(t3 - t2, 3)},
            "gemm_only_tflops": round(flop / (t2 - t1) / 1e12, 6)}


def run_reference(args):
    rank = int(os.environ.get("RANK", 0))
    if rank != 0:
        return
    from paper_2606_11718_b200 import synth
    from oracle import build as orc_build
    orc_build.build()
    X = synth.randn_bf16(SAMPLE_ROWS, H, synth.ACT_STD, 0, "bench/X")
    W = synth.randn_bf16(H, 2 * I, synth.WEIGHT_STD, 0, "bench/Wgu")
    host = {"X": X, "Wgu": W}
    for _ in range(args.warmup):
        oracle_sample(args.P, args.page, synth, host, REFERENCE_COLS)
    t0 = time.perf_counter()
    last = None
    for _ in range(args.steps):
        last = oracle_sample(args.P, args.page, synth, host, REFERENCE_COLS)
    ms_step = (time.perf_counter() - t0) * 1e3 / args.steps
    value = 2.0 * SAMPLE_ROWS * REFERENCE_COLS * H / (ms_step * 1e-3) / 1e12
    line = {"impl": "reference", "metric": METRIC, "value": round(value, 6), "unit": UNIT, "n_gpus": int(os.environ.get("WORLD_SIZE", 1)),
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(ms_step, 2), "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": "llama31_70b_ffn_fwd_8192tok (oracle on a bounded sample per step)", "P": args.P,
                       "page_bytes": args.page},
            "cpu_baseline": {"value": round(value, 6), "unit": UNIT, "cores": last["cores"], "kind": "oracle", "sample": last["sample"]},
            "e2e": {"value": round(value, 6), "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="ccl", choices=["ccl", "reference"])
    ap.add_argument("--P", type=int, default=4, help="chiplet count (the paper evaluates 4; B200 has 2 dies)")
    ap.add_argument("--page", type=int, default=4096, help="page / interleave bytes")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--tokens", type=int, default=8192, help="tokens per GPU (8192 = the benchmark workload)")
    args = ap.parse_args()
    set_tokens(args.tokens)
    if args.impl == "reference":
        args.steps = args.steps if args.steps is not None else 2
        args.warmup = args.warmup if args.warmup is not None else 1
        run_reference(args)
    else:
        args.steps = args.steps if args.steps is not None else 10
        args.warmup = max(3, args.warmup if args.warmup is not None else 3)
        run_cuda(args)


if __name__ == "__main__":
    main()
