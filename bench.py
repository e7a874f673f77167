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


def gemm_dram_traffic(tokens, P, page):
    """DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) of the two GEMM launches of one step, as measured by
    ncu: read from profiles/ccl_gemm_kernel_dram_traffic.json, which names the captured case, the capture command and the
    rule that scales a reduced capture to the full launch.  None when the file does not cover this configuration."""
    path = os.path.join(ROOT, "profiles", "ccl_gemm_kernel_dram_traffic.json")
    try:
        rec = json.load(open(path))
    except (OSError, ValueError):
        return None
    for row in rec.get("configs", []):
        if (row.get("tokens"), row.get("P"), row.get("page_bytes")) == (tokens, P, page):
            return row.get("bytes_per_step")
    return None


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
        return dict(hbm_gbs=p["hbm_gbs"], tf_burst=p["bf16_tflops"], tf_sustained=p["bf16_tflops_sustained"], source="measured",
                    sustained_sm_mhz=(p.get("clocks_under_load") or {}).get("sm_mhz_median"))
    return dict(hbm_gbs=6650.0, tf_burst=1590.0, tf_sustained=1400.0, source="fallback", sustained_sm_mhz=1300.0)


def tensor_peak(peaks, timed_seconds, sm_mhz):
    """Which measured bf16 peak a GEMM timed here is held against.  The sustained figure was taken in a seconds-long loop
    at the power cap (clock well below maximum); a timed region shorter than ~2 s, or one whose sampled SM clock is above the
    clock of that loop, ran in the burst regime and is held against the burst figure."""
    burst = timed_seconds < 2.0 or (sm_mhz is not None and peaks.get("sustained_sm_mhz") and sm_mhz > 1.05 * peaks["sustained_sm_mhz"])
    return (peaks["tf_burst"], "burst") if burst else (peaks["tf_sustained"], "sustained")


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
    peak_tf, peak_kind = tensor_peak(peaks, ms_total / 1e3, clocks.get("sm_mhz"))
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
        "roofline": {"kernel": "ccl_gemm_kernel", "bound": "tensor", "achieved": round(gemm_tf, 1), "peak": peak_tf,
                     "unit": "TFLOP/s", "frac": round(gemm_tf / peak_tf, 4), "traffic": gemm_dram_traffic(T, P, page),
                     "traffic_unit": "bytes per step (2 launches), ncu", "algorithmic_bytes_per_step": sum(2 * (g["M"] * g["K"] + g["K"] * g["N"] + g["M"] * g["N"]) for g in GEMMS),
                     "peak_source": f"bf16 {peak_kind}, {peaks['source']} (timed region {ms_total / 1e3:.2f} s at {clocks.get('sm_mhz')} MHz)",
                     "frac_of_burst": round(gemm_tf / peaks["tf_burst"], 4), "frac_of_sustained": round(gemm_tf / peaks["tf_sustained"], 4),
                     "frac_of_nominal_2250": round(gemm_tf / 2250.0, 4), "ms_per_step": round(kms["gemm"], 4)},
        "kernels": {"gemm_tflops": round(gemm_tf, 1), "repack_gbs": round(repack_gbs, 1),
                    "repack_frac_of_hbm": round(repack_gbs / peaks["hbm_gbs"], 4), "repack_frac_of_nominal_8TBs": round(repack_gbs / 8000.0, 4),
                    "repack_ms": round(kms["repack"], 4),
                    "traffic_ms": round(kms["traffic"], 4),
                    "remote_traffic_ratio_ccl_vs_rr4k": round(ratio, 4), "remote_bytes": remote},
    }
    if world == 1 and not args.no_by_config:
        line["kernels"]["by_config"] = by_config(ccl, torch, descs, devb, peaks, P, page, uuid)
    if rank == 0:
        if world == 1 and not args.no_cpu_baseline:
            # the step's own gate+up output, brought back to row-major by the library's repack, for the parity check
            # that the oracle leg makes on its slab
            d0 = descs[0]
            ccl.ccl_repack(d0["mB"], devb[d0["w"]], d0["w_ccl"], 0)
            ccl.ccl_gemm(d0["gd"], devb[d0["a"]], d0["w_ccl"], d0["c_ccl"])
            c_row = torch.empty(T * d0["g"]["N"], dtype=torch.bfloat16, device="cuda")
            ccl.ccl_repack(d0["mC"], d0["c_ccl"], c_row, 1)
            c_slab = c_row.view(T, d0["g"]["N"])[:SAMPLE_ROWS].float().cpu().numpy()
            line["cpu_baseline"], line["parity"] = oracle_sample(P, page, synth, host, c_slab=c_slab)
        print(json.dumps(line), flush=True)
    group.close()


# ---------------------------------------------------------------------------------------------
# the other configurations, kernel by kernel (outside the timed step and outside `value`)
# ---------------------------------------------------------------------------------------------
def by_config(ccl, torch, descs, devb, peaks, P, page, uuid):
    """GEMM TFLOP/s and repack GB/s of the configurations the step does not cover: the single Qwen expert GEMM, the six
    Qwen FFN GEMMs (forward, data and weight gradients), the Llama backward GEMMs and the weight-streaming rows
    (M = 1, 16, 128) of the token sweep on both Llama weights.  B and C in CCL (P strips aligned to the page size),
    grouped raster.  Each figure: CUDA events around back-to-back launches on one stream (100 for kernels under a
    millisecond, queued behind a device-side spin so that the host's issue rate does not show; 10 above), operands
    rotated through enough copies to exceed the L2 where one set would fit in it.
    roofline_frac = time at min(tensor, HBM) roofline / measured time, against the measured burst peaks."""
    from paper_2606_11718_b200 import synth
    L2_BYTES = 126e6
    sampler = ClockSampler(uuid)
    sampler.start()
    ev = lambda: torch.cuda.Event(enable_timing=True)

    def rand(rows, cols, std):
        return (torch.randn(rows, cols, device="cuda", dtype=torch.float32) * std).to(torch.bfloat16)

    def time_gemm(M, N, K, at, bt, a_src=None, b_src=None, P_=P):
        lay_b = ccl.Mat(N, K, 2, P_, ccl.PART_ROWS, ccl.CCL, page) if bt else ccl.Mat(K, N, 2, P_, ccl.PART_COLS, ccl.CCL, page)
        lay_c = ccl.Mat(M, N, 2, P_, ccl.PART_COLS, ccl.CCL, page)
        gd = ccl.GemmDesc()
        gd.M, gd.N, gd.K = M, N, K
        gd.A, gd.B, gd.C = ccl.Mat(K, M, 2) if at else ccl.Mat(M, K, 2), lay_b, lay_c
        gd.a_trans, gd.b_trans, gd.out_part, gd.P, gd.grouped_raster = at, bt, ccl.PART_COLS, P_, 1
        one_set = 2 * (M * K + K * N + M * N)
        copies = 1 if one_set > 2 * L2_BYTES else int(min(16, 2 * L2_BYTES // one_set + 2))
        sets = []
        for i in range(copies):
            a = a_src if a_src is not None else rand(K if at else M, M if at else K, synth.ACT_STD)
            if b_src is not None:
                b = b_src
            else:
                b_row = rand(N if bt else K, K if bt else N, synth.WEIGHT_STD)
                b = torch.empty(ccl.ccl_buffer_bytes(lay_b) // 2, dtype=torch.bfloat16, device="cuda")
                ccl.ccl_repack(lay_b, b_row, b, 0)
            c = torch.empty(ccl.ccl_buffer_bytes(lay_c) // 2, dtype=torch.bfloat16, device="cuda")
            sets.append((a, b, c))
        need = ccl.ccl_gemm_workspace(gd)
        ws = torch.empty(max(need, 16) // 4, dtype=torch.float32, device="cuda")
        flop = 2.0 * M * N * K
        n = 100 if flop / 1.4e15 < 1e-3 else 10
        for i in range(3):
            ccl.ccl_gemm(gd, *sets[i % copies], ws)
        e0, e1 = ev(), ev()
        torch.cuda.synchronize()
        if n == 100:
            torch.cuda._sleep(6_000_000)           # ~3 ms of device-side spin: the launches queue up behind it, so a kernel of
        e0.record()                                # a few microseconds is timed on the device, not at the host's issue rate
        for i in range(n):
            ccl.ccl_gemm(gd, *sets[i % copies], ws)
        e1.record()
        torch.cuda.synchronize()
        us = e0.elapsed_time(e1) * 1e3 / n
        roof_us = max(flop / (peaks["tf_burst"] * 1e12), one_set / (peaks["hbm_gbs"] * 1e9)) * 1e6
        return {"M": M, "N": N, "K": K, "us": round(us, 2), "tflops": round(flop / us / 1e6, 1), "roofline_frac": round(roof_us / us, 4),
                "bound": "tensor" if flop / (peaks["tf_burst"] * 1e12) > one_set / (peaks["hbm_gbs"] * 1e9) else "hbm",
                "launches": n, "operand_sets": copies}

    def time_repack(rows, cols):
        m = ccl.Mat(rows, cols, 2, P, ccl.PART_COLS, ccl.CCL, page)
        nbytes = rows * cols * 2
        copies = 1 if nbytes > L2_BYTES else int(2 * L2_BYTES // nbytes + 2)
        srcs = [rand(rows, cols, synth.WEIGHT_STD) for _ in range(copies)]
        dsts = [torch.empty(ccl.ccl_buffer_bytes(m) // 2, dtype=torch.bfloat16, device="cuda") for _ in range(copies)]
        n = 100 if nbytes < 1e8 else 20
        for i in range(3):
            ccl.ccl_repack(m, srcs[i % copies], dsts[i % copies], 0)
        e0, e1 = ev(), ev()
        torch.cuda.synchronize()
        if n == 100:
            torch.cuda._sleep(6_000_000)
        e0.record()
        for i in range(n):
            ccl.ccl_repack(m, srcs[i % copies], dsts[i % copies], 0)
        e1.record()
        torch.cuda.synchronize()
        us = e0.elapsed_time(e1) * 1e3 / n
        gbs = 2 * nbytes / us / 1e3
        return {"rows": rows, "cols": cols, "us": round(us, 2), "gbs": round(gbs, 1), "frac_of_hbm": round(gbs / peaks["hbm_gbs"], 4),
                "launches": n, "operand_sets": copies}

    out = {"layout": f"B and C in CCL, P={P}, strips aligned to {page} B, grouped raster", "peaks": "measured burst bf16 / measured HBM copy"}
    g = synth.config1_gemm()
    out["config1"] = {g["name"]: time_gemm(g["M"], g["N"], g["K"], g["a_trans"], g["b_trans"])}
    out["config2"] = {g["name"]: time_gemm(g["M"], g["N"], g["K"], g["a_trans"], g["b_trans"]) for g in synth.qwen_ffn_gemms()}
    out["config2_P2"] = {g["name"]: time_gemm(g["M"], g["N"], g["K"], g["a_trans"], g["b_trans"], P_=2) for g in synth.qwen_ffn_gemms()}
    X, Z = devb["X"], devb["Z"]
    wd_ccl = descs[1]["w_ccl"]
    out["config4"] = {"llama_dgrad": time_gemm(T, H, I, 0, 0, a_src=Z, b_src=wd_ccl)}
    x_ccl = torch.empty(ccl.ccl_buffer_bytes(ccl.Mat(T, H, 2, P, ccl.PART_COLS, ccl.CCL, page)) // 2, dtype=torch.bfloat16, device="cuda")
    ccl.ccl_repack(ccl.Mat(T, H, 2, P, ccl.PART_COLS, ccl.CCL, page), X, x_ccl, 0)
    out["config4"]["llama_wgrad"] = time_gemm(I, H, T, 1, 0, a_src=Z, b_src=x_ccl)
    del x_ccl
    out["config5"] = {}
    for d, nm in zip(descs, ("gateup", "down")):
        for M in (1, 16, 128):
            a = rand(M, d["g"]["K"], synth.ACT_STD)
            out["config5"][f"llama_{nm}_M{M}"] = time_gemm(M, d["g"]["N"], d["g"]["K"], 0, 0, a_src=a, b_src=d["w_ccl"])
    out["repack"] = {"qwen_gateup_weight": time_repack(2048, 1536), "qwen_down_weight": time_repack(768, 2048),
                     "llama_down_weight": time_repack(I, H), "llama_x": time_repack(T, H)}
    st, detail = ccl.ccl_gemm_status()
    if st != ccl.OK:
        raise SystemExit(f"bench.py: device-side wait expired in the per-configuration runs (code {detail})")
    out["clocks"] = sampler.stop()
    return out


# ---------------------------------------------------------------------------------------------
# the oracle on a bounded sample (cpu_baseline and --impl reference)
# ---------------------------------------------------------------------------------------------
SAMPLE_ROWS = 128          # GEMM slab: output rows [0, 128) of the gate+up GEMM, all 57344 columns
SAMPLE_REPACK_ROWS = 1024  # repack slab: the first 1024 rows of the gate+up weight
REFERENCE_COLS = 16384     # --impl reference: each step covers this many output columns of the slab


def oracle_sample(P, page, synth, host=None, ncols=None, c_slab=None):
    """Times the oracle, as it stands, on a slab of the workload.  Returns the cpu_baseline object; with c_slab (rows
    [0, SAMPLE_ROWS) of the gate+up output the CUDA path computed, fp32) also the parity of that slab against the
    oracle's fp32 sums, in the tolerance the tests use."""
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
    ref32, _, _ = orc.gemm(xb, wb, SAMPLE_ROWS, N, K, 0, 0, block=(0, SAMPLE_ROWS, 0, ncols), threads=cores)
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
    parity = None
    if c_slab is not None:
        import math
        import numpy as np
        err = np.abs(c_slab[:, :ncols] - ref32) / np.maximum(1.0, np.abs(ref32))
        tol = 1e-2 * math.sqrt(K / 1024.0)
        parity = {"max_err": float(err.max()), "tol": tol, "ok": bool(np.isfinite(c_slab).all() and err.max() <= tol),
                  "blocks": f"gate+up output rows [0,{SAMPLE_ROWS}) x all {ncols} columns ({SAMPLE_ROWS * ncols} elements, every strip), "
                            "err = |C - ref32| / max(1, |ref32|) against the fp32 oracle"}
    base = {"value": round(flop / total / 1e12, 6), "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"gate+up GEMM rows [0,{SAMPLE_ROWS}) x columns [0,{ncols}) of {N} (fp32 oracle, {cores} threads), repack of the first "
                      f"{SAMPLE_REPACK_ROWS} weight rows and the traffic count of one tile row (both single-threaded)",
            "seconds": {"repack": round(t1 - t0, 3), "gemm": round(t2 - t1, 3), "traffic": round(t3 - t2, 3)},
            "gemm_only_tflops": round(flop / (t2 - t1) / 1e12, 6)}
    return (base, parity) if c_slab is not None else base


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
    ap.add_argument("--no-by-config", action="store_true", help="skip the per-configuration kernel timings")
    args = ap.parse_args()
    set_tokens(args.tokens)
    from paper_2606_11718_b200 import dist as ccl_dist
    if args.impl == "ccl" and args.gpus > 1 and not ccl_dist.launched_by_a_launcher():
        # no launcher set the environment: start the ranks here, one per GPU; rank 0 prints the line
        env = {}
        if "NCCL_DEBUG" not in os.environ:       # the communicator's own log (rank count, transports), kept off stdout
            env = {"NCCL_DEBUG": "INFO", "NCCL_DEBUG_SUBSYS": "INIT", "NCCL_DEBUG_FILE": "/dev/stderr"}
        sys.exit(ccl_dist.spawn_ranks(args.gpus, [sys.executable, os.path.abspath(__file__)] + sys.argv[1:], extra_env=env))
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
