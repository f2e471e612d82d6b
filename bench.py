#!/usr/bin/env python
"""HGEMM benchmark: prints ONE JSON line.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--no-grid]

A "step" is one pass of the hot path over the square HGEMM sweep (M = N = K in
{1024, 2048, 4096, 8192}: one plan/launch per shape, fp16 operands uniform in [-1, 1]
seeded per shape, fp32 accumulation, fp16 result).  `value` is the whole-job TFLOP/s
(flops of the sweep / device time, max over ranks) with inputs resident in HBM; `e2e` is the
same metric through the host-buffer entry point with the copies inside the timed region.
Extra keys: per-shape TFLOP/s beside torch.matmul on the same box, the 729-shape grid
geomean against torch.matmul (single GPU only), the roofline of the dominant kernel, the CPU
oracle timed on the machine's cores, and SM clocks sampled during the timed region.

Timing follows the paper's listing (section 2.4): synchronise, record an event, launch, record
an event, synchronise; no side streams.  With N > 1 every rank runs the same sweep on its own
GPU (replicas: the path has no exchange step) and the slowest rank sets the time.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import random
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

SWEEP = [1024, 2048, 4096, 8192]
GRID = [64, 128, 256, 512, 1024, 2048, 4096, 8192, 12288]
L2_BYTES = 126 * (1 << 20)
SPEC_TFLOPS = 2250.0
SPEC_HBM_GBS = 8000.0
# dram__bytes_read.sum + dram__bytes_write.sum of one 8192^3 launch of the dominant kernel,
# from the ncu capture summarised in profiles/hgemm_umma_kernel_pair_8192x8192x8192.md
DOMINANT_KERNEL_DRAM_BYTES = 1.197085e9 + 0.130235e9
METRIC = "HGEMM TFLOP/s"
WORKLOAD = "square HGEMM sweep M=N=K in {1024,2048,4096,8192}, one launch per shape per step"


def measured_peaks() -> dict:
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return {"source": "measured", "hbm_gbs": d["hbm_gbs"], "tflops_burst": d["bf16_tflops"],
                "tflops_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"])}
    return {"source": "fallback", "hbm_gbs": 6650.0, "tflops_burst": 1590.0, "tflops_sustained": 1400.0}


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.rows = []
        self.proc = None
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "50"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), [c.strip() for c in line.split(",")]))

    def stop(self, t0: float, t1: float) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        rows = [r for (t, r) in self.rows if t0 <= t <= t1 + 0.2 and len(r) >= 7] or [r for (_, r) in self.rows if len(r) >= 7]
        sm, mx, pw, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            try:
                sm.append(float(r[0]))
                mx.append(float(r[1]))
                pw.append(float(r[2]))
            except ValueError:
                continue
            for name, v in zip(names, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(pw) if pw else None, "samples": len(sm), "reasons": sorted(reasons)}


def flops(M, N, K):
    return 2.0 * M * N * K


def compulsory_bytes(M, N, K):
    return 2.0 * (M * K + N * K + M * N)


# --------------------------------------------------------------------------------------------------
# the reference arm: the CPU oracle, as it stands, on bounded row slabs of the same sweep

def oracle_slab(oracle, inputs, S: int, rows: int):
    a = inputs.draw(inputs.shape_seed(S, S, S), inputs.TAG_A, S, S, "uniform", "cpu", row_index=list(range(rows)))
    b = inputs.draw(inputs.shape_seed(S, S, S), inputs.TAG_B, S, S, "uniform", "cpu")
    return inputs.bits(a), inputs.bits(b)


def run_reference(args) -> None:
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    from paper_2512_02551_b200 import inputs
    oracle.build()
    # rows of C per shape per step, sized so that warm-up + steps end within about a minute
    per_row_macs = sum(S * S for S in SWEEP)
    rows = max(1, min(96, int(60.0 * 15e9 / ((args.steps + args.warmup) * per_row_macs))))
    slabs = [(S, *oracle_slab(oracle, inputs, S, rows)) for S in SWEEP]
    macs = sum(rows * S * S for S in SWEEP)
    for _ in range(max(args.warmup, 1) if args.warmup else 0):
        for S, a, b in slabs:
            oracle.hgemm_full(a, b)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        for S, a, b in slabs:
            oracle.hgemm_full(a, b)
    dt = time.perf_counter() - t0
    value = 2.0 * macs * args.steps / dt / 1e12
    sample = f"per step: first {rows} rows of C for each sweep shape ({macs / 1e9:.1f} GMAC)"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": WORKLOAD, "sample": sample},
        "cpu_baseline": {"value": value, "unit": "TFLOP/s", "cores": oracle.max_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# --------------------------------------------------------------------------------------------------
# our arm

def run_ours(args) -> None:
    import torch
    from paper_2512_02551_b200 import build as hbuild
    from paper_2512_02551_b200 import hgemm, inputs, replicas

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a GPU (there is no CPU fallback)")
    if rank == 0:
        hbuild.build()
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
        dist.barrier()

    def barrier():
        replicas.barrier(dist)
        torch.cuda.synchronize()

    ctx = hgemm.Context(local)
    stream = torch.cuda.current_stream()

    # ---- buffers: enough distinct (A, B, C) sets per shape that the footprint exceeds 2x L2 ----
    work = []
    for S in SWEEP:
        sets = max(1, math.ceil(2 * L2_BYTES / compulsory_bytes(S, S, S)))
        A0, B0 = inputs.make_ab(S, S, S, "uniform", "cuda")
        bufs = []
        for r in range(sets):
            A = A0 if r == 0 else A0.clone()
            B = B0 if r == 0 else B0.clone()
            bufs.append((A, B, torch.empty(S, S, dtype=torch.float16, device="cuda")))
        work.append({"S": S, "plan": ctx.plan(S, S, S), "bufs": bufs})
    step_flops = sum(flops(S, S, S) for S in SWEEP)

    def one_step(i, events=None):
        for w in work:
            A, B, C = w["bufs"][i % len(w["bufs"])]
            if events is not None:
                e0 = torch.cuda.Event(enable_timing=True)
                e1 = torch.cuda.Event(enable_timing=True)
                e0.record(stream)
                w["plan"].run_ptr(A.data_ptr(), B.data_ptr(), C.data_ptr(), stream.cuda_stream)
                e1.record(stream)
                events.append((w["S"], e0, e1))
            else:
                w["plan"].run_ptr(A.data_ptr(), B.data_ptr(), C.data_ptr(), stream.cuda_stream)

    def timed(fn, steps, warmup, sampler=None, label="hgemm_timed_region"):
        for i in range(warmup):
            fn(i)
        barrier()
        t0w = time.time()
        if sampler:
            sampler.start()
            time.sleep(0.25)
            t0w = time.time()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.nvtx.range_push(label)
        e0.record(stream)
        for i in range(steps):
            fn(warmup + i)
        e1.record(stream)
        barrier()
        torch.cuda.nvtx.range_pop()
        t1w = time.time()
        ms = replicas.slowest_rank_ms(e0.elapsed_time(e1), dist, "cuda")
        return ms, t0w, t1w

    # ---- the timed region ---------------------------------------------------------------------
    sampler = ClockSampler(local) if rank == 0 else None
    events = []
    ms_total, t0w, t1w = timed(lambda i: one_step(i, events), args.steps, args.warmup, sampler)
    clocks = sampler.stop(t0w, t1w) if sampler else None
    st, code = ctx.last_device_status()
    if st != hgemm.OK:
        raise SystemExit(f"device status {st} code {code:#x}")
    ms_per_step = ms_total / args.steps
    value = replicas.job_throughput(step_flops, world, ms_per_step) / 1e12
    per_launch = {}
    for S, e0, e1 in events[-4 * args.steps:]:
        per_launch.setdefault(S, []).append(e0.elapsed_time(e1))
    per_shape = {}
    for S, v in per_launch.items():
        ms = statistics.mean(v)
        per_shape[str(S)] = {"us": ms * 1e3, "tflops": flops(S, S, S) / (ms * 1e-3) / 1e12,
                             "config": work[SWEEP.index(S)]["plan"].config.as_dict()}

    line = None
    if rank == 0:
        peaks = measured_peaks()
        dom = per_shape[str(SWEEP[-1])]
        timed_s = ms_total * 1e-3
        peak = peaks["tflops_sustained"] if timed_s > 1.0 else peaks["tflops_burst"]
        roofline = {"bound": "tensor", "kernel": "hgemm_umma_kernel, 8192^3 launch", "achieved": dom["tflops"], "peak": peak,
                    "unit": "TFLOP/s", "frac": dom["tflops"] / peak,
                    "peak_source": f"{peaks['source']} cuBLAS bf16 {'sustained' if timed_s > 1.0 else 'burst'} (fp16 dense = bf16 dense)",
                    "traffic": DOMINANT_KERNEL_DRAM_BYTES, "algorithmic_flops_per_launch": flops(8192, 8192, 8192),
                    "compulsory_bytes_per_launch": compulsory_bytes(8192, 8192, 8192),
                    "frac_of_spec_peak": dom["tflops"] / SPEC_TFLOPS}

    # ---- torch.matmul on the same buffers, same protocol (comparison point, single rank) --------
    torch_cmp = None
    if rank == 0:
        def torch_step(i):
            for w in work:
                A, B, C = w["bufs"][i % len(w["bufs"])]
                torch.matmul(A, B.T, out=C)
        tev = []

        def torch_step_ev(i):
            for w in work:
                A, B, C = w["bufs"][i % len(w["bufs"])]
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
                torch.matmul(A, B.T, out=C)
                e1.record(stream)
                tev.append((w["S"], e0, e1))
        for i in range(args.warmup):
            torch_step(i)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for i in range(args.steps):
            torch_step_ev(args.warmup + i)
        e1.record(stream)
        torch.cuda.synchronize()
        tms = e0.elapsed_time(e1) / args.steps
        tps = {}
        for S, a, b in tev:
            tps.setdefault(S, []).append(a.elapsed_time(b))
        torch_cmp = {"value": step_flops / (tms * 1e-3) / 1e12, "unit": "TFLOP/s",
                     "per_shape_tflops": {str(S): flops(S, S, S) / (statistics.mean(v) * 1e-3) / 1e12 for S, v in tps.items()}}

    # ---- end to end: host buffers, copies inside the timed region --------------------------------
    host = []
    for w in work:
        S = w["S"]
        A, B, _ = w["bufs"][0]
        hA = torch.empty(S, S, dtype=torch.float16).pin_memory()
        hB = torch.empty(S, S, dtype=torch.float16).pin_memory()
        hC = torch.empty(S, S, dtype=torch.float16).pin_memory()
        hA.copy_(A)
        hB.copy_(B)
        host.append((w["plan"], hA, hB, hC))
    h2d = sum(hA.numel() * 2 + hB.numel() * 2 for _, hA, hB, _ in host)
    d2h = sum(hC.numel() * 2 for *_, hC in host)

    def e2e_step(i):
        for plan, hA, hB, hC in host:
            plan.run_host(hA, hB, hC, stream.cuda_stream)
    e2e_steps = max(3, min(args.steps, 10))
    e2e_ms, _, _ = timed(e2e_step, e2e_steps, 2, label="hgemm_e2e_region")
    e2e_value = replicas.job_throughput(step_flops, world, e2e_ms / e2e_steps) / 1e12
    # the result that came back is the GEMM's (spot check against the device-resident run)
    if rank == 0:
        _, _, _, hC = host[0]
        _, _, C = work[0]["bufs"][0]
        work[0]["plan"].run(work[0]["bufs"][0][0], work[0]["bufs"][0][1], C)
        torch.cuda.synchronize()
        assert torch.equal(hC, C.cpu()), "host-buffer path returned a different result"
    del host

    # ---- the 729-shape grid against torch.matmul (single GPU) ------------------------------------
    grid = None
    if rank == 0 and world == 1 and not args.no_grid:
        grid = grid_sweep(ctx, torch, hgemm, inputs, stream)

    skinny = None
    if rank == 0 and world == 1 and not args.no_grid:
        skinny = skinny_report(ctx, torch, hgemm, inputs, stream)

    # ---- the CPU oracle on the machine's cores, on a bounded sample -------------------------------------
    cpu = None
    if rank == 0 and world == 1:
        import oracle
        oracle.build()
        rows = 384
        a, b = oracle_slab(oracle, inputs, 8192, rows)
        t0 = time.perf_counter()
        oracle.hgemm_full(a, b)
        dt = time.perf_counter() - t0
        cpu = {"value": 2.0 * rows * 8192 * 8192 / dt / 1e12, "unit": "TFLOP/s", "cores": oracle.max_threads(), "kind": "oracle",
               "sample": f"first {rows} rows of C for 8192^3 ({rows * 8192 * 8192 / 1e9:.1f} GMAC, {dt:.2f} s wall)"}

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f16",
            "data": "synthetic",
            "config": {"workload": WORKLOAD, "accumulate": "f32", "inputs": "uniform[-1,1) rounded to fp16, seeded per shape",
                       "l2": "inputs larger than L2: buffer sets rotate so that each shape's footprint exceeds 2x the 126 MB L2",
                       "parallelism": "replicas" if world > 1 else "single GPU"},
            "per_shape": per_shape, "pct_of_spec_peak": 100.0 * value / world / SPEC_TFLOPS,
            "roofline": roofline, "torch_matmul": torch_cmp, "grid": grid, "skinny": skinny, "cpu_baseline": cpu, "clocks": clocks,
            "e2e": {"value": e2e_value, "unit": "TFLOP/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": e2e_steps},
            "gpu_launches": args.steps * len(SWEEP),
        }
        print(json.dumps(line), flush=True)
    ctx.close()
    if dist is not None:
        dist.destroy_process_group()


def grid_sweep(ctx, torch, hgemm, inputs, stream) -> dict:
    """All 729 grid shapes, ours against torch.matmul on the same buffers: warm (back-to-back) calls,
    batches of n calls between two events, ours/torch batches interleaved in seeded random order,
    median over rounds.  Buffers are dense M x K / N x K / M x N prefixes of three maximal arrays."""
    mx = GRID[-1]
    A_all = inputs.draw(1, inputs.TAG_A, mx, mx, "uniform", "cuda")
    B_all = inputs.draw(1, inputs.TAG_B, mx, mx, "uniform", "cuda")
    C_all = torch.empty(mx * mx, dtype=torch.float16, device="cuda")
    rng = random.Random(729)
    ratios, rows = [], []
    server_ratios = []
    roof_frac = []
    peaks = measured_peaks()

    def batch_ms(fn, n):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(n):
            fn()
        e1.record(stream)
        e1.synchronize()
        return e0.elapsed_time(e1) / n

    for M in GRID:
        for N in GRID:
            for K in GRID:
                A = A_all.view(-1)[:M * K].view(M, K)
                B = B_all.view(-1)[:N * K].view(N, K)
                C = C_all[:M * N].view(M, N)
                plan = ctx.plan(M, N, K)
                a, b, c, s = A.data_ptr(), B.data_ptr(), C.data_ptr(), stream.cuda_stream
                ours = lambda: plan.run_ptr(a, b, c, s)          # noqa: E731
                Bt = B.T
                ref = lambda: torch.matmul(A, Bt, out=C)         # noqa: E731
                for fn in (ours, ref):
                    for _ in range(3):
                        fn()
                est = max(batch_ms(ours, 3), 1e-3)
                n = max(3, min(200, int(1.0 / est)))
                t = {"ours": [], "torch": []}
                for _ in range(3):
                    order = [("ours", ours), ("torch", ref)]
                    rng.shuffle(order)
                    for name, fn in order:
                        t[name].append(batch_ms(fn, n))
                to, tt = statistics.median(t["ours"]), statistics.median(t["torch"])
                ratios.append(tt / to)
                # server mode (paper section 2.4): single calls separated by random idle gaps that are not
                # timed; each call is bracketed by its own pair of events
                ts = {"ours": [], "torch": []}
                for _ in range(5):
                    order = [("ours", ours), ("torch", ref)]
                    rng.shuffle(order)
                    for name, fn in order:
                        gap = time.perf_counter() + rng.uniform(20e-6, 200e-6)
                        while time.perf_counter() < gap:
                            pass
                        ts[name].append(batch_ms(fn, 1))
                server_ratios.append(statistics.median(ts["torch"]) / statistics.median(ts["ours"]))
                t_roof = max(flops(M, N, K) / (peaks["tflops_burst"] * 1e12), compulsory_bytes(M, N, K) / (peaks["hbm_gbs"] * 1e9))
                roof_frac.append(t_roof / (to * 1e-3))
                rows.append((M, N, K, to * 1e3, tt * 1e3))
                plan.close()
    geo = math.exp(sum(math.log(r) for r in ratios) / len(ratios))
    worst = sorted(zip(ratios, rows))[:5]
    big = [(r, row) for r, row in zip(ratios, rows) if min(row[:3]) >= 4096]
    out_path = os.path.join(ROOT, "gpurun_out", "grid_times.csv")
    try:
        os.makedirs(os.path.dirname(out_path), exist_ok=True)
        with open(out_path, "w") as f:
            f.write("M,N,K,ours_us,torch_us,ratio\n")
            for r, (M, N, K, to, tt) in zip(ratios, rows):
                f.write(f"{M},{N},{K},{to:.3f},{tt:.3f},{r:.4f}\n")
    except OSError:
        pass
    return {
        "shapes": len(ratios), "regime": "warm, back-to-back calls (the paper's offline mode)",
        "geomean_torch_time_over_ours": geo, "wins": sum(r > 1.0 for r in ratios),
        "mean_speedup_minus_1": sum(r - 1.0 for r in ratios) / len(ratios),
        "geomean_fraction_of_measured_roofline": math.exp(sum(math.log(x) for x in roof_frac) / len(roof_frac)),
        "compute_bound_min_tflops": min(flops(*row[:3]) / (row[3] * 1e-6) / 1e12 for _, row in big),
        "compute_bound_geomean_vs_torch": math.exp(sum(math.log(r) for r, _ in big) / len(big)),
        "worst5": [{"shape": list(row[:3]), "ratio": r, "ours_us": row[3], "torch_us": row[4]} for r, row in worst],
        "server_mode": {"regime": "single calls after random idle gaps of 20-200 us, gap not timed, median of 5",
                        "geomean_torch_time_over_ours": math.exp(sum(math.log(r) for r in server_ratios) / len(server_ratios)),
                        "mean_speedup_minus_1": sum(r - 1.0 for r in server_ratios) / len(server_ratios),
                        "win_rate": sum(r > 1.0 for r in server_ratios) / len(server_ratios)},
        "offline_win_rate": sum(r > 1.0 for r in ratios) / len(ratios),
    }


def skinny_report(ctx, torch, hgemm, inputs, stream) -> dict:
    """The memory-bound LLM-projection shapes, M in {64, 128, 256} tokens x (N, K) in {(4096, 4096), (12288, 4096),
    (4096, 12288)}, entries N(0, 1) * K^-1/2: achieved GB/s of compulsory traffic against the HBM roofline, with B
    (the weight matrix) rotated through enough copies that it never comes from L2, torch.matmul beside it."""
    peaks = measured_peaks()
    base = inputs.draw(3, inputs.TAG_B, 4096, 4096, "normal", "cpu").cuda()          # N(0,1) / sqrt(4096)
    out = []

    def batch_ms(fn, n):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for i in range(n):
            fn(i)
        e1.record(stream)
        e1.synchronize()
        return e0.elapsed_time(e1) / n

    for (N, K) in ((4096, 4096), (12288, 4096), (4096, 12288)):
        scale = (4096.0 / K) ** 0.5
        tile = (base.float() * scale).half()
        B0 = tile.repeat(N // 4096, K // 4096).contiguous()
        copies = max(2, math.ceil(2 * L2_BYTES / (2.0 * N * K)) + 1)
        Bs = [B0] + [B0.clone() for _ in range(copies - 1)]
        for M in (64, 128, 256):
            A = (base[:M].float() * scale).half().repeat(1, K // 4096).contiguous()
            C = torch.empty(M, N, dtype=torch.float16, device="cuda")
            plan = ctx.plan(M, N, K)
            a, c, s = A.data_ptr(), C.data_ptr(), stream.cuda_stream
            ours = lambda i: plan.run_ptr(a, Bs[i % copies].data_ptr(), c, s)       # noqa: E731
            ref = lambda i: torch.matmul(A, Bs[i % copies].T, out=C)                # noqa: E731
            for fn in (ours, ref):
                batch_ms(fn, copies)
            n = 8 * copies
            to = statistics.median(batch_ms(ours, n) for _ in range(3))
            tt = statistics.median(batch_ms(ref, n) for _ in range(3))
            by = compulsory_bytes(M, N, K)
            out.append({"shape": [M, N, K], "us": to * 1e3, "gbs": by / (to * 1e-3) / 1e9,
                        "frac_of_measured_hbm": by / (to * 1e-3) / 1e9 / peaks["hbm_gbs"],
                        "frac_of_spec_hbm": by / (to * 1e-3) / 1e9 / SPEC_HBM_GBS, "torch_us": tt * 1e3,
                        "torch_time_over_ours": tt / to, "config": plan.config.as_dict()})
            plan.close()
        del Bs, B0
    return {"regime": "B rotates through copies totalling more than 2x L2 (cold weights), A and C stay hot",
            "inputs": "N(0,1) * K^-1/2 rounded to fp16", "shapes": out,
            "geomean_frac_of_measured_hbm": math.exp(sum(math.log(r["frac_of_measured_hbm"]) for r in out) / len(out)),
            "geomean_torch_time_over_ours": math.exp(sum(math.log(r["torch_time_over_ours"]) for r in out) / len(out))}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--no-grid", action="store_true", help="skip the 729-shape comparison against torch.matmul")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
