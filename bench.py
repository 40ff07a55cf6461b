#!/usr/bin/env python
"""Benchmark of the HARP apply hot path on B200.

One step = one pass of the apply path over one synthetic batch of the headline
workload (d = 4096 = 4^6, radix-4 schedule, sign diagonal, base-4 digit-reversal
permutation, 16384 bf16 rows): a forward apply (y = x Q) of the batch followed by a
transpose apply (x = y Q^T) of a batch.  `value` counts row-applies per second
(2 * n_rows per step), whole job.  Four device buffers (134 MB each) are rotated so a
buffer is touched again only after three others (> 3x the 126 MB L2) have streamed by.

Prints ONE JSON line (rank 0).  `--impl reference` times the CPU oracle instead.
The line carries a compact "per_config" object (forward / transpose rate of all five
configurations, decode latency, two-sided time; a few repetitions each, full row counts);
`--all-configs` adds the longer per-configuration measurements (gradient, CUDA-graph decode,
diagnostics) under "per_config_detail".  `--gpus N` without a launcher starts N ranks itself.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2605_29843_b200 import workloads as wl  # noqa: E402

METRIC = "harp_apply_rows_per_s"
UNIT = "rows/s"
WORKLOAD = "cfg2: d=4096 radix-4 x6, signs + digit-reversal perm, 16384 rows bf16, forward+transpose per step"
N_BUF = 4
# DRAM bytes per apply (dram__bytes_read.sum + dram__bytes_write.sum, summed over the launches of one
# apply, mean of forward and transpose) from one ncu capture per configuration of
# `bench.py --profile-config C --profile-rows R --profile-reps 2`: {config: (R, bytes)}.  Traffic grows in
# proportion to the rows, so a full launch is scaled by n_rows / R.  Write-back that is still in L2
# when a kernel ends is not in these figures (cfg1 and cfg2 read below their algorithmic bytes for
# that reason).
NCU_TRAFFIC = {1: (4096, 33.8e6), 2: (16384, 209.8e6), 3: (4096, 259.1e6), 4: (4096, 364.2e6), 5: (4096, 833.3e6)}


def ncu_traffic(cfg: int, n_rows: int):
    rows, nbytes = NCU_TRAFFIC[cfg]
    return nbytes * n_rows / rows


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        j = json.load(open(p))
        return float(j["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons in the background."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int, period_ms: int = 50):
        self.samples = []
        self.proc = None
        self.t0 = self.t1 = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-i", str(index), "-lms", str(period_ms)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL,
                text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.samples.append((time.time(), line.strip()))

    def mark_start(self):
        self.t0 = time.time()

    def mark_end(self):
        self.t1 = time.time()

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        time.sleep(0.06)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()
        inside = [s for t, s in self.samples if self.t0 is not None and self.t0 - 0.05 <= t <= self.t1 + 0.1]
        use = inside if inside else [s for _, s in self.samples]
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for s in use:
            f = [v.strip() for v in s.split(",")]
            try:
                sm.append(float(f[0]))
                smax.append(float(f[1]))
            except Exception:
                continue
            for name, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "reasons": sorted(reasons), "samples": len(use)}


# ------------------------------------------------------------------ reference arm

def oracle_step(cplan, x64, c_oracle):
    c_oracle.forward(cplan, x64)
    c_oracle.transpose(cplan, x64)


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import c_oracle
    w = wl.config(2)
    spec, data = w.plans["q"], w.data["x"]
    cplan = c_oracle.CPlan(spec)
    sample_rows = args.ref_rows
    x64 = data.rows_f64(0, sample_rows)
    for _ in range(max(1, min(args.warmup, 2))):
        oracle_step(cplan, x64, c_oracle)
    steps = max(1, min(args.steps, 20))
    t0 = time.perf_counter()
    for _ in range(steps):
        oracle_step(cplan, x64, c_oracle)
    dt = time.perf_counter() - t0
    val = 2 * sample_rows * steps / dt
    sample = f"{sample_rows} of {data.n_rows} rows per step, forward+transpose, {steps} steps"
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
            "steps": steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": WORKLOAD, "sample": sample},
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": c_oracle.threads(), "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ------------------------------------------------------------------ GPU arm

def cpu_baseline(spec, data):
    from oracle import c_oracle
    cplan = c_oracle.CPlan(spec)
    probe = 256
    x64 = data.rows_f64(0, probe)
    t0 = time.perf_counter()
    oracle_step(cplan, x64, c_oracle)
    dt = time.perf_counter() - t0
    rows = int(min(data.n_rows, max(probe, probe * 12.0 / max(dt, 1e-6))))
    rows = (rows // 256) * 256 or 256
    x64 = data.rows_f64(0, rows)
    t0 = time.perf_counter()
    oracle_step(cplan, x64, c_oracle)
    one = time.perf_counter() - t0
    reps = int(max(1, min(20, round(10.0 / max(one, 1e-3)))))
    t0 = time.perf_counter()
    for _ in range(reps):
        oracle_step(cplan, x64, c_oracle)
    dt = time.perf_counter() - t0
    return {"value": 2 * rows * reps / dt, "unit": UNIT, "cores": c_oracle.threads(), "kind": "oracle",
            "sample": f"first {rows} of {data.n_rows} rows, forward+transpose, {reps} passes, {dt:.1f} s"}


def time_region(torch, fn, iters):
    start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    start.record()
    for i in range(iters):
        fn(i)
    end.record()
    end.synchronize()
    return start.elapsed_time(end) * 1e-3


def bench_extra_configs(torch, harp, kernel, peak):
    """Per-configuration apply throughput (forward and transpose), decode latency and
    two-sided time.  Inputs are seeded device-side normals of the configuration's shape
    (throughput does not depend on the values; parity is covered by the tests)."""
    out = {}
    gen = torch.Generator(device="cuda")
    gen.manual_seed(1234)
    for cfg in (1, 2, 3, 4, 5):
        w = wl.config(cfg)
        spec = w.plans["in"] if cfg == 5 else w.plans["q"]
        data = w.data["x"]
        plan = harp.plan_from_spec(spec)
        tdt = torch.float32 if data.dtype == "f32" else torch.bfloat16
        es = 4 if data.dtype == "f32" else 2
        nbytes = data.n_rows * data.d * es
        nbuf = max(2, int(np.ceil(3 * 126e6 / nbytes)) + 1)
        bufs = [torch.randn((data.n_rows, data.d), generator=gen, device="cuda", dtype=torch.float32).to(tdt)
                for _ in range(nbuf)]
        res = {}
        for name, tr in (("forward", False), ("transpose", True)):
            for i in range(3):
                harp.apply_(plan, bufs[i % nbuf], transpose=tr, kernel=kernel)
            torch.cuda.synchronize()
            iters = max(5, min(200, int(0.3 / (2 * nbytes / (peak * 1e9) * 3))))
            dt = time_region(torch, lambda i: harp.apply_(plan, bufs[i % nbuf], transpose=tr, kernel=kernel), iters)
            gbs = 2 * nbytes * iters / dt / 1e9
            res[name] = {"rows_per_s": data.n_rows * iters / dt, "GBps": gbs, "frac_of_measured_peak": gbs / peak,
                         "frac_of_8TBps": gbs / 8000.0, "us_per_launch": 1e6 * dt / iters}
        if cfg == 2:
            # gradient of a loss with respect to the block kernels (chain rule through Algorithm 1)
            grad = torch.zeros(harp.harp_plan_n_params(plan), dtype=torch.float32, device="cuda")
            stream = torch.cuda.current_stream().cuda_stream
            gb = lambda i: harp.harp_grad_blocks(plan, bufs[0].data_ptr(), bufs[1].data_ptr(), data.n_rows, harp.HARP_BF16,
                                                 grad.data_ptr(), False, stream)
            for i in range(2):
                gb(i)
            dt = time_region(torch, gb, 5)
            res["grad_blocks"] = {"ms": 1e3 * dt / 5, "rows_per_s": data.n_rows * 5 / dt}
        if cfg == 4:
            dec = {}
            for n in w.extra["decode_rows"]:
                x = bufs[0][:n]
                for _ in range(5):
                    harp.apply_(plan, x, kernel=kernel)
                torch.cuda.synchronize()
                dt = time_region(torch, lambda i: harp.apply_(plan, x, kernel=kernel), 200)
                dec[str(n)] = {"us_per_call": 1e6 * dt / 200}
                # the same 100 calls replayed from one CUDA graph (no per-call launch cost on the host)
                side = torch.cuda.Stream()
                side.wait_stream(torch.cuda.current_stream())
                with torch.cuda.stream(side):
                    graph = torch.cuda.CUDAGraph()
                    with torch.cuda.graph(graph, stream=side):
                        for _ in range(100):
                            harp.apply_(plan, x, kernel=kernel)
                torch.cuda.current_stream().wait_stream(side)
                graph.replay()
                torch.cuda.synchronize()
                dtg = time_region(torch, lambda i: graph.replay(), 5)
                dec[str(n)]["us_per_call_cuda_graph"] = 1e6 * dtg / 500
            res["decode"] = dec
        if cfg == 5:
            del bufs
            wd = w.data["w"]
            p_out = harp.plan_from_spec(w.plans["out"])
            W = (torch.randn((wd.n_rows, wd.d), generator=gen, device="cuda") * 0.02).to(torch.bfloat16)
            scratch = torch.empty(harp.harp_two_sided_scratch_bytes(p_out, plan, harp.HARP_BF16), dtype=torch.uint8,
                                  device="cuda")
            for _ in range(2):
                harp.two_sided_(W, p_out, plan, scratch)
            torch.cuda.synchronize()
            dt = time_region(torch, lambda i: harp.two_sided_(W, p_out, plan, scratch), 10)
            wbytes = 2 * wd.n_rows * wd.d * 2
            res["two_sided"] = {"ms": 1e3 * dt / 10, "GBps_vs_1R1W": wbytes * 10 / dt / 1e9,
                                "frac_of_measured_peak_vs_1R1W": wbytes * 10 / dt / 1e9 / peak}
            # diagnostics of the processed weight (Eq. 4): one read of W per call
            acc = torch.zeros(4, dtype=torch.float64, device="cuda")
            stream = torch.cuda.current_stream().cuda_stream
            mu = lambda i: harp.harp_weight_incoherence(W.data_ptr(), wd.n_rows, wd.d, harp.HARP_BF16, acc.data_ptr(), stream)
            for i in range(2):
                mu(i)
            dt = time_region(torch, mu, 10)
            res["weight_incoherence"] = {"ms": 1e3 * dt / 10, "GBps_read": wbytes / 2 * 10 / dt / 1e9,
                                         "frac_of_measured_peak": wbytes / 2 * 10 / dt / 1e9 / peak,
                                         "mu_W": float(acc[0].item())}
        out[w.name] = res
        bufs = None
        torch.cuda.empty_cache()
    return out


def bench_compact(torch, harp, kernel, peak):
    """Forward / transpose rate of every configuration at its full row count, decode latency (cfg4,
    1 and 16 rows) and the two-sided product (cfg5): a few repetitions each, buffers rotated past L2."""
    out = {}
    gen = torch.Generator(device="cuda")
    gen.manual_seed(4321)
    for cfg in (1, 2, 3, 4, 5):
        w = wl.config(cfg)
        spec = w.plans["in"] if cfg == 5 else w.plans["q"]
        data = w.data["x"]
        plan = harp.plan_from_spec(spec)
        tdt = torch.float32 if data.dtype == "f32" else torch.bfloat16
        es = 4 if data.dtype == "f32" else 2
        nbytes = data.n_rows * data.d * es
        nbuf = max(2, min(6, int(np.ceil(2.5 * 126e6 / nbytes)) + 1))
        bufs = [torch.randn((data.n_rows, data.d), generator=gen, device="cuda", dtype=torch.float32).to(tdt)
                for _ in range(nbuf)]
        res = {"d": data.d, "n_rows": data.n_rows, "dtype": data.dtype, "algorithmic_bytes": 2 * nbytes,
               "traffic": ncu_traffic(cfg, data.n_rows)}
        for name, tr in (("forward", False), ("transpose", True)):
            for i in range(3):
                harp.apply_(plan, bufs[i % nbuf], transpose=tr, kernel=kernel)
            torch.cuda.synchronize()
            iters = max(4, min(40, int(0.05 / (2 * nbytes / (0.3 * peak * 1e9)))))
            dt = time_region(torch, lambda i: harp.apply_(plan, bufs[i % nbuf], transpose=tr, kernel=kernel), iters)
            gbs = 2 * nbytes * iters / dt / 1e9
            res[name] = {"GBps": round(gbs, 1), "frac": round(gbs / peak, 4), "frac_of_8TBps": round(gbs / 8000.0, 4),
                         "us": round(1e6 * dt / iters, 2)}
        if cfg == 4:
            stream = torch.cuda.current_stream().cuda_stream
            for n in (1, 16):
                ptr = bufs[0].data_ptr()
                call = lambda i: harp.harp_apply(plan, ptr, n, harp.HARP_BF16, i & 1, stream, kernel)   # raw binding: the host must not be the limit
                for i in range(20):
                    call(i)
                torch.cuda.synchronize()
                dt = time_region(torch, call, 400)
                res[f"decode_{n}_rows_us"] = round(1e6 * dt / 400, 2)
        if cfg == 4:
            # the same schedule behind a random permutation (a layer whose reshape permutes the coordinates):
            # one gather kernel and the two tensor-core passes
            import copy
            pspec = copy.copy(spec)
            pspec.perm = np.random.default_rng(977).permutation(spec.d).astype(np.int32)
            pplan = harp.plan_from_spec(pspec)
            for name, tr in (("forward", False), ("transpose", True)):
                for i in range(2):
                    harp.apply_(pplan, bufs[i % nbuf], transpose=tr, kernel=kernel)
                torch.cuda.synchronize()
                l0 = harp.harp_launch_count()
                dt = time_region(torch, lambda i: harp.apply_(pplan, bufs[i % nbuf], transpose=tr, kernel=kernel), 6)
                gbs = 2 * nbytes * 6 / dt / 1e9
                res.setdefault("random_permutation", {})[name] = {
                    "GBps": round(gbs, 1), "frac": round(gbs / peak, 4), "us": round(1e6 * dt / 6, 2),
                    "launches": (harp.harp_launch_count() - l0) // 6}
            del pplan
        if cfg == 5:
            del bufs
            torch.cuda.empty_cache()
            wd = w.data["w"]
            p_out = harp.plan_from_spec(w.plans["out"])
            W = (torch.randn((wd.n_rows, wd.d), generator=gen, device="cuda") * 0.02).to(torch.bfloat16)
            for _ in range(2):
                harp.two_sided_(W, p_out, plan)
            torch.cuda.synchronize()
            l0 = harp.harp_launch_count()
            dt = time_region(torch, lambda i: harp.two_sided_(W, p_out, plan), 5)
            wbytes = 2 * wd.n_rows * wd.d * 2
            res["two_sided"] = {"ms": round(1e3 * dt / 5, 4), "launches": (harp.harp_launch_count() - l0) // 5,
                                "algorithmic_bytes": wbytes, "frac_vs_1R1W": round(wbytes * 5 / dt / 1e9 / peak, 4)}
        out[f"cfg{cfg}"] = res
        bufs = None
        torch.cuda.empty_cache()
    return out


def relaunch_with_ranks(args):
    """`--gpus N` (N > 1) outside a launcher: start N ranks of this script on this node."""
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    raise SystemExit(subprocess.call(cmd))


def run_gpu(args):
    import torch
    import torch.distributed as dist
    import paper_2605_29843_b200 as harp

    if "WORLD_SIZE" not in os.environ and args.gpus > 1:
        relaunch_with_ranks(args)
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the HARP library has no CPU path")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    harp.lib()
    kernel = KERNELS(harp)[args.kernel]

    w = wl.config(2)
    spec, data = w.plans["q"], w.data["x"]
    n_rows, d = data.n_rows, data.d
    plan = harp.plan_from_spec(spec)
    # every rank works on a batch of the same shape (weak scaling); rank r draws its own rows
    host_bits = wl.DataSpec(n_rows, d, "bf16", "normal", seed=data.seed + 1000 * rank).rows(0, n_rows)
    host = torch.from_numpy(host_bits.view(np.int16)).view(torch.bfloat16)
    bufs = [host.cuda().clone() for _ in range(N_BUF)]
    stream = torch.cuda.current_stream()

    def step(i):
        harp.apply_(plan, bufs[(2 * i) % N_BUF], transpose=False, kernel=kernel)
        harp.apply_(plan, bufs[(2 * i + 1) % N_BUF], transpose=True, kernel=kernel)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local_rank) if rank == 0 else None
    for i in range(max(3, args.warmup)):
        step(i)
    barrier()
    launches0 = harp.harp_launch_count()
    if sampler:
        sampler.mark_start()
    dt = time_region(torch, step, args.steps)
    barrier()
    if sampler:
        sampler.mark_end()
    launches = harp.harp_launch_count() - launches0
    t = torch.tensor([dt], device="cuda", dtype=torch.float64)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dt_max = float(t.item())
    clocks = sampler.stop() if sampler else None

    # end to end through the host-buffer entry point: pinned host rows in, results back
    pinned = [host.clone().pin_memory() for _ in range(2)]
    e2e_steps = max(2, min(args.steps, 10))

    def e2e_step(i):
        harp.harp_apply_host(plan, pinned[0].data_ptr(), n_rows, harp.HARP_BF16, False)
        harp.harp_apply_host(plan, pinned[1].data_ptr(), n_rows, harp.HARP_BF16, True)

    e2e_step(0)
    barrier()
    t0 = time.perf_counter()
    for i in range(e2e_steps):
        e2e_step(i)
    torch.cuda.synchronize()
    e2e_dt = time.perf_counter() - t0
    te = torch.tensor([e2e_dt], device="cuda", dtype=torch.float64)
    if world > 1:
        dist.all_reduce(te, op=dist.ReduceOp.MAX)
    e2e_dt = float(te.item())

    if rank == 0:
        peak, peak_kind = measured_peaks()
        row_bytes = d * 2 * 2                                     # bf16 read + write
        per_launch_s = dt_max / (2 * args.steps)
        achieved = n_rows * row_bytes / per_launch_s / 1e9
        line = {
            "metric": METRIC, "value": world * 2 * n_rows * args.steps / dt_max, "unit": UNIT,
            "n_gpus": world, "steps": args.steps, "warmup": max(3, args.warmup),
            "ms_per_step": 1e3 * dt_max / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": WORKLOAD, "n_rows": n_rows, "d": d, "kernel": args.kernel,
                       "arithmetic": "bf16 operands (fused blocks rounded to bf16 at plan time), fp32 accumulate, "
                                     "rows rounded to bf16 after each of the three fused phases",
                       "l2": f"{N_BUF} rotating 134 MB buffers (inputs larger than L2)", "parallelism": f"rows x{world}"},
            "clocks": clocks,
            "e2e": {"value": world * 2 * n_rows * e2e_steps / e2e_dt, "unit": UNIT,
                    "h2d_bytes_per_step": 2 * n_rows * d * 2, "d2h_bytes_per_step": 2 * n_rows * d * 2,
                    "api": "harp_apply_host (pinned host rows, chunked copy/compute overlap)"},
            "gpu_launches": int(launches),
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                         "frac": achieved / peak, "peak_kind": f"of {peak_kind}", "frac_of_8TBps": achieved / 8000.0,
                         "traffic": ncu_traffic(2, n_rows),
                         "algorithmic_bytes_per_launch": n_rows * row_bytes,
                         "us_per_launch": 1e6 * per_launch_s},
        }
        if not args.no_cpu and world == 1:
            line["cpu_baseline"] = cpu_baseline(spec, data)
        if world == 1 and not args.no_per_config:
            del bufs, pinned
            torch.cuda.empty_cache()
            line["per_config"] = bench_compact(torch, harp, kernel, peak)
        if args.all_configs and world == 1:
            torch.cuda.empty_cache()
            line["per_config_detail"] = bench_extra_configs(torch, harp, kernel, peak)
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def KERNELS(harp):
    return {"auto": harp.KERNEL_AUTO, "generic": harp.KERNEL_GENERIC, "fast": harp.KERNEL_FAST,
            "split": harp.KERNEL_SPLIT, "tmem": harp.KERNEL_TMEM}


def run_profile_case(args):
    """Small case for profilers: `--profile-config C` applies configuration C's processor to
    `--profile-rows` seeded device rows, alternating forward and transpose, `--profile-reps` times."""
    import torch
    import paper_2605_29843_b200 as harp
    kernel = KERNELS(harp)[args.kernel]
    gen = torch.Generator(device="cuda")
    gen.manual_seed(7)
    if args.profile_config == 6:          # two-sided processing of configuration 5's weight matrix
        w = wl.config(5)
        p_out, p_in = harp.plan_from_spec(w.plans["out"]), harp.plan_from_spec(w.plans["in"])
        W = (torch.randn((p_out.d, p_in.d), generator=gen, device="cuda") * 0.02).to(torch.bfloat16)
        for _ in range(args.profile_reps):
            harp.two_sided_(W, p_out, p_in)
        torch.cuda.synchronize()
        print(json.dumps({"profile_case": "two_sided_8192x28672", "reps": args.profile_reps,
                          "launches": harp.harp_launch_count()}))
        return
    w = wl.config(args.profile_config)
    spec = w.plans["in"] if args.profile_config == 5 else w.plans["q"]
    plan = harp.plan_from_spec(spec)
    tdt = torch.float32 if w.data["x"].dtype == "f32" else torch.bfloat16
    x = torch.randn((args.profile_rows, spec.d), generator=gen, device="cuda").to(tdt)
    if args.profile_grad:                 # gradient with respect to the block kernels instead of the apply
        G = torch.randn((args.profile_rows, spec.d), generator=gen, device="cuda").to(tdt)
        grad = torch.zeros(harp.harp_plan_n_params(plan), dtype=torch.float32, device="cuda")
        for i in range(args.profile_reps):
            harp.harp_grad_blocks(plan, x.data_ptr(), G.data_ptr(), args.profile_rows,
                                  harp.HARP_F32 if tdt == torch.float32 else harp.HARP_BF16, grad.data_ptr(), False,
                                  torch.cuda.current_stream().cuda_stream)
        torch.cuda.synchronize()
        print(json.dumps({"profile_case": w.name + "_grad_blocks", "rows": args.profile_rows, "reps": args.profile_reps,
                          "launches": harp.harp_launch_count()}))
        return
    for i in range(args.profile_reps):
        harp.apply_(plan, x, transpose=bool(i & 1), kernel=kernel)
    torch.cuda.synchronize()
    print(json.dumps({"profile_case": w.name, "rows": args.profile_rows, "reps": args.profile_reps,
                      "launches": harp.harp_launch_count()}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="harp", choices=["harp", "reference"])
    ap.add_argument("--kernel", default="auto", choices=["auto", "generic", "fast", "split", "tmem"])
    ap.add_argument("--no-per-config", action="store_true", help="headline only: skip the compact per-configuration block")
    ap.add_argument("--profile-config", type=int, default=0, help="run a small profiling case of this configuration and exit")
    ap.add_argument("--profile-rows", type=int, default=8192)
    ap.add_argument("--profile-reps", type=int, default=2)
    ap.add_argument("--profile-grad", action="store_true", help="the profiling case calls harp_grad_blocks")
    ap.add_argument("--all-configs", action="store_true")
    ap.add_argument("--no-cpu", action="store_true", help="skip the timed CPU-oracle baseline")
    ap.add_argument("--ref-rows", type=int, default=2048)
    args = ap.parse_args()
    if args.profile_config:
        run_profile_case(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
