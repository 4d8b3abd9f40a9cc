#!/usr/bin/env python
"""Benchmark of the shared-prefix attention hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

One step = one forward (`pskv_attn_fwd`: out, lse) plus one backward (`pskv_attn_bwd`: dq,
dk_suffix, dv_suffix) of one attention layer of the Llama-3-8B-shaped GQA workload (C2:
B=512 candidates, 32 query / 8 KV heads, d=128, prefix 256, suffix-side 48, outlier key
channels), all inputs resident in HBM.  Prints ONE JSON line on rank 0.  With N > 1 each
rank runs the same step on its own B candidates against its own replica of the prefix cache
(candidates are independent given the prefix; there is no collective on the data path): started
under torchrun the script is one rank of N; started plainly with --gpus N it launches the N ranks
itself (one process per GPU, NCCL for the barrier and the max over ranks only).
`--impl reference` times the fp64 CPU oracle on a bounded sample instead.
"""
from __future__ import annotations

import argparse
import dataclasses
import json
import os
import subprocess
import sys
import threading
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2603_13420_b200 import inputs as wl  # noqa: E402

METRIC = "shared-prefix attention TFLOP/s (fwd+bwd, one layer)"
MAIN = "C2"


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm_gbs=float(p["hbm_gbs"]), bf16_tflops=float(p["bf16_tflops"]),
                    bf16_tflops_sustained=float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                    source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int, trim: int = 0):
        self.gpu = gpu_index
        self.trim = trim
        self.lines = []
        self.proc = None
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.gpu), "--query-gpu=" + self.FIELDS,
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, smax, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.lines:
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 9:
                continue
            try:
                sm.append(float(parts[1]))
                smax = float(parts[2])
            except ValueError:
                continue
            for name, val in zip(names, parts[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        n_all = len(sm)
        if self.trim and len(sm) > 2 * self.trim + 4:
            sm = sm[self.trim:-self.trim]  # the samples at both ends may lie outside the loop
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_min_mhz": sm[0] if sm else None,
                "sm_max_mhz": smax, "samples": n_all, "reasons": sorted(reasons)}


def dist_env():
    return int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)), \
        int(os.environ.get("WORLD_SIZE", 1))


def launch_ranks(n, argv):
    """Start this script once per rank (RANK / LOCAL_RANK / WORLD_SIZE / MASTER_* in the environment, as
    torchrun would set them) and wait for all of them; rank 0 prints the JSON line.  Returns the largest
    exit code."""
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    procs = []
    for r in range(n):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE=str(n),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, os.path.abspath(__file__)] + list(argv), env=env))
    rc = 0
    for pr in procs:
        rc = max(rc, abs(pr.wait()))
    return rc


def run_stub(args):
    """The multi-rank plumbing without a GPU: every rank 'computes' for stub_step_ms * (rank + 1)
    milliseconds per step; barrier, timing of exactly K steps, max over ranks and the one JSON line of
    rank 0 are those of the real benchmark, over the gloo backend.  Used by the CPU test of the launcher."""
    import torch.distributed as dist
    rank, _, world = dist_env()
    if world > 1:
        dist.init_process_group("gloo")
        dist.barrier()
    for _ in range(args.warmup):
        time.sleep(1e-3 * args.stub_step_ms * (rank + 1))
    if world > 1:
        dist.barrier()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        time.sleep(1e-3 * args.stub_step_ms * (rank + 1))
    ms = torch.tensor([(time.perf_counter() - t0) * 1e3], dtype=torch.float64)
    if world > 1:
        dist.barrier()
        dist.all_reduce(ms, op=dist.ReduceOp.MAX)
    if rank == 0:
        print(json.dumps({"stub": True, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
                          "ms_per_step": ms.item() / args.steps, "scaling": "weak"}), flush=True)
    if world > 1:
        dist.destroy_process_group()


# ----------------------------------------------------------------------------- reference arm

def run_reference(args):
    """The fp64 CPU oracle, as it stands, on a bounded sample of the same workload."""
    rank, _, world = dist_env()
    if rank != 0:
        return
    import oracle
    w = wl.WORKLOADS[MAIN]
    cand = args.ref_candidates
    sub = w.with_candidates(cand)
    t = wl.make_inputs(sub, with_dout=True)
    f = {k: v.to(torch.float64).numpy() for k, v in t.items()}

    def step():
        oracle.attn_fwd(f["q"], f["prefix_k"], f["prefix_v"], f["suffix_k"], f["suffix_v"], w.scale)
        oracle.attn_bwd(f["dout"], f["q"], f["prefix_k"], f["prefix_v"], f["suffix_k"], f["suffix_v"],
                        w.scale)

    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    dt = (time.perf_counter() - t0) / args.steps
    flops = wl.fwd_flops(sub) + wl.bwd_flops(sub)
    value = flops / dt / 1e12
    cores = oracle.num_threads()
    sample = "%d of %d candidates of %s per step, fwd+bwd, fp64" % (cand, w.B, MAIN)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": workload_config(w, 1),
        "candidates_per_s": cand / dt,
        "cpu_baseline": {"value": value, "unit": "TFLOP/s", "cores": cores, "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def workload_config(w, world):
    return {"workload": "%s: %s" % (w.name, w.note), "B_per_gpu": w.B, "Hq": w.Hq, "Hkv": w.Hkv,
            "d": w.d, "P": w.P, "S": w.S, "step": "pskv_attn_fwd + pskv_attn_bwd, one layer",
            "parallelism": "candidates sharded over %d GPU(s), prefix cache replicated" % world,
            "l2": "inputs larger than L2 (%.0f MB touched per step vs 126 MB L2)"
                  % ((wl.fwd_bytes(w) + wl.bwd_bytes(w)) / 1e6)}


# ----------------------------------------------------------------------------- CUDA arm

E2E_CHUNKS = 8  # candidate chunks of the end-to-end leg


def time_calls(fn, iters, warmup):
    """Median-free plain average over `iters` calls with CUDA events on the current stream."""
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    e0 = torch.cuda.Event(enable_timing=True)
    e1 = torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(iters):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / iters  # ms


def device_inputs(w, seed, device):
    """Same distribution as inputs.make_inputs, drawn on the device (kernel-only timing legs)."""
    gen = torch.Generator(device=device)
    gen.manual_seed(seed)

    def draw(shape, outliers=False):
        x = torch.randn(shape, generator=gen, device=device, dtype=torch.float32)
        if outliers:
            for c in wl.OUTLIER_CHANNELS:
                x[..., c] *= wl.OUTLIER_GAIN
        return x.to(torch.bfloat16)

    t = {"q": draw((w.B, w.Hq, w.S, w.d)),
         "prefix_k": draw((w.Hkv, w.P, w.d), w.outlier_keys),
         "prefix_v": draw((w.Hkv, w.P, w.d)),
         "suffix_k": draw((w.B, w.Hkv, w.S, w.d), w.outlier_keys),
         "suffix_v": draw((w.B, w.Hkv, w.S, w.d)),
         "dout": draw((w.B, w.Hq, w.S, w.d))}
    return t


class Layer:
    """Device buffers of one attention layer call (inputs, outputs, workspaces)."""

    def __init__(self, pskv, w, t):
        self.pskv, self.w, self.t = pskv, w, t
        dev = t["q"].device
        dims = (w.B, w.Hq, w.Hkv, w.S, w.P, w.d)
        self.out = torch.empty_like(t["q"])
        self.lse = torch.empty((w.B, w.Hq, w.S), dtype=torch.float32, device=dev)
        self.dq = torch.empty_like(t["q"])
        self.dk = torch.empty_like(t["suffix_k"])
        self.dv = torch.empty_like(t["suffix_v"])
        self.ws_f = torch.empty(max(pskv.pskv_attn_fwd_workspace_bytes(*dims), 256), dtype=torch.uint8, device=dev)
        self.ws_b = torch.empty(max(pskv.pskv_attn_bwd_workspace_bytes(*dims), 256), dtype=torch.uint8, device=dev)

    def fwd(self):
        t = self.t
        self.pskv.pskv_attn_fwd(t["q"], t["prefix_k"], t["prefix_v"], t["suffix_k"], t["suffix_v"],
                                self.w.scale, out=self.out, lse=self.lse, workspace=self.ws_f)

    def bwd(self):
        t = self.t
        self.pskv.pskv_attn_bwd(t["dout"], t["q"], t["prefix_k"], t["prefix_v"], t["suffix_k"],
                                t["suffix_v"], self.out, self.lse, self.w.scale,
                                dq=self.dq, dk_suffix=self.dk, dv_suffix=self.dv, workspace=self.ws_b)


def run_cuda(args):
    rank, local_rank, world = dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    import paper_2603_13420_b200 as pskv
    pskv.pskv_enable_cta_pairs(args.cta_pairs)
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=device)
    peaks = load_peaks()
    w = wl.WORKLOADS[MAIN]

    # ---- inputs: seeded on the host (pinned, reused by the end-to-end leg), then resident in HBM
    host = wl.make_inputs(w, seed=w.seed + 1000 * rank, with_dout=True)
    host = {k: v.pin_memory() for k, v in host.items()}
    dev = {k: v.to(device, non_blocking=True) for k, v in host.items()}
    torch.cuda.synchronize()
    layer = Layer(pskv, w, dev)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- main timed region: K steps, device-resident inputs
    for _ in range(max(args.warmup, 3)):
        layer.fwd()
        layer.bwd()
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    barrier()
    for kid in range(pskv.pskv_kernel_timing_count()):
        pskv.pskv_kernel_timing_read(kid)  # forget launches recorded so far
    pskv.pskv_kernel_timing_enable(True)
    launches0 = pskv.pskv_kernel_launches()
    e_start = torch.cuda.Event(enable_timing=True)
    e_stop = torch.cuda.Event(enable_timing=True)
    e_start.record()
    for k in range(args.steps):
        ev[k][0].record()
        layer.fwd()
        ev[k][1].record()
        layer.bwd()
        ev[k][2].record()
    e_stop.record()
    barrier()
    launches = pskv.pskv_kernel_launches() - launches0
    pskv.pskv_kernel_timing_enable(False)
    kernels = {}
    for kid in range(pskv.pskv_kernel_timing_count()):
        ms, n = pskv.pskv_kernel_timing_read(kid)
        if n:
            kernels[pskv.pskv_kernel_timing_name(kid)] = {"launches": n, "total_ms": ms, "avg_us": 1e3 * ms / n}
    total_ms = e_start.elapsed_time(e_stop)
    fwd_ms = sum(e[0].elapsed_time(e[1]) for e in ev) / args.steps
    bwd_ms = sum(e[1].elapsed_time(e[2]) for e in ev) / args.steps
    if rank == 0:
        time.sleep(0.2)
    clocks = sampler.stop() if rank == 0 else None
    status = pskv.pskv_poll_device_status()
    if status != pskv.PSKV_OK:
        raise SystemExit("device status after timed region: %s" % pskv.pskv_status_string(status))

    # ---- sustained leg: the same step in a loop of a few seconds, clocks sampled throughout.  The K timed
    # steps above last some ten milliseconds (a burst, at boost clocks); under sustained load the part runs
    # into its power cap and clocks lower.  Both are reported; the clock record of the line comes from
    # this loop, whose duration holds enough nvidia-smi samples.
    sustained = None
    if args.sustained_s > 0:
        burst_step_ms = total_ms / args.steps

        def loop(fn, seconds, per_ms):
            n = max(10, int(seconds * 1e3 / per_ms))
            smp = ClockSampler(local_rank, trim=2)
            if rank == 0:
                smp.start()
                time.sleep(0.25)
            barrier()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            for _ in range(n):
                fn()
            b.record()
            barrier()
            ck = smp.stop() if rank == 0 else None
            return a.elapsed_time(b) / n, n, ck

        def one_step():
            layer.fwd()
            layer.bwd()

        s_ms, s_n, s_clk = loop(one_step, args.sustained_s, burst_step_ms)
        f_ms, f_n, f_clk = loop(layer.fwd, args.sustained_s / 2, fwd_ms)
        sustained = {"step": {"ms_per_step": s_ms, "steps": s_n, "clocks": s_clk},
                     "fwd": {"ms": f_ms, "calls": f_n, "clocks": f_clk}}

    # ---- end-to-end leg: host buffers, H2D and D2H inside the timed region
    houts = {"out": torch.empty_like(host["q"]).pin_memory(),
             "lse": torch.empty((w.B, w.Hq, w.S), dtype=torch.float32).pin_memory(),
             "dq": torch.empty_like(host["q"]).pin_memory(),
             "dk": torch.empty_like(host["suffix_k"]).pin_memory(),
             "dv": torch.empty_like(host["suffix_v"]).pin_memory()}
    h2d = sum(v.numel() * v.element_size() for v in host.values())
    d2h = sum(v.numel() * v.element_size() for v in houts.values())

    # The public call for host-resident data: candidate chunks through upload, compute and download streams, so that the copies of
    # neighbouring chunks overlap the kernels (every chunk still goes through pskv_attn_fwd / pskv_attn_bwd).
    from paper_2603_13420_b200.host_step import HostStep
    hstep = HostStep(w.B, w.Hq, w.Hkv, w.S, w.P, w.d, w.scale, device, chunks=E2E_CHUNKS)

    def e2e_step():
        hstep.run(host, houts)

    e2e_steps = max(3, min(args.steps, 10))
    barrier()
    e2e_ms = time_calls(e2e_step, e2e_steps, 2) if not args.no_e2e else float("nan")
    barrier()

    # ---- max over ranks
    sus = [sustained["step"]["ms_per_step"], sustained["fwd"]["ms"]] if sustained else [0.0, 0.0]
    times = torch.tensor([total_ms, fwd_ms, bwd_ms, e2e_ms] + sus, dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(times, op=dist.ReduceOp.MAX)
    total_ms, fwd_ms, bwd_ms, e2e_ms, sus_step_ms, sus_fwd_ms = times.tolist()
    step_ms = total_ms / args.steps
    flops_f, flops_b = wl.fwd_flops(w), wl.bwd_flops(w)
    value = world * (flops_f + flops_b) / (step_ms * 1e-3) / 1e12
    e2e_value = world * (flops_f + flops_b) / (e2e_ms * 1e-3) / 1e12

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    line = {
        "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": step_ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": workload_config(w, world),
        "candidates_per_s": world * w.B / (step_ms * 1e-3),
        "pct_bf16_peak": 100.0 * value / world / peaks["bf16_tflops"],
        "parts": {
            "fwd": {"ms": fwd_ms, "tflops": flops_f / fwd_ms / 1e9, "candidates_per_s": w.B / fwd_ms * 1e3,
                    "pct_bf16_peak": 100.0 * flops_f / fwd_ms / 1e9 / peaks["bf16_tflops"],
                    "hbm_gbs": wl.fwd_bytes(w) / fwd_ms / 1e6,
                    "kernel_family": pskv.pskv_kernel_family(0, w.B, w.Hq, w.Hkv, w.S, w.P, w.d)},
            "bwd": {"ms": bwd_ms, "tflops": flops_b / bwd_ms / 1e9, "candidates_per_s": w.B / bwd_ms * 1e3,
                    "pct_bf16_peak": 100.0 * flops_b / bwd_ms / 1e9 / peaks["bf16_tflops"],
                    "hbm_gbs": wl.bwd_bytes(w) / bwd_ms / 1e6,
                    "kernel_family": pskv.pskv_kernel_family(1, w.B, w.Hq, w.Hkv, w.S, w.P, w.d)},
        },
        "e2e": {"value": e2e_value, "unit": "TFLOP/s", "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms,
                "how": "HostStep: %d candidate chunks through upload, compute and download streams, pinned host buffers" % E2E_CHUNKS},
        "gpu_launches": int(launches),
        "clocks": clocks,
        "peaks": peaks,
    }
    if args.no_e2e:
        line["e2e"] = None
    line["clocks"]["window"] = "the %d timed steps (%.1f ms)" % (args.steps, total_ms)
    if sustained:
        sc, fc = sustained["step"]["clocks"], sustained["fwd"]["clocks"]
        s_val = world * (flops_f + flops_b) / (sus_step_ms * 1e-3) / 1e12
        f_val = flops_f / sus_fwd_ms / 1e9
        line["sustained"] = {
            "what": "the same step (and the forward call alone) in a loop of seconds; clocks sampled every 100 ms inside the loop",
            "step": {"ms_per_step": sus_step_ms, "steps": sustained["step"]["steps"], "value": s_val, "unit": "TFLOP/s",
                     "sm_mhz_median": sc["sm_mhz"], "sm_mhz_min": sc["sm_min_mhz"], "clock_samples": sc["samples"],
                     "ms_x_mhz": sus_step_ms * sc["sm_mhz"] if sc["sm_mhz"] else None,
                     "frac_bf16_sustained_peak": s_val / world / peaks["bf16_tflops_sustained"],
                     "reasons": sc["reasons"]},
            "fwd": {"ms": sus_fwd_ms, "calls": sustained["fwd"]["calls"], "tflops": f_val,
                    "sm_mhz_median": fc["sm_mhz"], "sm_mhz_min": fc["sm_min_mhz"], "clock_samples": fc["samples"],
                    "ms_x_mhz": sus_fwd_ms * fc["sm_mhz"] if fc["sm_mhz"] else None,
                    "frac_bf16_sustained_peak": f_val / peaks["bf16_tflops_sustained"],
                    "frac_bf16_burst_peak": f_val / peaks["bf16_tflops"], "reasons": fc["reasons"]},
            "burst": {"ms_per_step": step_ms, "fwd_ms": fwd_ms,
                      "fwd_frac_bf16_burst_peak": flops_f / fwd_ms / 1e9 / peaks["bf16_tflops"]},
        }
        # the clock record the line is judged by: samples taken INSIDE a timed loop (the K steps above are
        # shorter than one nvidia-smi sample)
        burst_clocks = line["clocks"]
        line["clocks"] = {"sm_mhz": sc["sm_mhz"], "sm_max_mhz": sc["sm_max_mhz"], "samples": sc["samples"],
                          "reasons": sorted(set(sc["reasons"]) | set(burst_clocks["reasons"])),
                          "window": "sustained loop of %d steps (%.2f s); around the %d timed steps (%.1f ms): %s MHz, %d samples"
                                    % (sustained["step"]["steps"], sus_step_ms * sustained["step"]["steps"] * 1e-3,
                                       args.steps, total_ms, burst_clocks["sm_mhz"], burst_clocks["samples"])}
    tot = sum(k["total_ms"] for k in kernels.values()) or 1.0
    for k in kernels.values():
        k["share"] = k["total_ms"] / tot
    line["kernels"] = kernels
    line["roofline"] = roofline(w, kernels, peaks)

    if world == 1 and not args.no_detail:
        line["detail"] = detail_runs(pskv, device, peaks)
    if world == 1 and not args.no_cpu:
        line["cpu_baseline"] = cpu_baseline(w, args.cpu_candidates, host,
                                            {"out": layer.out, "lse": layer.lse, "dq": layer.dq, "dk": layer.dk, "dv": layer.dv})
        if "checked" in line["cpu_baseline"]:
            line["checked"] = line["cpu_baseline"]["checked"]["ok"]
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def roofline(w, kernels, peaks):
    """Roofline of the dominant kernel of the step: the kernel with the largest summed device time
    in the timed region (CUDA events around each launch, on the launch stream).  Algorithmic bytes
    and flops per launch come from inputs.kernel_work; the binding roof is the slower of
    bytes / measured HBM peak and flops / measured bf16 peak."""
    work = wl.kernel_work(w)
    cands = {k: v for k, v in kernels.items() if k in work}
    if not cands:
        return None
    name = max(cands, key=lambda k: cands[k]["total_ms"])
    sec = cands[name]["avg_us"] * 1e-6
    t_hbm = work[name]["bytes"] / (peaks["hbm_gbs"] * 1e9)
    t_mma = work[name]["flops"] / (peaks["bf16_tflops"] * 1e12)
    traffic = TRAFFIC_BYTES_PER_LAUNCH.get((name, w.name))
    common = {"kernel": name, "avg_us": cands[name]["avg_us"], "share_of_step": cands[name]["share"],
              "algorithmic_bytes": work[name]["bytes"], "algorithmic_flops": work[name]["flops"],
              "traffic": traffic}
    if t_hbm >= t_mma:
        ach = work[name]["bytes"] / sec / 1e9
        common.update({"bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                       "frac": ach / peaks["hbm_gbs"], "peak_source": peaks["source"] + " (of measured), burst copy"})
    else:
        ach = work[name]["flops"] / sec / 1e12
        common.update({"bound": "tensor", "achieved": ach, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                       "frac": ach / peaks["bf16_tflops"], "peak_source": peaks["source"] + " (of measured), burst"})
    return common


# dram__bytes_read.sum + dram__bytes_write.sum per launch, from the ncu captures summarised under
# profiles/ (kernel, workload) -> bytes.
TRAFFIC_BYTES_PER_LAUNCH = {
    ("tc_fwd_kernel", "C2"): 475.3e6,        # profiles/tc_fwd_kernel_C2.md
    ("tc_bwd_dq_kernel", "C2"): 691.0e6,     # profiles/tc_bwd_dq_kernel_C2.md
    ("tc_bwd_dkv_kernel", "C2"): 823.0e6,    # profiles/tc_bwd_dkv_kernel_C2.md (with the row statistic D)
}


MULTI_LENS = [256, 240, 224, 208, 192, 176, 160, 144]
MULTI_LENS_UNEQUAL = [256, 32, 32, 32, 200, 100, 16, 64]


def multi_run(pskv, device, lens, iters, warmup):
    """pskv_attn_fwd_multi / pskv_attn_bwd_multi at the C2 shape: len(lens) instructions, B / len(lens)
    candidates each, one left-padded prefix cache per instruction."""
    w = wl.WORKLOADS["C2"]
    Bp, Pmax = len(lens), w.P
    gen = torch.Generator(device="cpu")
    gen.manual_seed(w.seed + 500)

    def draw(*shape):
        return torch.randn(shape, generator=gen, dtype=torch.float32).to(torch.bfloat16).to(device)

    q, sk, sv, do = draw(w.B, w.Hq, w.S, w.d), draw(w.B, w.Hkv, w.S, w.d), draw(w.B, w.Hkv, w.S, w.d), draw(w.B, w.Hq, w.S, w.d)
    pk, pv = draw(Bp, w.Hkv, Pmax, w.d), draw(Bp, w.Hkv, Pmax, w.d)
    out = torch.empty_like(q)
    lse = torch.empty((w.B, w.Hq, w.S), dtype=torch.float32, device=device)
    dq, dk, dv = torch.empty_like(q), torch.empty_like(sk), torch.empty_like(sv)
    mdims = (w.B, Bp, w.Hq, w.Hkv, w.S, Pmax, w.d)
    ws_f = torch.empty(max(pskv.pskv_attn_fwd_multi_workspace_bytes(*mdims), 256), dtype=torch.uint8, device=device)
    ws_b = torch.empty(max(pskv.pskv_attn_bwd_multi_workspace_bytes(*mdims), 256), dtype=torch.uint8, device=device)

    def mfwd():
        pskv.pskv_attn_fwd_multi(q, pk, pv, lens, sk, sv, w.scale, out=out, lse=lse, workspace=ws_f)

    def mbwd():
        pskv.pskv_attn_bwd_multi(do, q, pk, pv, lens, sk, sv, out, lse, w.scale, dq=dq, dk_suffix=dk, dv_suffix=dv,
                                 workspace=ws_b)

    mfwd()
    kq = w.B // Bp
    fl_f = sum(wl.fwd_flops(dataclasses.replace(w, B=kq, P=n)) for n in lens)
    fl_b = sum(wl.bwd_flops(dataclasses.replace(w, B=kq, P=n)) for n in lens)
    ms_f = time_calls(mfwd, iters, warmup)
    ms_b = time_calls(mbwd, iters, warmup)
    return {"prefix_len": list(lens),
            "fwd": {"ms": ms_f, "tflops": fl_f / ms_f / 1e9, "candidates_per_s": w.B / ms_f * 1e3},
            "bwd": {"ms": ms_b, "tflops": fl_b / ms_b / 1e9, "candidates_per_s": w.B / ms_b * 1e3}}


def detail_runs(pskv, device, peaks):
    """Kernel-only timings of every workload (forward; backward where the workload asks for it)."""
    res = {}
    for name in ("C1", "C2", "C3", "C4"):
        w = wl.WORKLOADS[name]
        layer = Layer(pskv, w, device_inputs(w, w.seed, device))
        layer.fwd()
        entry = {}
        ms = time_calls(layer.fwd, 20, 3)
        entry["fwd"] = {"ms": ms, "tflops": wl.fwd_flops(w) / ms / 1e9,
                        "candidates_per_s": w.B / ms * 1e3,
                        "pct_bf16_peak": 100 * wl.fwd_flops(w) / ms / 1e9 / peaks["bf16_tflops"],
                        "hbm_gbs": wl.fwd_bytes(w) / ms / 1e6,
                        "pct_hbm_peak": 100 * wl.fwd_bytes(w) / ms / 1e6 / peaks["hbm_gbs"]}
        if name in ("C4", "C2"):
            ms = time_calls(layer.bwd, 20, 3)
            entry["bwd"] = {"ms": ms, "tflops": wl.bwd_flops(w) / ms / 1e9,
                            "candidates_per_s": w.B / ms * 1e3,
                            "pct_bf16_peak": 100 * wl.bwd_flops(w) / ms / 1e9 / peaks["bf16_tflops"],
                            "hbm_gbs": wl.bwd_bytes(w) / ms / 1e6,
                            "pct_hbm_peak": 100 * wl.bwd_bytes(w) / ms / 1e6 / peaks["hbm_gbs"]}
        res[name] = entry
        del layer
        torch.cuda.empty_cache()
    res["C2_prefix_gradients"] = prefix_grad_run(pskv, device, peaks, 10, 3)
    # C2 over 32 layers back to back: 32 calls on distinct per-layer tensors, one stream, no host sync
    w = wl.WORKLOADS["C2"]
    layers = [Layer(pskv, w, device_inputs(w, w.seed + 100 + i, device)) for i in range(32)]

    def stack():
        for L in layers:
            L.fwd()

    ms = time_calls(stack, 3, 1)
    res["C2_32_layers_fwd"] = {"ms": ms, "ms_per_layer": ms / 32, "tflops": 32 * wl.fwd_flops(w) / ms / 1e9,
                               "candidates_per_s": w.B / ms * 1e3}
    del layers
    torch.cuda.empty_cache()
    # Batched multi-instruction variant (Sec. 4.3) at the C2 shape: 8 instructions x 64 candidates, one
    # left-padded prefix cache per instruction, true lengths 144..256; then very unequal lengths (padding is
    # more than half of the padded keys)
    res["C2_multi_8x64"] = multi_run(pskv, device, MULTI_LENS, 20, 3)
    res["C2_multi_8x64_unequal"] = multi_run(pskv, device, MULTI_LENS_UNEQUAL, 20, 3)
    for Bd in (512, 2048):
        res["C2_decode_1of48_B%d" % Bd] = decode_run(pskv, device, peaks, Bd, 40, 4)
    res["prefix_prefill_P%d" % wl.WORKLOADS["C3"].P] = prefill_run(pskv, device, peaks, 40, 4)
    res["target_ce_512x20_Dm4096_V128256"] = ce_run(pskv, device, peaks, 5, 3)
    return res


def _draw_on(device, seed):
    gen = torch.Generator(device="cpu")
    gen.manual_seed(seed)

    def draw(*shape):
        return torch.randn(shape, generator=gen, dtype=torch.float32).to(torch.bfloat16).to(device)

    return draw, gen


def decode_run(pskv, device, peaks, Bd, iters, warmup):
    """Decode-shaped variant at the C2 layer shape: one new token per candidate on top of a suffix cache of up
    to 48 tokens (uniform ragged lengths), forward only (the attacks that grow suffixes token by token are
    gradient-free).  The call is bound by reading each candidate's suffix K/V once, so it is reported
    against the HBM roofline; four input sets are rotated so that every call reads from HBM, not L2."""
    w = wl.WORKLOADS["C2"]
    draw, gen = _draw_on(device, w.seed + 600 + Bd)
    Sq, Skv = 1, 48
    sets = []
    for i in range(4):
        sets.append((draw(Bd, w.Hq, Sq, w.d), draw(Bd, w.Hkv, Skv, w.d), draw(Bd, w.Hkv, Skv, w.d),
                     torch.randint(Sq, Skv + 1, (Bd,), generator=gen, dtype=torch.int32).to(device)))
    pk, pv = draw(w.Hkv, w.P, w.d), draw(w.Hkv, w.P, w.d)
    out = torch.empty_like(sets[0][0])
    lse = torch.empty((Bd, w.Hq, Sq), dtype=torch.float32, device=device)
    ws = torch.empty(256, dtype=torch.uint8, device=device)
    turn = [0]

    def dfwd():
        qd, skd, svd, ln = sets[turn[0] % 4]
        turn[0] += 1
        pskv.pskv_attn_fwd_decode(qd, pk, pv, skd, svd, ln, w.scale, out=out, lse=lse, workspace=ws)

    ms = time_calls(dfwd, iters, warmup)
    nbytes = (2 * Bd * w.Hq * Sq * w.d + 2 * Bd * w.Hkv * Skv * w.d + 2 * w.Hkv * w.P * w.d) * 2 + Bd * w.Hq * Sq * 4
    return {"Sq": Sq, "Skv": Skv, "B": Bd, "algorithmic_bytes": nbytes,
            "fwd": {"ms": ms, "candidates_per_s": Bd / ms * 1e3, "hbm_gbs": nbytes / ms / 1e6,
                    "pct_hbm_peak": 100 * nbytes / ms / 1e6 / peaks["hbm_gbs"]},
            "roofline": {"kernel": "tc_fwd_kernel<128, 2>", "bound": "hbm", "achieved": nbytes / ms / 1e6,
                         "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": nbytes / ms / 1e6 / peaks["hbm_gbs"],
                         "traffic": 449.3e6 if Bd == 2048 else None,  # profiles/tc_fwd_kernel_decode_B2048.md
                         "note": "whole call timed with CUDA events (one kernel launch); peak = measured copy bandwidth"}}


def prefill_run(pskv, device, peaks, iters, warmup):
    """Prefix prefill, attention step: the causal self-attention of one 2048-token sequence (B = 1, P = 0, the
    sequence's K/V passed as the suffix), i.e. what produces a C3-sized prefix cache in the first place."""
    w3 = wl.WORKLOADS["C3"]
    draw, _ = _draw_on(device, w3.seed + 700)
    Sp = w3.P
    qp, kp, vp = draw(1, w3.Hq, Sp, w3.d), draw(1, w3.Hkv, Sp, w3.d), draw(1, w3.Hkv, Sp, w3.d)
    outp = torch.empty_like(qp)
    lsep = torch.empty((1, w3.Hq, Sp), dtype=torch.float32, device=device)
    wsp = torch.empty(256, dtype=torch.uint8, device=device)

    def prefill():
        pskv.pskv_attn_fwd(qp, None, None, kp, vp, w3.scale, out=outp, lse=lsep, workspace=wsp)

    ms = time_calls(prefill, iters, warmup)
    fl = 4.0 * w3.d * ((Sp + 1) / 2) * w3.Hq * Sp
    return {"fwd": {"ms": ms, "tflops": fl / ms / 1e9, "pct_bf16_peak": 100 * fl / ms / 1e9 / peaks["bf16_tflops"],
                    "kernel_family": pskv.pskv_kernel_family(0, 1, w3.Hq, w3.Hkv, Sp, 0, w3.d)},
            "roofline": {"kernel": "tc_fwd_kernel<128, 2>", "bound": "tensor", "achieved": fl / ms / 1e9,
                         "peak": peaks["bf16_tflops"], "unit": "TFLOP/s", "frac": fl / ms / 1e9 / peaks["bf16_tflops"],
                         "traffic": None, "note": "causal-visible flops; inputs (34 MB) are L2 resident as in use"}}


def ce_run(pskv, device, peaks, iters, warmup, with_library=True):
    """Masked target cross-entropy fused with the vocabulary projection at the Llama-3-8B head (hidden 4096,
    vocabulary 128256), 512 candidates x 20 target positions.  A dense contraction: reported against the
    bf16 tensor peak (sustained figure: the launch runs for milliseconds under the power cap).  For context
    the library pipeline on the same inputs: one bf16 GEMM that writes the logits, then float cross-entropy."""
    import math
    N, Lr, Dm, V = 512, 20, 4096, 128256
    gen = torch.Generator(device=device)
    gen.manual_seed(wl.WORKLOADS["C2"].seed + 800)
    h = torch.randn((N, Lr, Dm), generator=gen, device=device).to(torch.bfloat16)
    wt = (torch.randn((V, Dm), generator=gen, device=device) / math.sqrt(Dm)).to(torch.bfloat16)
    t = torch.randint(0, V, (N, Lr), generator=gen, device=device, dtype=torch.int32)
    m = (torch.rand((N, Lr), generator=gen, device=device) < 0.8).to(torch.float32)
    f32 = dict(dtype=torch.float32, device=device)
    nll, lse, loss = torch.empty((N, Lr), **f32), torch.empty((N, Lr), **f32), torch.empty((N,), **f32)
    ws = torch.empty(pskv.pskv_target_ce_fwd_workspace_bytes(N, Lr, Dm, V), dtype=torch.uint8, device=device)

    def fused():
        pskv.pskv_target_ce_fwd(h, wt, t, m, nll=nll, lse=lse, loss=loss, workspace=ws)

    ms = time_calls(fused, iters, warmup)
    fl = 2.0 * N * Lr * Dm * V
    out = {"N": N, "Lr": Lr, "Dm": Dm, "V": V, "algorithmic_flops": fl,
           "fwd": {"ms": ms, "tflops": fl / ms / 1e9, "candidates_per_s": N / ms * 1e3,
                   "pct_bf16_peak_sustained": 100 * fl / ms / 1e9 / peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"]),
                   "pct_bf16_peak_burst": 100 * fl / ms / 1e9 / peaks["bf16_tflops"],
                   "logits_bytes_never_written": 2.0 * N * Lr * V},
           "roofline": {"kernel": "ce_fwd_kernel", "bound": "tensor", "achieved": fl / ms / 1e9, "peak": peaks["bf16_tflops"],
                        "unit": "TFLOP/s", "frac": fl / ms / 1e9 / peaks["bf16_tflops"],
                        "traffic": 3.65e9,  # profiles/ce_fwd_kernel_512x20_V128256.md (algorithmic 1.13 GB)
                        "note": "call = GEMM kernel + a 40 us finalize kernel; peak = measured bf16 burst (a library GEMM)"}}
    if with_library:
        tl = t.view(-1).long()

        def library():
            logits = h.view(-1, Dm) @ wt.T
            return torch.nn.functional.cross_entropy(logits.float(), tl, reduction="none")

        out["library_gemm_plus_ce_ms"] = time_calls(library, 3, 2)
    return out


def prefix_grad_run(pskv, device, peaks, iters, warmup):
    """Gradients of the shared prefix cache at C2 (optional path: the search keeps the prefix frozen)."""
    w = wl.WORKLOADS["C2"]
    layer = Layer(pskv, w, device_inputs(w, w.seed, device))
    layer.fwd()
    dkp, dvp = torch.empty_like(layer.t["prefix_k"]), torch.empty_like(layer.t["prefix_v"])
    ws_p = torch.empty(pskv.pskv_attn_bwd_prefix_workspace_bytes(w.B, w.Hq, w.Hkv, w.S, w.P, w.d), dtype=torch.uint8,
                       device=device)

    def pgrad():
        t = layer.t
        pskv.pskv_attn_bwd_prefix(t["dout"], None, t["q"], t["prefix_k"], t["prefix_v"], layer.out, layer.lse, w.scale,
                                  dk_prefix=dkp, dv_prefix=dvp, workspace=ws_p)

    ms = time_calls(pgrad, iters, warmup)
    fl = 8.0 * w.d * w.P * w.B * w.Hq * w.S  # four contractions over (rows x prefix keys x d)
    return {"ms": ms, "tflops": fl / ms / 1e9, "pct_bf16_peak": 100 * fl / ms / 1e9 / peaks["bf16_tflops"],
            "algorithmic_flops": fl}


def run_variant(args):
    """One variant's timing loop alone (for profiling it without the rest of the benchmark)."""
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    import paper_2603_13420_b200 as pskv
    device = torch.device("cuda", 0)
    torch.cuda.set_device(device)
    peaks = load_peaks()
    if args.variant == "prefill":
        res = prefill_run(pskv, device, peaks, args.steps, max(args.warmup, 3))
    elif args.variant == "prefix_grad":
        res = prefix_grad_run(pskv, device, peaks, args.steps, max(args.warmup, 3))
    elif args.variant == "multi":
        res = multi_run(pskv, device, MULTI_LENS, args.steps, max(args.warmup, 3))
    elif args.variant == "target_ce":
        res = ce_run(pskv, device, peaks, args.steps, max(args.warmup, 3), with_library=False)
    else:
        res = decode_run(pskv, device, peaks, int(args.variant.split("_B")[1]), args.steps, max(args.warmup, 3))
    status = pskv.pskv_poll_device_status()
    if status != pskv.PSKV_OK:
        raise SystemExit("device status: %s" % pskv.pskv_status_string(status))
    print(json.dumps({"variant": args.variant, "steps": args.steps, **res}))


def cpu_baseline(w, cand, host, houts):
    """The oracle, as it stands, on the first `cand` candidates of the benchmark's own host inputs
    (candidates are independent, so a prefix of the batch is a valid sample).  Its results also check
    the results the timed full-size launches left in the device buffers for those candidates."""
    import oracle
    sub = w.with_candidates(cand)
    f = {k: (v if k.startswith("prefix") else v[:cand]).to(torch.float64).numpy() for k, v in host.items()}
    t0 = time.perf_counter()
    ro, rl = oracle.attn_fwd(f["q"], f["prefix_k"], f["prefix_v"], f["suffix_k"], f["suffix_v"], w.scale)
    rq, rk, rv = oracle.attn_bwd(f["dout"], f["q"], f["prefix_k"], f["prefix_v"], f["suffix_k"], f["suffix_v"], w.scale)
    dt = time.perf_counter() - t0
    flops = wl.fwd_flops(sub) + wl.bwd_flops(sub)
    res = {"value": flops / dt / 1e12, "unit": "TFLOP/s", "cores": oracle.num_threads(), "kind": "oracle",
           "sample": "first %d of %d candidates of %s, fwd+bwd once, fp64, %.1f s" % (cand, w.B, w.name, dt),
           "candidates_per_s": cand / dt}
    if houts is not None:
        import numpy as np
        errs, ok = {}, True
        for name, got, ref in (("out", houts["out"], ro), ("dq", houts["dq"], rq), ("dk_suffix", houts["dk"], rk),
                               ("dv_suffix", houts["dv"], rv)):
            g = got[:cand].cpu().to(torch.float64).numpy()
            e = float(np.max(np.abs(g - ref)))
            errs[name] = e
            ok = ok and np.isfinite(g).all() and e <= 2e-2 * max(1.0, float(np.max(np.abs(ref))))
        e = float(np.max(np.abs(houts["lse"][:cand].cpu().to(torch.float64).numpy() - rl) / np.maximum(np.abs(rl), 1.0)))
        errs["lse_rel"] = e
        ok = ok and e <= 1e-3
        res["checked"] = {"ok": bool(ok), "candidates": cand, "max_abs_err": errs,
                          "what": "device buffers of the timed full-size launches against the oracle"}
    return res


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--ref-candidates", type=int, default=32,
                    help="candidates per step of the CPU oracle sample (--impl reference)")
    ap.add_argument("--cpu-candidates", type=int, default=256,
                    help="candidates of the one-off CPU oracle sample reported as cpu_baseline")
    ap.add_argument("--no-detail", action="store_true", help="skip the per-workload kernel timings")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU oracle baseline")
    ap.add_argument("--cta-pairs", action="store_true",
                    help="use the opt-in CTA-pair forward kernel (pskv_enable_cta_pairs) instead of the default one")
    ap.add_argument("--no-e2e", action="store_true",
                    help="skip the end-to-end leg (profiling captures that should hold full-size steps only)")
    ap.add_argument("--sustained-s", type=float, default=2.0,
                    help="seconds of the sustained leg (the step in a loop, clocks sampled throughout); 0 skips it")
    ap.add_argument("--stub-step-ms", type=float, default=0.0,
                    help="CPU-only check of the multi-rank launcher: sleep this long per step instead of computing")
    ap.add_argument("--variant", default=None, choices=["decode_B512", "decode_B2048", "prefill", "target_ce", "prefix_grad", "multi"],
                    help="time only this variant of the detail runs (1 GPU) and print its entry")
    args = ap.parse_args()
    if args.gpus < 1:
        raise SystemExit("--gpus must be at least 1")
    if "WORLD_SIZE" in os.environ:
        if int(os.environ["WORLD_SIZE"]) != args.gpus:
            raise SystemExit("--gpus %d does not match WORLD_SIZE=%s of the launcher" % (args.gpus, os.environ["WORLD_SIZE"]))
    elif args.gpus > 1 and not args.variant:
        # started plainly: this process only launches the ranks (one per GPU) and waits for them
        if args.impl == "cuda" and args.stub_step_ms <= 0 and torch.cuda.device_count() < args.gpus:
            raise SystemExit("--gpus %d asked for, %d CUDA device(s) visible" % (args.gpus, torch.cuda.device_count()))
        sys.exit(launch_ranks(args.gpus, sys.argv[1:]))
    if args.stub_step_ms > 0:
        run_stub(args)
    elif args.impl == "reference":
        run_reference(args)
    elif args.variant:
        run_variant(args)
    else:
        run_cuda(args)


if __name__ == "__main__":
    main()
