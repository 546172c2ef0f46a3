#!/usr/bin/env python
"""Benchmark of the attention-JVP hot path (one step = one attn_jvp_fwd call over one synthetic batch).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

Prints ONE JSON line (rank 0).  `value` is TFLOP/s counted as 12*B*H*Lq*Lk*D per call with the inputs
resident in HBM; `e2e` is the same metric with pinned-host inputs copied in and O, tO, LSE copied out inside
the timed region; `roofline` relates the kernel's average launch time (CUDA events on the launching stream)
to the measured dense bf16 tensor peak; `cpu_baseline` times the fp64 oracle on the host cores on a bounded
sample of the same workload.  With N > 1 every rank runs an independent replica (the path has no exchange
step); the timed region is bracketed by a barrier and the time is the max over ranks.

`--impl reference` times the fp64 oracle (there is no reference implementation to install: the paper
ships no code), each step a bounded row sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402
import torch  # noqa: E402

from paper_2510_08431_b200 import replicas, synth  # noqa: E402

METRIC = "attention-JVP TFLOP/s (12*B*H*Lq*Lk*D)"
UNIT = "TFLOP/s"
FALLBACK_BF16_TFLOPS = 1590.0   # earlier measurement on this machine, used only if MEASURED_PEAKS.json is absent
DATASHEET_BF16_TFLOPS = 2250.0

# DRAM bytes per launch of attn_jvp_fwd_kernel<128, jvp> measured with ncu (dram__bytes_read.sum +
# dram__bytes_write.sum), see profiles/.  One capture per sequence-length class: whether the K/V re-reads of a
# head stay in L2 depends on the sequence length, so a workload takes the capture of its own class and scales it
# by algorithmic bytes (within a class traffic is proportional to the tensors streamed once from HBM).
NCU_TRAFFIC_BYTES = {
    "short": {"workload": "image_dit_2b", "bytes": 256.0e6},     # L = 4096: 204.4 MB read + 51.6 MB written (two launches)
    "long": {"workload": "video_dit_1p3b", "bytes": 1030.5e6},   # L = 32760: 820.1 MB read + 210.4 MB written (one launch)
}


def traffic_class(w) -> str:
    return "long" if w.Lk > 8192 else "short"


def algorithmic_bytes(w) -> int:
    """Bytes that must cross HBM once: the six inputs, O, tO (bf16) and LSE (fp32)."""
    q = w.B * w.Lq * w.H * w.D * 2
    k = w.B * w.Lk * w.H * w.D * 2
    n_in = 2 * q + (2 if w.kv_tangent_free else 4) * k
    return n_in + 2 * q + w.B * w.H * w.Lq * 4


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"bf16_tflops": float(p["bf16_tflops"]), "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", 0)),
                "source": "measured"}
    return {"bf16_tflops": FALLBACK_BF16_TFLOPS, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

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
        sm, mx, pw, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.lines:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1])); pw.append(float(parts[2]))
            except ValueError:
                continue
            for nm, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "power_w_max": max(pw),
                "samples": len(sm), "reasons": sorted(reasons)}


def time_oracle(w, x_host, budget_s: float):
    """Times the fp64 oracle (as it stands) on a row sample sized for about `budget_s` seconds."""
    from oracle import attn_jvp_oracle as orc
    orc.build()
    bits = {k: (None if t is None else synth.bf16_bits(t)) for k, t in x_host.items()}
    n_total = w.B * w.H * w.Lq
    per_row = (8 if w.kv_tangent_free else 12) * w.Lk * w.D

    def run(n):
        # rows of one head, spread over the sequence (one head => one K/V widening, like a real call per head)
        rows = np.unique(np.linspace(0, w.Lq - 1, num=min(n, w.Lq)).astype(np.int64))
        t0 = time.perf_counter()
        orc.attn_jvp_def_bf16_rows(bits["q"], bits["k"], bits["v"], bits["tq"], bits["tk"], bits["tv"],
                                   w.B, w.H, w.Lq, w.Lk, w.D, w.scale, rows)
        return len(rows), time.perf_counter() - t0

    # two probes: the first one mostly measures the one-off widening of K, V, tK, tV to fp64
    n0, t_probe = run(64)
    n1, t_probe = run(int(max(64, min(w.Lq, 64 / max(t_probe, 1e-6) * 2.0))))
    rate = n1 / max(t_probe, 1e-6)
    n = int(max(64, min(n_total, w.Lq, rate * budget_s)))
    n, dt = run(n)
    nominal_per_row = 12 * w.Lk * w.D
    return {"value": n * nominal_per_row / dt / 1e12, "unit": UNIT, "cores": orc.threads(), "kind": "oracle",
            "sample": f"{n} query rows of head (b=0,h=0) against all {w.Lk} keys, fp64, {dt:.1f} s "
                      f"({n / dt:.1f} rows/s; executed {per_row} flop/row, counted {nominal_per_row})",
            "seconds": dt, "rows": n}


def run_reference(args, w):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    x = synth.make_workload(w)
    times, rows = [], 0
    budget = max(2.0, min(20.0, 120.0 / max(1, args.steps + args.warmup)))
    res = None
    for i in range(args.warmup + args.steps):
        res = time_oracle(w, x, budget)
        if i >= args.warmup:
            times.append(res["seconds"]); rows += res["rows"]
    total = sum(times)
    value = rows * 12 * w.Lk * w.D / total / 1e12
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT,
            "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": workload_config(w, extra={"reference": "fp64 CPU oracle; each step a bounded row sample"}),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": res["cores"], "kind": "oracle",
                             "sample": res["sample"]},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def run_qknorm(args, w, aj):
    """Side benchmark of the RMS-norm JVP kernel on the q tensor of the workload: rows = B*Lq*H, memory bound."""
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device (sm_100a); there is no CPU path")
    dev = torch.device("cuda", int(os.environ.get("LOCAL_RANK", "0")))
    torch.cuda.set_device(dev)
    g = torch.Generator(device="cpu").manual_seed(w.seed)
    x = torch.randn((w.B, w.Lq, w.H, w.D), generator=g).to(torch.bfloat16).to(dev)
    tx = (torch.randn((w.B, w.Lq, w.H, w.D), generator=g) * w.sigma_tangent).to(torch.bfloat16).to(dev)
    wt = torch.ones(w.D, device=dev)
    rows = w.B * w.Lq * w.H
    nbytes = 4 * rows * w.D * 2
    flush = torch.empty(512 * 1024 * 1024, dtype=torch.uint8, device=dev) if nbytes <= 2 * 126e6 else None
    y = torch.empty_like(x); ty = torch.empty_like(x)
    stream = torch.cuda.current_stream()

    def step():
        rc = aj.attn_jvp_qknorm_fwd(x, tx, wt, y, ty, rows, w.D, 1e-6, stream.cuda_stream)
        if rc != 0:
            raise RuntimeError(aj.attn_jvp_strerror(rc))

    for _ in range(max(3, args.warmup)):
        step()
    torch.cuda.synchronize()
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    for a, b in evs:
        if flush is not None:
            flush.zero_()
        a.record(stream); step(); b.record(stream)
    torch.cuda.synchronize()
    ms = [a.elapsed_time(b) for a, b in evs]
    mean_ms = sum(ms) / len(ms)
    hbm = 6549.1
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    src = "fallback"
    if os.path.exists(path):
        with open(path) as f:
            hbm = float(json.load(f)["hbm_gbs"]); src = "measured"
    else:
        hbm = 6650.0
    achieved = nbytes / (mean_ms * 1e-3) / 1e9
    line = {"metric": "qknorm-JVP GB/s (4 tensors x rows x D x 2 B)", "value": achieved, "unit": "GB/s", "n_gpus": 1,
            "steps": args.steps, "warmup": max(3, args.warmup), "ms_per_step": mean_ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": f"qknorm on the q tensor of {w.name}", "rows": rows, "D": w.D,
                       "l2": "tensors larger than L2" if flush is None else "L2 flushed between timed iterations"},
            "gpu_launches": args.steps,
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": hbm, "unit": "GB/s", "frac": achieved / hbm,
                         "traffic": None, "peak_source": f"{src} copy bandwidth", "kernel": "qknorm_jvp_kernel",
                         "algorithmic_bytes": nbytes}}
    print(json.dumps(line), flush=True)


def workload_config(w, extra=None):
    cfg = {"workload": w.name, "B": w.B, "H": w.H, "Lq": w.Lq, "Lk": w.Lk, "D": w.D, "scale": w.scale,
           "kv_tangent_free": w.kv_tangent_free, "layout": "BLHD bf16", "seed": w.seed,
           "parallelism": "replicas only (no collective on the path)",
           "l2": "inputs larger than L2 (no flush needed)" if algorithmic_bytes(w) > 2 * 126e6 else "L2 flushed between timed iterations"}
    if extra:
        cfg.update(extra)
    return cfg


def run_cp_ranks(args, w, aj):
    """--cp P with P ranks: one step = exchange the sequence slices all-to-all, run the kernel on this rank's H/P
    heads over the whole sequence, exchange O, tO, LSE back (strong scaling: the workload is fixed, the ranks
    share it).  Time = max over ranks; value = the whole workload's flops over it."""
    import torch.distributed as dist
    from paper_2510_08431_b200.ulysses import UlyssesAttentionJVP
    rank, local_rank, P = int(os.environ["RANK"]), int(os.environ.get("LOCAL_RANK", "0")), args.cp
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist.init_process_group("nccl", device_id=dev)
    if w.Lq % P or w.Lk % P or w.H % P:
        raise RuntimeError(f"--cp {P} needs Lq, Lk and H to be multiples of {P}")
    # this rank's sequence slices, all heads; a replicated constant context for the tangent-free workload
    xs = synth.make_inputs(w.B, w.H, w.Lq // P, w.Lk if w.kv_tangent_free else w.Lk // P, w.D, w.sigma_primal,
                           w.sigma_tangent, w.seed + (0 if w.kv_tangent_free else 1000 * rank), w.kv_tangent_free,
                           pin_memory=True)
    if w.kv_tangent_free:   # queries differ per rank, the context does not
        xq = synth.make_inputs(w.B, w.H, w.Lq // P, 1, w.D, w.sigma_primal, w.sigma_tangent, w.seed + 1000 * rank + 1,
                               True, pin_memory=True)
        xs["q"], xs["tq"] = xq["q"], xq["tq"]
    g = {k: (None if t is None else t.to(dev)) for k, t in xs.items()}
    layer = UlyssesAttentionJVP(scale=w.scale)
    stream = torch.cuda.current_stream()

    def step(x):
        return layer(x["q"], x["k"], x["v"], x["tq"], x["tk"], x["tv"], kv_replicated=w.kv_tangent_free)

    def bracket(fn, n):
        dist.barrier(); torch.cuda.synchronize()
        a = torch.cuda.Event(enable_timing=True); b = torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for _ in range(n):
            fn()
        b.record(stream)
        dist.barrier(); torch.cuda.synchronize()
        return replicas.max_over_ranks(a.elapsed_time(b), dist, dev) / n

    for _ in range(args.warmup):
        step(g)
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    ms = bracket(lambda: step(g), args.steps)
    clocks = sampler.stop() if rank == 0 else None

    # end to end: pinned host slices in, results out to pinned host memory, every step
    ho = torch.empty(xs["q"].shape, dtype=torch.bfloat16, pin_memory=True)
    hto = torch.empty_like(ho).pin_memory()
    hl = torch.empty((w.B, w.H, w.Lq // P), dtype=torch.float32, pin_memory=True)

    def e2e_step():
        x = {k: (None if t is None else t.to(dev, non_blocking=True)) for k, t in xs.items()}
        o, to, lse = step(x)
        ho.copy_(o, non_blocking=True); hto.copy_(to, non_blocking=True); hl.copy_(lse, non_blocking=True)

    e2e_step()
    n_e2e = max(2, min(args.steps, 5))
    e2e_ms = bracket(e2e_step, n_e2e)
    st = aj.attn_jvp_device_status()
    if st != 0:
        raise RuntimeError(aj.attn_jvp_strerror(st))
    if rank == 0:
        h2d = sum(t.numel() * 2 for t in xs.values() if t is not None)
        d2h = ho.numel() * 4 + hl.numel() * 4
        line = {"metric": METRIC, "value": w.flops / (ms * 1e-3) / 1e12, "unit": UNIT, "n_gpus": P,
                "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
                "scaling": "strong", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
                "config": workload_config(w, extra={"parallelism": f"ulysses context parallel, P = {P}: all-to-all "
                                                    "of the inputs, kernel on H/P heads, all-to-all of the outputs"}),
                "clocks": clocks,
                "e2e": {"value": w.flops / (e2e_ms * 1e-3) / 1e12, "unit": UNIT, "h2d_bytes_per_step": h2d,
                        "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms, "steps": n_e2e},
                "gpu_launches": args.steps, "roofline": None}
        print(json.dumps(line), flush=True)
    dist.destroy_process_group()


def relaunch_with_ranks(n: int) -> int:
    """`python bench.py --gpus N` without a launcher: start N ranks of this script under torchrun and wait."""
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="video_dit_14b", choices=sorted(synth.WORKLOADS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--splits", type=int, default=1, help="key chunks (split-KV entry point) for few-query workloads")
    ap.add_argument("--op", default="attention", choices=["attention", "qknorm"],
                    help="attention = the hot path (default); qknorm = the RMS-norm JVP that feeds it (memory bound)")
    ap.add_argument("--cp", type=int, default=1,
                    help="Ulysses context-parallel size P: every rank's call covers H/P heads and the whole sequence "
                         "(the paper trains the 14B video model with P = 10, i.e. 4 heads per GPU and call).  With "
                         "P ranks launched (--gpus P) the all-to-all exchange of the six inputs and of O, tO, LSE is "
                         "inside the timed step; with one rank only the per-rank kernel shape is timed")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    w = synth.WORKLOADS[args.workload]

    world_env = os.environ.get("WORLD_SIZE")
    if args.impl == "ours" and args.gpus > 1 and world_env is None:
        if not torch.cuda.is_available() or torch.cuda.device_count() < args.gpus:
            raise RuntimeError(f"--gpus {args.gpus} needs that many CUDA devices on this node")
        sys.exit(relaunch_with_ranks(args.gpus))
    if world_env is not None and int(world_env) != args.gpus:
        raise RuntimeError(f"--gpus {args.gpus} does not match the {world_env} ranks that were launched")

    if args.impl == "reference":
        run_reference(args, w)
        return

    import paper_2510_08431_b200 as aj
    aj.load()   # raises if the CUDA library is missing: there is no fallback
    if args.op == "qknorm":
        run_qknorm(args, w, aj)
        return
    cp_note = None
    if args.cp > 1:
        if int(os.environ.get("WORLD_SIZE", "1")) == args.cp:
            run_cp_ranks(args, w, aj)
            return
        if int(os.environ.get("WORLD_SIZE", "1")) != 1 or w.H % args.cp:
            raise RuntimeError("--cp P runs with P ranks (--gpus P) or with one rank, and needs H to be a multiple of P")
        # one rank: the per-rank call of a context-parallel group of P (H/P heads, whole sequence), no exchange
        import dataclasses
        w = dataclasses.replace(w, name=f"{w.name}/cp{args.cp}", H=w.H // args.cp)
        cp_note = {"cp": args.cp, "cp_note": "per-rank kernel shape of a context-parallel group (H/P heads); "
                                             "the all-to-all exchange is not part of this one-rank run"}

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device (sm_100a); there is no CPU path")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    # each rank draws its own replica of the workload (seed offset by rank)
    x_host = synth.make_inputs(w.B, w.H, w.Lq, w.Lk, w.D, w.sigma_primal, w.sigma_tangent, w.seed + 1000 * rank,
                               w.kv_tangent_free, pin_memory=not args.no_e2e)
    g = {k: (None if t is None else t.to(dev)) for k, t in x_host.items()}
    o = torch.empty_like(g["q"]); to = torch.empty_like(g["q"])
    lse = torch.empty((w.B, w.H, w.Lq), dtype=torch.float32, device=dev)
    flush = None
    if algorithmic_bytes(w) <= 2 * 126e6:
        flush = torch.empty(512 * 1024 * 1024, dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream()
    workspace = None
    if args.splits > 1:
        need = aj.attn_jvp_splitkv_workspace_bytes(w.B, w.H, w.Lq, w.Lk, w.D, args.splits)
        workspace = torch.empty(max(need, 16), dtype=torch.uint8, device=dev)

    def step(fwd_only=False):
        aj.attention_jvp(g["q"], g["k"], g["v"], g["tq"], g["tk"], g["tv"], scale=w.scale, fwd_only=fwd_only,
                         out=(o, None if fwd_only else to, lse), splits=args.splits, workspace=workspace)

    def timed(n_steps, fwd_only=False):
        """Per-launch CUDA-event durations (ms) on the launching stream."""
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n_steps)]
        for a, b in evs:
            if flush is not None:
                flush.zero_()
            a.record(stream)
            step(fwd_only)
            b.record(stream)
        torch.cuda.synchronize()
        return [a.elapsed_time(b) for a, b in evs]

    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize()
    st = aj.attn_jvp_device_status()
    if st != 0:
        raise RuntimeError(aj.attn_jvp_strerror(st))

    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    barrier()
    t_begin = torch.cuda.Event(enable_timing=True); t_end = torch.cuda.Event(enable_timing=True)
    t_begin.record(stream)
    per_launch = timed(args.steps)
    t_end.record(stream)
    barrier()
    clocks = sampler.stop() if rank == 0 else None
    kernel_ms = sum(per_launch) / len(per_launch)
    total_ms = t_begin.elapsed_time(t_end) if flush is None else sum(per_launch)
    flops_per_s, ms_per_step, _ = replicas.aggregate_throughput(w.flops, total_ms, args.steps, dist, dev)
    value = flops_per_s / 1e12

    # forward-only of the same kernel, for the JVP / forward cost ratio
    fwd_ms = None
    if not w.kv_tangent_free:
        timed(2, fwd_only=True)
        f = timed(max(3, args.steps // 2), fwd_only=True)
        fwd_ms = sum(f) / len(f)

    # end to end: pinned host inputs -> device, kernel, O / tO / LSE -> pinned host, every step
    e2e = None
    if not args.no_e2e:
        ho = torch.empty(o.shape, dtype=o.dtype, pin_memory=True)
        hto = torch.empty(o.shape, dtype=o.dtype, pin_memory=True)
        hl = torch.empty(lse.shape, dtype=lse.dtype, pin_memory=True)
        names = [k for k in ("q", "k", "v", "tq", "tk", "tv") if x_host[k] is not None]
        h2d = sum(x_host[k].numel() * 2 for k in names)
        d2h = ho.numel() * 2 + hto.numel() * 2 + hl.numel() * 4

        # the library's host entry point: groups of heads are copied in, computed and copied out in a pipeline
        ws = torch.empty(aj.attn_jvp_host_workspace_bytes(w.B, w.H, w.Lq, w.Lk, w.D, 0), dtype=torch.uint8, device=dev)

        def e2e_step():
            aj.attention_jvp_host(x_host["q"], x_host["k"], x_host["v"], x_host["tq"], x_host["tk"], x_host["tv"],
                                  scale=w.scale, device=dev, out=(ho, hto, hl), workspace=ws, synchronize=False)

        e2e_step(); torch.cuda.synchronize()
        barrier()
        a = torch.cuda.Event(enable_timing=True); b = torch.cuda.Event(enable_timing=True)
        n_e2e = max(2, min(args.steps, 5))
        a.record(stream)
        for _ in range(n_e2e):
            e2e_step()
        b.record(stream)
        barrier()
        e2e_ms = replicas.max_over_ranks(a.elapsed_time(b), dist, dev) / n_e2e
        e2e = {"value": world * w.flops / (e2e_ms * 1e-3) / 1e12, "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms, "steps": n_e2e}
    st = aj.attn_jvp_device_status()
    if st != 0:
        raise RuntimeError(aj.attn_jvp_strerror(st))

    if rank == 0:
        peaks = measured_peaks()
        flops = w.executed_flops
        achieved = flops / (kernel_ms * 1e-3) / 1e12
        cap = NCU_TRAFFIC_BYTES[traffic_class(w)]
        wt = synth.WORKLOADS[cap["workload"]]
        traffic = cap["bytes"] * algorithmic_bytes(w) / algorithmic_bytes(wt)
        # clock-normalised work: SM cycles one CTA spends per 64-key tile of a 128-row query tile (kernel time x
        # sampled median SM clock x SMs / tiles), which separates the power state from the kernel's own cycles
        tiles = w.B * w.H * ((w.Lq + 127) // 128) * ((w.Lk + 63) // 64)
        sm_count = torch.cuda.get_device_properties(dev).multi_processor_count
        cycles_per_tile = None
        if clocks and clocks.get("sm_mhz"):
            cycles_per_tile = kernel_ms * 1e-3 * clocks["sm_mhz"] * 1e6 * sm_count / tiles
        roofline = {"bound": "tensor", "achieved": achieved, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                    "frac": achieved / peaks["bf16_tflops"], "traffic": traffic,
                    "peak_source": f"{peaks['source']} burst cuBLAS bf16 (MEASURED_PEAKS.json)",
                    "kernel": "attn_jvp_fwd_kernel", "kernel_ms": kernel_ms, "flops_per_launch": flops,
                    "frac_of_sustained": achieved / peaks["bf16_tflops_sustained"] if peaks["bf16_tflops_sustained"] else None,
                    "frac_of_datasheet": achieved / DATASHEET_BF16_TFLOPS,
                    "algorithmic_bytes": algorithmic_bytes(w),
                    "traffic_source": f"ncu capture on {cap['workload']} scaled by algorithmic bytes"
                                      if cap["workload"] != w.name else f"ncu capture on {w.name}",
                    "sm_cycles_per_key_tile": cycles_per_tile,
                    "mma_cycles_per_key_tile_ideal": (w.executed_flops / (w.B * w.H * w.Lq * w.Lk * w.D)) * 128 * 64 * w.D / 8192.0}
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
                "config": workload_config(w, extra=dict(({"splits": args.splits} if args.splits > 1 else {}),
                                                        **(cp_note or {}))),
                "clocks": clocks, "e2e": e2e, "gpu_launches": args.steps * (2 if args.splits > 1 else 1),
                "roofline": roofline,
                "jvp_over_fwd": (kernel_ms / fwd_ms) if fwd_ms else None, "fwd_only_ms": fwd_ms,
                "per_launch_ms": {"median": statistics.median(per_launch), "best": min(per_launch)}}
        if world == 1 and not args.no_cpu_baseline:
            cb = time_oracle(w, x_host, 15.0)
            line["cpu_baseline"] = {k: cb[k] for k in ("value", "unit", "cores", "kind", "sample")}
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
