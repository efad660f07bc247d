#!/usr/bin/env python
"""Benchmark of the APMSqueeze compression-phase step on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config IDX] [--impl ours|reference]

A step is one pass of the whole hot path (worker momentum + error-compensated 1-bit
compression for all n simulated workers, server average + recompression, model update) over
one set of n synthetic gradients.  Default workload: the BERT-Large-shaped parameter set,
n = 16 workers, chunk = 32768 (the configuration the metric is quoted on).  Gradients are
resident in HBM before the timed region (a ring of two distinct sets); the working set of a
step (~73 GB) is far larger than L2, so no flush is needed between steps.

Prints ONE JSON line.  With --gpus N > 1 (launched by torchrun) every rank runs an independent
replica of the same single-GPU job - the measured path keeps all n workers on one GPU - and the
value is the aggregate over ranks, timed as the maximum over ranks.

--path sharded | peer (under torchrun) runs the paper's own layout instead: the workload's n workers
are split over the processes, one GPU each, every process serves a range of chunks, and the 1-bit
messages are exchanged (Section 3.3 steps 3 and 5) over torch.distributed (sharded) or by the server
kernel's own loads from the peers' mapped workspaces (peer).  The total work is fixed ("scaling": "strong").
--one-gpu puts every process on cuda:0 (peer form only; host flags over gloo): the code path of a
one-process-per-GPU run where only one GPU is at hand.

--impl reference times the CPU oracle (oracle/) on a bounded sample of the same workload on the
host cores; it is a deliberately plain program, reported as a baseline.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "compressed_step_worker_elements_per_s"
UNIT = "worker-elements/s"

# DRAM traffic of the worker kernel measured once with ncu (dram__bytes_read.sum +
# dram__bytes_write.sum per launch) on a smaller case of the same kernel, in bytes per
# worker-element; scaled by n*d for the benchmarked launch.  Source: profiles/*.md.
NCU_WORKER_TRAFFIC_BYTES_PER_WORKER_ELEMENT = 11.96    # k_worker_fine, profiles/k_worker_fine_small_case.md
# The fused server + update kernel, same kind of capture at n = 8 workers (profiles/k_server_staged_small_case.md):
# 19.49 B per element; each further worker adds its sign words, 1/8 B per element (the traffic grows in proportion).
NCU_SERVER_FUSED_TRAFFIC_BYTES_PER_ELEMENT_N8 = 19.49


def algorithmic_bytes(d: int, n: int, chunk: int, grad_bytes: int = 4) -> dict:
    """Bytes each kernel must move per step (state kept as compensated vectors + messages)."""
    C = -(-d // chunk)
    W4 = 4 * -(-d // 32)
    worker = n * ((8 + grad_bytes) * d + W4) + W4 + n * 8 * C + 4 * C      # g, z read, z write, bits out; Bbar once; scales
    server = n * (W4 + 4 * C) + 8 * d + W4 + 8 * C           # n bit streams + scales in; zbar r/w; Bbar, Sbar
    apply_ = W4 + 4 * C + 12 * d                             # Bbar, Sbar, v, x in; x out
    return {"worker": worker, "server": server, "apply": apply_, "step": worker + server + apply_,
            "warmup_adam": (grad_bytes * n + 24) * d}


def measured_peaks() -> dict:
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            p = json.load(fh)
        return {"hbm_gbs": float(p["hbm_gbs"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs (read-only)."""

    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown",
               0x40: "hw_thermal_slowdown", 0x80: "hw_power_brake_slowdown", 0x2: "applications_clocks_setting"}

    def __init__(self, index: int, period_s: float = 0.02):
        self.index, self.period = index, period_s
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None

    def __enter__(self):
        try:
            import pynvml

            pynvml.nvmlInit()
            vis = os.environ.get("CUDA_VISIBLE_DEVICES")
            phys = self.index
            if vis:
                ids = [v for v in vis.split(",") if v.strip()]
                if self.index < len(ids) and ids[self.index].strip().isdigit():
                    phys = int(ids[self.index])
            h = pynvml.nvmlDeviceGetHandleByIndex(phys)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(h, pynvml.NVML_CLOCK_SM))

            def loop():
                while not self._stop.is_set():
                    try:
                        self.samples.append(int(pynvml.nvmlDeviceGetClockInfo(h, pynvml.NVML_CLOCK_SM)))
                        mask = int(pynvml.nvmlDeviceGetCurrentClocksThrottleReasons(h))
                        for bit, name in self.REASONS.items():
                            if mask & bit:
                                self.reasons.add(name)
                    except Exception:
                        pass
                    self._stop.wait(self.period)

            self._thread = threading.Thread(target=loop, daemon=True)
            self._thread.start()
        except Exception:
            self._thread = None
        return self

    def __exit__(self, *exc):
        self._stop.set()
        if self._thread:
            self._thread.join(timeout=2)

    def summary(self) -> dict:
        return {"sm_mhz": statistics.median(self.samples) if self.samples else None,
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


def max_over_ranks(seconds: float, dist) -> float:
    """Slowest rank's time (a job is as fast as its slowest rank)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return seconds
    import torch

    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([seconds], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, dist) -> float:
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return value
    import torch

    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([value], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


# ------------------------------------------------------------------------------------------ CPU oracle leg

def cpu_model() -> str:
    try:
        with open("/proc/cpuinfo") as f:
            for line in f:
                if line.lower().startswith("model name"):
                    return line.split(":", 1)[1].strip()
    except OSError:
        pass
    return "unknown"


def oracle_sample_workload(w, max_chunks: int = 48):
    from paper_2008_11343_b200 import workloads as wl

    chunks = min(max_chunks, w.n_chunks)
    return wl.sliced(w, min(w.d, chunks * w.chunk), name=f"{w.name}: first {chunks} chunks")


def time_oracle(w, steps: int, warmup: int, budget_s: float = 20.0) -> dict:
    """The CPU oracle, as it stands, on the first chunks of the workload, all host cores."""
    from oracle import apms_oracle as ao
    from paper_2008_11343_b200 import workloads as wl

    ws = oracle_sample_workload(w)
    orc = ao.Oracle(ws.d, ws.n, ws.beta1, ws.beta2, ws.eps, ws.lr, ws.chunk)
    threads = orc.max_threads()
    orc.set_threads(threads)
    orc.set_params(wl.initial_params(ws))
    ring = [wl.host_gradients(ws, s) for s in range(2)]
    orc.warmup_step(ring[0])
    orc.warmup_step(ring[1])
    orc.freeze_v()
    for k in range(max(1, warmup)):
        orc.compressed_step(ring[k % 2])
    times = []
    t_begin = time.perf_counter()
    for k in range(steps):
        t0 = time.perf_counter()
        orc.compressed_step(ring[k % 2])
        times.append(time.perf_counter() - t0)
        if time.perf_counter() - t_begin > budget_s and len(times) >= 3:
            break
    per_step = sum(times) / len(times)
    # the same sample on one thread (a few steps), for the per-core rate
    orc.set_threads(1)
    single = []
    t_begin = time.perf_counter()
    for k in range(3):
        t0 = time.perf_counter()
        orc.compressed_step(ring[k % 2])
        single.append(time.perf_counter() - t0)
        if time.perf_counter() - t_begin > budget_s / 2:
            break
    per_step_1 = sum(single) / len(single)
    return {"value": ws.d * ws.n / per_step, "unit": UNIT, "cores": threads, "kind": "oracle",
            "sample": f"{ws.name} (d={ws.d}, n={ws.n}, chunk={ws.chunk}), {len(times)} steps, "
                      f"{per_step * 1e3:.1f} ms/step, OpenMP over chunks",
            "ms_per_step": per_step * 1e3, "steps": len(times),
            "single_thread_value": ws.d * ws.n / per_step_1, "cpu_model": cpu_model()}


# ------------------------------------------------------------------------------------------ GPU leg

def measure(w, args, rank, world, local_rank, dist, want_adam=False, want_e2e=True) -> dict:
    """Set up one workload on this rank's GPU and time K compressed steps (device-resident
    gradients, CUDA events on the context's stream), optionally the Adam step and the e2e path."""
    import torch

    from paper_2008_11343_b200 import binding as B
    from paper_2008_11343_b200 import workloads as wl

    dev = torch.device("cuda", local_rank)
    split = args.path in ("sharded", "peer")          # the workload's workers are split over the processes
    n_total = w.n
    if split:
        assert n_total % world == 0, "the worker count must be a multiple of the number of processes"
        w = w.with_(n=n_total // world)
    ctx = B.Context(w.d, w.n, w.beta1, w.beta2, w.eps, w.lr, w.chunk, device=f"cuda:{local_rank}",
                    library_workspace=(args.path == "peer" and args.compressor == "onebit"))   # top-k: the peers share receive rows, not workspaces
    if args.compressor == "topk":
        ctx.set_compressor(B.COMPRESSOR_TOPK, args.topk_fraction)
    x0 = torch.empty(w.d, dtype=torch.float32, device=dev).normal_(0.0, w.x0_std)
    ctx.set_params(x0)
    del x0
    gdt = getattr(torch, args.grad_dtype)
    gbytes = 4 if gdt == torch.float32 else 2
    ring = []
    scratch = torch.empty(w.d, dtype=torch.float32, device=dev) if gbytes == 2 else None
    for r in range(2):
        gs = [torch.empty(w.d, dtype=gdt, device=dev) for _ in range(w.n)]
        for i in range(w.n):
            if scratch is None:
                wl.device_gradient(w, r + 1000 * rank, i, gs[i])
            else:                                    # drawn in binary32, rounded once to the 16-bit type
                wl.device_gradient(w, r + 1000 * rank, i, scratch)
                gs[i].copy_(scratch)
        ring.append(gs)
    del scratch
    torch.cuda.synchronize()
    group = dist if world > 1 else None

    # warmup phase (timed alone when asked), phase switch, first compressed step
    adam = None
    for k in range(3):
        ctx.warmup_step(ring[k % 2])
    if want_adam:
        ctx.set_timing(True)
        for k in range(10):
            ctx.warmup_step(ring[k % 2])
        ms, cnt = ctx.kernel_time(B.KERNEL_WARMUP_ADAM)
        ctx.set_timing(False)
        ab = algorithmic_bytes(w.d, w.n, w.chunk, gbytes)["warmup_adam"]
        adam = {"ms_per_step": ms / cnt, "achieved_gbs": ab / (ms / cnt * 1e-3) / 1e9,
                "worker_elements_per_s": w.d * w.n / (ms / cnt * 1e-3)}
    ctx.freeze_v()
    if args.path == "phases":
        # the step as a one-process-per-GPU run makes it (worker phase, server phase over rows given by address,
        # apply phase), here with one process that serves every chunk from its own workers' messages
        own_bits = [ctx.message_ptrs(i)[0] for i in range(w.n)]
        own_scales = [ctx.message_ptrs(i)[1] for i in range(w.n)]

        def step(gs):
            ctx.worker_phase(gs)
            ctx.server_phase_rows(own_bits, own_scales, 0, ctx.C)
            ctx.apply_phase()
    elif split:
        from paper_2008_11343_b200 import sharded

        stepper = (sharded.PeerShardedStep if args.path == "peer" else sharded.ShardedStep)(ctx)
        step = stepper.step
    else:
        step = ctx.compressed_step
    step(ring[0])                            # reads the binary32 momentum once; not representative
    for k in range(args.warmup):
        step(ring[(k + 1) % 2])
    torch.cuda.synchronize()

    # timed region: K steps between two events on the context's stream
    ctx.set_timing(True)
    for kid in range(len(B.KERNEL_NAMES)):
        ctx.kernel_time(kid)
    if args.compressor == "topk":
        ctx.topk_route_counts()                        # reset: the counts below are those of the timed steps
    launches0 = ctx.launch_count
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    with ClockSampler(local_rank) as clocks:
        marks = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps - 1)]
        e0.record(ctx.stream)
        for k in range(args.steps):
            step(ring[k % 2])
            if k < args.steps - 1:
                marks[k].record(ctx.stream)          # per-step times (min, median); the value comes from e0..e1
        e1.record(ctx.stream)
        torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    seconds = max_over_ranks(e0.elapsed_time(e1) * 1e-3, group)
    edges = [e0] + marks + [e1]
    per_step_ms = sorted(a.elapsed_time(b) for a, b in zip(edges, edges[1:]))
    launches = ctx.launch_count - launches0
    kernel_ms = {}
    for kid, name in enumerate(B.KERNEL_NAMES):
        ms, cnt = ctx.kernel_time(kid)
        if cnt:
            kernel_ms[name] = ms / cnt
    ctx.set_timing(False)
    routes = None
    if args.compressor == "topk":                     # how the chunks' selections were settled (exact on every route)
        names = ("predicted_list", "two_passes", "general", "missed_above", "missed_below", "missed_overflow")
        wr, sr = ctx.topk_route_counts()
        routes = {"worker": dict(zip(names, wr)), "server": dict(zip(names, sr))}
    work = n_total if split else world * w.n          # worker vectors the whole job compresses per step
    out = {"ms_per_step": seconds * 1e3 / args.steps, "value": work * w.d * args.steps / seconds,
           "ms_per_step_min": per_step_ms[0], "ms_per_step_median": per_step_ms[len(per_step_ms) // 2],
           "kernel_ms": kernel_ms, "launches": launches, "clocks": clocks.summary(), "adam": adam, "e2e": None,
           "topk_routes": routes}

    # end to end through the host-gradient entry point: H2D of the n gradients and D2H of x
    # inside the timed region, every step
    if split:
        out["wire_bytes_per_step"] = stepper.wire_bytes_per_step()
        stepper.close() if args.path == "peer" else None
    if want_e2e and not split:
        try:
            host = [torch.empty(w.d, dtype=gdt).pin_memory() for _ in range(w.n)]
            for i in range(w.n):
                host[i].copy_(ring[0][i])
            x_host = torch.empty(w.d, dtype=torch.float32).pin_memory()
            torch.cuda.synchronize()
            ctx.compressed_step_host(host, x_host)
            if world > 1:
                dist.barrier()
            t0 = time.perf_counter()
            e0.record(ctx.stream)
            for _ in range(args.e2e_steps):
                ctx.compressed_step_host(host, x_host)
            e1.record(ctx.stream)
            torch.cuda.synchronize()
            wall = time.perf_counter() - t0
            secs = max_over_ranks(max(e0.elapsed_time(e1) * 1e-3, wall), group)
            out["e2e"] = {"value": world * w.d * w.n * args.e2e_steps / secs, "unit": UNIT,
                          "h2d_bytes_per_step": gbytes * w.d * w.n, "d2h_bytes_per_step": 4 * w.d,
                          "ms_per_step": secs * 1e3 / args.e2e_steps, "steps": args.e2e_steps,
                          "api": "apms_compressed_step_host (pinned host gradients in, x out)"}
            del host, x_host
        except RuntimeError as exc:      # e.g. not enough host memory to pin n*d floats
            out["e2e"] = {"value": None, "unit": UNIT, "error": str(exc)[:200]}
    ctx.close()
    del ring, ctx
    torch.cuda.empty_cache()
    return out


# ------------------------------------------------------------------------------------------ main

def main(argv=None) -> int:
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--config", type=int, default=3, help="workload index (3 = BERT-Large-shaped, n=16)")
    ap.add_argument("--n", type=int, default=None, help="override the number of simulated workers")
    ap.add_argument("--chunk", type=int, default=None, help="override the chunk length")
    ap.add_argument("--d", type=int, default=None, help="use only the first d elements of the parameter set")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--compressor", default="onebit", choices=["onebit", "topk"],
                    help="the compression operator (the configurations of record use the 1-bit compressor)")
    ap.add_argument("--topk-fraction", type=float, default=0.01)
    ap.add_argument("--path", default="whole", choices=["whole", "phases", "sharded", "peer"],
                    help="whole: apms_compressed_step (the configurations of record); phases: the same step through "
                         "apms_worker_phase / apms_server_phase_rows / apms_apply_phase (1-bit compressor only); "
                         "sharded / peer: the workers split over the processes of a torchrun launch, messages exchanged")
    ap.add_argument("--one-gpu", action="store_true", help="every process on cuda:0 (--path peer only)")
    ap.add_argument("--grad-dtype", default="float32", choices=["float32", "bfloat16", "float16"],
                    help="element type of the gradient arrays (the configurations of record use float32)")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--adam", action="store_true", help="also time the warmup-phase Adam step alone")
    ap.add_argument("--sweep", action="store_true",
                    help="n in {2,4,8,16,32} x chunk in {1K,4K,16K,64K} on the chosen parameter set")
    args = ap.parse_args(argv)
    if args.warmup < 3:
        args.warmup = 3

    from paper_2008_11343_b200 import workloads as wl

    w = wl.config(args.config)
    if args.d:
        w = wl.sliced(w, args.d)
    if args.n:
        w = w.with_(n=args.n)
    if args.chunk:
        w = w.with_(chunk=args.chunk)
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = 0 if args.one_gpu else int(os.environ.get("LOCAL_RANK", "0"))
    split = args.path in ("sharded", "peer")
    if args.one_gpu and args.path != "peer":
        raise SystemExit("--one-gpu exists for --path peer only (NCCL wants one GPU per process)")
    config = {"workload": f"{w.name}: d={w.d}, n={w.n} simulated workers, chunk={w.chunk}, {w.dist} gradients",
              "d": w.d, "n_workers": w.n, "chunk": w.chunk, "gradient_dtype": args.grad_dtype,
              "compressor": args.compressor if args.compressor == "onebit" else f"topk {args.topk_fraction}",
              "path": args.path,
              "parallelism": (f"{world} processes x {w.n // world} workers, {args.path} exchange"
                              + (", all on one GPU" if args.one_gpu else "")) if split else f"replicas x{world}",
              "l2_policy": "inputs_exceed_l2" if 12 * w.d * w.n > (256 << 20) else "l2_resident",
              "gradient_ring": 2}

    if args.impl == "reference":
        if rank != 0:
            return 0
        r = time_oracle(w, steps=args.steps, warmup=args.warmup, budget_s=90.0)
        line = {"impl": "reference", "metric": METRIC, "value": r["value"], "unit": UNIT, "n_gpus": args.gpus,
                "steps": r["steps"], "warmup": args.warmup, "ms_per_step": r["ms_per_step"],
                "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
                "data": "synthetic", "config": config,
                "cpu_baseline": {k: r[k] for k in ("value", "unit", "cores", "kind", "sample", "single_thread_value", "cpu_model")},
                "e2e": {"value": r["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
                "gpu_launches": 0}
        print(json.dumps(line))
        return 0

    import torch
    import torch.distributed as dist

    from paper_2008_11343_b200 import build as libbuild

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the path has no CPU fallback")
    if libbuild.is_stale():
        libbuild.build()
    torch.cuda.set_device(local_rank)
    if world > 1 or split:
        if args.one_gpu or world == 1:
            if world == 1 and "MASTER_ADDR" not in os.environ:      # a plain `python bench.py --path sharded`
                import socket

                with socket.socket() as sock:
                    sock.bind(("127.0.0.1", 0))
                    port = sock.getsockname()[1]
                os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK="0", WORLD_SIZE="1")
            dist.init_process_group("gloo")           # handles and host flags only; every exchange is a load or a store
        else:
            dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    peaks = measured_peaks()

    if args.sweep:
        rows = []
        for n in (2, 4, 8, 16, 32):
            for chunk in (1024, 4096, 16384, 65536):
                ws = w.with_(n=n, chunk=chunk)
                m = measure(ws, args, rank, world, local_rank, dist, want_adam=(chunk == 1024), want_e2e=False)
                ab = algorithmic_bytes(ws.d, n, chunk, 4 if args.grad_dtype == "float32" else 2)
                gbs = ab["step"] / (m["ms_per_step"] * 1e-3) / 1e9
                row = {"n": n, "chunk": chunk, "ms_per_step": m["ms_per_step"], "value": m["value"],
                       "step_gbs": gbs, "step_frac": gbs / peaks["hbm_gbs"], "kernel_ms": m["kernel_ms"]}
                if m["adam"]:
                    row["warmup_adam"] = m["adam"]
                rows.append(row)
        if rank == 0:
            print(json.dumps({"sweep": rows, "workload": w.name, "d": w.d, "unit": UNIT, "peak_gbs": peaks["hbm_gbs"],
                              "peak_source": peaks["source"]}))
        if world > 1:
            dist.destroy_process_group()
        return 0

    m = measure(w, args, rank, world, local_rank, dist, want_adam=args.adam, want_e2e=not args.no_e2e)
    ms_per_step, kernel_ms = m["ms_per_step"], m["kernel_ms"]
    n_local = w.n // world if split else w.n           # what one process's kernels move
    ab = algorithmic_bytes(w.d, n_local, w.chunk, 4 if args.grad_dtype == "float32" else 2)
    if split:                                          # a process serves 1 / world of the chunks, from all n workers' rows
        full = algorithmic_bytes(w.d, w.n, w.chunk, 4 if args.grad_dtype == "float32" else 2)
        ab["server"] = full["server"] // world
        ab["step"] = ab["worker"] + ab["server"] + ab["apply"]
    if args.compressor == "topk":
        # g, z read, z write and both masks per worker, the binary32 momentum once; masks, the kept values,
        # zbar read + write, new momentum, v, x read, x write, server mask
        gb = 4 if args.grad_dtype == "float32" else 2
        ab["worker"] = w.n * ((8 + gb) * w.d + w.d // 4) + 4 * w.d
        ab["server"] = w.n * (w.d // 8 + int(4 * args.topk_fraction * w.d)) + (8 + 4 + 12) * w.d + w.d // 8
        ab["step"] = ab["worker"] + ab["server"]
    elif "apply" not in kernel_ms:          # steps 4-6 ran as one kernel: it moves both kernels' bytes (Bbar is not re-read)
        ab["server"] = ab["server"] + ab["apply"] - 4 * -(-w.d // 32)
        ab["step"] = ab["worker"] + ab["server"]
    wk_gbs = ab["worker"] / (kernel_ms["worker"] * 1e-3) / 1e9
    step_gbs = ab["step"] / (ms_per_step * 1e-3) / 1e9
    # the ncu figures are those of k_worker_fine (chunks of 512 elements and more) and of the per-chunk fused server kernel
    traffic = (NCU_WORKER_TRAFFIC_BYTES_PER_WORKER_ELEMENT * w.d * n_local
               if NCU_WORKER_TRAFFIC_BYTES_PER_WORKER_ELEMENT and args.grad_dtype == "float32"
               and args.compressor == "onebit" and w.chunk >= 512 else None)
    fused = args.compressor == "onebit" and "apply" not in kernel_ms and not split and 2048 <= w.chunk <= 65536
    traffic_by_kernel = {"worker": traffic,
                         "server": ((NCU_SERVER_FUSED_TRAFFIC_BYTES_PER_ELEMENT_N8 + (w.n - 8) / 8.0) * w.d
                                    if fused and args.grad_dtype == "float32" else None)}
    roofline = {"bound": "hbm", "kernel": "k_worker", "achieved": wk_gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": wk_gbs / peaks["hbm_gbs"], "peak_source": peaks["source"], "traffic": traffic,
                "traffic_by_kernel": traffic_by_kernel,
                "algorithmic_bytes_per_launch": ab["worker"],
                "whole_step": {"algorithmic_bytes": ab["step"], "achieved": step_gbs,
                               "frac": step_gbs / peaks["hbm_gbs"], "frac_of_8TBs_nominal": step_gbs / 8000.0},
                "kernel_ms": kernel_ms,
                "kernel_gbs": {k: ab[k] / (v * 1e-3) / 1e9 for k, v in kernel_ms.items() if k in ab}}

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu = time_oracle(w, steps=50, warmup=1, budget_s=15.0)
        cpu = {k: cpu[k] for k in ("value", "unit", "cores", "kind", "sample", "single_thread_value", "cpu_model")}

    if rank == 0:
        line = {"metric": METRIC, "value": m["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
                "scaling": "strong" if split else "weak",
                "vs_baseline": None, "dtype": "f32", "data": "synthetic", "config": config,
                "roofline": roofline, "cpu_baseline": cpu, "e2e": m["e2e"], "gpu_launches": m["launches"],
                "clocks": m["clocks"],
                "ms_per_step_min": m["ms_per_step_min"], "ms_per_step_median": m["ms_per_step_median"]}
        if m["adam"]:
            line["warmup_adam"] = m["adam"]
        if m.get("topk_routes"):
            line["topk_routes"] = m["topk_routes"]
        if "wire_bytes_per_step" in m:
            line["wire_bytes_per_step_per_process"] = m["wire_bytes_per_step"]
        print(json.dumps(line))
    if dist.is_initialized():
        dist.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
