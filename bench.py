#!/usr/bin/env python
"""Benchmark of the WP-SGD hot path on B200.

One "step" = one pass of the whole path over one synthetic batch: sample-stream kernel, the k
per-node SGD chains, and the weighted combination. Prints ONE JSON line (rank 0).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload 2|3|5|1] [--impl ours|reference]

N > 1 is launched with torch.distributed.run (one rank per GPU). Every rank then runs its own
set of nodes of a cluster that is N times larger (weak scaling) and the partial combinations are
added with one all-reduce of d floats, the only exchange the method has.

--impl reference times the CPU checker (plain single-threaded C++) on the host cores, on the same
workload, as the baseline this box can offer; rank 0 only.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

METRIC = "sgd_sample_updates_per_s"
UNIT = "sample-updates/s"
FALLBACK_HBM_GBS = 6650.0

# DRAM bytes (read + write) per launch of the chain kernel from an ncu capture, with the hash of the
# kernel sources the capture was taken from; reported as null once the sources have changed.
NCU_TRAFFIC = {"config2": {"src_sha": "caf6ef3dd3dddded", "bytes_per_launch": 601684224}}


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--workload", type=int, default=2, help="benchmark configuration (default 2)")
    ap.add_argument("--rho", type=float, default=4.0, help="speed ratio of workload 5")
    ap.add_argument("--small", action="store_true", help="scaled-down copy of the workload (profiling captures)")
    ap.add_argument("--rows", type=int, default=0, help="rows per node override (smaller device footprint for profiler captures)")
    ap.add_argument("--also", default="3,5,4", help="further workloads measured after the main one at 1 GPU and reported "
                    "under other_workloads (device-resident timing only); empty to skip")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--option", action="append", default=[], help="name=value passed to wpsgd_set_option")
    return ap.parse_args()


def kernel_src_sha() -> str:
    h = hashlib.sha256()
    csrc = os.path.join(ROOT, "paper_1708_04801_b200", "csrc")
    for f in sorted(os.listdir(csrc)):
        h.update(open(os.path.join(csrc, f), "rb").read())
    return h.hexdigest()[:16]


def make_workload(args, rank: int, device):
    import wpsgd_inputs as wi

    cfg = args.workload
    seed_shift = 1000 * rank
    if args.small:
        wl = wi.small(cfg, device=device)
    elif cfg == 5:
        kw = {"m": args.rows} if args.rows else {}
        wl = wi.config5(rho=args.rho, device=device, data_seed=1005 + seed_shift, **kw)
    elif cfg in (1, 2, 3, 4):
        kw = {"m": args.rows} if args.rows else {}
        wl = wi.FULL[cfg](device=device, data_seed=1000 + cfg + seed_shift, **kw)
    else:
        raise SystemExit(f"unknown workload {cfg}")
    return wl


def describe(wl, args) -> str:
    kind = "csr" if wl.sparse else ("bf16" if wl.xtype == 1 else "fp32")
    loss = ["hinge", "logistic", "squared"][wl.loss]
    return (f"config{args.workload}{'-small' if args.small else ''}: k={wl.k} d={wl.d} {kind} {loss} "
            f"rows/node={int(wl.shard_off[1] - wl.shard_off[0])} steps={int(wl.n_steps.min())}..{int(wl.n_steps.max())} "
            f"total={wl.total_steps}")


def bytes_per_update(wl) -> float:
    """Algorithmic bytes one sample-update must move: the row, its label and its sample index."""
    if wl.sparse:
        nnz = float(wl.col_idx.numel()) / float(wl.y.numel())
        return 16.0 + nnz * 8.0 + nnz * 8.0  # row extents, (col, val), model read + write on the nonzeros
    es = 2 if wl.xtype == 1 else 4
    return wl.d * es + 4 + 4


class ClockSampler:
    """nvidia-smi clocks and throttle reasons while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.lines = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "100"], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._pump, daemon=True).start()
        except OSError:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            parts = [p.strip() for p in ln.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for nm, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def measure_other(P, args, cfg: int, dev, peak: float):
    """Device-resident timing of one more workload: chains + combination, 3 warm-up and 3 timed steps."""
    import argparse as _ap

    import torch

    a2 = _ap.Namespace(**vars(args))
    a2.workload, a2.small, a2.rows = cfg, False, 0
    wl = make_workload(a2, 0, dev)
    with P.Context(wl.k, wl.d, device=dev.index) as ctx:
        ctx.set_option("timing", 1)
        v = torch.empty(wl.d, dtype=torch.float32, device=dev)
        for _ in range(3):
            ctx.run_workload(wl)
            ctx.combine(out=v)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        chain = []
        e0.record()
        for _ in range(3):
            ctx.run_workload(wl)
            ctx.combine(out=v)
        e1.record()
        torch.cuda.synchronize()
        for _ in range(3):
            ctx.run_workload(wl)
            chain.append(ctx.last_chain_ms())
        ctx.check()
    ms = e0.elapsed_time(e1) / 3
    cms = float(np.mean(chain))
    achieved = bytes_per_update(wl) * wl.total_steps / (cms * 1e-3) / 1e9
    out = {"workload": describe(wl, a2), "value": wl.total_steps / (ms * 1e-3), "unit": UNIT, "ms_per_step": ms,
           "steps": 3, "warmup": 3, "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                                                 "frac": achieved / peak, "kernel_ms": cms,
                                                 "bytes_per_sample_update": bytes_per_update(wl)}}
    del wl
    torch.cuda.empty_cache()
    return out


def cpu_baseline(wl_cpu, min_seconds=10.0, max_passes=30):
    """The CPU checker as it stands, single-threaded, on whole passes of the same workload."""
    import oracle

    oracle.build()
    t0 = time.perf_counter()
    passes = 0
    while True:
        oracle.solve(wl_cpu)
        passes += 1
        el = time.perf_counter() - t0
        if el >= min_seconds or passes >= max_passes:
            break
    return {"value": wl_cpu.total_steps * passes / el, "unit": UNIT, "cores": 1, "kind": "oracle",
            "sample": f"{passes} full pass(es) of the workload ({wl_cpu.total_steps} sample-updates each) in {el:.1f} s"}


def cpu_sample_of(wl_cpu, budget_updates: float):
    """A bounded copy of a workload that is too large for the host: same k, d and rows, step counts
    scaled down so that about budget_updates sample-updates remain."""
    import dataclasses

    f = min(1.0, budget_updates / max(1, wl_cpu.total_steps))
    if f >= 1.0:
        return wl_cpu, "the full workload"
    n = np.maximum(1, np.floor(wl_cpu.n_steps * f)).astype(np.int64)
    return dataclasses.replace(wl_cpu, n_steps=n), f"step counts scaled by {f:.4f} (same k, d, rows)"


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    import wpsgd_inputs as wi  # noqa: F401

    oracle.build()
    wl = make_workload(args, 0, "cpu") if args.workload in (1, 2) or args.small else None
    note = "the full workload"
    if wl is None:
        # large workloads: generate a host-sized copy with fewer rows per node and fewer steps
        import wpsgd_inputs as wi2

        if args.workload == 3:
            wl = wi2.config3(m=1024)
            note = "rows/node reduced to 1024 for host memory"
        elif args.workload == 4:
            wl = wi2.config4(m=4096)
            note = "rows/node reduced to 4096 for host memory"
        else:
            wl = wi2.config5(rho=args.rho)
    wl, n2 = cpu_sample_of(wl, 2.0e5 if not wl.sparse else 2.0e6)
    if n2 != "the full workload":
        note = note + "; " + n2 if note != "the full workload" else n2
    for _ in range(args.warmup):
        oracle.solve(wl)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle.solve(wl)
    el = time.perf_counter() - t0
    value = wl.total_steps * args.steps / el
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": 1e3 * el / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": describe(wl, args), "sample": note},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": note},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
        return

    import torch
    import torch.distributed as dist

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if world != args.gpus and world > 1:
        raise SystemExit(f"--gpus {args.gpus} but WORLD_SIZE={world}")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    from paper_1708_04801_b200 import build as lib_build

    if rank == 0 or not os.path.exists(lib_build.LIB):
        lib_build.build()
    if world > 1:
        dist.barrier()
    import paper_1708_04801_b200 as P
    from paper_1708_04801_b200 import multi

    # ---- workload: host copy where it fits (CPU baseline, host-buffer path), device copy for the kernels
    host_sized = args.small or args.workload in (1, 2, 5)
    wl_cpu = make_workload(args, rank, "cpu") if host_sized else None
    wl = wl_cpu.to(dev) if wl_cpu is not None else make_workload(args, rank, dev)
    # the cluster has world * k nodes with the same pattern of step counts; this rank holds k of them
    n_global = np.tile(wl.n_steps, world)
    owned = np.arange(rank * wl.k, (rank + 1) * wl.k)
    w_local = multi.local_weights(n_global, owned, wl.eta0, wl.sched, wl.lam)

    ctx = P.Context(wl.k, wl.d, device=local_rank)
    ctx.set_node_ids(owned)
    ctx.set_option("timing", 1)
    for opt in args.option:
        name, val = opt.split("=")
        ctx.set_option(name, int(val))
    v = torch.empty(wl.d, dtype=torch.float32, device=dev)

    def step():
        ctx.run_workload(wl)
        ctx.combine_weighted(w_local, out=v)
        multi.allreduce_sum(v)

    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize()
    ctx.check()

    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    launches0 = ctx.launch_count()
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
    chain_ms = []
    ev[0].record()
    for i in range(args.steps):
        step()
        ev[i + 1].record()
    torch.cuda.synchronize()
    # per-launch device time of the chain kernel: a second pass of the same steps, read back one by one
    total_ms = ev[0].elapsed_time(ev[-1])
    launches = ctx.launch_count() - launches0
    for i in range(min(args.steps, 10)):
        ctx.run_workload(wl)
        chain_ms.append(ctx.last_chain_ms())
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    ctx.check()
    if world > 1:
        t = torch.tensor([total_ms], device=dev, dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        total_ms = float(t.item())
    updates_all = float(wl.total_steps) * world
    value = updates_all * args.steps / (total_ms * 1e-3)

    # ---- end to end through the host-buffer entry point (dense workloads that fit the host) ----------------
    e2e = None
    if wl_cpu is not None and not wl.sparse:
        Xh, yh = wl_cpu.X.pin_memory(), wl_cpu.y.pin_memory()
        vh = torch.empty(wl.d, dtype=torch.float32).pin_memory()
        n_e2e = max(3, min(args.steps, 10))
        for _ in range(2):
            ctx.solve_host(Xh, yh, wl.shard_off, wl.n_steps, wl.eta0, wl.sched, wl.lam, wl.loss, wl.seed, out=vh)
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(n_e2e):
            ctx.solve_host(Xh, yh, wl.shard_off, wl.n_steps, wl.eta0, wl.sched, wl.lam, wl.loss, wl.seed, out=vh)
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1)
        if world > 1:
            t = torch.tensor([ms], device=dev, dtype=torch.float64)
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            ms = float(t.item())
        e2e = {"value": updates_all * n_e2e / (ms * 1e-3), "unit": UNIT,
               "h2d_bytes_per_step": int(Xh.numel() * Xh.element_size() + yh.numel() * 4) * world,
               "d2h_bytes_per_step": int(wl.d * 4) * world, "steps": n_e2e}

    clocks = sampler.stop() if rank == 0 else None  # sampled across the device-timed and the end-to-end loops
    if rank == 0:
        peaks_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
        if os.path.exists(peaks_path):
            peak, peak_src = float(json.load(open(peaks_path))["hbm_gbs"]), "measured"
        else:
            peak, peak_src = FALLBACK_HBM_GBS, "fallback"
        chain = float(np.mean(chain_ms))
        alg_bytes = bytes_per_update(wl) * wl.total_steps
        achieved = alg_bytes / (chain * 1e-3) / 1e9
        tr = NCU_TRAFFIC.get(f"config{args.workload}", {})
        traffic = tr.get("bytes_per_launch") if tr.get("src_sha") == kernel_src_sha() and not args.small else None
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": total_ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic",
            "config": {"workload": describe(wl, args), "parallelism": f"nodes sharded over {world} GPU(s)",
                       "l2": "inputs larger than L2; no flush" if (wl.sparse or wl.X.numel() * wl.X.element_size() > 126e6)
                       else "inputs fit in L2 (correctness-sized workload)"},
            "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches),
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                         "traffic": traffic, "peak_source": f"of {peak_src}", "kernel": "chain kernel (per-node SGD loops)",
                         "kernel_ms": chain, "algorithmic_bytes_per_launch": alg_bytes,
                         "bytes_per_sample_update": bytes_per_update(wl)},
        }
        if not args.no_cpu_baseline:
            if wl_cpu is not None:
                line["cpu_baseline"] = cpu_baseline(wl_cpu)
            else:
                line["cpu_baseline"] = None
        if world == 1 and args.also and not args.small and not args.rows:
            ctx.destroy()
            del wl, v
            torch.cuda.empty_cache()
            others = []
            for tok in args.also.split(","):
                cfg = int(tok)
                if cfg == args.workload:
                    continue
                try:
                    others.append(measure_other(P, args, cfg, dev, peak))
                except Exception as exc:  # e.g. not enough device memory for the 32 GiB workload
                    others.append({"workload": f"config{cfg}", "error": str(exc)[:200]})
            line["other_workloads"] = others
        print(json.dumps(line), flush=True)
    ctx.destroy()
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
