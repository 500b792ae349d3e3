#!/usr/bin/env python
"""Benchmark of the WP-SGD hot path on B200.

One "step" = one pass of the whole path over one synthetic batch: sample-stream kernel, the k
per-node SGD chains, and the weighted combination. Prints ONE JSON line (rank 0).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload 3|2|5|4|1] [--impl ours|reference]

The headline workload is configuration 3 (k=128, d=4096 bf16, 32 GiB of rows): the largest of the five that
fits one GPU. At one GPU the other configurations (2, 5 at five speed ratios, 4) are measured after it
and reported under "other_workloads" in the same line.

N > 1 is launched with torch.distributed.run (one rank per GPU). The cluster then has N times the nodes
(the pattern of step counts repeated N times); the nodes are dealt to the ranks by longest processing
time, every rank runs its own nodes, and the partial combinations are added with one all-reduce of d
floats, the only exchange the method has.

--impl reference times the CPU checker (plain single-threaded C++) on the host cores, on a bounded
sample of the same workload, as the baseline this box can offer; rank 0 only.
"""
from __future__ import annotations

import argparse
import dataclasses
import hashlib
import json
import os
import subprocess
import sys
import threading
import time
from concurrent.futures import ThreadPoolExecutor

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

METRIC = "sgd_sample_updates_per_s"
UNIT = "sample-updates/s"
FALLBACK_HBM_GBS = 6650.0
N_SMS = 148

# DRAM bytes (read + write) per launch of the chain kernel from an ncu capture, with the hash of the
# kernel sources the capture was taken from; reported as null once the sources have changed.
NCU_TRAFFIC = {
    "config3": {"src_sha": "5464430f1e53acb2", "bytes_per_launch": 26347713776,
                "note": "captured with 2048 rows per node (2 GiB on the device): same step counts and kernel work per launch, no scaling"},
    "config5": {"src_sha": "5464430f1e53acb2", "bytes_per_launch": 15943503448, "note": "full-size capture"},
    "config4": {"src_sha": "5464430f1e53acb2", "bytes_per_launch": 4299267560, "note": "full-size capture"},
    "config2": {"src_sha": "5464430f1e53acb2", "bytes_per_launch": 604431360, "note": "full-size capture"},
}


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--workload", type=int, default=3, help="benchmark configuration (default 3)")
    ap.add_argument("--rho", type=float, default=4.0, help="speed ratio of workload 5")
    ap.add_argument("--small", action="store_true", help="scaled-down copy of the workload (profiling captures)")
    ap.add_argument("--rows", type=int, default=0, help="rows per node override (smaller device footprint for profiler captures)")
    ap.add_argument("--also", default="2,5,4", help="further workloads measured after the main one at 1 GPU and reported "
                    "under other_workloads; empty to skip")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--option", action="append", default=[], help="name=value passed to wpsgd_set_option")
    return ap.parse_args()


def kernel_src_sha() -> str:
    h = hashlib.sha256()
    csrc = os.path.join(ROOT, "paper_1708_04801_b200", "csrc")
    for f in sorted(os.listdir(csrc)):
        h.update(open(os.path.join(csrc, f), "rb").read())
    return h.hexdigest()[:16]


def make_workload(cfg: int, device, rho=4.0, small=False, rows=0, rank=0, k=None, n_steps=None):
    """Workload `cfg` on `device`. k / n_steps override the node count and step counts (multi-GPU sharding)."""
    import wpsgd_inputs as wi

    seed_shift = 1000 * rank
    if small:
        return wi.small(cfg, device=device)
    kw = {"m": rows} if rows else {}
    if k is not None:
        kw["k"] = int(k)
    if cfg == 5:
        wl = wi.config5(rho=rho, device=device, data_seed=1005 + seed_shift, **kw)
    elif cfg in (1, 2, 3, 4):
        wl = wi.FULL[cfg](device=device, data_seed=1000 + cfg + seed_shift, **kw)
    else:
        raise SystemExit(f"unknown workload {cfg}")
    if n_steps is not None:
        wl = dataclasses.replace(wl, n_steps=np.asarray(n_steps, dtype=np.int64))
    return wl


def describe(wl, cfg, small=False) -> str:
    kind = "csr" if wl.sparse else ("bf16" if wl.xtype == 1 else "fp32")
    loss = ["hinge", "logistic", "squared"][wl.loss]
    return (f"config{cfg}{'-small' if small else ''}: k={wl.k} d={wl.d} {kind} {loss} "
            f"rows/node={int(wl.shard_off[1] - wl.shard_off[0])} steps={int(wl.n_steps.min())}..{int(wl.n_steps.max())} "
            f"total={wl.total_steps}")


def bytes_per_update(wl) -> float:
    """Algorithmic bytes one sample-update must move: the row, its label and its sample index."""
    if wl.sparse:
        nnz = float(wl.col_idx.numel()) / float(wl.y.numel())
        return 16.0 + nnz * 8.0 + nnz * 8.0  # row extents, (col, val), model read + write on the nonzeros
    es = 2 if wl.xtype == 1 else 4
    return wl.d * es + 4 + 4


def input_bytes(wl) -> int:
    if wl.sparse:
        return int(wl.col_idx.numel() * 8 + wl.row_ptr.numel() * 8 + wl.y.numel() * 4)
    return int(wl.X.numel() * wl.X.element_size() + wl.y.numel() * 4)


def ctas_of(wl) -> int:
    """CTAs the default chain kernel of this workload launches (for the SM coverage figure)."""
    if wl.sparse:
        return wl.k
    chunks = wl.d // (8 if wl.xtype == 1 else 4)
    if wl.xtype != 1 and chunks >= 128:   # few wide fp32 chains: a cluster of 4 or 8 CTAs per node when the SMs allow
        c = 8
        while c > 1 and (wl.k * c > N_SMS or (chunks + c - 1) // c < 8):
            c //= 2
        if c >= 4 and (chunks + c - 1) // c <= 64:
            return wl.k * c
    if chunks <= 64:
        return (wl.k + 3) // 4            # four nodes (warps) per CTA
    if wl.xtype == 1 and chunks >= 256:
        c = 1
        while (chunks + c - 1) // c > 256 and c < 8:
            c *= 2
        return wl.k * c                   # cluster of c CTAs per node
    return wl.k


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
        return self

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


# ---- the CPU checker as a baseline ------------------------------------------------------------------------------
def cpu_sample_of(wl_cpu, budget_updates: float):
    """A bounded copy of a workload: same k, d and rows, step counts scaled down so that about
    budget_updates sample-updates remain."""
    f = min(1.0, budget_updates / max(1, wl_cpu.total_steps))
    if f >= 1.0:
        return wl_cpu, "all step counts"
    n = np.maximum(1, np.floor(wl_cpu.n_steps * f)).astype(np.int64)
    return dataclasses.replace(wl_cpu, n_steps=n), f"step counts scaled by {f:.4f}"


def host_copy_for_cpu(cfg: int, rho: float, small: bool):
    """Host-resident copy of a workload for the CPU checker, with fewer rows per node where the full rows do not
    fit or take minutes to generate on the host (same k, d and step counts)."""
    import wpsgd_inputs as wi

    if small:
        return wi.small(cfg), "scaled-down copy"
    if cfg == 3:
        return wi.config3(m=1024), "rows/node 1024 instead of 32768 (host memory)"
    if cfg == 4:
        return wi.config4(m=4096), "rows/node 4096 instead of 65536 (host generation time)"
    if cfg == 5:
        return wi.config5(rho=rho), "all rows"
    return wi.FULL[cfg](), "all rows"


def oracle_chains_one_node(wl, j):
    """The checker's chain of node j alone (its number still enters the sample stream)."""
    import oracle

    n = np.zeros(wl.k, dtype=np.int64)
    n[j] = wl.n_steps[j]
    if wl.sparse:
        return oracle.run_csr(wl.row_ptr, wl.col_idx, wl.val, wl.y, wl.shard_off, n, wl.d, wl.eta0, wl.sched, wl.lam,
                              wl.loss, wl.seed, wl.w0, one_node=j)
    return oracle.run_dense(wl.X, wl.y, wl.shard_off, n, wl.d, wl.eta0, wl.sched, wl.lam, wl.loss, wl.seed, wl.w0)[j]


def cpu_baseline(wl_cpu, note: str, seconds: float):
    """The CPU checker as it stands on a bounded sample: (i) its own single thread; (ii) the same function called
    for one node per host thread over all cores (nodes are independent until the combination)."""
    import oracle

    oracle.build()
    per_core = 0.6e6 if not wl_cpu.sparse else 6e6  # rough sample-updates/s of one core at d = 1024, for sizing only
    if not wl_cpu.sparse:
        per_core *= 1024.0 / max(64, wl_cpu.d)
    sample, how = cpu_sample_of(wl_cpu, per_core * seconds)
    t0 = time.perf_counter()
    oracle.solve(sample)
    el1 = time.perf_counter() - t0
    cores = os.cpu_count() or 1
    t0 = time.perf_counter()
    with ThreadPoolExecutor(max_workers=cores) as ex:
        W = list(ex.map(lambda j: oracle_chains_one_node(sample, j), range(sample.k)))
    wts, _, _ = oracle.weights(sample.n_steps, sample.eta0, sample.sched, sample.lam)
    oracle.combine(np.stack(W), wts)
    eln = time.perf_counter() - t0
    text = f"{sample.total_steps} sample-updates ({note}; {how})"
    return {"value": sample.total_steps / el1, "unit": UNIT, "cores": 1, "kind": "oracle",
            "sample": f"{text} in {el1:.1f} s on one core",
            "all_cores": {"value": sample.total_steps / eln, "unit": UNIT, "cores": min(cores, sample.k),
                          "host_cores": cores, "kind": "oracle, one node per thread",
                          "sample": f"{text} in {eln:.1f} s"}}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle

    oracle.build()
    wl, note = host_copy_for_cpu(args.workload, args.rho, args.small)
    wl, n2 = cpu_sample_of(wl, 2.0e5 * 1024.0 / max(64, wl.d) if not wl.sparse else 2.0e6)
    note = f"{note}; {n2}"
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
            "config": {"workload": describe(wl, args.workload, args.small), "sample": note},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": note},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ---- device measurements ------------------------------------------------------------------------------------------
def measure(P, multi, wl, cfg, dev, steps, warmup, peak, peak_src, options, world=1, weights=None, node_ids=None,
            small=False):
    """Warm-up, then `steps` timed passes (sample stream + chains + combination [+ all-reduce]); afterwards per-phase
    device times of up to 10 more passes. Returns (entry, ctx) with the context still open."""
    import torch
    import torch.distributed as dist

    ctx = P.Context(wl.k, wl.d, device=dev.index)
    if node_ids is not None:
        ctx.set_node_ids(node_ids)
    ctx.set_option("timing", 1)
    for name, val in options:
        ctx.set_option(name, val)
    v = torch.empty(wl.d, dtype=torch.float32, device=dev)

    def step():
        ctx.run_workload(wl)
        if weights is not None:
            ctx.combine_weighted(weights, out=v)
            multi.allreduce_sum(v)
        else:
            ctx.combine(out=v)

    for _ in range(max(warmup, 1)):
        step()
    torch.cuda.synchronize()
    ctx.check()
    sampler = ClockSampler(dev.index).start()
    launches0 = ctx.launch_count()
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        step()
    e1.record()
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    total_ms = e0.elapsed_time(e1)
    launches = ctx.launch_count() - launches0
    # phases, one pass at a time: run (plan upload + sample stream + chains), chains alone, combination
    run_ms, chain_ms, comb_ms = [], [], []
    for _ in range(min(max(steps, 3), 10)):
        a, b, c = (torch.cuda.Event(enable_timing=True) for _ in range(3))
        a.record()
        ctx.run_workload(wl)
        b.record()
        ctx.combine(out=v)
        c.record()
        torch.cuda.synchronize()
        run_ms.append(a.elapsed_time(b))
        comb_ms.append(b.elapsed_time(c))
        chain_ms.append(ctx.last_chain_ms())
    clocks = sampler.stop()
    ctx.check()
    if world > 1:
        t = torch.tensor([total_ms], device=dev, dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        total_ms = float(t.item())
    chain_med, chain_best = float(np.median(chain_ms)), float(np.min(chain_ms))
    alg_bytes = bytes_per_update(wl) * wl.total_steps
    achieved = alg_bytes / (chain_med * 1e-3) / 1e9
    ctas = ctas_of(wl)
    mhz = clocks.get("sm_mhz") or 1965.0
    longest = int(wl.n_steps.max())
    roof = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
            "traffic": None, "peak_source": f"of {peak_src}", "kernel": "chain kernel (per-node SGD loops)",
            "kernel_ms": chain_med, "kernel_ms_best": chain_best, "algorithmic_bytes_per_launch": alg_bytes,
            "bytes_per_sample_update": bytes_per_update(wl),
            # mean chain length over the longest: the busy share of a schedule that gives every chain its own SMs for
            # the whole launch (chains that take turns on the same SMs, as the cluster kernels' do, can exceed it);
            # and how much of the GPU the launch covers
            "mean_over_longest_chain": float(wl.total_steps) / float(wl.k * max(longest, 1)),
            "ctas": ctas, "sm_coverage": min(1.0, ctas / N_SMS),
            # the serial side of the same kernel: device cycles per sample-update of the longest chain
            "cycles_per_update_longest_chain": chain_med * 1e-3 * mhz * 1e6 / max(longest, 1)}
    # which side of the kernel holds it back: the memory system, or the dependent steps of one chain
    roof["limiter"] = ("chain latency: the longest chain's dependent steps, not a memory level"
                       if (roof["frac"] < 0.2 or ctas < N_SMS) else "dependent loop of a block and HBM together (see the profile)")
    tr = NCU_TRAFFIC.get(f"config{cfg}", {})
    # (config 5 was captured at speed ratio 4: the workload's name carries the ratio)
    if tr.get("src_sha") == kernel_src_sha() and not small and (cfg != 5 or wl.name == "config5_rho4"):
        roof["traffic"] = tr.get("bytes_per_launch")
        roof["traffic_note"] = tr.get("note")
    entry = {"workload": describe(wl, cfg, small), "value": float(wl.total_steps) * world * steps / (total_ms * 1e-3),
             "unit": UNIT, "ms_per_step": total_ms / steps, "steps": steps, "warmup": max(warmup, 1),
             "gpu_launches": int(launches), "clocks": clocks,
             "phases_ms": {"run_median": float(np.median(run_ms)), "run_best": float(np.min(run_ms)),
                           "chains_median": chain_med, "chains_best": chain_best,
                           "plan_upload_and_sample_stream_median": float(np.median(np.array(run_ms) - np.array(chain_ms))),
                           "combine_median": float(np.median(comb_ms)), "combine_best": float(np.min(comb_ms))},
             "l2": "inputs larger than L2; no flush" if input_bytes(wl) > 126e6 else "inputs fit in L2 (correctness-sized workload)",
             "roofline": roof}
    return entry, ctx


def measure_e2e(ctx, wl, host, n_e2e, world, dev):
    """The same metric through wpsgd_solve_host: pinned host rows in, combined model out, copies inside the call."""
    import torch
    import torch.distributed as dist

    vh = torch.empty(wl.d, dtype=torch.float32, pin_memory=True)
    solve = ctx.solve_host_csr if wl.sparse else ctx.solve_host
    args = tuple(host) + (wl.shard_off, wl.n_steps, wl.eta0, wl.sched, wl.lam, wl.loss, wl.seed)
    for _ in range(2):
        solve(*args, out=vh)
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(n_e2e):
        solve(*args, out=vh)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1)
    if world > 1:
        t = torch.tensor([ms], device=dev, dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms = float(t.item())
    return {"value": float(wl.total_steps) * world * n_e2e / (ms * 1e-3), "unit": UNIT,
            "h2d_bytes_per_step": int(sum(t.numel() * t.element_size() for t in host)) * world,
            "d2h_bytes_per_step": int(wl.d * 4) * world, "steps": n_e2e}


def pinned_host_rows(wl):
    """Pinned host copies of a workload's rows and labels (dense rows chunked, so no second pageable copy is needed)."""
    import torch

    if wl.sparse:
        out = []
        for t in (wl.row_ptr, wl.col_idx, wl.val, wl.y):
            h = torch.empty(t.shape, dtype=t.dtype, pin_memory=True)
            h.copy_(t)
            out.append(h)
        torch.cuda.synchronize()
        return tuple(out)

    Xh = torch.empty(wl.X.shape, dtype=wl.X.dtype, pin_memory=True)
    rows = max(1, (1 << 28) // max(1, wl.X.shape[1] * wl.X.element_size()))
    for r0 in range(0, wl.X.shape[0], rows):
        Xh[r0:r0 + rows].copy_(wl.X[r0:r0 + rows])
    yh = torch.empty(wl.y.shape, dtype=wl.y.dtype, pin_memory=True)
    yh.copy_(wl.y)
    torch.cuda.synchronize()
    return Xh, yh


def host_memory_available() -> int:
    try:
        for line in open("/proc/meminfo"):
            if line.startswith("MemAvailable:"):
                return int(line.split()[1]) * 1024
    except OSError:
        pass
    return 0


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

    peaks_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(peaks_path):
        peak, peak_src = float(json.load(open(peaks_path))["hbm_gbs"]), "measured"
    else:
        peak, peak_src = FALLBACK_HBM_GBS, "fallback"
    options = [(o.split("=")[0], int(o.split("=")[1])) for o in args.option]
    cfg = args.workload

    # ---- this rank's nodes: the cluster has world x k nodes (the pattern of step counts repeated), dealt to the ranks
    # by longest processing time; a rank generates the shards of its own nodes only
    weights = node_ids = None
    if world > 1:
        base_n = make_workload(cfg, "cpu", rho=args.rho, rows=2).n_steps  # the pattern of step counts of one GPU's share
        n_global = np.tile(base_n, world)
        owned = multi.partition_nodes(n_global, world)[rank]
        wl = make_workload(cfg, dev, rho=args.rho, small=args.small, rows=args.rows, rank=rank, k=len(owned),
                           n_steps=n_global[owned])
        weights = multi.local_weights(n_global, owned, wl.eta0, wl.sched, wl.lam)
        node_ids = owned
    else:
        wl = make_workload(cfg, dev, rho=args.rho, small=args.small, rows=args.rows)

    entry, ctx = measure(P, multi, wl, cfg, dev, args.steps, args.warmup, peak, peak_src, options, world, weights,
                         node_ids, args.small)
    updates_all = float(wl.total_steps)
    if world > 1:
        t = torch.tensor([updates_all], device=dev, dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.SUM)
        updates_all = float(t.item())
        entry["value"] = updates_all * args.steps / (entry["ms_per_step"] * args.steps * 1e-3)

    # ---- end to end through the host-buffer entry point (dense rows; pinned host memory must hold them) -------------
    e2e = None
    if not args.no_e2e:
        if input_bytes(wl) * 1.2 > host_memory_available():
            e2e = {"value": None, "unit": UNIT,
                   "note": f"host buffer of {input_bytes(wl) / 2**30:.1f} GiB not attempted: "
                           f"{host_memory_available() / 2**30:.1f} GiB of host memory available"}
        else:
            try:
                host = pinned_host_rows(wl)
                e2e = measure_e2e(ctx, wl, host, max(3, min(args.steps, 5 if input_bytes(wl) > 4e9 else 10)), world, dev)
                del host
            except RuntimeError as exc:  # e.g. the pinned allocation was refused
                e2e = {"value": None, "unit": UNIT, "note": f"host-buffer run failed: {str(exc)[:160]}"}
    ctx.destroy()

    if rank == 0:
        line = {
            "metric": METRIC, "value": entry["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": entry["ms_per_step"], "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": entry["workload"],
                       "parallelism": f"nodes dealt to {world} GPU(s) by longest processing time, one all-reduce of d floats"
                       if world > 1 else "all nodes on 1 GPU", "l2": entry["l2"]},
            "clocks": entry["clocks"], "e2e": e2e, "gpu_launches": entry["gpu_launches"], "phases_ms": entry["phases_ms"],
            "roofline": entry["roofline"],
        }
        if not args.no_cpu_baseline:
            wl_cpu, note = host_copy_for_cpu(cfg, args.rho, args.small)
            line["cpu_baseline"] = cpu_baseline(wl_cpu, note, 12.0)
            del wl_cpu
        if world == 1 and args.also and not args.small and not args.rows:
            del wl
            torch.cuda.empty_cache()
            others = []
            todo = []
            for tok in args.also.split(","):
                c2 = int(tok)
                if c2 == cfg:
                    continue
                todo += [(5, r) for r in (1.0, 2.0, 4.0, 8.0, 16.0)] if c2 == 5 else [(c2, args.rho)]
            for c2, rho in todo:
                try:
                    w2 = make_workload(c2, dev, rho=rho)
                    ent, ctx2 = measure(P, multi, w2, c2, dev, 10, 3, peak, peak_src, options)
                    if c2 == 5:
                        ent["rho"] = rho
                    if not args.no_e2e and (c2 != 5 or rho == args.rho):
                        ent["e2e"] = measure_e2e(ctx2, w2, pinned_host_rows(w2), 5, 1, dev)
                    ctx2.destroy()
                    if not args.no_cpu_baseline and (c2 != 5 or rho == args.rho):
                        wc, note = host_copy_for_cpu(c2, rho, False)
                        ent["cpu_baseline"] = cpu_baseline(wc, note, 3.0)
                        del wc
                    others.append(ent)
                    del w2
                    torch.cuda.empty_cache()
                except Exception as exc:  # a workload that does not fit this device is reported, not fatal
                    others.append({"workload": f"config{c2}", "error": str(exc)[:200]})
            line["other_workloads"] = others
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
