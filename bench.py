#!/usr/bin/env python
"""Benchmark of the batched adaptive filtered beam search (BOA / BOA+) on B200.

One step = one boa_search over one batch of synthetic queries: every phase of
Algorithm 1, all kernels of the hot path.  The workload is the 1M-point, 128-d,
two-attribute configuration with a 10,000-query batch.  Prints ONE JSON line.

  python bench.py [--gpus N] [--steps K] [--warmup W]        this library (CUDA)
  python bench.py --impl reference ...                        the CPU oracle, timed

With N > 1 (under torchrun) every rank holds a full replica of the index and
searches its own batch; there is no exchange step, so no collective on the data
path -- only the barrier and the max-over-ranks of the timing.
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

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "queries/sec at recall@10>=0.95 (10k-query batch)"
UNIT = "queries/s"

# dram__bytes_read.sum + dram__bytes_write.sum of the search kernel per scored neighbour
# record, from the full-size ncu capture summarised in
# profiles/boa_search_kernel_c2_dram_traffic.md (38.24 GB for 91.20 M records).  It holds
# for the default workload and table size only.
NCU_DRAM_BYTES_PER_SCORED = {"c2": 419.3}


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c2")
    ap.add_argument("--scale-n", type=int, default=0, help="debug: shrink the data set")
    ap.add_argument("--queries", type=int, default=0, help="debug: shrink the batch")
    ap.add_argument("--eps", type=float, default=0.03)
    ap.add_argument("--mode", default="resume", choices=["restart", "resume"])
    ap.add_argument("--schedule", default="16,512")
    ap.add_argument("--plus-k", type=int, default=0)
    ap.add_argument("--expand-w", type=int, default=1, choices=[1, 2],
                    help="nodes expanded per iteration: 1 = Algorithm 2 as printed, 2 = extension")
    ap.add_argument("--lam", type=float, default=float("inf"),
                    help="weight of the filter penalty; default infinity = lexicographic keys")
    ap.add_argument("--table-kb", type=int, default=0)
    ap.add_argument("--table-tags", type=int, default=0, choices=[0, 16])
    ap.add_argument("--max-warps", type=int, default=0)
    ap.add_argument("--fixed-L", type=int, default=0,
                    help="the paper's Fixed-L baseline: one phase at this beamwidth for every query")
    ap.add_argument("--no-extras", action="store_true", help="debug: skip recall/e2e/cpu legs")
    ap.add_argument("--cpu-seconds", type=float, default=12.0)
    ap.add_argument("--seed", type=int, default=0)
    return ap.parse_args()


def dist_env():
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    return rank, world, local


def get_workload(args):
    from boa_synth import ALL
    w = ALL[args.workload]
    if args.scale_n:
        w = w.scaled(args.scale_n, args.queries or w.Q)
    elif args.queries:
        w = dataclasses.replace(w, Q=args.queries)
    return w


def schedule_of(args, w):
    if getattr(args, "fixed_L", 0):
        return [int(args.fixed_L)]
    s = [int(x) for x in args.schedule.split(",") if x]
    if s[0] != w.L0 or s[-1] != w.Lmax:
        s = [w.L0] + [x for x in s[1:-1] if w.L0 < x < w.Lmax] + [w.Lmax]
    return s


class ClockSampler:
    """nvidia-smi clocks and throttle reasons sampled while the timed region runs."""
    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-i", str(self.index), "-lms", "50"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, smax, reasons, power = [], [], set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); smax.append(float(f[2])); power.append(float(f[3]))
            except ValueError:
                continue
            for nm, v in zip(names, f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": float(np.median(sm)) if sm else None,
                "sm_max_mhz": float(np.max(smax)) if smax else None,
                "power_w_max": float(np.max(power)) if power else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def max_over_ranks(local_ms: float, device, world: int) -> float:
    """Time of the slowest rank (all ranks get it)."""
    import torch
    import torch.distributed as dist
    t = torch.tensor([local_ms], dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(queries_per_rank: int, world: int, ms_per_step: float) -> float:
    """Queries per second of the whole job: every rank searched its own batch."""
    return world * queries_per_rank / (ms_per_step / 1e3)


def measured_peak_gbs():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return float(json.load(open(p))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return 6650.0, "fallback"


def algorithmic_bytes(w, st, scored_unique_ratio, mode, widths):
    """Bytes the method must move for one batch: query + bounds, one adjacency row per
    expansion, one record (vector + attribute cells) per neighbour scored for the first
    time, the outputs, and in resume mode the pool spill and reload of escalated queries."""
    sv = 1 if w.vec_dtype == "u8" else 4
    Q = st["n_expand"].shape[0]
    per_query = w.D * 4 + 8 * w.m + 8 * w.k
    rec = w.D * sv + 4 * w.m
    total = Q * per_query
    total += float(st["n_expand"].sum()) * 4 * w.R
    total += float(st["n_scored"].sum()) * scored_unique_ratio * rec
    if mode == "resume":
        esc = st["final_L"] > widths[0]
        pool = np.minimum(widths[-1], st["n_scored"][esc] + 1)
        total += float(pool.sum()) * 8 * 2
    return total


def run_oracle_sample(w, d, widths, args, seconds, dist_mode=1):
    """The CPU oracle, as it stands, on a leading slice of the batch sized for `seconds`."""
    from oracle.boa_oracle import OracleIndex
    orc = OracleIndex(d["vectors"], d["attrs"], d["attr_types"], d["graph"])
    probe = min(8, w.Q)
    t0 = time.perf_counter()
    orc.search(d["queries"][:probe], d["lo"][:probe], d["hi"][:probe], w.k, widths, eps=args.eps,
               mode=args.mode, dist_mode=dist_mode, expand_w=args.expand_w, lam=args.lam)
    per = max((time.perf_counter() - t0) / probe, 1e-6)
    n = int(max(8, min(w.Q, seconds / per)))
    t0 = time.perf_counter()
    o = orc.search(d["queries"][:n], d["lo"][:n], d["hi"][:n], w.k, widths, eps=args.eps,
                   mode=args.mode, dist_mode=dist_mode, expand_w=args.expand_w, lam=args.lam)
    dt = time.perf_counter() - t0
    return orc, o, n, dt


def reference_arm(args):
    """--impl reference: the oracle timed on the host cores, same workload and metric."""
    rank, world, local = dist_env()
    if rank != 0:
        return
    from boa_synth import make_workload
    w = get_workload(args)
    widths = schedule_of(args, w)
    d = make_workload(w, seed=args.seed)
    per_step = max(2.0, min(10.0, 150.0 / max(1, args.steps + args.warmup)))
    from oracle.boa_oracle import OracleIndex
    orc = OracleIndex(d["vectors"], d["attrs"], d["attr_types"], d["graph"])
    probe = min(8, w.Q)
    t0 = time.perf_counter()
    orc.search(d["queries"][:probe], d["lo"][:probe], d["hi"][:probe], w.k, widths, eps=args.eps,
               mode=args.mode, dist_mode=1, expand_w=args.expand_w, lam=args.lam)
    per = max((time.perf_counter() - t0) / probe, 1e-6)
    n = int(max(4, min(w.Q, per_step / per)))
    times = []
    for s in range(args.warmup + args.steps):
        a = (s * n) % max(1, w.Q - n + 1)
        t0 = time.perf_counter()
        orc.search(d["queries"][a:a + n], d["lo"][a:a + n], d["hi"][a:a + n], w.k, widths,
                   eps=args.eps, mode=args.mode, dist_mode=1, expand_w=args.expand_w, lam=args.lam)
        if s >= args.warmup:
            times.append(time.perf_counter() - t0)
    ms = 1e3 * float(np.mean(times))
    qps = n / (ms / 1e3)
    sample = f"{n} consecutive queries of the {w.Q}-query batch per step, full index"
    line = {"impl": "reference", "metric": METRIC, "value": qps, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": config_dict(w, widths, args),
            "cpu_baseline": {"value": qps, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
            "e2e": {"value": qps, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def config_dict(w, widths, args):
    return {"workload": f"{w.name}: N={w.N} D={w.D} {w.vec_dtype} m={w.m} R={w.R} Q={w.Q} k={w.k} "
                        f"L0={w.L0} Lmax={w.Lmax}",
            "schedule": widths, "eps": args.eps, "mode": args.mode, "plus_k": args.plus_k,
            "expand_w": args.expand_w, "lambda": "inf" if np.isinf(args.lam) else args.lam,
            "selectivity": f"{w.sel_kind} {w.sel_lo}-{w.sel_hi}", "seed": args.seed,
            "l2": "inputs larger than L2: records + graph are read by random access from a "
                  "working set far above 126 MB; no flush between steps"}


def main():
    args = parse_args()
    if args.impl == "reference":
        reference_arm(args)
        return

    import torch
    import torch.distributed as dist
    from boa_synth import make_workload
    from boa_synth.groundtruth import filtered_topk, recall_against
    from paper_2609_16175_b200 import BoaIndex

    rank, world, local = dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the search has no CPU path")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    w = get_workload(args)
    widths = schedule_of(args, w)
    d = make_workload(w, seed=args.seed, device=str(dev))
    t = {k: torch.from_numpy(v.view(np.int32) if v.dtype == np.uint32 else v).to(dev)
         for k, v in d.items() if k in ("vectors", "attrs", "graph", "queries", "lo", "hi")}
    ix = BoaIndex(t["vectors"], t["attrs"], d["attr_types"].tolist(), t["graph"])
    ix.set_param("mode", 1 if args.mode == "resume" else 0)
    ix.set_param("eps", args.eps)
    ix.set_param("plus_k", args.plus_k)
    ix.set_param("expand_w", args.expand_w)
    ix.set_param("lam", args.lam)
    ix.set_param("table_kb", args.table_kb)
    ix.set_param("table_tags", args.table_tags)
    ix.set_param("max_warps_per_sm", args.max_warps)
    ix.set_schedule(widths)
    Q, k = w.Q, w.k
    out_ids = torch.empty((Q, k), dtype=torch.int32, device=dev)
    out_d2 = torch.empty((Q, k), dtype=torch.float32, device=dev)

    def step():
        ix.search(t["queries"], t["lo"], t["hi"], k, widths[0], widths[-1], out_ids, out_d2)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- device-resident timing: W warm-up steps, then exactly K timed steps
    for _ in range(max(3, args.warmup)):
        step()
    barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
    barrier()
    ev[0].record()
    for s in range(args.steps):
        step()
        ev[s + 1].record()
    torch.cuda.synchronize()
    barrier()
    total_ms = ev[0].elapsed_time(ev[-1])
    step_ms = [ev[i].elapsed_time(ev[i + 1]) for i in range(args.steps)]
    launches = ix.last_launch_count * args.steps
    ms_per_step = max_over_ranks(total_ms, dev, world) / args.steps
    value = whole_job_value(Q, world, ms_per_step)

    # ---- statistics of the batch (outside the timed region)
    st = {kk: v.cpu().numpy() for kk, v in ix.stats().items()}
    phase_counts = ix.phase_counts()
    ids_np = out_ids.cpu().numpy().view(np.uint32)
    d2_np = out_d2.cpu().numpy()

    if args.no_extras:
        if rank == 0:
            sampler.stop()
            print(json.dumps({"ms_per_step": ms_per_step, "value": value, "table_kb": args.table_kb,
                              "schedule": widths, "mode": args.mode,
                              "plus_k": args.plus_k, "expand_w": args.expand_w, "mean_scored": float(st["n_scored"].mean()),
                              "status": ix.device_status()}))
        return

    # ---- end to end through the public call: pinned host inputs in, results out, every step
    hq = torch.from_numpy(d["queries"]).pin_memory()
    hlo = torch.from_numpy(d["lo"]).pin_memory()
    hhi = torch.from_numpy(d["hi"]).pin_memory()
    h_ids = torch.empty((Q, k), dtype=torch.int32).pin_memory()
    h_d2 = torch.empty((Q, k), dtype=torch.float32).pin_memory()
    dq, dlo, dhi = torch.empty_like(t["queries"]), torch.empty_like(t["lo"]), torch.empty_like(t["hi"])

    def e2e_step():
        dq.copy_(hq, non_blocking=True)
        dlo.copy_(hlo, non_blocking=True)
        dhi.copy_(hhi, non_blocking=True)
        ix.search(dq, dlo, dhi, k, widths[0], widths[-1], out_ids, out_d2)
        h_ids.copy_(out_ids, non_blocking=True)
        h_d2.copy_(out_d2, non_blocking=True)
        torch.cuda.synchronize()          # the caller reads the results of every step

    for _ in range(2):
        e2e_step()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        e2e_step()
    e1.record()
    torch.cuda.synchronize()
    barrier()
    clocks = sampler.stop() if rank == 0 else None     # sampled over both timed regions
    e2e_value = whole_job_value(Q, world, max_over_ranks(e0.elapsed_time(e1), dev, world) / args.steps)
    h2d = hq.numel() * 4 + hlo.numel() * 4 + hhi.numel() * 4
    d2h = h_ids.numel() * 4 + h_d2.numel() * 4
    assert (h_ids.numpy().view(np.uint32) == ids_np).all()

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- recall against exact filtered top-k (torch brute force: harness, not search path)
    gt_ids, gt_d2, gt_nv = filtered_topk(t["vectors"], t["attrs"], d["attr_types"], t["queries"],
                                         t["lo"], t["hi"], k)
    rec = recall_against(ids_np, d2_np, gt_d2.cpu().numpy(), gt_nv.cpu().numpy(), k)
    recall = float(np.nanmean(rec))

    # ---- CPU baseline: the oracle on a bounded sample; also gives the exact scored counts
    orc, o, n_s, dt_s = run_oracle_sample(w, d, widths, args, args.cpu_seconds)
    parity_ok = bool((o["ids"] == ids_np[:n_s]).all() and (o["final_L"] == st["final_L"][:n_s]).all()
                     and (o["n_expand"] == st["n_expand"][:n_s]).all())
    ratio = float(o["n_scored"].sum()) / max(1.0, float(st["n_scored"][:n_s].sum()))
    cpu_qps = n_s / dt_s

    # ---- roofline of the search kernel (HBM-bound random gather)
    peak, peak_kind = measured_peak_gbs()
    alg_bytes = algorithmic_bytes(w, st, ratio, args.mode, widths)
    kernel_ms = float(np.mean(step_ms))
    achieved = alg_bytes / (kernel_ms / 1e3) / 1e9
    traffic = None
    if (args.workload in NCU_DRAM_BYTES_PER_SCORED and not args.scale_n and not args.table_kb and not args.table_tags
            and args.expand_w == 1):
        traffic = NCU_DRAM_BYTES_PER_SCORED[args.workload] * float(st["n_scored"].sum())

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(3, args.warmup), "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": config_dict(w, widths, args),
        "recall_at_10": recall, "recall_ok": recall >= 0.95,
        "avg_beamwidth": float(st["final_L"].mean()),
        "phase_active": phase_counts,
        "mean_expansions": float(st["n_expand"].mean()), "mean_scored": float(st["n_scored"].mean()),
        "rescored_fraction": 1.0 - ratio, "capped_fraction": float((st["flags"] & 1).mean()),
        "parity_with_oracle_on_sample": parity_ok,
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                     "frac": achieved / peak, "traffic": traffic, "peak_kind": peak_kind,
                     "kernel": "boa_search_kernel, all phase launches of one step",
                     "kernel_ms_per_step": kernel_ms, "algorithmic_bytes_per_step": alg_bytes},
        "cpu_baseline": {"value": cpu_qps, "unit": UNIT, "cores": 1, "kind": "oracle",
                         "sample": f"first {n_s} queries of the batch, full index, {dt_s:.1f} s"},
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
        "gpu_launches": launches,
        "clocks": clocks,
    }
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
