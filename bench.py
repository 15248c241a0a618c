#!/usr/bin/env python
"""Benchmark of the batched adaptive filtered beam search (BOA / BOA+) on B200.

One step = one boa_search over one batch of synthetic queries: every phase of
Algorithm 1, all kernels of the hot path.  The headline workload is the 1M-point, 128-d,
two-attribute configuration with a 10,000-query batch; on one GPU the other
configurations are measured too and reported under "per_config".  Prints ONE JSON line.

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
# record, from the ncu captures summarised under profiles/ (file named beside each figure),
# together with the digest of the kernel source the capture was taken with.  A figure is
# used only while the kernel source still has that digest; after any change to the kernel
# the line reports "traffic": null until the capture is repeated.
NCU_DRAM_BYTES_PER_SCORED = {
    # workload: (bytes per scored record, sha256[:12] of csrc/boa_search.cuh, summary file)
    "c2": (409.8, "bd70335f918a", "profiles/boa_search_kernel_c2_dram_traffic.md"),
    "c3": (312.7, "bd70335f918a", "profiles/boa_search_kernel_c3_dram_traffic.md"),
}

# Operating point of each workload: explicit phase widths and eps, chosen from the sweeps in
# the design notes as the fastest setting of the adaptive method with recall@10 >= 0.95
# (c5: the configuration's own 16 -> 512, recall below the bar, reported beside fixed 500).
OPERATING = {
    "c1": dict(schedule=[16, 64, 128], eps=0.05, steps=20),    # literal, disconnected graph: parity only
    "c1b": dict(schedule=[16, 128], eps=0.02, steps=20),
    "c2": dict(schedule=[16, 80], eps=0.02, steps=20),
    "c3": dict(schedule=[16, 96], eps=0.03, steps=20),
    "c4": dict(schedule=[32, 96], eps=0.05, steps=20),
    "c5": dict(schedule=[16, 512], eps=0.03, steps=4),
}
# The schedule that runs each configuration's own L0 -> Lmax = 512 (most queries end at 512:
# the wide-beam regime, where one query expands about 500 nodes).
WIDE = {"c2": dict(schedule=[16, 512], eps=0.03), "c3": dict(schedule=[16, 512], eps=0.03),
        "c4": dict(schedule=[32, 512], eps=0.05)}


# What per_config measures beside each workload's operating point: the wide schedule for
# c2-c4, the operating point with two nodes expanded per iteration for c2 (tag w2), the configuration's own fixed beamwidth of 500 for c5, and for c5 the same two runs
# with PQ traversal (48 subspaces of 20 dimensions, 64 centroids each; exact final ranking).
PER_CONFIG_VARIANTS = {
    "c2": (dict(WIDE["c2"], tag="wide"), dict(expand_w=2, tag="w2")),
    "c3": ({}, dict(WIDE["c3"], tag="wide")),
    "c4": ({}, dict(WIDE["c4"], tag="wide")),
    "c5": ({}, {"fixed_L": 500}, {"pq": "48,64"}, {"pq": "48,64", "fixed_L": 500}),
}


# Graphs made by the library's own builder (boa_graph_build) instead of the fixture graph:
# build parameters (attribute thresholds in rank space, sized to the workload's query
# windows) and the settings timed over the built graph: the fastest adaptive schedule and
# the fastest fixed beamwidth with recall@10 >= 0.95 from the sweeps in the design notes.
# GPU-only figures: the oracle never sees a graph the CUDA builder made.
INF = float("inf")
BUILT_GRAPH = {
    "c2": dict(build=dict(R=32, Lb=64, alpha=1.2, thresholds=(INF, 0.3, 0.05), B=8192, passes=2),
               runs=(dict(schedule=[16, 32], eps=0.02), dict(schedule=[28], eps=0.05))),
    "c3": dict(build=dict(R=32, Lb=64, alpha=1.2, thresholds=(INF, 0.2, 0.08), B=8192, passes=2),
               runs=(dict(schedule=[16, 48], eps=0.02), dict(schedule=[48], eps=0.05))),
    "c4": dict(build=dict(R=64, Lb=64, alpha=1.2, thresholds=(INF, 0.3, 0.05), B=16384, passes=1),
               runs=(dict(schedule=[16, 48], eps=0.05), dict(schedule=[24], eps=0.05))),
    "c5": dict(build=dict(R=32, Lb=64, alpha=1.2, thresholds=(INF, 0.3, 0.12), B=8192, passes=2),
               runs=(dict(schedule=[16, 128], eps=0.005), dict(schedule=[96], eps=0.05),
                     dict(schedule=[256], eps=0.05, pq="48,64"))),
}


def kernel_source_digest() -> str:
    import hashlib
    with open(os.path.join(ROOT, "paper_2609_16175_b200", "csrc", "boa_search.cuh"), "rb") as f:
        return hashlib.sha256(f.read()).hexdigest()[:12]


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c2")
    ap.add_argument("--scale-n", type=int, default=0, help="debug: shrink the data set")
    ap.add_argument("--queries", type=int, default=0, help="debug: shrink the batch")
    ap.add_argument("--eps", type=float, default=None, help="default: the workload's operating point")
    ap.add_argument("--mode", default="resume", choices=["restart", "resume"])
    ap.add_argument("--schedule", default="", help="phase widths; default: the workload's operating point")
    ap.add_argument("--built-graph", default="c2,c3,c4,c5",
                    help="workloads of per_config also measured over a graph built by boa_graph_build "
                         "(comma list; the 10M-point build of c4 takes about 40 s, c5's 960-d one about 25 s)")
    ap.add_argument("--graph-build-only", action="store_true",
                    help="time boa_graph_build on the workload (with --scale-n for a small case), search the "
                         "built graph at BUILT_GRAPH's settings and print that entry alone")
    ap.add_argument("--no-per-config", action="store_true",
                    help="measure the headline workload only (always so with more than one GPU)")
    ap.add_argument("--plus-k", type=int, default=0)
    ap.add_argument("--chains", type=int, default=0, choices=[0, 1, 2],
                    help="2: the halves of a batch go through their phases on two streams; 1: the batch as one; "
                         "0 (the library's default): 2 while the widest phase is at most 128 (BOA_PARAM_CHAINS)")
    ap.add_argument("--plus-min-sub", type=int, default=0,
                    help="BOA+: fewest queries per sub-batch (0 = the library's default, twice the resident "
                         "query warps; 1 = always K sub-batches)")
    ap.add_argument("--expand-w", type=int, default=1, choices=[1, 2],
                    help="nodes expanded per iteration: 1 = Algorithm 2 as printed, 2 = extension")
    ap.add_argument("--lam", type=float, default=float("inf"),
                    help="weight of the filter penalty; default infinity = lexicographic keys")
    ap.add_argument("--table-kb", type=int, default=0)
    ap.add_argument("--table-tags", type=int, default=0, choices=[0, 16])
    ap.add_argument("--max-warps", type=int, default=0)
    ap.add_argument("--fixed-L", type=int, default=0,
                    help="the paper's Fixed-L baseline: one phase at this beamwidth for every query")
    ap.add_argument("--pq", default="", help="M[,K]: traverse on product-quantised distances with a codebook "
                    "of M subspaces and K centroids (default 256) trained on the fixture; exact final ranking")
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
    if not args.schedule:
        op = OPERATING.get(args.workload)
        return list(op["schedule"]) if op and not args.scale_n else [w.L0, w.Lmax]
    s = [int(x) for x in args.schedule.split(",") if x]
    if s[0] != w.L0:
        s = [w.L0] + [x for x in s[1:] if x > w.L0]
    return s


def eps_of(args):
    if args.eps is not None:
        return args.eps
    op = OPERATING.get(args.workload)
    return op["eps"] if op else 0.05


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


def algorithmic_bytes(w, st, scored_unique_ratio, mode, widths, pq_M=0, n_rerank=None):
    """Bytes the method must move for one batch: query + bounds, one adjacency row per
    expansion, one record (vector + attribute cells) per neighbour scored for the first
    time, the outputs, and in resume mode the pool spill and reload of escalated queries.
    With PQ traversal a scored neighbour costs its code (pq_M bytes) and attribute cells, and
    every row of the final exact ranking one vector; the codebook itself (K*D*4 bytes, read by
    every query) stays in L2 and is not counted against HBM."""
    sv = 1 if w.vec_dtype == "u8" else 4
    Q = st["n_expand"].shape[0]
    per_query = w.D * 4 + 8 * w.m + 8 * w.k
    rec = (pq_M if pq_M else w.D * sv) + 4 * w.m
    total = Q * per_query
    total += float(st["n_expand"].sum()) * 4 * w.R
    total += float(st["n_scored"].sum()) * scored_unique_ratio * rec
    if mode == "resume":
        esc = st["final_L"] > widths[0]
        pool = np.minimum(widths[-1], st["n_scored"][esc] + 1)
        total += float(pool.sum()) * 8 * 2
    if pq_M and n_rerank is not None:
        total += float(n_rerank.sum()) * w.D * sv
    return total


def parse_pq(args):
    if not getattr(args, "pq", ""):
        return 0, 0
    f = [int(x) for x in str(args.pq).split(",")]
    return f[0], (f[1] if len(f) > 1 else 256)


def codebook(d, args, dev=None):
    """The fixture's PQ codebook for this run (trained once per process and workload)."""
    M, K = parse_pq(args)
    key = ("pq", M, K)
    if key not in d:
        from boa_synth.pq import train_pq
        d[key] = train_pq(d["vectors"], M=M, K=K, iters=6, seed=args.seed, device=dev)
    return d[key]


def run_oracle_sample(w, d, widths, args, seconds, dist_mode=1):
    """The CPU oracle, as it stands, on a leading slice of the batch sized for `seconds`."""
    from oracle.boa_oracle import OracleIndex
    orc = OracleIndex(d["vectors"], d["attrs"], d["attr_types"], d["graph"])
    if parse_pq(args)[0]:
        orc.attach_pq(*codebook(d, args))
    probe = min(8, w.Q)
    t0 = time.perf_counter()
    pq = bool(parse_pq(args)[0])
    orc.search(d["queries"][:probe], d["lo"][:probe], d["hi"][:probe], w.k, widths, eps=args.eps,
               mode=args.mode, dist_mode=dist_mode, expand_w=args.expand_w, lam=args.lam, pq=pq)
    per = max((time.perf_counter() - t0) / probe, 1e-6)
    n = int(max(8, min(w.Q, seconds / per)))
    t0 = time.perf_counter()
    o = orc.search(d["queries"][:n], d["lo"][:n], d["hi"][:n], w.k, widths, eps=args.eps,
                   mode=args.mode, dist_mode=dist_mode, expand_w=args.expand_w, lam=args.lam, pq=pq)
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
    pq = bool(parse_pq(args)[0])
    if pq:
        orc.attach_pq(*codebook(d, args, "cpu"))
    probe = min(8, w.Q)
    t0 = time.perf_counter()
    orc.search(d["queries"][:probe], d["lo"][:probe], d["hi"][:probe], w.k, widths, eps=args.eps,
               mode=args.mode, dist_mode=1, expand_w=args.expand_w, lam=args.lam, pq=pq)
    per = max((time.perf_counter() - t0) / probe, 1e-6)
    n = int(max(4, min(w.Q, per_step / per)))
    times = []
    for s in range(args.warmup + args.steps):
        a = (s * n) % max(1, w.Q - n + 1)
        t0 = time.perf_counter()
        orc.search(d["queries"][a:a + n], d["lo"][a:a + n], d["hi"][a:a + n], w.k, widths,
                   eps=args.eps, mode=args.mode, dist_mode=1, expand_w=args.expand_w, lam=args.lam, pq=pq)
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
            "pq": (dict(zip(("M", "K"), parse_pq(args))) if parse_pq(args)[0] else None),
            "selectivity": f"{w.sel_kind} {w.sel_lo}-{w.sel_hi}", "seed": args.seed,
            "l2": "inputs larger than L2: records + graph are read by random access from a "
                  "working set far above 126 MB; no flush between steps"}


def to_device(d, dev):
    import torch
    return {k: torch.from_numpy(v.view(np.int32) if v.dtype == np.uint32 else v).to(dev)
            for k, v in d.items() if k in ("vectors", "attrs", "graph", "queries", "lo", "hi")}


def configure(ix, args, widths, d=None):
    if parse_pq(args)[0] and d is not None:
        import torch
        if ("attached",) + parse_pq(args) not in d:
            piv, codes = codebook(d, args, str(ix.device))
            ix.attach_pq(torch.from_numpy(piv).to(ix.device), torch.from_numpy(codes).to(ix.device))
            d[("attached",) + parse_pq(args)] = True
    ix.set_param("pq", 1 if parse_pq(args)[0] else 0)
    ix.set_param("mode", 1 if args.mode == "resume" else 0)
    ix.set_param("eps", args.eps)
    ix.set_param("plus_k", args.plus_k)
    ix.set_param("plus_min_sub", getattr(args, "plus_min_sub", 0))
    ix.set_param("chains", getattr(args, "chains", 0))
    ix.set_param("expand_w", args.expand_w)
    ix.set_param("lam", args.lam)
    ix.set_param("table_kb", args.table_kb)
    ix.set_param("table_tags", args.table_tags)
    ix.set_param("max_warps_per_sm", args.max_warps)
    ix.set_schedule(widths)


def timed_steps(ix, t, k, widths, out_ids, out_d2, steps, warmup, barrier):
    """W untimed steps, then exactly `steps` timed ones: CUDA events on the launching stream
    around every step.  Returns (total ms, per-step ms list)."""
    import torch
    for _ in range(max(3, warmup)):
        ix.search(t["queries"], t["lo"], t["hi"], k, widths[0], widths[-1], out_ids, out_d2)
    barrier()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
    barrier()
    ev[0].record()
    for s in range(steps):
        ix.search(t["queries"], t["lo"], t["hi"], k, widths[0], widths[-1], out_ids, out_d2)
        ev[s + 1].record()
    torch.cuda.synchronize()
    barrier()
    return ev[0].elapsed_time(ev[-1]), [ev[i].elapsed_time(ev[i + 1]) for i in range(steps)]


def quality(w, d, t, ix, args, widths, ids_np, d2_np, st, gt_queries, cpu_seconds):
    """Recall against exact filtered top-k (on the first gt_queries queries), the oracle on a
    bounded sample (parity, exact scored counts, CPU timing) and the algorithmic bytes."""
    from boa_synth.groundtruth import filtered_topk, recall_against
    n_gt = min(gt_queries, ids_np.shape[0])
    gt_ids, gt_d2, gt_nv = filtered_topk(t["vectors"], t["attrs"], d["attr_types"], t["queries"][:n_gt],
                                         t["lo"][:n_gt], t["hi"][:n_gt], w.k)
    rec = recall_against(ids_np[:n_gt], d2_np[:n_gt], gt_d2.cpu().numpy(), gt_nv.cpu().numpy(), w.k)
    del gt_ids, gt_d2, gt_nv
    orc, o, n_s, dt_s = run_oracle_sample(w, d, widths, args, cpu_seconds)
    parity_ok = bool((o["ids"] == ids_np[:n_s]).all() and (o["final_L"] == st["final_L"][:n_s]).all()
                     and (o["n_expand"] == st["n_expand"][:n_s]).all()
                     and (o["d2"].view(np.uint32) == d2_np[:n_s].view(np.uint32)).all())
    ratio = float(o["n_scored"].sum()) / max(1.0, float(st["n_scored"][:n_s].sum()))
    del orc
    return dict(recall=float(np.nanmean(rec)), recall_queries=n_gt, parity=parity_ok, unique_ratio=ratio,
                cpu_qps=n_s / dt_s, cpu_n=n_s, cpu_dt=dt_s)


def measure_config(name, args, dev, steps, cpu_seconds, variants=({},), gt_queries=10_000):
    """One workload at its operating point and in every variant asked for (fixed beamwidth,
    PQ traversal), on one build of its inputs: the entries of per_config (keys name,
    name_fixed<L>, name_pq<M>, name_pq<M>_fixed<L>)."""
    import copy
    import torch
    from boa_synth import ALL, make_workload
    from paper_2609_16175_b200 import BoaIndex
    w = ALL[name]
    t0 = time.perf_counter()
    d = make_workload(w, seed=args.seed, device=str(dev))
    t_build = time.perf_counter() - t0
    t = to_device(d, dev)
    ix = BoaIndex(t["vectors"], t["attrs"], d["attr_types"].tolist(), t["graph"])
    out_ids = torch.empty((w.Q, w.k), dtype=torch.int32, device=dev)
    out_d2 = torch.empty((w.Q, w.k), dtype=torch.float32, device=dev)
    peak, peak_kind = measured_peak_gbs()
    res = {}
    for var in variants:
        fixed_L, pq = var.get("fixed_L", 0), var.get("pq", "")
        a = copy.copy(args)
        a.workload, a.scale_n, a.queries, a.schedule, a.fixed_L, a.pq = name, 0, 0, "", fixed_L, pq
        a.eps = var.get("eps", OPERATING[name]["eps"])
        a.plus_k, a.expand_w, a.lam, a.table_kb, a.table_tags, a.max_warps = 0, var.get("expand_w", 1), float("inf"), 0, 0, 0
        widths = var.get("schedule") or schedule_of(a, w)
        configure(ix, a, widths, d)
        n_steps = steps if not fixed_L else max(3, steps // 2)
        total_ms, step_ms = timed_steps(ix, t, w.k, widths, out_ids, out_d2, n_steps, 3, torch.cuda.synchronize)
        st = {kk: v.cpu().numpy() for kk, v in ix.stats().items()}
        counts = ix.phase_counts()
        ids_np, d2_np = out_ids.cpu().numpy().view(np.uint32), out_d2.cpu().numpy()
        ql = quality(w, d, t, ix, a, widths, ids_np, d2_np, st, gt_queries, cpu_seconds)
        pq_M = parse_pq(a)[0]
        n_rr = ix.rerank_counts().cpu().numpy() if pq_M else None
        alg = algorithmic_bytes(w, st, ql["unique_ratio"], a.mode, widths, pq_M, n_rr)
        ms = total_ms / n_steps
        in_flight = None
        if not var and name in ("c2", "c3", "c4"):
            a.chains = 0
            in_flight = two_in_flight(ix, t, w.k, widths, a, n_steps, 4, out_ids, out_d2, ids_np)
        key = name + (f"_pq{pq_M}" if pq_M else "") + (f"_fixed{fixed_L}" if fixed_L else "") + \
            (f"_{var['tag']}" if var.get("tag") else "")
        res[key] = {
            "pq": config_dict(w, widths, a)["pq"],
            "mean_rows_reranked": float(n_rr.mean()) if pq_M else None,
            "workload": config_dict(w, widths, a)["workload"], "schedule": widths, "eps": a.eps, "mode": a.mode,
            "steps": n_steps, "ms_per_step": ms, "queries_per_s": w.Q / (ms / 1e3),
            "recall_at_10": ql["recall"], "recall_queries": ql["recall_queries"],
            "avg_beamwidth": float(st["final_L"].mean()), "phase_active": counts,
            "mean_expansions": float(st["n_expand"].mean()), "mean_scored": float(st["n_scored"].mean()),
            "rescored_fraction": 1.0 - ql["unique_ratio"], "capped_fraction": float((st["flags"] & 1).mean()),
            "algorithmic_bytes_per_step": alg, "achieved_gbs": alg / (ms / 1e3) / 1e9,
            "traffic": (NCU_DRAM_BYTES_PER_SCORED[name][0] * float(st["n_scored"].sum())
                        if name in NCU_DRAM_BYTES_PER_SCORED and not var
                        and NCU_DRAM_BYTES_PER_SCORED[name][1] == kernel_source_digest() else None),
            "frac": alg / (ms / 1e3) / 1e9 / peak, "peak_kind": peak_kind,
            "parity_with_oracle_on_sample": ql["parity"], "oracle_sample_queries": ql["cpu_n"],
            "cpu_oracle_queries_per_s": ql["cpu_qps"], "gpu_launches_per_step": ix.last_launch_count,
            "two_batches_in_flight": ({"ms_per_step": in_flight["ms_per_step"], "queries_per_s": in_flight["value"],
                                       "same_results": in_flight["same_results"]} if in_flight else None),
            "device_status": ix.device_status(), "fixture_build_s": round(t_build, 1)}
    ix.close()
    del ix, out_ids, out_d2
    torch.cuda.empty_cache()
    if name in BUILT_GRAPH and name in [x for x in args.built_graph.split(",") if x]:
        try:
            res[name + "_built_graph"] = measure_built_graph(name, args, dev, w, d, t, max(3, steps // 2), gt_queries)
        except Exception as e:
            res[name + "_built_graph"] = {"error": f"{type(e).__name__}: {e}"}
    del t, d
    torch.cuda.empty_cache()
    return res


def two_in_flight(ix, t, k, widths, args, steps, warmup, out_ids, out_d2, ids_np):
    """The same steps with two batches in flight: two handles on the index (boa_index_share),
    steps alternating between two streams, so that the partly empty last wave of one batch's
    wide phase overlaps the narrow phase of the next batch.  Each batch runs as one chain: the
    other batch already fills the tails."""
    import torch
    Q = t["queries"].shape[0]
    ix2 = ix.share()
    configure(ix2, args, widths)
    ix.set_param("chains", 1)
    ix2.set_param("chains", 1)
    pair = ((ix, torch.cuda.Stream(), out_ids, out_d2),
            (ix2, torch.cuda.Stream(), torch.empty_like(out_ids), torch.empty_like(out_d2)))

    def run(n):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _, s_, _, _ in pair:
            s_.wait_event(e0)
        for i in range(n):
            h_, s_, oi, od = pair[i % 2]
            h_.search(t["queries"], t["lo"], t["hi"], k, widths[0], widths[-1], oi, od, stream=s_)
        for _, s_, _, _ in pair:
            ev = torch.cuda.Event()
            ev.record(s_)
            torch.cuda.current_stream().wait_event(ev)
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1)

    run(warmup)
    p_ms = run(steps) / steps
    same = bool((pair[1][2].cpu().numpy().view(np.uint32) == ids_np).all()
                and (pair[0][2].cpu().numpy().view(np.uint32) == ids_np).all())
    ix2.close()
    ix.set_param("chains", getattr(args, "chains", 0))
    return {"handles": 2, "streams": 2, "steps": steps, "ms_per_step": p_ms, "value": Q / (p_ms / 1e3),
            "unit": UNIT, "same_results": same,
            "note": "value above is one batch at a time on one stream; this is the same work with the next "
                    "batch's launches enqueued on a second stream and handle (each batch as one chain)"}


def attribute_positions(attrs, types):
    """rank / N of every point in every attribute column (stable order): the builder's attr_pos."""
    import torch
    n, m = attrs.shape
    pos = torch.empty((n, m), dtype=torch.float32, device=attrs.device)
    for j in range(m):
        col = attrs[:, j].view(torch.float32) if int(types[j]) == 1 else attrs[:, j]
        order = torch.argsort(col, stable=True)
        pos[order, j] = torch.arange(n, dtype=torch.float32, device=attrs.device) / n
    return pos


def measure_built_graph(name, args, dev, w, d, t, steps, gt_queries=10_000):
    """per_config[name + "_built_graph"]: the graph built on the GPU by boa_graph_build from the
    workload's vectors and attributes, then the search over it at the settings of
    BUILT_GRAPH[name].  No oracle run here."""
    import copy
    import torch
    from boa_synth.groundtruth import filtered_topk, recall_against
    from paper_2609_16175_b200 import BoaIndex, build_graph
    spec = BUILT_GRAPH[name]
    pos = attribute_positions(t["attrs"], d["attr_types"])
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    g = build_graph(t["vectors"], pos, **spec["build"])
    torch.cuda.synchronize()
    build_s = time.perf_counter() - t0
    del pos
    ix = BoaIndex(t["vectors"], t["attrs"], d["attr_types"].tolist(), g)
    out_ids = torch.empty((w.Q, w.k), dtype=torch.int32, device=dev)
    out_d2 = torch.empty((w.Q, w.k), dtype=torch.float32, device=dev)
    n_gt = min(gt_queries, w.Q)
    _, gt_d2, gt_nv = filtered_topk(t["vectors"], t["attrs"], d["attr_types"], t["queries"][:n_gt],
                                    t["lo"][:n_gt], t["hi"][:n_gt], w.k)
    gt_d2, gt_nv = gt_d2.cpu().numpy(), gt_nv.cpu().numpy()
    runs = []
    for run in spec["runs"]:
        a = copy.copy(args)
        a.workload, a.pq, a.eps = name, run.get("pq", ""), run["eps"]
        a.plus_k, a.expand_w, a.lam, a.table_kb, a.table_tags, a.max_warps = 0, 1, float("inf"), 0, 0, 0
        widths = run["schedule"]
        # the codebook cached beside the workload is reused; "attached" marks belong to another index
        configure(ix, a, widths, {k: v for k, v in d.items() if not (isinstance(k, tuple) and k[0] == "attached")}
                  if a.pq else None)
        total_ms, _ = timed_steps(ix, t, w.k, widths, out_ids, out_d2, steps, 3, torch.cuda.synchronize)
        st = {kk: v.cpu().numpy() for kk, v in ix.stats().items()}
        rec = recall_against(out_ids.cpu().numpy().view(np.uint32)[:n_gt], out_d2.cpu().numpy()[:n_gt], gt_d2, gt_nv, w.k)
        ms = total_ms / steps
        runs.append({"schedule": widths, "eps": a.eps, "mode": a.mode, "pq": a.pq or None, "steps": steps, "ms_per_step": ms,
                     "queries_per_s": w.Q / (ms / 1e3), "recall_at_10": float(np.nanmean(rec)), "recall_queries": n_gt,
                     "avg_beamwidth": float(st["final_L"].mean()), "mean_expansions": float(st["n_expand"].mean()),
                     "mean_scored": float(st["n_scored"].mean()), "gpu_launches_per_step": ix.last_launch_count,
                     "device_status": ix.device_status()})
    degree = float((g != -1).sum(1).float().mean().item())
    ix.close()
    del g, out_ids, out_d2
    build = dict(spec["build"])
    build["thresholds"] = [str(x) for x in build["thresholds"]]
    return {"graph": "boa_graph_build", "build": build, "build_s": round(build_s, 2), "mean_degree": degree,
            "points_per_s": w.N / build_s, "runs": runs}


def main():
    args = parse_args()
    args.eps = eps_of(args)
    if args.impl == "reference":
        reference_arm(args)
        return

    import torch
    import torch.distributed as dist
    from boa_synth import make_workload
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
    if args.graph_build_only:
        d = make_workload(w, seed=args.seed, device=str(dev), with_graph=False)
        d["graph"] = np.zeros((w.N, 1), np.uint32)
        t = to_device(d, dev)
        entry = measure_built_graph(args.workload, args, dev, w, d, t, max(3, args.steps // 2))
        print(json.dumps({"metric": "graph_build_points_per_s", "value": entry["points_per_s"], "unit": "points/s",
                          "n_gpus": 1, "config": config_dict(w, widths, args), "built_graph": entry}))
        return
    d = make_workload(w, seed=args.seed, device=str(dev))
    t = to_device(d, dev)
    ix = BoaIndex(t["vectors"], t["attrs"], d["attr_types"].tolist(), t["graph"])
    configure(ix, args, widths, d)
    Q, k = w.Q, w.k
    out_ids = torch.empty((Q, k), dtype=torch.int32, device=dev)
    out_d2 = torch.empty((Q, k), dtype=torch.float32, device=dev)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- device-resident timing: W warm-up steps, then exactly K timed steps
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    total_ms, step_ms = timed_steps(ix, t, k, widths, out_ids, out_d2, args.steps, args.warmup, barrier)
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

    # ---- the same K steps with two batches in flight: two handles on the index (boa_index_share),
    # steps alternating between two streams, so that the partly empty last wave of one batch's
    # wide phase overlaps the narrow phase of the next batch
    pipelined = None
    if world == 1:
        pipelined = two_in_flight(ix, t, k, widths, args, args.steps, max(4, 2 * args.warmup), out_ids, out_d2, ids_np)

    # ---- end to end through the public call: pinned host inputs in, results out, every step
    hq = torch.from_numpy(d["queries"]).pin_memory()
    hlo = torch.from_numpy(d["lo"]).pin_memory()
    hhi = torch.from_numpy(d["hi"]).pin_memory()
    h_ids = torch.empty((Q, k), dtype=torch.int32).pin_memory()
    h_d2 = torch.empty((Q, k), dtype=torch.float32).pin_memory()

    def e2e_step():
        # boa_search_host: the library copies the host inputs in, searches, copies the results
        # out and returns when they are readable
        ix.search_host(hq, hlo, hhi, k, widths[0], widths[-1], h_ids, h_d2)

    for _ in range(2):
        e2e_step()

    # two host threads, each with its own handle, stream and result buffers, each making half of
    # the same boa_search_host calls: the end-to-end figure with two batches in flight
    if pipelined is not None:
        ix3 = ix.share()
        configure(ix3, args, widths)
        ix.set_param("chains", 1)
        ix3.set_param("chains", 1)
        lanes = ((ix, torch.cuda.Stream(), h_ids, h_d2),
                 (ix3, torch.cuda.Stream(), torch.empty_like(h_ids).pin_memory(), torch.empty_like(h_d2).pin_memory()))
        def lane_steps(lane, n):
            h_, s_, oi, od = lane
            torch.cuda.set_device(dev)
            for _ in range(n):
                h_.search_host(hq, hlo, hhi, k, widths[0], widths[-1], oi, od, stream=s_)
        def threaded(n):
            th = [threading.Thread(target=lane_steps, args=(ln, n)) for ln in lanes]
            t0 = time.perf_counter()
            for x in th:
                x.start()
            for x in th:
                x.join()
            return time.perf_counter() - t0
        threaded(2)
        half = max(1, args.steps // 2)
        dt = threaded(half)
        pipelined["e2e_value"] = 2 * half * Q / dt
        pipelined["e2e_same_results"] = bool((lanes[1][2].numpy().view(np.uint32) == ids_np).all())
        pipelined["e2e_note"] = (f"{2 * half} boa_search_host calls from two host threads (wall clock: every call "
                                 "returns with its results readable)")
        ix3.close()
        ix.set_param("chains", getattr(args, "chains", 0))
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
    # the page-locked buffers are read in place: every phase fetches the queries it searches
    # (vector and bounds) over the host link, the results are written back once
    h2d = int(sum(ix.phase_counts())) * (w.D * 4 + 2 * 4 * w.m)
    d2h = h_ids.numel() * 4 + h_d2.numel() * 4
    assert (h_ids.numpy().view(np.uint32) == ids_np).all()

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- recall, oracle sample (parity, CPU baseline, exact scored counts)
    ql = quality(w, d, t, ix, args, widths, ids_np, d2_np, st, 10_000, args.cpu_seconds)
    recall = ql["recall"]

    # ---- roofline of the search kernel (HBM-bound random gather)
    peak, peak_kind = measured_peak_gbs()
    pq_M = parse_pq(args)[0]
    alg_bytes = algorithmic_bytes(w, st, ql["unique_ratio"], args.mode, widths, pq_M,
                                  ix.rerank_counts().cpu().numpy() if pq_M else None)
    kernel_ms = float(np.mean(step_ms))
    achieved = alg_bytes / (kernel_ms / 1e3) / 1e9
    traffic, traffic_note = None, "no ncu capture on file for this workload and kernel source"
    cap = NCU_DRAM_BYTES_PER_SCORED.get(args.workload)
    plain = not (args.scale_n or args.table_kb or args.table_tags or args.expand_w != 1 or args.fixed_L
                 or args.pq)
    if cap and plain and cap[1] == kernel_source_digest() and widths == OPERATING[args.workload]["schedule"]:
        traffic = cap[0] * float(st["n_scored"].sum())
        traffic_note = f"{cap[0]} DRAM bytes per scored record ({cap[2]}) x records scored in this run"

    # ---- the fastest fixed beamwidth that reaches the same recall bar, for comparison
    fixed_same = None
    if plain and not args.scale_n and world == 1:
        from boa_synth.groundtruth import filtered_topk, recall_against
        gt_ids, gt_d2, gt_nv = filtered_topk(t["vectors"], t["attrs"], d["attr_types"], t["queries"],
                                             t["lo"], t["hi"], k)
        gt_d2, gt_nv = gt_d2.cpu().numpy(), gt_nv.cpu().numpy()
        ix.set_param("mode", 0)
        for L in (48, 56, 64, 72, 80, 96, 128, 192, 256, 512):
            if L < w.L0:
                continue
            ix.set_schedule([L])
            tot, _ = timed_steps(ix, t, k, [L], out_ids, out_d2, 5, 3, torch.cuda.synchronize)
            r = float(np.nanmean(recall_against(out_ids.cpu().numpy().view(np.uint32), out_d2.cpu().numpy(),
                                                gt_d2, gt_nv, k)))
            if r >= 0.95:
                fixed_same = {"L": L, "recall_at_10": r, "ms_per_step": tot / 5, "queries_per_s": Q / (tot / 5 / 1e3)}
                break
        configure(ix, args, widths, d)
        del gt_ids, gt_d2, gt_nv

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(3, args.warmup), "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": config_dict(w, widths, args),
        "recall_at_10": recall, "recall_ok": recall >= 0.95,
        "avg_beamwidth": float(st["final_L"].mean()),
        "phase_active": phase_counts,
        "mean_expansions": float(st["n_expand"].mean()), "mean_scored": float(st["n_scored"].mean()),
        "rescored_fraction": 1.0 - ql["unique_ratio"], "capped_fraction": float((st["flags"] & 1).mean()),
        "parity_with_oracle_on_sample": ql["parity"],
        "fixed_L_at_same_recall": fixed_same,
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                     "frac": achieved / peak, "traffic": traffic, "traffic_note": traffic_note,
                     "peak_kind": peak_kind,
                     "kernel": "boa_search_kernel, all phase launches of one step",
                     "kernel_ms_per_step": kernel_ms, "algorithmic_bytes_per_step": alg_bytes},
        "cpu_baseline": {"value": ql["cpu_qps"], "unit": UNIT, "cores": 1, "kind": "oracle",
                         "sample": f"first {ql['cpu_n']} queries of the batch, full index, {ql['cpu_dt']:.1f} s"},
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "call": "boa_search_host on page-locked host buffers (read and written in place by the kernels), "
                        "stream synchronised inside every call"},
        "gpu_launches": launches,
        "pipelined": pipelined,
        "clocks": clocks,
    }
    ix.close()
    del t, d, ix
    torch.cuda.empty_cache()

    # ---- the other configurations, one GPU only
    if world == 1 and plain and not args.no_per_config and args.workload == "c2":
        per = {}
        for name in ("c1", "c1b", "c2", "c3", "c4", "c5"):
            try:
                per.update(measure_config(name, args, dev, OPERATING[name]["steps"], 3.0,
                                          variants=PER_CONFIG_VARIANTS.get(name, ({},))))
            except Exception as e:           # one workload failing must not lose the line
                per[name] = {"error": f"{type(e).__name__}: {e}"}
        line["per_config"] = per
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
