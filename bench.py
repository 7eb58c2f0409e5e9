"""Benchmark of the selection hot path: (problem, candidate) pairs ranked per second through
the fused featurize + score + top-k call, on seeded synthetic inputs shaped like the paper's
full configuration space (1,024 problems x 60,000 candidates, 500 trees of depth 8, top-10).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload 1]

One step = one pass of the whole path over the batch. With N > 1 (under torchrun, or started
here when no launcher is around) every rank ranks its own batch of problems (weak scaling; the
only exchange is the all-gather of the [P, k] result blocks) and rank 0 prints the line. The
default N = 1 line also carries short runs of the other configurations under "extra".
`--impl reference` times the CPU oracle on a bounded sample of the same workload instead.
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

METRIC = "problem x candidate pairs ranked/sec (fused featurize+score+top-k)"
UNIT = "pairs/s"
# Issue-rate roofline of the tree walk: 148 SMs x 4 schedulers x 32 lanes x 1.965 GHz
# thread-instructions per second, 4 thread-instructions per node visit.
ISSUE_PEAK = 148 * 4 * 32 * 1.965e9
INSTR_PER_VISIT = 4


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            d = json.load(fh)
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained"), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples during the timed region (read-only query)."""
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.rows = []
        self.proc = None
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.gpu}", f"--query-gpu={self.QUERY}",
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            f = [x.strip() for x in r.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                smax.append(float(f[2]))
            except ValueError:
                continue
            for n, v in zip(names, f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None,
                "sm_max_mhz": float(max(smax)) if smax else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def workload_config(cfg: int):
    from paper_2609_35587_b200 import workloads as wl
    spec = wl.CONFIGS[cfg]
    return spec


def run_reference(args, rank, world):
    """CPU-oracle arm: each step ranks a bounded sample of the workload on the host cores."""
    if rank != 0:
        return
    import oracle
    from paper_2609_35587_b200 import workloads as wl
    cfg = args.workload
    spec = wl.CONFIGS[cfg]
    cores = oracle.threads()
    w = wl.make_workload(cfg, P=max(2, min(spec["P"], args.ref_problems)), law=args.law)
    kw = dict(gbdt=w.gbdt, mlp=w.mlp, seg_off=w.seg_offsets, seg_idx=w.seg_index)
    for _ in range(args.warmup):
        oracle.select(w.problems[:1], w.candidates, w.desc, w.k, gbdt=w.gbdt, mlp=w.mlp,
                      seg_off=None if w.seg_offsets is None else w.seg_offsets[:2],
                      seg_idx=w.seg_index)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle.select(w.problems, w.candidates, w.desc, w.k, **kw)
    dt = (time.perf_counter() - t0) / args.steps
    value = w.pairs / dt
    sample = f"{len(w.problems)} problems x {w.pairs // len(w.problems)} candidates per step"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
            "data": "synthetic", "config": config_dict(cfg, spec, args),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def config_dict(cfg, spec, args):
    d = {"workload": f"config {cfg} ({spec['name']})", "problems": args.problems or spec["P"],
         "candidates_per_problem": spec["seg"] or spec["C"], "k": spec["k"],
         "l2": "flushed between steps (256 MiB write)"}
    if spec["trees"]:
        d.update(scorer="gbdt", trees=spec["trees"], depth=spec["depth"], threshold_law=args.law)
        d["workload"] += f", thresholds: {args.law}"
    else:
        d.update(scorer="mlp 64-256-256-1 bf16")
    return d


def cpu_baseline(cfg, law, budget_s=15.0):
    """The oracle as it stands on this machine's host cores, on a bounded sample of the workload."""
    import oracle
    from paper_2609_35587_b200 import workloads as wl
    spec = wl.CONFIGS[cfg]
    cores = oracle.threads()
    probe_p = max(1, min(cores, spec["P"]))
    w = wl.make_workload(cfg, P=max(probe_p, 2), law=law)
    kw = dict(gbdt=w.gbdt, mlp=w.mlp)

    def run(n):
        so = None if w.seg_offsets is None else w.seg_offsets[:n + 1]
        t0 = time.perf_counter()
        oracle.select(w.problems[:n], w.candidates, w.desc, w.k, seg_off=so, seg_idx=w.seg_index, **kw)
        return time.perf_counter() - t0

    per = w.pairs // len(w.problems)
    t_probe = run(probe_p)
    n = int(max(probe_p, min(spec["P"], probe_p * budget_s / max(t_probe, 1e-3))))
    n = max(cores, n // cores * cores)
    if n > len(w.problems):
        w = wl.make_workload(cfg, P=n, law=law)
    dt = run(n)
    return {"value": n * per / dt, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"first {n} problems x {per} candidates of the workload, {dt:.1f} s"}


def run_latency_stream(args, rank, local_rank, dev):
    """Workload 3: a stream of single problems, each ranked against the 60,000-candidate
    catalogue with the 500-tree ensemble through the synchronous ks_select_one call. Reports
    p50 / p99 per-call latency (host clock around the call: problem by value in, k results
    visible in host memory out) and sustained problems per second."""
    if rank != 0:
        return
    import torch
    from paper_2609_35587_b200 import binding as ks
    from paper_2609_35587_b200 import workloads as wl
    n_warm, n = (1000 if args.calls >= 1000 else 10), args.calls
    w = wl.make_workload(3, P=n_warm + n, law=args.law)
    ctx = ks.Context(w.desc, local_rank)
    model = ctx.model_create_gbdt(*w.gbdt)
    d_c = ks.to_device(w.candidates, dev)
    C, k = len(w.candidates), w.k
    h_idx = torch.empty(k, dtype=torch.int32).pin_memory()
    h_sc = torch.empty(k, dtype=torch.float32).pin_memory()
    # the C call itself is what is timed: pointers and the by-value structs are prepared once
    cat = None if args.unprepared else ctx.catalogue_prepare(d_c, C, model)
    call = ctx.select_one_caller(d_c, C, model, k, h_idx, h_sc, catalogue=cat)
    structs = ks.problem_structs(w.problems)
    for i in range(n_warm):
        call(structs[i])
    lat = np.empty(n)
    sampler = ClockSampler(local_rank)
    sampler.start()
    launches0 = ctx.launch_count()
    t_all = time.perf_counter()
    for i in range(n):
        t0 = time.perf_counter()
        call(structs[n_warm + i])
        lat[i] = time.perf_counter() - t0
    total = time.perf_counter() - t_all
    clocks = sampler.stop()
    visits = C * 500 * 8
    line = {"metric": "problems/sec, single-problem stream (ks_select_one: featurize+score+top-k of one problem)",
            "value": n / total, "unit": "problems/s", "n_gpus": 1, "steps": n, "warmup": n_warm,
            "ms_per_step": total / n * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic",
            "config": {"workload": f"config 3 (dynamic), thresholds: {args.law}", "candidates": C, "trees": 500, "depth": 8, "k": k,
                       "call": "ks_select_one" if args.unprepared else "ks_select_one_prepared", "kernel": model.describe(),
                       "l2": "catalogue and model are L2-resident by design (re-used every call)"},
            "latency_us": {"p50": float(np.percentile(lat, 50) * 1e6), "p99": float(np.percentile(lat, 99) * 1e6),
                           "mean": float(lat.mean() * 1e6)},
            "pairs_per_s": C * n / total, "clocks": clocks, "gpu_launches": int(ctx.launch_count() - launches0),
            "roofline": {"bound": "alu", "achieved": visits * INSTR_PER_VISIT / (total / n) / 1e12,
                         "peak": ISSUE_PEAK / 1e12, "unit": "T thread-instr/s (4 per node visit)",
                         "frac": visits * INSTR_PER_VISIT / (total / n) / ISSUE_PEAK,
                         "note": "whole call incl. launch, sync and host read-back", "traffic": None},
            "e2e": {"value": n / total, "unit": "problems/s", "h2d_bytes_per_step": 16, "d2h_bytes_per_step": k * 8}}
    print(json.dumps(line), flush=True)


def run_catalogue(args, rank, local_rank, dev):
    """The steps in front of the path: the four layouts' valid catalogues built from the
    534,600-id search space (generate each candidate from its id, test the validity rules,
    pack the survivors in id order). One step = the four layouts; timed with CUDA events."""
    if rank != 0:
        return
    import torch
    from paper_2609_35587_b200 import binding as ks
    from paper_2609_35587_b200 import workloads as wl
    desc = wl.gpu_desc()
    ctx = ks.Context(desc, local_rank)
    probs = np.zeros(4, wl.PROBLEM_DT)
    probs["m"] = probs["n"] = probs["k"] = 4096
    probs["layout"] = np.arange(4)
    probs["dtype_ab"] = probs["dtype_d"] = 1
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    def step():
        return [ctx.valid_catalogue(probs[i:i + 1], ks.KS_VALID_COUPLED, sync=False) for i in range(4)]
    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    sampler = ClockSampler(local_rank)
    sampler.start()
    launches0 = ctx.launch_count()
    ms = []
    for _ in range(args.steps):
        flush.fill_(1)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        res = step()
        e1.record()
        torch.cuda.synchronize()
        ms.append(e0.elapsed_time(e1))
    clocks = sampler.stop()
    launches = int(ctx.launch_count() - launches0)
    t = float(np.mean(ms)) * 1e-3
    tested = 4 * ks.KS_CATALOGUE_SIZE
    kept = sum(int(r[2].item()) for r in res)
    out_bytes = kept * 20
    cpu = None
    if not args.no_cpu_baseline:
        import oracle
        t0 = time.perf_counter()
        n_ref = sum(len(oracle.valid_catalogue(probs[i:i + 1], desc, 1, dtype=wl.CANDIDATE_DT)[1])
                    for i in range(4))
        t_ref = time.perf_counter() - t0
        assert n_ref == kept, (n_ref, kept)
        cpu = {"value": tested / t_ref, "unit": "candidates/s", "cores": 1, "kind": "oracle",
               "sample": f"the same four layouts, {t_ref:.2f} s"}
    peaks = load_peaks()
    line = {"metric": "candidates/sec tested (enumerate + validity rules + ordered compaction, 4 layouts)",
            "value": tested / t, "unit": "candidates/s", "n_gpus": 1, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": t * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "int32", "data": "synthetic",
            "config": {"workload": "search space of Table Configuration knobs, 534,600 ids x 4 layouts",
                       "valid": kept, "l2": "256 MiB flush between steps"},
            "clocks": clocks, "gpu_launches": launches,
            "roofline": {"bound": "hbm", "achieved": out_bytes / t / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                         "frac": out_bytes / t / 1e9 / peaks["hbm_gbs"], "traffic": None,
                         "note": "20 B written per valid candidate, nothing read: twelve launches of a few "
                                 "microseconds each, launch-latency bound"},
            "cpu_baseline": cpu, "e2e": None}
    print(json.dumps(line), flush=True)


def run_stages(args, rank, local_rank, dev):
    """The unfused calls of the boundary, one at a time: `ks_featurize` writes the padded feature
    rows of every pair to HBM (256 B each), `ks_score` reads them back and scores them with the
    tree ensemble of config 1 and with the MLP of config 4. The fused `ks_select` never does this
    round trip; these lines say what it would cost. Each call is timed alone with CUDA events,
    with a 256 MiB L2 flush in front (the feature matrix is far larger than L2 anyway)."""
    if rank != 0:
        return
    import torch
    from paper_2609_35587_b200 import binding as ks
    from paper_2609_35587_b200 import workloads as wl
    P = args.problems or 64
    w = wl.make_workload(1, P=P)
    w4 = wl.make_workload(4, P=1)
    C = len(w.candidates)
    pairs = P * C
    ctx = ks.Context(w.desc, local_rank)
    gbdt = ctx.model_create_gbdt(*w.gbdt)
    mlp = ctx.model_create_mlp(w4.mlp)
    d_p, d_c = ks.to_device(w.problems, dev), ks.to_device(w.candidates, dev)
    feat = torch.empty((pairs, ks.KS_F_PAD), dtype=torch.float32, device=dev)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    peaks = load_peaks()
    row_bytes = 4 * ks.KS_F_PAD
    calls = [
        ("ks_featurize", lambda: ctx.featurize(d_p, P, d_c, C, out=feat), pairs * row_bytes + C * 16 + P * 16),
        ("ks_score (500 trees, depth 8)", lambda: ctx.score(feat, gbdt), pairs * (row_bytes + 4)),
        ("ks_score (MLP 64-256-256-1)", lambda: ctx.score(feat, mlp), pairs * (row_bytes + 4)),
    ]
    sampler = ClockSampler(local_rank)
    sampler.start()
    launches0 = ctx.launch_count()
    stages = []
    for name, fn, nbytes in calls:
        for _ in range(max(args.warmup, 3)):
            fn()
        torch.cuda.synchronize()
        ms = []
        for _ in range(args.steps):
            flush.fill_(1)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            fn()
            e1.record()
            torch.cuda.synchronize()
            ms.append(e0.elapsed_time(e1))
        t = float(np.mean(ms)) * 1e-3
        stages.append({"call": name, "ms": t * 1e3, "pairs_per_s": pairs / t,
                       "roofline": {"bound": "hbm", "achieved": nbytes / t / 1e9, "peak": peaks["hbm_gbs"],
                                    "unit": "GB/s", "frac": nbytes / t / 1e9 / peaks["hbm_gbs"],
                                    "peak_source": peaks["source"]}})
    clocks = sampler.stop()
    line = {"metric": "unfused boundary calls, each timed alone (feature rows through HBM)",
            "value": stages[0]["pairs_per_s"], "unit": "pairs/s (ks_featurize)", "n_gpus": 1, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": stages[0]["ms"], "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": "config 1 (full_space) catalogue and ensemble, config 4 MLP", "problems": P,
                       "candidates_per_problem": C, "l2": "256 MiB flush before every call"},
            "clocks": clocks, "gpu_launches": int(ctx.launch_count() - launches0), "stages": stages,
            "cpu_baseline": None, "e2e": None}
    print(json.dumps(line), flush=True)


def measure_select(ks, ctx, w, model, steps, warm, dev, flush, world=1, gather=None):
    """K timed passes of ks_select over workload `w` (inputs resident on the device), each
    bracketed by CUDA events on the launching stream with an L2 flush in front. Returns the
    per-step times, the dominant kernel's own times, and the launches counted."""
    import torch
    import torch.distributed as dist
    P, C, k = len(w.problems), len(w.candidates), w.k
    d_p, d_c = ks.to_device(w.problems, dev), ks.to_device(w.candidates, dev)
    d_so = None if w.seg_offsets is None else ks.to_device(w.seg_offsets, dev)
    d_si = None if w.seg_index is None else ks.to_device(w.seg_index, dev)
    out_idx = torch.empty((P, k), dtype=torch.int32, device=dev)
    out_sc = torch.empty((P, k), dtype=torch.float32, device=dev)

    def step():
        ctx.select(d_p, P, d_c, C, model, k, d_so, d_si, w.pairs, out_idx, out_sc)
        if gather is not None:  # N > 1: the one exchange of the sharded path
            gather(out_idx, out_sc)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(warm):
        step()
    barrier()
    ctx.profile_enable(True)
    launches0 = ctx.launch_count()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    kern_ms = []
    barrier()
    for i in range(steps):
        flush.fill_(i & 0xFF)
        ev[i][0].record()
        step()
        ev[i][1].record()
        kern_ms.append(ctx.profile_last_ms())
    barrier()
    ctx.profile_enable(False)
    return {"step_ms": [a.elapsed_time(b) for a, b in ev], "kernel_ms": kern_ms,
            "launches": int(ctx.launch_count() - launches0)}


def tree_roofline(pairs, trees, depth, kms):
    achieved = pairs * trees * depth * INSTR_PER_VISIT / (kms * 1e-3)
    return achieved, achieved / ISSUE_PEAK


def walk_floor(ks, ctx, w, model, dev):
    """The tree walk stripped to its gather and instruction stream (ks_debug_walk_floor): feature
    rows of the workload's first problems, 592 blocks of 1,024 rows (whole waves of 148 or 296
    CTAs); the time of one pass over the ensemble is the difference of two calls that differ in
    their number of passes only, so tile building, launches and the first copies cancel. The rows
    are those of the catalogue in similarity order, as the product kernel's tiles are."""
    import torch
    rows = 592 * 1024
    C = len(w.candidates)
    P = -(-rows // C)
    # the catalogue in the similarity order the product ranks it in (the same sort keys), so that a
    # warp's lanes hold neighbouring candidates here as they do there
    c = w.candidates
    order = np.lexsort((c["instr_n"] != c["tile_n"], c["tile_sched"], c["epi_sched"], c["kernel_sched"],
                        c["cluster_n"], c["cluster_m"], c["stages"], c["tile_k"], c["tile_n"], c["tile_m"]))
    d_p, d_c = ks.to_device(w.problems[:P], dev), ks.to_device(np.ascontiguousarray(c[order]), dev)
    feat = ctx.featurize(d_p, P, d_c, C)[:rows]
    out = torch.empty(rows, dtype=torch.float32, device=dev)
    lo, hi = 2, 10

    def timed(repeat):
        best = float("inf")
        for _ in range(4):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            e0.record()
            ctx.debug_walk_floor(feat, model, repeat, out)
            e1.record()
            torch.cuda.synchronize()
            best = min(best, e0.elapsed_time(e1))
        return best

    timed(lo)
    t_lo, t_hi = timed(lo), timed(hi)
    pass_ms = (t_hi - t_lo) / (hi - lo)
    trees, depth = len(w.gbdt[0]) - 1, 8  # config 1's ensemble: complete trees of depth 8
    return {"rows": rows, "pass_ms": pass_ms, "passes": [lo, hi], "call_ms": [t_lo, t_hi],
            "frac": tree_roofline(rows, trees, depth, pass_ms)[1], "kernel": model.describe()}


def extra_runs(ks, ctx, dev, flush, args, peaks):
    """Short runs of the other configurations and threshold laws, so that one default line carries
    them: config 1 under the other two laws, config 2, config 4 (5 / 3 timed steps each), a
    short latency stream, and the oracle on one host thread."""
    import torch
    from paper_2609_35587_b200 import workloads as wl
    out = {}
    for law in [l for l in wl.LAWS if l != args.law]:
        w = wl.make_workload(1, law=law)
        model = ctx.model_create_gbdt(*w.gbdt)
        m = measure_select(ks, ctx, w, model, 5, 3, dev, flush)
        kms = float(np.mean(m["kernel_ms"]))
        out[f"config1_{law}"] = {"pairs_per_s": w.pairs / (np.mean(m["step_ms"]) * 1e-3), "ms_per_step": float(np.mean(m["step_ms"])),
                                 "kernel_ms": kms, "frac": tree_roofline(w.pairs, 500, 8, kms)[1], "kernel": model.describe()}
        out[f"walk_floor_{law}"] = walk_floor(ks, ctx, w, model, dev)
        model.close()
    w = wl.make_workload(1, law=args.law)
    model = ctx.model_create_gbdt(*w.gbdt)
    out[f"walk_floor_{args.law}"] = walk_floor(ks, ctx, w, model, dev)
    model.close()
    w = wl.make_workload(2, law=args.law)
    model = ctx.model_create_gbdt(*w.gbdt)
    m = measure_select(ks, ctx, w, model, 3, 3, dev, flush)
    kms = float(np.mean(m["kernel_ms"]))
    out[f"config2_{args.law}"] = {"pairs_per_s": w.pairs / (np.mean(m["step_ms"]) * 1e-3), "ms_per_step": float(np.mean(m["step_ms"])),
                                  "kernel_ms": kms, "frac": tree_roofline(w.pairs, 1000, 8, kms)[1], "kernel": model.describe()}
    model.close()
    del w
    w = wl.make_workload(4)
    model = ctx.model_create_mlp(w.mlp)
    m = measure_select(ks, ctx, w, model, 5, 3, dev, flush)
    kms = float(np.mean(m["kernel_ms"]))
    tflops = w.pairs * 2.0 * (64 * 256 + 256 * 256) / (kms * 1e-3) / 1e12
    out["config4"] = {"pairs_per_s": w.pairs / (np.mean(m["step_ms"]) * 1e-3), "ms_per_step": float(np.mean(m["step_ms"])),
                      "kernel_ms": kms, "tflops": tflops, "frac_of_sustained_bf16": tflops / peaks["bf16_tflops_sustained"],
                      "frac_of_burst_bf16": tflops / peaks["bf16_tflops"], "kernel": model.describe()}
    model.close()
    # latency stream, short
    w = wl.make_workload(3, P=2200, law=args.law)
    model = ctx.model_create_gbdt(*w.gbdt)
    d_c = ks.to_device(w.candidates, dev)
    cat = ctx.catalogue_prepare(d_c, len(w.candidates), model)
    call = ctx.select_one_caller(d_c, len(w.candidates), model, w.k, catalogue=cat)
    structs = ks.problem_structs(w.problems)
    for i in range(200):
        call(structs[i])
    lat = np.empty(2000)
    t_all = time.perf_counter()
    for i in range(2000):
        t0 = time.perf_counter()
        call(structs[200 + i])
        lat[i] = time.perf_counter() - t0
    total = time.perf_counter() - t_all
    out[f"config3_{args.law}"] = {"problems_per_s": 2000 / total, "p50_us": float(np.percentile(lat, 50) * 1e6),
                                  "p99_us": float(np.percentile(lat, 99) * 1e6), "calls": 2000}
    model.close()
    # the oracle on one host thread (config 1, first two problems)
    import oracle
    w = wl.make_workload(1, P=2, law=args.law)
    n_thr = oracle.threads()
    oracle.set_threads(1)
    t0 = time.perf_counter()
    oracle.select(w.problems, w.candidates, w.desc, w.k, gbdt=w.gbdt)
    dt = time.perf_counter() - t0
    oracle.set_threads(n_thr)
    out["oracle_1_thread"] = {"value": w.pairs / dt, "unit": UNIT, "cores": 1, "sample": f"2 problems x 60000 candidates of config 1, {dt:.1f} s"}
    return out


def spawn_ranks(args):
    """`python bench.py --gpus N` with N > 1 and no launcher around it: start the N ranks here, one
    process per GPU, the way the multi-rank launch line does."""
    import socket
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", type=int, default=1, choices=[0, 1, 2, 3, 4])
    ap.add_argument("--law", default="pernode", choices=["pernode", "hist256", "slots128"],
                    help="threshold law of the synthetic tree ensemble (workloads.LAWS)")
    ap.add_argument("--calls", type=int, default=100000, help="latency stream (workload 3): timed calls")
    ap.add_argument("--unprepared", action="store_true",
                    help="latency stream: plain ks_select_one instead of the prepared-catalogue call")
    ap.add_argument("--ref-problems", type=int, default=16)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extra", action="store_true",
                    help="leave out the short runs of the other configurations that the default line carries")
    ap.add_argument("--problems", type=int, default=None,
                    help="profiling aid: rank only the first N problems of the workload (not a bench line)")
    ap.add_argument("--skip-e2e", action="store_true", help="profiling aid: skip the host-buffer leg")
    ap.add_argument("--catalogue", action="store_true",
                    help="measure the search-space enumeration + validity filter instead of a selection workload")
    ap.add_argument("--stages", action="store_true",
                    help="time the unfused calls (ks_featurize, ks_score) one at a time instead of ks_select")
    ap.add_argument("--floor", action="store_true",
                    help="measure the tree walk's gather stream alone (ks_debug_walk_floor) on config 1's ensemble")
    args = ap.parse_args()

    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(spawn_ranks(args))
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        run_reference(args, rank, world)
        return

    import torch
    import torch.distributed as dist
    from paper_2609_35587_b200 import binding as ks
    from paper_2609_35587_b200 import sharding
    from paper_2609_35587_b200 import workloads as wl

    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    cfg = args.workload
    spec = wl.CONFIGS[cfg]
    if world > 1 and cfg != 3 and not args.catalogue and not args.stages and not args.floor:
        dist.init_process_group("nccl", device_id=dev)
    if args.catalogue:
        run_catalogue(args, rank, local_rank, dev)
        return
    if args.stages:
        run_stages(args, rank, local_rank, dev)
        return
    if args.floor:
        if rank == 0:
            w = wl.make_workload(1, P=12, law=args.law)
            ctx = ks.Context(w.desc, local_rank)
            model = ctx.model_create_gbdt(*w.gbdt)
            f = walk_floor(ks, ctx, w, model, dev)
            print(json.dumps({"metric": "tree walk, gather stream alone (fraction of the issue roofline)", "value": f["frac"],
                              "unit": "fraction", "n_gpus": 1, "higher_is_better": True, "data": "synthetic",
                              "config": {"workload": f"config 1 ensemble, thresholds: {args.law}", **f}}), flush=True)
        return
    if cfg == 3:
        run_latency_stream(args, rank, local_rank, dev)
        return
    # weak scaling: every rank ranks its own batch of problems against the shared catalogue; with
    # N > 1 the [P, k] result blocks are all-gathered at the end of every step (the only exchange)
    w = wl.make_workload(cfg, P=args.problems, seed=wl.BASE_SEED, law=args.law)
    if rank != 0:
        w.problems = wl.make_inputs(cfg, P=args.problems, seed=wl.BASE_SEED + 7919 * rank)[0]
    P, C, k = len(w.problems), len(w.candidates), w.k
    ctx = ks.Context(w.desc, local_rank)
    model = ctx.model_create_gbdt(*w.gbdt) if w.gbdt is not None else ctx.model_create_mlp(w.mlp)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    pairs = w.pairs
    gather = (lambda i, s: sharding.all_gather_topk(i, s, P * world, k)) if world > 1 else None

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    n_warm = args.warmup if args.problems else max(args.warmup, 3)
    sampler = ClockSampler(local_rank)
    sampler.start()
    m = measure_select(ks, ctx, w, model, args.steps, n_warm, dev, flush, world, gather)
    clocks = sampler.stop()
    launches, kern_ms = m["launches"], m["kernel_ms"]
    total_ms = float(sum(m["step_ms"]))
    if world > 1:
        total_ms = sharding.max_over_ranks(total_ms, dev)
    ms_per_step = total_ms / args.steps
    value = world * pairs / (ms_per_step * 1e-3)

    # ---- end to end: host buffers in, host results out, through the C ABI ------------------------
    h_p = torch.from_numpy(w.problems.view(np.uint8).reshape(P, 16).copy()).pin_memory()
    h_c = torch.from_numpy(w.candidates.view(np.uint8).reshape(C, 16).copy()).pin_memory()
    h_so = None if w.seg_offsets is None else torch.from_numpy(w.seg_offsets.copy()).pin_memory()
    h_si = None if w.seg_index is None else torch.from_numpy(w.seg_index.copy()).pin_memory()
    h_idx = torch.empty((P, k), dtype=torch.int32).pin_memory()
    h_sc = torch.empty((P, k), dtype=torch.float32).pin_memory()
    e2e_steps = 0 if args.skip_e2e else max(3, min(args.steps, 10))
    for _ in range(0 if args.skip_e2e else 2):
        ctx.select_host(h_p, P, h_c, C, model, k, h_so, h_si, pairs, h_idx, h_sc)
    barrier()
    t0 = time.perf_counter()
    for i in range(e2e_steps):
        flush.fill_(i & 0xFF)
        ctx.select_host(h_p, P, h_c, C, model, k, h_so, h_si, pairs, h_idx, h_sc)
    barrier()
    e2e_s = (time.perf_counter() - t0) / max(e2e_steps, 1)
    if world > 1:
        e2e_s = sharding.max_over_ranks(e2e_s, dev)
    e2e_value = world * pairs / e2e_s
    h2d = P * 16 + C * 16 + (0 if h_so is None else h_so.numel() * 8 + h_si.numel() * 4)
    d2h = P * k * 8

    if rank == 0:
        peaks = load_peaks()
        kms = float(np.mean(kern_ms))
        cfgd = config_dict(cfg, spec, args)
        cfgd["l2"] = "flushed before every step of both legs (256 MiB write)"
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": n_warm, "ms_per_step": ms_per_step, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "data": "synthetic",
                "config": cfgd, "clocks": clocks, "gpu_launches": int(launches),
                "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": int(h2d),
                        "d2h_bytes_per_step": int(d2h)}}
        if w.gbdt is not None:
            achieved, frac = tree_roofline(pairs, spec["trees"], spec["depth"], kms)
            line["dtype"] = "f32"
            line["roofline"] = {"bound": "alu", "kernel": model.describe(),
                                "achieved": achieved / 1e12, "peak": ISSUE_PEAK / 1e12,
                                "unit": "T thread-instr/s (4 per node visit)",
                                "frac": frac, "kernel_ms": kms,
                                "peak_source": "derived: 148 SMs x 4 schedulers x 32 lanes x 1.965 GHz",
                                "traffic": TRAFFIC_BYTES.get((cfg, args.law))}
        else:
            flops = pairs * 2.0 * (64 * 256 + 256 * 256)
            achieved = flops / (kms * 1e-3)
            line["dtype"] = "bf16"
            line["roofline"] = {"bound": "tensor", "kernel": model.describe(),
                                "achieved": achieved / 1e12, "peak": peaks["bf16_tflops_sustained"],
                                "unit": "TFLOP/s", "frac": achieved / 1e12 / peaks["bf16_tflops_sustained"],
                                "frac_of_burst": achieved / 1e12 / peaks["bf16_tflops"],
                                "kernel_ms": kms, "peak_source": peaks["source"] + " (sustained bf16)",
                                "traffic": TRAFFIC_BYTES.get((cfg, None))}
        if not args.no_cpu_baseline and world == 1:
            line["cpu_baseline"] = cpu_baseline(cfg, args.law)
        if world == 1 and cfg == 1 and not args.problems and not args.no_extra:
            model.close()
            line["extra"] = extra_runs(ks, ctx, dev, flush, args, peaks)
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


# dram__bytes_read.sum + dram__bytes_write.sum of the dominant kernel per full-size step, from the
# ncu captures of the 48-problem case under profiles/, scaled by the problems (None: no capture
# for that workload). Config 1, per-node law: 15.7 MB read in the small case (catalogue, model,
# per-call tables, the class records of 48 problems) + 0.24 MB of class records per further
# problem (written by the table kernel, read once) + 4.8 MB of partial lists written.
TRAFFIC_BYTES = {(1, "pernode"): 255e6, (1, "slots128"): 229e6, (4, None): 5.7e6}

if __name__ == "__main__":
    main()
