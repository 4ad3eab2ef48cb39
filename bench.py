#!/usr/bin/env python
"""Benchmark of the sparsified-SGD compress + aggregate step on B200.

One "step" is one pass of the whole hot path over one batch of synthetic
gradients: for each sparsifier of the workload (top-k, random-k, block-random-k)
W workers are compressed (error-feedback add, selection, packing, residual
writeback) and their messages are aggregated into one dense average.  The
metric is gradient elements compressed per second (W * n * schemes / time).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Prints ONE JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "compress+aggregate gradient elements/s"
UNIT = "elements/s"
CONTRACT_PEAK_GBS = 8000.0        # the nominal B200 HBM figure the target is stated against
FALLBACK_PEAK_GBS = 6650.0        # used only if MEASURED_PEAKS.json is absent
# DRAM bytes per gradient element of the streaming kernels, measured once with ncu on a small case
NCU_DRAM_BYTES_PER_ELEMENT = {"topk_main": 11.84, "randk_pack": 11.94, "randblock": 11.80}


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c5", help="c1..c5 (default: the largest, flat 350M x 16 workers)")
    ap.add_argument("--density", default="1/100", help="kept fraction num/den (default: the paper's 1 %%)")
    ap.add_argument("--schemes", default="", help="comma list; default: all schemes of the workload")
    ap.add_argument("--n", type=int, default=0, help="override elements per worker (flat workloads only)")
    ap.add_argument("--workers", type=int, default=0, help="override W")
    ap.add_argument("--pool", type=int, default=2, help="distinct gradient sets cycled through the steps")
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-kernel-events", action="store_true",
                    help="do not bracket every kernel with events in the timed region (no roofline object)")
    ap.add_argument("--cpu-sample-div", type=int, default=1, help="oracle sample = n / this of one worker")
    ap.add_argument("--scope", default="layerwise", choices=["layerwise", "flat"],
                    help="one k per tensor of the workload, or one segment over the whole vector")
    ap.add_argument("--no-sweep", action="store_true",
                    help="skip the sweep over the other densities and workloads that follows the default run")
    ap.add_argument("--sweep-steps", type=int, default=10)
    ap.add_argument("--selftest-dist", action="store_true",
                    help="CPU-only check of the multi-rank plumbing (gloo): barrier, max over ranks, aggregate value")
    return ap.parse_args()


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_PEAK_GBS, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, uuid: str):
        self.uuid, self.proc, self.path = uuid, None, None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(prefix="sc_clocks_", suffix=".csv")
            self.proc = subprocess.Popen(["nvidia-smi", "-i", self.uuid, f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=fd, stderr=subprocess.DEVNULL)
            os.close(fd)
            time.sleep(0.3)
        except Exception:
            self.proc = None

    def stop(self) -> dict:
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        try:
            rows = [r.strip().split(",") for r in open(self.path) if r.strip()]
            os.unlink(self.path)
        except Exception:
            return out
        sm, mx, pw, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1])); pw.append(float(r[2]))
                for name, v in zip(names, r[3:7]):
                    if v.strip().lower().startswith("active"):
                        reasons.add(name)
            except Exception:
                continue
        if sm:
            busy = [c for c, p in zip(sm, pw) if p >= 0.5 * max(pw)] or sm
            out.update(sm_mhz=statistics.median(busy), sm_max_mhz=max(mx), reasons=sorted(reasons),
                       samples=len(sm), power_w_max=max(pw))
        return out


def algorithmic_bytes(kind: str, n: int, W: int, K: int, shared: bool) -> float:
    """Bytes one launch of a kernel must move by the definition of its step
    (operands read once, results written once)."""
    return {
        "randk_pack": 12.0 * n * W + n / 8.0 * W + 8.0 * K * W,  # read g, e, mask; write e', vals, idx
        "mask_count": n / 8.0, "row_scan": 8.0 * (n / 4096.0),
        "randblock": 12.0 * n * W + 8.0 * K * W,
        "randk_scatter": 4.0 * K,
        "agg_tiles": 4.0 * n + (4.0 * K * W + 4.0 * K if shared else 8.0 * K * W),
        "agg_warp": 4.0 * n + 8.0 * K * W, "agg_fine": 4.0 * n + 8.0 * K * W,     # private coordinates (top-k)
        "agg_bounds": 4.0 * (n / 4096.0) * (1 if shared else W),
        "topk_main": 12.0 * n * W + 8.0 * K * W,          # read g, e; write e' and the flagged (value, coordinate) list
        "topk_emit": 16.0 * K * W,                        # read the flagged list, write vals and idx
    }.get(kind, 0.0)


def step_min_bytes(scheme: str, n: int, W: int, K: int, shared: bool) -> float:
    """Minimum traffic of one whole step: read g and e, write e', write and read the messages,
    write the dense average."""
    if scheme == "topk" or not shared:
        return 12.0 * n * W + 16.0 * K * W + 4.0 * n
    return 12.0 * n * W + 8.0 * K * W + 8.0 * K + 4.0 * n


class Ranks:
    """Process-group plumbing of the benchmark: one process per GPU, no data-path collective.
    Only the timing is reduced (max over ranks) and the per-rank work summed."""

    def __init__(self, world: int, backend: str, device=None):
        self.world, self.dist, self.device = world, None, device
        if world > 1:
            import torch.distributed as dist
            kwargs = {"device_id": device} if backend == "nccl" and device is not None else {}
            dist.init_process_group(backend, **kwargs)
            self.dist = dist

    def barrier(self):
        if self.dist is not None:
            self.dist.barrier()

    def max_ms(self, ms: float) -> float:
        if self.dist is None:
            return ms
        import torch
        t = torch.tensor([ms], dtype=torch.float64, device=self.device if self.device is not None else "cpu")
        self.dist.all_reduce(t, op=self.dist.ReduceOp.MAX)
        return float(t.item())

    def whole_job_value(self, units_per_rank_per_step: float, steps: int, ms: float) -> float:
        """Units all ranks processed divided by the slowest rank's time."""
        return self.world * units_per_rank_per_step * steps / (self.max_ms(ms) * 1e-3)

    def close(self):
        if self.dist is not None:
            self.dist.barrier()
            self.dist.destroy_process_group()


def run_selftest_dist(args, rank: int, world: int):
    """No GPU: every rank pretends to have timed `steps` steps in (10 + 5 rank) ms."""
    ranks = Ranks(world, "gloo")
    ranks.barrier()
    value = ranks.whole_job_value(1000.0, args.steps, 10.0 + 5.0 * rank)
    ranks.barrier()
    if rank == 0:
        print(json.dumps({"selftest": "dist", "n_gpus": world, "value": value,
                          "max_ms": 10.0 + 5.0 * (world - 1)}), flush=True)
    ranks.close()


def build_problem(args):
    import workloads as wl
    w = wl.workload(args.workload)
    num, den = (int(x) for x in args.density.split("/"))
    sizes = list(w.sizes)
    if args.n:
        sizes = [args.n]
    W = args.workers or w.W
    schemes = [s for s in (args.schemes.split(",") if args.schemes else w.schemes) if s]
    segs = wl.flat_table(sum(sizes), num, den) if args.scope == "flat" else wl.segment_table(sizes, num, den)
    return w, sizes, W, schemes, segs, (num, den)



# The other configurations of the metric: every (workload, scope, density) below is timed like the
# headline (W workers per step, CUDA events around `steps` whole steps of one scheme, a fresh gradient
# set every step out of `pool`, residuals carried, clocks sampled), without per-kernel events.
SWEEP_PLAN = (
    ("c5", "flat", ((1, 10000), (1, 1000), (1, 10))),          # 1/100 is the headline itself
    ("c1", "flat", ((1, 100),)),
    ("c2", "layerwise", ((1, 100),)),
    ("c3", "layerwise", ((1, 1000),)),
    ("c4", "layerwise", ((1, 1000), (1, 100), (1, 10))),
    ("c4", "flat", ((1, 1000), (1, 100), (1, 10))),
)


def time_schemes(torch, sc, ctx, wl, w, W, n, schemes, seg_t, K, grads, res, vals, idx, out, steps, warmup, peak, uuid):
    """One sweep entry: per scheme `warmup` untimed steps, then `steps` timed ones."""
    pool = len(grads)
    sampler = ClockSampler(uuid)
    sampler.start()
    per, paths = {}, None
    for s in schemes:
        code = sc.SCHEMES[s]
        for t in range(warmup):
            ctx.sc_step(code, grads[t % pool], res[s], seg_t, [wl.step_seed(w.base_seed, t)] * W, vals, idx, out)
        if s == "topk":
            paths = dict(zip(("radix_small", "one_pass", "radix_after_missed_bracket"), ctx.sc_topk_path_counts()))
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for t in range(steps):
            ctx.sc_step(code, grads[(warmup + t) % pool], res[s], seg_t,
                        [wl.step_seed(w.base_seed, warmup + t)] * W, vals, idx, out)
        b.record()
        torch.cuda.synchronize()
        ms = a.elapsed_time(b) / steps
        bmin = step_min_bytes(s, n, W, K, shared=True)
        per[s] = {"ms": round(ms, 4), "elements_per_s": W * n / (ms * 1e-3), "min_GB": round(bmin / 1e9, 4),
                  "frac_of_8000": round(bmin / (ms * 1e-3) / 1e9 / CONTRACT_PEAK_GBS, 4),
                  "frac_of_measured": round(bmin / (ms * 1e-3) / 1e9 / peak, 4)}
    status = ctx.sc_sync_status()
    if status != 0:
        raise RuntimeError(f"device status in the sweep: {sc.strerror(status)}")
    return per, paths, sampler.stop()


def run_sweep(args, torch, sc, wl, dev, peak, uuid, c5_state):
    """Returns the list of sweep entries.  c5_state = (ctx, grads, res, out) of the headline run, reused for
    the other densities of the largest workload; the smaller workloads get buffers of their own."""
    entries = []
    for name, scope, densities in SWEEP_PLAN:
        w = wl.workload(name)
        n, W = w.n, w.W
        if name == "c5":
            ctx, grads, res, out = c5_state
            own = False
        else:
            ctx = sc.Context(max_n=n, max_W=W, max_segments=len(w.sizes))
            grads = []
            for t in range(max(1, args.pool)):
                g = torch.empty(W, n, device=dev)
                for ww in range(W):
                    g[ww] = wl.generate(w, ww, t, dev)
                grads.append(g)
            res = {s: torch.zeros(W, n, device=dev) for s in w.schemes}
            out = torch.empty(n, device=dev)
            own = True
        for num, den in densities:
            segs = wl.flat_table(n, num, den) if scope == "flat" else wl.segment_table(w.sizes, num, den)
            seg_t = [(s.offset, s.n, s.k) for s in segs]
            K = sum(s.k for s in segs)
            vals = torch.empty(W, max(K, 1), device=dev)
            idx = torch.empty(W, max(K, 1), device=dev, dtype=torch.int32)
            for s in w.schemes:
                res[s].zero_()
            per, paths, clocks = time_schemes(torch, sc, ctx, wl, w, W, n, w.schemes, seg_t, K, grads, res, vals, idx,
                                              out, args.sweep_steps, max(3, args.warmup), peak, uuid)
            entries.append({"config": name, "scope": scope, "density": f"{num}/{den}", "n": n, "W": W,
                            "segments": len(segs), "k": K, "steps": args.sweep_steps,
                            "l2": "working set fits L2" if 8.0 * n * W < 100e6 else "inputs larger than L2",
                            "schemes": per, "topk_paths": paths, "clocks": clocks})
            del vals, idx
        if own:
            ctx.close()
            del grads, res, out
            torch.cuda.empty_cache()
    return entries


def run_reference(args, rank: int):
    """Times the CPU oracle, as it stands, on a bounded sample of the same workload."""
    if rank != 0:
        return
    import numpy as np
    import torch
    import workloads as wl
    from oracle import sparsify_oracle as O
    w, sizes, W, schemes, segs, (num, den) = build_problem(args)
    n_full = sum(sizes)
    # sample: one worker, the first n/div elements of a flat vector (or the whole table if it is small)
    if len(sizes) == 1 and n_full > 50_000_000:
        sizes = [n_full // args.cpu_sample_div]
    segs = wl.segment_table(sizes, num, den)
    n = sum(sizes)
    seg_t = [(s.offset, s.n, s.k) for s in segs]
    torch.manual_seed(0)
    times = []
    e = {s: np.zeros(n, np.float32) for s in schemes}
    for t in range(args.warmup + args.steps):
        g = wl.generate(w, 0, t, "cpu", sizes=sizes).numpy()
        t0 = time.perf_counter()
        for s in schemes:
            v, i, e_new = O.compress_segments(O.SCHEMES[s], g, e[s], seg_t, wl.step_seed(w.base_seed, t))
            O.aggregate([v], [i], n)
            e[s] = e_new
        if t >= args.warmup:
            times.append(time.perf_counter() - t0)
    total = sum(times)
    value = n * len(schemes) * len(times) / total
    sample = (f"worker 0 only, {n} of {n_full} elements per step, schemes {','.join(schemes)}, density {num}/{den}, "
              f"compress + aggregate of that one message (W=1)")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / len(times),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": f"{w.name}: n={n_full} W={W} density={num}/{den}", "kind": "numpy oracle on host cores"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def run_ours(args, rank: int, world: int, local_rank: int):
    import torch
    import paper_2009_09271_b200 as sc
    import workloads as wl

    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    ranks = Ranks(world, "nccl", dev)

    def barrier():
        torch.cuda.synchronize()
        ranks.barrier()
        torch.cuda.synchronize()

    w, sizes, W, schemes, segs, (num, den) = build_problem(args)
    n = sum(sizes)
    K = sum(s.k for s in segs)
    seg_t = [(s.offset, s.n, s.k) for s in segs]
    codes = [sc.SCHEMES[s] for s in schemes]
    pool = max(1, args.pool)

    ctx = sc.Context(max_n=n, max_W=W, max_segments=len(segs))
    grads = []
    for t in range(pool):
        g = torch.empty(W, n, device=dev)
        for ww in range(W):
            g[ww] = wl.generate(w, ww + 1000 * rank, t, dev, sizes=sizes)
        grads.append(g)
    res = {s: torch.zeros(W, n, device=dev) for s in schemes}
    vals = torch.empty(W, max(K, 1), device=dev)
    idx = torch.empty(W, max(K, 1), device=dev, dtype=torch.int32)
    out = torch.empty(n, device=dev)

    def seeds(t):
        return [wl.step_seed(w.base_seed, t)] * W          # shared coordinates (the paper's allReduce mode)

    def one_step(t, marks=None):
        for s, code in zip(schemes, codes):
            ctx.sc_step(code, grads[t % pool], res[s], seg_t, seeds(t), vals, idx, out)
            if marks is not None:
                ev = torch.cuda.Event(enable_timing=True)
                ev.record()
                marks.append(ev)

    for t in range(args.warmup):
        one_step(t)
    topk_paths = None
    if "topk" in schemes:                       # which top-k path served the segments (not timed)
        ctx.sc_step(sc.SC_TOPK, grads[0], res["topk"], seg_t, seeds(0), vals, idx, out)
        topk_paths = dict(zip(("radix_small", "one_pass", "radix_after_missed_bracket"), ctx.sc_topk_path_counts()))
    status = ctx.sc_sync_status()
    if status != 0:
        raise RuntimeError(f"device status after warm-up: {sc.strerror(status)}")

    sampler = ClockSampler(str(torch.cuda.get_device_properties(dev).uuid))
    if not sampler.uuid.startswith("GPU-"):
        sampler.uuid = "GPU-" + sampler.uuid
    # The timed region.  A measurement taken while the GPU reported a hardware or thermal slowdown, or with
    # the SM clock far below its maximum for no stated reason, is thrown away and taken once more (every rank
    # repeats, so that the collective calls stay matched); sw_power_cap is kept and reported.
    remeasured = False
    for attempt in range(2):
        barrier()
        if rank == 0:
            sampler.start()
        ctx.sc_profile(not args.no_kernel_events)
        launches0 = ctx.launch_count
        marks = []
        start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        start.record()
        for t in range(args.steps):
            one_step(args.warmup + t, marks)
        end.record()
        barrier()
        elapsed_ms = start.elapsed_time(end)
        launches = ctx.launch_count - launches0
        prof = ctx.sc_profile_read()
        ctx.sc_profile(False)
        clocks = sampler.stop() if rank == 0 else {}
        status = ctx.sc_sync_status()
        if status != 0:
            raise RuntimeError(f"device status after the timed region: {sc.strerror(status)}")
        elapsed_ms = ranks.max_ms(elapsed_ms)
        bad = 0.0
        if rank == 0 and clocks.get("samples"):
            slow = {"hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown"} & set(clocks["reasons"])
            stuck = (not clocks["reasons"]) and clocks["sm_mhz"] < 0.8 * clocks["sm_max_mhz"]
            bad = 1.0 if (slow or stuck) else 0.0
        bad = ranks.max_ms(bad)                               # rank 0 decides for everyone
        if bad == 0.0 or attempt == 1:
            break
        remeasured = True
    if rank == 0 and clocks:
        clocks["remeasured"] = remeasured

    # per-scheme device time from the marks
    per_scheme_ms = {s: 0.0 for s in schemes}
    prev = start
    step_ms, acc = [], 0.0
    for i, ev in enumerate(marks):
        dt = prev.elapsed_time(ev)
        per_scheme_ms[schemes[i % len(schemes)]] += dt
        acc += dt
        if (i + 1) % len(schemes) == 0:                        # the last scheme of a step
            step_ms.append(acc)
            acc = 0.0
        prev = ev

    peak, peak_src = measured_peak()
    elems_per_step = W * n * len(schemes)
    value = world * elems_per_step * args.steps / (elapsed_ms * 1e-3)

    kernels = {}
    for kind, (ms, cnt) in prof.items():
        if cnt:
            b = algorithmic_bytes(kind, n, W, K, shared=True)
            kernels[kind] = {"launches": int(cnt), "ms_total": round(ms, 4), "ms_avg": round(ms / cnt, 5),
                             "share": round(ms / max(elapsed_ms, 1e-9), 4),
                             "alg_GBps": round(b / (ms / cnt * 1e-3) / 1e9, 1) if ms > 0 else None}
    dom = max(kernels, key=lambda k_: kernels[k_]["ms_total"]) if kernels else None
    roofline = None
    if dom:
        ach = kernels[dom]["alg_GBps"]
        roofline = {"bound": "hbm", "kernel": dom, "achieved": ach, "peak": peak, "unit": "GB/s",
                    "frac": round(ach / peak, 4), "peak_source": peak_src, "traffic": None}
        per_elem = NCU_DRAM_BYTES_PER_ELEMENT.get(dom)
        if per_elem is not None:
            roofline["traffic"] = per_elem * n * W
            roofline["traffic_note"] = ("dram__bytes_read.sum + dram__bytes_write.sum per element from one ncu capture "
                                        "of this kernel at n=1e8, W=2, scaled by n*W (traffic grows with n*W)")
        else:
            roofline["traffic_note"] = (f"no ncu capture of {dom} is on record: DRAM traffic per element was captured "
                                        "for the streaming kernels only (" + ", ".join(NCU_DRAM_BYTES_PER_ELEMENT) + ")")
    step_roof = {}
    for s in schemes:
        t_s = per_scheme_ms[s] / args.steps * 1e-3
        bmin = step_min_bytes(s, n, W, K, shared=True)
        step_roof[s] = {"ms": round(t_s * 1e3, 4), "elements_per_s": W * n / t_s, "min_GB": round(bmin / 1e9, 3),
                        "GBps_min_bytes": round(bmin / t_s / 1e9, 1),
                        "frac_of_8000": round(bmin / t_s / 1e9 / CONTRACT_PEAK_GBS, 4),
                        "frac_of_measured": round(bmin / t_s / 1e9 / peak, 4)}

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": elapsed_ms / args.steps,
        "ms_per_step_median": round(statistics.median(step_ms), 4) if step_ms else None,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic",
        "config": {"workload": f"{w.name}: flat n={n} x W={W} simulated workers per GPU, {w.values} values, "
                               f"density {num}/{den} (k={K}), schemes {','.join(schemes)}, shared seed per step, "
                               f"error feedback on, {pool} gradient sets cycled",
                   "segments": len(segs), "l2": "inputs (%.1f GB per scheme pass) far larger than L2" % (8e-9 * n * W),
                   "replicas": world},
        "gpu_launches": int(launches),
        "topk_paths": topk_paths,
        "clocks": clocks,
        "roofline": roofline,
        "per_scheme": step_roof,
        "kernels": kernels,
    }

    # ---- next row: aggregate fused with the model update (not part of the metric) ------------
    if rank == 0 and K > 0:
        xmodel = torch.zeros(n, device=dev)
        tim = {}
        for name, shared in (("aggregate_apply_ms", False), ("aggregate_apply_shared_ms", True)):
            ctx.sc_aggregate_apply(W, vals, idx, K, n, xmodel, shared=shared)          # warm-up
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            for _ in range(3):
                ctx.sc_aggregate_apply(W, vals, idx, K, n, xmodel, shared=shared)
            b.record()
            torch.cuda.synchronize()
            tim[name] = round(a.elapsed_time(b) / 3, 4)
        tim["note"] = ("x <- x - average applied at sent coordinates only, on the last scheme's messages; "
                       "the dense sc_aggregate of the same messages is in kernels.agg_tiles")

        # ---- next row: the block that wraps around, and the accumulate line with a step size -------
        def timed_step(code, gamma):
            e_tmp = res[schemes[-1]]                           # any residual buffer: the metric's run is over
            ctx.sc_set_gamma(gamma)
            ctx.sc_step(code, grads[0], e_tmp, seg_t, seeds(0), vals, idx, out)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            for t in range(3):
                ctx.sc_step(code, grads[t % pool], e_tmp, seg_t, seeds(t + 1), vals, idx, out)
            b.record()
            torch.cuda.synchronize()
            ctx.sc_set_gamma(1.0)
            return round(a.elapsed_time(b) / 3, 4)
        def timed_step_apply(code):
            e_tmp = res[schemes[-1]]
            xm = torch.zeros(n, device=dev)
            ctx.sc_step_apply(code, grads[0], e_tmp, seg_t, seeds(0), vals, idx, xm)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            for t in range(3):
                ctx.sc_step_apply(code, grads[t % pool], e_tmp, seg_t, seeds(t + 1), vals, idx, xm)
            b.record()
            torch.cuda.synchronize()
            return round(a.elapsed_time(b) / 3, 4)
        for s_ in schemes:
            tim[f"{s_}_step_apply_ms"] = timed_step_apply(sc.SCHEMES[s_])
        tim["note_step_apply"] = ("sc_step_apply: the whole step with x <- x - average applied at the sent coordinates "
                                  "instead of writing the dense average (compare per_scheme.*.ms)")
        tim["randblock_wrap_step_ms"] = timed_step(sc.SC_RANDBLOCK_WRAP, 1.0)
        tim["topk_step_gamma_0.1_ms"] = timed_step(sc.SC_TOPK, 0.1)
        tim["note_steps"] = ("whole sc_step (compress + aggregate) on this workload: wrap-around block scheme; "
                             "top-k with p = fma(0.1, g, e)")
        line["next_rows"] = tim
        del xmodel

    # ---- the other densities and workloads of the metric (not part of `value`) ------------------
    default_run = (args.workload == "c5" and args.density == "1/100" and not args.n and not args.workers
                   and not args.schemes and args.scope == "layerwise")
    if rank == 0 and world == 1 and default_run and not args.no_sweep:
        del vals, idx
        line["sweep"] = run_sweep(args, torch, sc, wl, dev, peak, sampler.uuid, (ctx, grads, res, out))

    # ---- end to end through the C ABI with host buffers ------------------------------------
    if not args.no_e2e and rank == 0:
        line["e2e"] = run_e2e(args, ctx, sc, wl, w, sizes, W, schemes, codes, seg_t, res, n, dev)
    elif rank == 0:
        line["e2e"] = None

    # ---- CPU oracle on a bounded sample -----------------------------------------------------
    if not args.no_cpu_baseline and rank == 0 and world == 1:
        line["cpu_baseline"] = run_cpu_baseline(args, wl, w, sizes, schemes, num, den, grads[0])

    ranks.close()
    if rank == 0:
        print(json.dumps(line), flush=True)


def run_e2e(args, ctx, sc, wl, w, sizes, W, schemes, codes, seg_t, res, n, dev):
    import psutil
    import torch
    need = 4 * n * (W + 1)
    if psutil.virtual_memory().available < 2 * need + (8 << 30):
        return {"value": None, "unit": UNIT, "note": "not enough host memory for pinned staging"}
    h_grads = torch.empty(W, n, dtype=torch.float32).pin_memory()
    h_out = torch.empty(n, dtype=torch.float32).pin_memory()
    for ww in range(W):
        h_grads[ww].copy_(wl.generate(w, ww, 7, dev, sizes=sizes))
    torch.cuda.synchronize()
    steps = max(1, args.e2e_steps)

    def one(t):
        for s, code in zip(schemes, codes):
            ctx.sc_step_host(code, h_grads, res[s], seg_t, [wl.step_seed(w.base_seed, 1000 + t)] * W, h_out)

    one(0)                                                # warm-up (allocates the device staging)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for t in range(steps):
        one(1 + t)
    torch.cuda.synchronize()
    dt = time.perf_counter() - t0
    status = ctx.sc_sync_status()
    if status != 0:
        raise RuntimeError(f"device status after the end-to-end run: {sc.strerror(status)}")
    h2d, d2h = 4 * n * W * len(schemes), 4 * n * len(schemes)
    return {"value": W * n * len(schemes) * steps / dt, "unit": UNIT, "steps": steps,
            "ms_per_step": 1e3 * dt / steps,
            "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
            "host_link_GBps": round((h2d + d2h) * steps / dt / 1e9, 2),
            "note": "sc_step_host: pinned host gradients copied per worker, overlapped with compression; "
                    "dense average copied back.  Every step uploads W*n fresh floats, so this number is the rate "
                    "of the host link (host_link_GBps = bytes copied / time), not of the kernels"}


def run_cpu_baseline(args, wl, w, sizes, schemes, num, den, grads0):
    import numpy as np
    from oracle import sparsify_oracle as O
    n_full = sum(sizes)
    if len(sizes) == 1 and n_full > 50_000_000:
        sizes_s = [n_full // args.cpu_sample_div]
    else:
        sizes_s = sizes
    n = sum(sizes_s)
    segs = [(s.offset, s.n, s.k) for s in wl.segment_table(sizes_s, num, den)]
    g = grads0[0, :n].cpu().numpy()
    e = np.zeros(n, np.float32)
    t0 = time.perf_counter()
    for s in schemes:
        v, i, _ = O.compress_segments(O.SCHEMES[s], g, e, segs, wl.step_seed(w.base_seed, 0))
        O.aggregate([v], [i], n)
    dt = time.perf_counter() - t0
    base = {"value": n * len(schemes) / dt, "unit": UNIT, "cores": 1, "kind": "oracle", "seconds": round(dt, 2),
            "sample": f"worker 0, first {n} of {n_full} elements, schemes {','.join(schemes)}, density {num}/{den}, "
                      f"compress + aggregate of that one message"}
    # the same oracle with one thread per worker (workers are independent), on a quarter of each row
    try:
        from concurrent.futures import ThreadPoolExecutor
        cores = len(os.sched_getaffinity(0))
        Wt = max(1, min(grads0.shape[0], cores))
        nq = max(1, n // 4)
        segq = [(s.offset, s.n, s.k) for s in wl.segment_table([nq], num, den)] if len(sizes_s) == 1 else segs
        nq = sum(s[1] for s in segq)
        rows = [grads0[ww, :nq].cpu().numpy() for ww in range(Wt)]
        seed = wl.step_seed(w.base_seed, 0)

        def one_worker(g_row):
            e_row = np.zeros(nq, np.float32)
            return [O.compress_segments(O.SCHEMES[s], g_row, e_row, segq, seed)[:2] for s in schemes]

        t0 = time.perf_counter()
        with ThreadPoolExecutor(max_workers=Wt) as ex:
            msgs = list(ex.map(one_worker, rows))
        for si in range(len(schemes)):
            O.aggregate([m[si][0] for m in msgs], [m[si][1] for m in msgs], nq)
        dtq = time.perf_counter() - t0
        base["threads"] = {"value": Wt * nq * len(schemes) / dtq, "unit": UNIT, "cores": Wt, "kind": "oracle",
                           "seconds": round(dtq, 2),
                           "sample": f"{Wt} workers in {Wt} threads (host has {cores} cores), first {nq} elements "
                                     f"of each, then one aggregate of the {Wt} messages per scheme"}
    except Exception as ex_:                                    # the single-core figure stands on its own
        base["threads"] = {"value": None, "note": f"not timed: {ex_}"}
    return base


def main():
    args = parse_args()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.selftest_dist:
        run_selftest_dist(args, rank, world)
        return
    if args.impl == "reference":
        run_reference(args, rank)
        return
    if world == 1 and args.gpus > 1:
        sys.stderr.write("bench.py: --gpus > 1 expects to be launched by torch.distributed.run; running 1 GPU\n")
    run_ours(args, rank, world, local_rank)


if __name__ == "__main__":
    main()
