#!/usr/bin/env python
"""Benchmark of the span-restricted decode-attention step on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                    [--cfg 2] [--sweep auto|none|all] [--regions R]
    python bench.py --probe gather              # plain loads against bulk copies for the row gather
    python bench.py --profile-step --cfg 2 ...  # a few untimed steps, for use under a profiler

One step = one decode step of the method over one batch through the library's
one-call entry point (ssa_decode_step): span lists -> index lists and
span-restricted attention over the selected rows of the KV cache.  The metric
is the effective KV bandwidth: bytes of the selected K and V rows divided by
the step time.  The dense baseline (ssa_decode_attn_dense) is timed beside it
for the speedup.

The K-step timed region is repeated R times (barrier + synchronize on both
sides of every region, device time from CUDA events, maximum over ranks); the
reported step time is the median region divided by K.

With N > 1 every rank (one per GPU) runs its own batch of the same workload
(requests are independent: no collective on the data path); started without
torchrun, the script starts the N ranks itself.

Prints ONE JSON line on rank 0; tables too long for that line go to stderr.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import socket
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "span-sparse decode attn: effective KV GB/s (% HBM peak); speedup vs dense"
SPEC_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
WORKLOAD_TEXT = {
    1: "cfg1 tiny: B=1 H=8 D=64 ctx=512 fp16",
    2: "cfg2 arithmetic-style: B=64 H=32 D=128 ragged ctx 256-1024 bf16, prefix 64 + 1-4 spans of 4-32 + last 32",
    3: "cfg3 summarization-style: B=16 H=32 D=128 ctx=4096 bf16",
    4: "cfg4 long context: B=8 H=32 D=128 ctx=16384 bf16",
    5: "cfg5 density sweep: B=32 H=32 D=128 ctx=8192 bf16",
}

# DRAM traffic of one launch of the dominant kernel at cfg 2, the index-list kernel of the two-kernel step
# (dram__bytes_read.sum + dram__bytes_write.sum of one ncu capture: 148 970 496 + 3 003 904), valid only for the
# kernel sources it was captured from and for that form of the step.
NCU_TRAFFIC = {"source_sha256_16": "941e3aca0e20f476", "cfg": 2, "bytes_per_launch": 151974400}


def log(*a):
    print(*a, file=sys.stderr, flush=True)


def kernel_source_hash():
    import hashlib
    h = hashlib.sha256()
    for name in ("decode_attn.cu", "span_merge.cuh", "ssa_common.cuh"):
        h.update(open(os.path.join(ROOT, "paper_2404_09336_b200", "csrc", name), "rb").read())
    return h.hexdigest()[:16]


def hbm_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        return float(json.load(open(path))["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


# ---------------------------------------------------------------------------------------
# clocks
# ---------------------------------------------------------------------------------------
class ClockSampler:
    FIELDS = ("clocks.mem,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.rows, self.proc, self.thread = [], None, None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "50",
                 "-i", str(gpu_index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), line.strip()))

    def stop(self, windows):
        """windows: (t0, t1) wall-clock intervals of the timed regions.  Every sample between the start of
        the first and the end of the last region counts as taken under load: the regions follow one another
        within milliseconds, each far shorter than the sampling period."""
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                self.proc.kill()
        return summarize_clock_rows(self.rows, windows)


def summarize_clock_rows(rows, windows):
    t_lo = min((a for a, _ in windows), default=0.0)
    t_hi = max((b for _, b in windows), default=0.0)
    sm, mem, mx, reasons, n_all = [], [], 0.0, set(), 0
    names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
    for t, line in rows:
        parts = [p.strip() for p in line.split(",")]
        if len(parts) < 9:
            continue
        n_all += 1
        if not (t_lo <= t <= t_hi + 0.05):
            continue
        try:
            sm.append(float(parts[1]))
            mem.append(float(parts[0]))
            mx = max(mx, float(parts[2]))
        except ValueError:
            continue
        for name, val in zip(names, parts[5:9]):
            if val.lower().startswith("active"):
                reasons.add(name)
    return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": mx or None,
            "mem_mhz": statistics.median(mem) if mem else None,
            "reasons": sorted(reasons), "samples_under_load": len(sm), "samples": n_all}


# ---------------------------------------------------------------------------------------
# the CPU oracle as a timed baseline (cpu_baseline leg and the reference arm)
# ---------------------------------------------------------------------------------------
def oracle_step(O, wl, q, k, v, n_seq, stride):
    """One decode step of the oracle over the first n_seq requests."""
    index, counts, _ = O.spans_to_index_batch(wl.span_offsets[: n_seq + 1], wl.spans, wl.ctx_lens[:n_seq], stride)
    O.decode_attn_sparse(q[:n_seq], k[:n_seq], v[:n_seq], wl.ctx_lens[:n_seq], index, counts,
                         1.0 / math.sqrt(wl.D), wl.dtype)
    return int(counts.sum()) * wl.kv_bytes_per_token()


_POOL_BARRIER = None


def _pool_init(barrier):
    global _POOL_BARRIER
    _POOL_BARRIER = barrier


def _oracle_worker(task):
    """One process of the all-cores oracle run: its share of the sample's requests, numpy kept to one thread.
    Inputs are drawn before the barrier; only the oracle's own work lies between the two time stamps."""
    cfg, density, n_seq, rank, world, warmup, steps = task
    from threadpoolctl import threadpool_limits

    from oracle import ssa_oracle as O
    from paper_2404_09336_b200 import inputs
    wl = inputs.make_config(cfg, density=density, B=n_seq).shard(rank, world)
    stride = (max(wl.selected_upper_bound(), 1) + 31) // 32 * 32
    with threadpool_limits(limits=1):
        q, (k, v) = wl.q_bits(), wl.kv_bits(threads=1)
        for _ in range(warmup):
            oracle_step(O, wl, q, k, v, wl.B, stride)
        _POOL_BARRIER.wait()
        t0 = time.time()
        nbytes = 0
        for _ in range(steps):
            nbytes += oracle_step(O, wl, q, k, v, wl.B, stride)
        t1 = time.time()
    return t0, t1, nbytes


def host_cores():
    try:
        return len(os.sched_getaffinity(0))
    except Exception:
        return os.cpu_count() or 1


def time_oracle_one_thread(cfg, density, n_seq, steps, warmup=0):
    from threadpoolctl import threadpool_limits

    from oracle import ssa_oracle as O
    from paper_2404_09336_b200 import inputs
    wl = inputs.make_config(cfg, density=density, B=n_seq)
    stride = (max(wl.selected_upper_bound(), 1) + 31) // 32 * 32
    with threadpool_limits(limits=1):
        q, (k, v) = wl.q_bits(), wl.kv_bits()
        for _ in range(warmup):
            oracle_step(O, wl, q, k, v, n_seq, stride)
        t0 = time.perf_counter()
        nbytes = sum(oracle_step(O, wl, q, k, v, n_seq, stride) for _ in range(steps))
        el = time.perf_counter() - t0
    return {"gbs": nbytes / el / 1e9, "seconds": el, "bytes_per_step": nbytes // max(steps, 1)}


def time_oracle_all_cores(cfg, density, n_seq, steps, warmup=0):
    """The oracle's (request, head) loop spread over the host's cores: a pool of spawned processes, each with
    an even share of the sample's requests.  The oracle itself is untouched."""
    import multiprocessing as mp
    world = max(1, min(host_cores(), n_seq))
    ctx = mp.get_context("spawn")
    barrier = ctx.Barrier(world)
    with ctx.Pool(world, initializer=_pool_init, initargs=(barrier,)) as pool:
        res = pool.map(_oracle_worker, [(cfg, density, n_seq, r, world, warmup, steps) for r in range(world)],
                       chunksize=1)
    t0, t1 = min(r[0] for r in res), max(r[1] for r in res)
    nbytes = sum(r[2] for r in res)
    return {"gbs": nbytes / (t1 - t0) / 1e9, "seconds": t1 - t0, "processes": world,
            "bytes_per_step": nbytes // max(steps, 1)}


def oracle_sample(cfg, budget_s, steps):
    """How many requests of workload `cfg` one timed oracle step covers so that `steps` steps on one thread
    stay near budget_s (whole batch when it fits)."""
    from paper_2404_09336_b200 import inputs
    density = 0.10 if cfg == 5 else None
    full = inputs.make_config(cfg, density=density)
    probe = time_oracle_one_thread(cfg, density, min(2, full.B), 1)
    per_seq = probe["seconds"] / min(2, full.B)
    n_seq = int(max(1, min(full.B, budget_s / max(steps, 1) / max(per_seq, 1e-9))))
    return density, n_seq, full


def cpu_baseline(cfg, budget_s=12.0):
    density, n_seq, full = oracle_sample(cfg, budget_s, steps=3)
    one = time_oracle_one_thread(cfg, density, n_seq, steps=3)
    cores = host_cores()
    reps = int(max(1, min(200, 4.0 / max(one["seconds"] / 3 / max(min(cores, n_seq), 1), 1e-4))))
    allc = time_oracle_all_cores(cfg, density, n_seq, steps=reps)
    name = WORKLOAD_TEXT[cfg].split(":")[0]
    return {"value": allc["gbs"], "unit": "GB/s", "cores": allc["processes"], "kind": "oracle",
            "host_cores": cores,
            "sample": f"{reps} steps over the first {n_seq} of {full.B} requests x {full.H} heads of {name} "
                      f"({allc['bytes_per_step']} selected KV bytes per step), numpy fp64, one process per core "
                      f"({allc['processes']} processes, requests split evenly), {allc['seconds']:.1f} s",
            "one_thread": {"value": one["gbs"], "unit": "GB/s", "seconds": round(one["seconds"], 2), "steps": 3}}


def run_reference(args):
    """The reference arm: there is no reference implementation (the paper's kernel is not available), so the
    oracle, as it stands, is timed on the host cores on the same workload, metric and unit."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    world = int(os.environ.get("WORLD_SIZE", "1"))
    density, n_seq, full = oracle_sample(args.cfg, 60.0, args.steps + args.warmup)
    r = time_oracle_all_cores(args.cfg, density, n_seq, steps=args.steps, warmup=args.warmup)
    name = WORKLOAD_TEXT[args.cfg].split(":")[0]
    sample = (f"{args.steps} steps, each over the first {n_seq} of {full.B} requests x {full.H} heads of {name} "
              f"({r['bytes_per_step']} selected KV bytes per step), numpy fp64, one process per core "
              f"({r['processes']} processes)")
    line = {"impl": "reference", "metric": METRIC, "value": r["gbs"], "unit": "GB/s", "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": r["seconds"] / args.steps * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic",
            "config": {"workload": WORKLOAD_TEXT[args.cfg] + (" (10% point)" if args.cfg == 5 else "")},
            "cpu_baseline": {"value": r["gbs"], "unit": "GB/s", "cores": r["processes"], "kind": "oracle",
                             "host_cores": host_cores(), "sample": sample},
            "e2e": {"value": r["gbs"], "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ---------------------------------------------------------------------------------------
# GPU arm
# ---------------------------------------------------------------------------------------
class Timer:
    def __init__(self, torch, dist, world, device="cuda"):
        self.torch, self.dist, self.world, self.device = torch, dist, world, device
        self.windows = []

    def max_over_ranks(self, x):
        if self.world > 1:
            t = self.torch.tensor([float(x)], dtype=self.torch.float64, device=self.device)
            self.dist.all_reduce(t, op=self.dist.ReduceOp.MAX)
            return float(t.item())
        return float(x)

    def sync(self):
        self.torch.cuda.synchronize()
        if self.world > 1:
            self.dist.barrier()
        self.torch.cuda.synchronize()

    def run(self, fn, steps):
        """Device time (ms) of `steps` calls of fn(i): events on the launching stream, a barrier +
        synchronize on both sides, maximum over ranks."""
        torch = self.torch
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        self.sync()
        w0 = time.time()
        e0.record()
        for i in range(steps):
            fn(i)
        e1.record()
        self.sync()
        self.windows.append((w0, time.time()))
        return self.max_over_ranks(e0.elapsed_time(e1))

    def regions(self, fn, steps, n_regions):
        """n_regions timed regions of `steps` calls each -> per-call microseconds of every region."""
        return [self.run(fn, steps) / steps * 1e3 for _ in range(n_regions)]

    def median_us(self, fn, steps, n_regions):
        return statistics.median(self.regions(fn, steps, n_regions))

    def total(self, x):
        if self.world > 1:
            t = self.torch.tensor([float(x)], dtype=self.torch.float64, device=self.device)
            self.dist.all_reduce(t, op=self.dist.ReduceOp.SUM)
            return float(t.item())
        return float(x)


def l2_bytes(torch):
    return int(torch.cuda.get_device_properties(torch.cuda.current_device()).L2_cache_size)


def copies_for(selected_bytes, cache_bytes, l2, cap_bytes=40e9):
    want = max(2, math.ceil(2 * l2 / max(selected_bytes, 1)) + 1)
    return int(max(1, min(want, 8, cap_bytes // max(cache_bytes, 1))))


def capture_graphs(torch, ds, fn):
    """One CUDA graph per KV copy replaying fn() (the library's launches)."""
    graphs = []
    side = torch.cuda.Stream()
    for c in range(len(ds.k_store)):
        ds.select_copy(c)
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            fn()
        graphs.append(g)
    torch.cuda.synchronize()
    return graphs


def kernel_time_us(torch, ssa, timer, ds, fn, n):
    """Duration of the main (split-KV) kernel of fn()'s attention call: events the library records right
    around that kernel on the call's stream; median over n launches over rotating KV copies."""
    ncopy = len(ds.k_store)
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n)]
    for a, b in evs:
        a.record()
        b.record()
    torch.cuda.synchronize()

    def with_events(i):
        ds.select_copy(i % ncopy)
        ssa.set_kernel_events(*evs[i])
        fn()

    timer.run(with_events, n)
    durs = [a.elapsed_time(b) * 1e3 for a, b in evs]
    return statistics.median(durs), statistics.mean(durs)


def measure(torch, ssa, timer, ds, steps, warmup, regions, pieces=True):
    """All timings of the workload held by `ds`.  Inputs are larger than L2: consecutive steps rotate over
    the KV copies.  Returns a dict (microseconds are medians over `regions` timed regions)."""
    ncopy = len(ds.k_store)

    def rotating(fn):
        return lambda i: (ds.select_copy(i % ncopy), fn())

    for i in range(max(warmup, 3)):
        ds.select_copy(i % ncopy)
        ds.step()
        ds.attend_dense()
    torch.cuda.synchronize()
    l0 = ssa.launch_count()
    ds.step()
    launches_per_step = ssa.launch_count() - l0
    l0 = ssa.launch_count()
    ds.step(kernels="two")
    launches_two = ssa.launch_count() - l0
    torch.cuda.synchronize()
    status = int(ds.status.item())
    sel = ds.selected_bytes()
    ctx_tokens = int(ds.ctx_lens.sum().item())
    dense_bytes = ctx_tokens * ds.wl.kv_bytes_per_token()
    res = {"selected_bytes": sel, "dense_bytes": dense_bytes, "density": sel / max(dense_bytes, 1),
           "kv_copies": ncopy, "launches_per_step": launches_per_step, "dev_status": status,
           "path": "one kernel" if launches_per_step < launches_two else "index + attention"}

    # the step as the library runs it (ssa_decode_step decides between one kernel and index + attention)
    reg = timer.regions(rotating(ds.step), steps, regions)
    res["step_regions_us"] = reg
    res["step_us"] = statistics.median(reg)
    one_kernel = res["path"] == "one kernel"
    if pieces:
        res["step_two_kernels_us"] = timer.median_us(rotating(lambda: ds.step(kernels="two")), steps, regions)
        if ds.max_spans <= 128:
            res["step_one_kernel_us"] = timer.median_us(rotating(lambda: ds.step(kernels="one")), steps, regions)
        # the same step without rotating: every step re-reads copy 0 (L2-warm where the selection fits the L2)
        ds.select_copy(0)
        res["warm_us"] = timer.median_us(lambda i: ds.step(), steps, regions)
        # the step replayed from CUDA graphs (one per KV copy)
        graphs = capture_graphs(torch, ds, ds.step)
        for g in graphs:
            g.replay()
        res["graph_us"] = timer.median_us(lambda i: graphs[i % ncopy].replay(), steps, regions)
        del graphs
        # index expansion alone (graph replays: the launch is too short for back-to-back direct calls)
        gs = capture_graphs(torch, ds, ds.build_index)
        for g in gs:
            g.replay()
        res["index_us"] = timer.median_us(lambda i: gs[i % ncopy].replay(), steps, regions)
        del gs
    n_dense = max(10, min(steps, int(steps * sel / max(dense_bytes, 1)) + 10))
    res["dense_us"] = timer.median_us(rotating(ds.attend_dense), n_dense, max(3, regions // 3))
    # The dominant kernel: a timed region of nothing but the attention call of the step's form, launched back
    # to back (CUDA events around the region on the launching stream; region / launches).  Where the lists span
    # several chunks the call's small second pass rides along, so the figure errs on the long side.
    ds.build_index()
    attend = (lambda: ds.step(kernels="one")) if one_kernel else ds.attend_sparse   # one kernel: the step is the call
    for i in range(3):
        attend()
    res["kernel_us"] = timer.median_us(rotating(attend), steps, regions)
    res["sparse_attn_us"] = res["kernel_us"] if not one_kernel else timer.median_us(rotating(ds.attend_sparse), steps, regions)
    # for context: one launch on its own, between events the library records right around the kernel (nothing
    # overlaps its ramp-up and drain then, and the two event records cost a few microseconds themselves)
    ds.step()
    res["kernel_isolated_us"], _ = kernel_time_us(torch, ssa, timer, ds, ds.step, min(max(steps, 50), 300))
    res["gbs"] = sel / res["step_us"] / 1e3
    res["dense_gbs"] = dense_bytes / res["dense_us"] / 1e3
    res["speedup_vs_dense"] = res["dense_us"] / res["step_us"]
    return res


def roofline_entry(name, r, peak):
    kb = r["selected_bytes"] / r["kernel_us"] / 1e3
    return {"workload": name, "density": round(r["density"], 4), "bytes": r["selected_bytes"],
            "kernel_us": round(r["kernel_us"], 2), "step_us": round(r["step_us"], 2),
            "frac": round(kb / peak, 4), "frac_spec": round(kb / SPEC_HBM_GBS, 4),
            "step_frac": round(r["gbs"] / peak, 4), "step_frac_spec": round(r["gbs"] / SPEC_HBM_GBS, 4),
            "speedup_vs_dense": round(r["speedup_vs_dense"], 3), "path": r["path"]}


def mixed_batches(torch, ssa, timer, steps, regions, l2):
    """A batch in which some requests are at a "determine span" step (full context) and the others generate
    with their selected spans, served by ONE launch sized for the longest list - against the same requests
    served by two launches, each sized for its own class (the other class's requests given nothing to do)."""
    from paper_2404_09336_b200 import inputs
    from paper_2404_09336_b200.runner import DecodeStep
    rows = []
    for every in (2, 8):
        wl = inputs.make_mixed(every)
        cache = 2 * wl.B * wl.H * wl.max_ctx * wl.D * 2
        ds = DecodeStep(wl, kv_copies=copies_for(cache // 4, cache, l2))
        ncopy = len(ds.k_store)
        full = torch.arange(wl.B, device=ds.device) % every == 0
        ds.step()
        torch.cuda.synchronize()
        sel = ds.selected_bytes()
        one = timer.median_us(lambda i: (ds.select_copy(i % ncopy), ds.step()), steps, regions)
        # class by class: the dense kernel over the full-context requests (context length 0 for the others) ...
        ctx_all = ds.ctx_lens.clone()
        ctx_dense = torch.where(full, ctx_all, torch.zeros_like(ctx_all))
        base = inputs.make_config(2)
        sp = DecodeStep.__new__(DecodeStep)              # ... and a restricted step over the others' span lists
        sp.__dict__.update(ds.__dict__)
        sp._steps = {}
        sp.wl = base
        sp.max_selected = max(base.selected_upper_bound(), 1)
        sp.max_spans = int(np.diff(base.span_offsets).max())
        offs, spans = [0], []
        for b in range(base.B):
            if b % every != 0:
                spans += [tuple(x) for x in base.spans_of(b)]
            offs.append(len(spans))
        sp.span_offsets = torch.tensor(offs, dtype=torch.int32, device=ds.device)
        sp.spans = torch.tensor(spans, dtype=torch.int32, device=ds.device)

        def by_class(i):
            ds.select_copy(i % ncopy)
            sp.k, sp.v = ds.k, ds.v
            ds.ctx_lens.copy_(ctx_dense)
            ds.attend_dense()
            ds.ctx_lens.copy_(ctx_all)
            sp.step()

        for i in range(3):
            by_class(i)
        two = timer.median_us(by_class, steps, regions)
        rows.append({"full_context_every": every, "selected_bytes": sel, "one_launch_us": round(one, 2),
                     "per_class_launches_us": round(two, 2), "one_over_per_class": round(one / two, 3),
                     "gbs": round(sel / one / 1e3)})
        del ds, sp
        torch.cuda.empty_cache()
    return {"what": "cfg 2 shapes with every k-th request attending to its full context (a 'determine span' step) and "
                    "the rest to their spans: one ssa_decode_step over the mixed batch against a dense launch over the "
                    "full-context requests plus a restricted step over the others (two context-length copies included)",
            "rows": rows}


def paper_microbench(torch, ssa, timer, n_iter=20):
    """The paper's kernel micro-benchmark (50 % of the preceding tokens ignored, mask made of
    blocks of ones of a given size, batch 64, 1024..8192 preceding tokens): speedup of the
    span-restricted step over this library's dense kernel, through the index list and through
    the paper's blocked (index, bitmask) encoding with 256-position blocks."""
    from paper_2404_09336_b200 import inputs
    from paper_2404_09336_b200.runner import DecodeStep
    T, B = 8192, 64
    base = inputs.make_microbench(T, 256, B=B, max_ctx=T)
    ds = DecodeStep(base, kv_copies=1, index_stride=T // 2, max_selected=T // 2, span_capacity=B * (T // 64))
    ds.enable_blockmask(256)
    rows = []
    for ctx in (1024, 2048, 4096, 8192):
        for sb in (32, 64, 128, 256):
            ds.set_spans(inputs.make_microbench(ctx, sb, B=B, max_ctx=T))
            for fn in (ds.step, ds.step_blockmask, ds.attend_dense):
                fn()
            torch.cuda.synchronize()
            if int(ds.status.item()) != 0:
                raise SystemExit("micro-benchmark raised a device status flag")
            t_idx = timer.run(lambda i: ds.step(), n_iter) / n_iter * 1e3
            t_bm = timer.run(lambda i: ds.step_blockmask(), n_iter) / n_iter * 1e3
            t_dense = timer.run(lambda i: ds.attend_dense(), n_iter) / n_iter * 1e3
            sel = B * (ctx // 2) * base.kv_bytes_per_token()
            rows.append({"ctx": ctx, "sparsity_block": sb, "dense_us": round(t_dense, 2),
                         "index_path_us": round(t_idx, 2), "blockmask_path_us": round(t_bm, 2),
                         "speedup_index": round(t_dense / t_idx, 3), "speedup_blockmask": round(t_dense / t_bm, 3),
                         "index_path_gbs": round(sel / t_idx / 1e3, 1)})
    geo = lambda xs: float(np.exp(np.mean(np.log(xs))))
    summary = {"geomean_speedup_index": round(geo([r["speedup_index"] for r in rows]), 3),
               "geomean_speedup_blockmask": round(geo([r["speedup_blockmask"] for r in rows]), 3)}
    for sb in (32, 64, 128, 256):
        summary[f"geomean_speedup_index_sb{sb}"] = round(
            geo([r["speedup_index"] for r in rows if r["sparsity_block"] == sb]), 3)
        summary[f"geomean_speedup_blockmask_sb{sb}"] = round(
            geo([r["speedup_blockmask"] for r in rows if r["sparsity_block"] == sb]), 3)
    del ds
    torch.cuda.empty_cache()
    log("paper micro-benchmark rows:")
    for r in rows:
        log("  " + json.dumps(r))
    return {"what": "paper kernel micro-benchmark: batch 64, 32 heads x 128, 50% of tokens ignored, speedup vs "
                    "ssa_decode_attn_dense (the paper compares with HF attention on an A100: 1.29x overall, "
                    "0.97/1.2/1.6/1.6x at sparsity block 32/64/128/256); per-row figures on stderr",
            "summary": summary}


def variants_outside_the_paper(torch, ssa, timer, n_iter=100):
    """Grouped query heads, several query tokens per step and a paged cache, all outside the paper: B = 32
    requests, 32 query heads x 128, context 8192, 10 % selected (the cfg 5 recipe), L2-cold by rotating copies."""
    from paper_2404_09336_b200 import inputs
    from paper_2404_09336_b200.runner import DecodeStep
    dev = torch.device("cuda", torch.cuda.current_device())
    B, H, D, T = 32, 32, 128, 8192
    rows = []
    for hkv in (8, 4, 2):
        wl = inputs.make_config(5, density=0.10, B=B, H=hkv)
        ncopy = max(2, min(8, int(3e9 // (2 * B * hkv * T * D * 2))))
        ds = DecodeStep(wl, kv_copies=ncopy, query_heads=H)
        ds.build_index()
        torch.cuda.synchronize()
        sel = int(ds.counts.sum().item()) * 2 * hkv * D * 2

        def sparse(i):
            ds.select_copy(i % ncopy)
            ds.attend_sparse()

        def dense(i):
            ds.select_copy(i % ncopy)
            ds.attend_dense()

        for i in range(3):
            sparse(i), dense(i)
        ts = timer.run(sparse, n_iter) / n_iter * 1e3
        td = timer.run(dense, n_iter // 4) / (n_iter // 4) * 1e3
        rows.append({"H": H, "H_kv": hkv, "sparse_attn_us": round(ts, 2), "dense_us": round(td, 2),
                     "kv_gbs_sparse": round(sel / ts / 1e3), "kv_gbs_dense": round(B * T * 2 * hkv * D * 2 / td / 1e3)})
        del ds
        torch.cuda.empty_cache()
    # 8-bit (e4m3) cache storage against the 16-bit cache: same shapes and lists (cfg 5 at 10 %, multi-head)
    wl = inputs.make_config(5, density=0.10)
    ncopy = 3
    ds = DecodeStep(wl, kv_copies=ncopy)
    ds.build_index()
    torch.cuda.synchronize()
    rows_sel, rows_all = int(ds.counts.sum().item()), wl.B * wl.max_ctx
    k8 = [k.to(torch.float8_e4m3fn) for k in ds.k_store]
    v8 = [v.to(torch.float8_e4m3fn) for v in ds.v_store]
    desc8 = ssa.make_desc(ds.q, k8[0], v8[0], ds.out, max_ctx=wl.max_ctx)

    def sparse8(i):
        ssa.decode_attn_sparse(desc8, ds.q, k8[i % ncopy], v8[i % ncopy], ds.ctx_lens, ds.index, ds.counts,
                               ds.max_selected, ds.out, ds.lse, ds.workspace, ds.status)

    def dense8(i):
        ssa.decode_attn_dense(desc8, ds.q, k8[i % ncopy], v8[i % ncopy], ds.ctx_lens, ds.out, ds.lse, ds.workspace,
                              ds.status)

    def sparse16(i):
        ds.select_copy(i % ncopy)
        ds.attend_sparse()

    def dense16(i):
        ds.select_copy(i % ncopy)
        ds.attend_dense()

    for i in range(3):
        sparse8(i), dense8(i), sparse16(i), dense16(i)
    t8s = timer.run(sparse8, n_iter) / n_iter * 1e3
    t8d = timer.run(dense8, n_iter // 4) / (n_iter // 4) * 1e3
    t16s = timer.run(sparse16, n_iter) / n_iter * 1e3
    t16d = timer.run(dense16, n_iter // 4) / (n_iter // 4) * 1e3
    row8 = 2 * wl.H * wl.D                               # K + V bytes of one position over all heads, one byte each
    fp8 = {"workload": "cfg5 10%: B=32, 32 heads x 128, ctx 8192; cache stored as e4m3 bytes, bf16 queries",
           "sparse_attn_us": round(t8s, 2), "dense_us": round(t8d, 2),
           "kv_gbs_sparse": round(rows_sel * row8 / t8s / 1e3), "kv_gbs_dense": round(rows_all * row8 / t8d / 1e3),
           "bf16_cache_sparse_attn_us": round(t16s, 2), "bf16_cache_dense_us": round(t16d, 2)}
    del ds, k8, v8
    torch.cuda.empty_cache()
    # paged cache: cfg 2 shapes, token-major pool, 16-row pages in shuffled order, against the contiguous call
    wl = inputs.make_config(2)
    ncopy = 4
    ds = DecodeStep(wl, kv_copies=ncopy, layout="bthd")
    ds.build_index()
    B, H, D, T, ps = wl.B, wl.H, wl.D, wl.max_ctx, 16
    n_pages = B * T // ps
    perm = torch.randperm(n_pages, generator=torch.Generator().manual_seed(1)).to(dev)
    table = perm.to(torch.int32).view(B, T // ps)
    pools = []
    for c in range(ncopy):
        kp = torch.empty((n_pages, ps, H, D), dtype=ds.k_store[c].dtype, device=dev)
        vp = torch.empty_like(kp)
        kp[perm] = ds.k_store[c].view(n_pages, ps, H, D)
        vp[perm] = ds.v_store[c].view(n_pages, ps, H, D)
        pools.append((kp, vp))
    desc = ssa.make_desc_paged(ds.q, pools[0][0], pools[0][1], ds.out, max_ctx=T)
    pg = ssa.make_paging(table, ps, n_pages)

    def paged(i):
        kp, vp = pools[i % ncopy]
        ssa.decode_attn_sparse_paged(desc, ds.q, kp, vp, pg, ds.ctx_lens, ds.index, ds.counts, ds.max_selected,
                                     ds.out, ds.lse, ds.workspace, ds.status)

    def contiguous(i):
        ds.select_copy(i % ncopy)
        ds.attend_sparse()

    for i in range(3):
        paged(i), contiguous(i)
    tp = timer.run(paged, 4 * n_iter) / (4 * n_iter) * 1e3
    tc = timer.run(contiguous, 4 * n_iter) / (4 * n_iter) * 1e3
    del ds, pools
    torch.cuda.empty_cache()
    return {"what": "outside the paper: grouped query heads (B=32, 32 query heads x 128, ctx 8192, 10% selected; rows "
                    "of a K/V head are read once for its whole group), an 8-bit cache and a paged cache (cfg 2 shapes, "
                    "16-row pages in shuffled order, attention call alone)",
            "grouped_heads": rows, "fp8_cache": fp8,
            "paged_cfg2": {"page_size": ps, "paged_attn_us": round(tp, 2), "contiguous_attn_us": round(tc, 2)}}


def run_dry(args):
    """The multi-rank plumbing without a GPU (SSA_BENCH_DRY_RUN=1): process group over gloo, the same
    barrier / maximum / sum reductions, a stand-in for the measurement (rank r: 10 + r ms per region of
    1000 * (r + 1) bytes per step).  Rank 0 prints the JSON line."""
    import torch
    import torch.distributed as dist
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if world > 1:
        dist.init_process_group("gloo")
    timer = Timer(torch, dist, world, device="cpu")
    ms = timer.max_over_ranks(10.0 + rank)
    total = timer.total(1000.0 * (rank + 1))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps({"metric": METRIC, "value": total * args.steps / (ms * 1e-3) / 1e9, "unit": "GB/s",
                          "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms / args.steps,
                          "dry_run": True}), flush=True)


def run_ours(args):
    if os.environ.get("SSA_BENCH_DRY_RUN") == "1":
        return run_dry(args)
    import torch
    import torch.distributed as dist

    from paper_2404_09336_b200 import inputs, ssa
    from paper_2404_09336_b200.runner import DecodeStep

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    # the oracle's process pool is started (spawn) and finished before this process touches the GPU
    baseline = cpu_baseline(args.cfg) if (rank == 0 and world == 1) else None
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    peak, peak_kind = hbm_peak()
    timer = Timer(torch, dist, world)
    l2 = l2_bytes(torch)
    steps, warmup, regions = args.steps, max(args.warmup, 3), max(args.regions, 1)

    try:
        gpu_id = f"GPU-{torch.cuda.get_device_properties(local).uuid}"
    except Exception:
        gpu_id = str(local)
    sampler = ClockSampler(gpu_id)
    density = 0.10 if args.cfg == 5 else None
    wl = inputs.make_config(args.cfg, density=density, first_id=rank * 1000)
    sel_guess = wl.selected_upper_bound() * wl.B * wl.kv_bytes_per_token() // 2
    cache = 2 * wl.B * wl.H * wl.max_ctx * wl.D * 2
    ds = DecodeStep(wl, device=f"cuda:{local}", kv_copies=copies_for(sel_guess, cache, l2))
    ncopy = len(ds.k_store)
    main = measure(torch, ssa, timer, ds, steps, warmup, regions)
    if main["dev_status"] != 0:
        raise SystemExit(f"device status word is {main['dev_status']}: the workload raised a data flag")

    # the headline: `regions` timed regions of exactly `steps` steps; the median region is the figure
    for i in range(warmup):
        ds.select_copy(i % ncopy)
        ds.step()
    l0 = ssa.launch_count()
    reg = timer.regions(lambda i: (ds.select_copy(i % ncopy), ds.step()), steps, regions)
    launches = (ssa.launch_count() - l0) // regions
    step_us = statistics.median(reg)
    total_sel = timer.total(main["selected_bytes"])
    value = total_sel / step_us / 1e3

    # end to end: per-step inputs from pinned host memory, result back to the host
    h2d, d2h = ds.make_host_buffers()
    # two ways of moving the same bytes: copy-engine transfers around the kernels, or copies done by kernels
    # with the output rows stored straight into the pinned buffer; both are reported, the figure is the
    # kernel-copy form (the one a latency-bound decode loop would use)
    e2e_us = {}
    for how, direct in (("copy_engine", False), ("kernels", True)):
        for i in range(max(3, warmup)):
            ds.step_from_host(direct=direct)
        e2e_us[how] = statistics.median(timer.regions(
            lambda i: (ds.select_copy(i % ncopy), ds.step_from_host(direct=direct)), steps, max(3, regions // 2)))
    e2e_how = "kernels"
    e2e_value = total_sel / e2e_us[e2e_how] / 1e3
    clocks = sampler.stop(timer.windows)

    if rank != 0:
        if world > 1:
            dist.barrier()
            dist.destroy_process_group()
        return

    kernel_us = main["kernel_us"]
    traffic = NCU_TRAFFIC["bytes_per_launch"] if (args.cfg == NCU_TRAFFIC["cfg"] and main["path"] == "index + attention"
                                                  and kernel_source_hash() == NCU_TRAFFIC["source_sha256_16"]) else None
    kernel_name = ("decode_partial_kernel<spans> (ssa_decode_attn_spans)" if main["path"] == "one kernel"
                   else "decode_partial_kernel<index> (ssa_decode_attn_sparse)")
    roofline = {"bound": "hbm", "kernel": kernel_name,
                "achieved": main["selected_bytes"] / kernel_us / 1e3,
                "peak": peak, "unit": "GB/s", "peak_kind": f"of {peak_kind}",
                "frac": main["selected_bytes"] / kernel_us / 1e3 / peak,
                "frac_of_spec_8000": main["selected_bytes"] / kernel_us / 1e3 / SPEC_HBM_GBS,
                "traffic": traffic, "kernel_us": kernel_us,
                "kernel_us_how": "timed region of back-to-back launches of the step's attention call alone (CUDA events "
                                 "on the launching stream, region / launches, median of the regions), L2-cold",
                "kernel_isolated_us": main["kernel_isolated_us"],
                "kernel_isolated_how": "one launch on its own between events the library records around the kernel "
                                       "(ssa_set_kernel_events): includes its undisturbed ramp-up and drain and the "
                                       "cost of the event records",
                "algorithmic_bytes_per_launch": main["selected_bytes"],
                "by_config": [roofline_entry(WORKLOAD_TEXT[args.cfg].split(":")[0], main, peak)]}
    line = {
        "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": steps, "warmup": warmup,
        "ms_per_step": step_us * 1e-3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic",
        "config": {"workload": WORKLOAD_TEXT[args.cfg] + (" (10% point)" if args.cfg == 5 else ""),
                   "layout": "[B,H,T,D]", "kv_dtype": wl.dtype, "launch": "direct calls of ssa_decode_step",
                   "step_path": main["path"],
                   "l2": f"inputs larger than L2: {ncopy} rotating KV copies, "
                         f"{ncopy * main['selected_bytes'] / 1e6:.0f} MB of selected rows between reuses "
                         f"(L2 {l2 / 1e6:.0f} MB)",
                   "per_gpu_batch": wl.B},
        "timed_regions": {"n": regions, "steps_each": steps, "us_per_step_median": round(step_us, 3),
                          "us_per_step_min": round(min(reg), 3), "us_per_step_max": round(max(reg), 3)},
        "pct_hbm_peak_measured": 100 * value / world / peak, "pct_hbm_peak_spec": 100 * value / world / SPEC_HBM_GBS,
        "speedup_vs_dense": main["dense_us"] / step_us, "density": main["density"],
        "us_per_step": step_us,
        "breakdown_us": {k: round(main[k], 3) for k in ("step_us", "step_two_kernels_us", "step_one_kernel_us",
                                                         "graph_us", "warm_us", "index_us", "sparse_attn_us",
                                                         "dense_us", "kernel_us", "kernel_isolated_us") if k in main},
        "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": "GB/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "us_per_step": e2e_us[e2e_how], "copies": e2e_how,
                "us_per_step_by_copy_mode": {k: round(v, 3) for k, v in e2e_us.items()},
                "note": "ssa_decode_step from pinned host buffers: query rows + context lengths + span lists in, "
                        "output rows + lse + counts + status back, every step; copy_engine = two cudaMemcpyAsync "
                        "transfers, kernels = SSA_STEP_COPY_BY_KERNEL with out/lse stored straight into the "
                        "pinned buffer; the KV cache is resident state"},
        "gpu_launches": int(launches),
        "roofline": roofline,
    }

    if world == 1:
        sweep = []
        want = {"auto": [1, 3, 4, 5], "all": [1, 3, 4, 5], "none": []}[args.sweep]
        sweep_steps, sweep_regions = max(20, min(steps, 100)), max(3, min(regions, 9))
        del ds
        torch.cuda.empty_cache()
        for cfg in want:
            if cfg == args.cfg:
                continue
            if cfg == 5:
                wls = {f: inputs.make_config(5, density=f) for f in inputs.DENSITIES}
                cap = max(len(w.spans) for w in wls.values())
                d5 = DecodeStep(wls[1.0], kv_copies=6, index_stride=8192, max_selected=8192, span_capacity=cap)
                for f in inputs.DENSITIES:
                    d5.set_spans(wls[f])
                    r = measure(torch, ssa, timer, d5, sweep_steps, 3, sweep_regions, pieces=(f <= 0.10))
                    r["workload"] = f"cfg5 density {int(f * 100)}%"
                    sweep.append(r)
                del d5
            else:
                w = inputs.make_config(cfg)
                sg = w.selected_upper_bound() * w.B * w.kv_bytes_per_token() // 2
                cb = 2 * w.B * w.H * w.max_ctx * w.D * 2
                d = DecodeStep(w, kv_copies=copies_for(sg, cb, l2))
                r = measure(torch, ssa, timer, d, sweep_steps, 3, sweep_regions)
                r["workload"] = WORKLOAD_TEXT[cfg].split(":")[0]
                sweep.append(r)
                del d
            torch.cuda.empty_cache()
        for r in sweep:
            roofline["by_config"].append(roofline_entry(r["workload"], r, peak))
            log("sweep " + json.dumps({k: (round(v, 3) if isinstance(v, float) else v) for k, v in r.items()
                                        if k != "step_regions_us"}))
        if sweep:
            read_peak = max(r["dense_gbs"] for r in sweep)
            roofline["read_stream_gbs"] = round(read_peak, 1)
            roofline["read_stream_how"] = ("best rate of this library's full-context kernel in this run (a read-only "
                                           "stream; the measured peak above is a copy, which a read-only stream exceeds)")
            roofline["frac_of_read_stream"] = round(roofline["achieved"] / read_peak, 4)
            for e in roofline["by_config"]:            # no workload exceeds this denominator
                e["frac_of_read_stream"] = round(e["bytes"] / e["kernel_us"] / 1e3 / read_peak, 4)
        five = [r for r in sweep if r["workload"].startswith("cfg5")]
        line["crossover_density"] = next((r["density"] for r in five if r["speedup_vs_dense"] < 1.0), None)
        if args.sweep != "none":
            line["mixed"] = mixed_batches(torch, ssa, timer, sweep_steps, sweep_regions, l2)
            line["paper_microbench"] = paper_microbench(torch, ssa, timer)
            line["variants"] = variants_outside_the_paper(torch, ssa, timer)
        line["cpu_baseline"] = baseline
    else:
        dist.barrier()
        dist.destroy_process_group()
    print(json.dumps(line), flush=True)


# ---------------------------------------------------------------------------------------
# other modes
# ---------------------------------------------------------------------------------------
def run_profile_step(args):
    """A few decode steps of one workload, nothing timed: the command profiler captures are taken from."""
    import torch

    from paper_2404_09336_b200 import inputs
    from paper_2404_09336_b200.runner import DecodeStep
    wl = inputs.make_config(args.cfg, density=args.density if args.cfg == 5 else None, B=args.batch, H=args.heads)
    ds = DecodeStep(wl, layout=args.layout, kv_copies=1, query_heads=args.query_heads)
    for _ in range(args.steps):
        ds.step(kernels=args.kernels)
        if args.dense:
            ds.attend_dense()
    torch.cuda.synchronize()
    print(f"{wl.name}: {args.steps} steps, status {int(ds.status.item())}, "
          f"{ds.selected_bytes()} selected KV bytes per step")


def spawn_ranks(n):
    """Started as a plain script with --gpus N > 1: run the same command as N ranks (one per GPU) under
    torch.distributed.run on this node and return its exit code."""
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__), *sys.argv[1:]]
    return subprocess.call(cmd)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=500)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--regions", type=int, default=31, help="timed regions of --steps steps; the median is reported")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--cfg", type=int, default=2, choices=[1, 2, 3, 4, 5])
    ap.add_argument("--sweep", default="auto", choices=["auto", "none", "all"])
    ap.add_argument("--probe", default=None, choices=["gather"])
    ap.add_argument("--profile-step", action="store_true")
    ap.add_argument("--density", type=float, default=0.10, help="--profile-step: point of the cfg 5 sweep")
    ap.add_argument("--batch", type=int, default=None, help="--profile-step: batch size override")
    ap.add_argument("--heads", type=int, default=None, help="--profile-step: cache heads override")
    ap.add_argument("--query-heads", type=int, default=None, help="--profile-step: query heads (grouped heads)")
    ap.add_argument("--layout", default="bhtd", choices=["bhtd", "bthd"])
    ap.add_argument("--kernels", default="auto", choices=["auto", "one", "two"], help="--profile-step: step form")
    ap.add_argument("--dense", action="store_true", help="--profile-step: also run the full-context kernel")
    args = ap.parse_args()
    if args.profile_step:
        return run_profile_step(args)
    if args.probe == "gather":
        from paper_2404_09336_b200 import gather_probe
        return gather_probe.main()
    if args.impl == "reference":
        return run_reference(args)
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(spawn_ranks(args.gpus))
    run_ours(args)


if __name__ == "__main__":
    main()
