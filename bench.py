#!/usr/bin/env python
"""Benchmark of the quantized-GBDT hot path on B200.

A step is one boosting iteration (one tree) of the whole path -- gradients, quantization,
leaf-wise growth with integer histograms, subtraction, split search, partition, refit, score
update -- on a synthetic workload shaped like the paper's largest dense dataset
(10.5 M rows x 28 features, 255 bins, squared loss, 4-bit gradients, 255 leaves).

Metric: histogram row-features per second = rows x features that Algorithm 1 has to visit
(the root plus the smaller child of every split) divided by the time of the WHOLE step.
ms_per_step is ms per tree.  `roofline` is the histogram kernel alone: algorithmic bytes of
all its launches inside the timed region over their summed CUDA-event durations, against the
measured HBM copy bandwidth; `tree_roofline` is the whole step: the algorithmic bytes of every
kernel family of the timed trees over the step time.  `cpu_baseline` is the CPU oracle.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

WORKLOAD_ROWS = {"large": 10_500_000, "tall": 1_000_000, "tiny": 50_000, "wide": 400_000}
# rows of the CPU arm: the same rows as the GPU arm (one oracle tree: about 9 s on 'large', 15 s on 'wide')
CPU_SAMPLE_ROWS = dict(WORKLOAD_ROWS)
FALLBACK_HBM_GBS = 6650.0
# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) of the histogram kernels on the 'large'
# workload, per build, averaged over the builds of one tree, from an ncu capture of the same kernels on
# 4 M rows scaled by the rows (traffic grows in proportion to them).  Valid only for the kernel sources
# the capture was taken with.
HIST_TRAFFIC = {"workload": "large", "bytes_per_launch": 11.01e6,
                "sources_sha1": "0ba02b51281a9401982eb480d803ad5ff840cfbe"}


def hist_traffic(workload, rows):
    import hashlib
    h = hashlib.sha1()
    try:
        for f in ("hist_cta.cuh", "hist.cu"):   # the sources of the histogram kernels
            h.update(open(os.path.join(ROOT, "paper_2207_09682_b200", "csrc", f), "rb").read())
    except OSError:
        return None
    if workload != HIST_TRAFFIC["workload"] or rows != WORKLOAD_ROWS[workload] or h.hexdigest() != HIST_TRAFFIC["sources_sha1"]:
        return None      # the kernel changed since the counters were taken (or another workload)
    return HIST_TRAFFIC["bytes_per_launch"]


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        return float(json.load(open(path))["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.FIELDS,
                                          "--format=csv,noheader,nounits", "-lms", "100"], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None
        return self

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def __exit__(self, *a):
        if self.proc:
            time.sleep(0.15)
            self.proc.terminate()
            self.thread.join(timeout=2)

    def summary(self) -> dict:
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0]))
                mx.append(float(r[1]))
                for name, v in zip(names, r[2:6]):
                    if v.lower().startswith("active"):
                        reasons.add(name)
            except Exception:
                pass
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def tree_rows(tree: dict, n_rows: int) -> tuple[int, int]:
    """Rows one tree must visit: (histogram rows = the root plus the smaller child of every split,
    partition rows = the rows of every leaf that was split)."""
    nl = tree["num_leaves"]
    if nl <= 1:
        return n_rows, 0
    count = {}

    def size(c):
        if c < 0:
            return int(tree["leaf_count"][~c])
        if c not in count:
            count[c] = size(int(tree["left"][c])) + size(int(tree["right"][c]))
        return count[c]

    hist, part = n_rows, 0
    for i in range(nl - 1):
        a, b = size(int(tree["left"][i])), size(int(tree["right"][i]))
        hist += min(a, b)
        part += a + b
    return hist, part


def needed_hist_rows(tree: dict, n_rows: int) -> int:
    return tree_rows(tree, n_rows)[0]


def code_bytes(bits: int) -> int:
    """Packed gradient + hessian code per row that the method has to move: one byte up to 4 bits, two beyond."""
    return 1 if bits <= 4 else 2


def tree_algorithmic_bytes(trees: list, n: int, features: int, n_bins: int, bits: int, const_hessian: bool) -> dict:
    """Bytes every step of the path must move for the given trees (per kernel family, summed over the trees):
    histogram builds  rows * (F + c [+ 4 row index for a child]) + F * bins * 8 per build
    partition         parent rows * (4 index in + 1 bin code + 4 index out)
    quantizer         N * (4 per gradient array read + c written)
    gradients         N * (scores + labels read, one or two arrays written)
    refit, scores     N * (gradient arrays + 4 row index) resp. N * 8
    split search      2 * F * bins * 8 per split; subtraction 3 * F * bins * 8 per split"""
    c = code_bytes(bits)
    arrays = 1 if const_hessian else 2
    hb = features * n_bins * 8
    out = dict.fromkeys(("histogram", "partition", "quantize", "gradients", "refit", "score_update", "split_search",
                         "subtraction"), 0)
    for t in trees:
        hist_rows, part_rows = tree_rows(t, n)
        splits = max(int(t["num_leaves"]) - 1, 0)
        out["histogram"] += n * (features + c) + (hist_rows - n) * (features + c + 4) + (splits + 1) * hb
        out["partition"] += part_rows * 9
        out["quantize"] += n * (4 * arrays + c)
        out["gradients"] += n * (8 + 4 * arrays)
        out["refit"] += n * (4 * arrays + 4)
        out["score_update"] += n * 8
        out["split_search"] += (2 * splits + 1) * hb
        out["subtraction"] += 3 * splits * hb
    return out


def oracle_leg(wl_name: str, rows: int, steps: int, warmup: int, data=None, y=None, n_bins=None, params=None) -> dict:
    """Times the CPU oracle (as it stands, one thread): whole boosting iterations."""
    import numpy as np
    import oracle
    from paper_2207_09682_b200 import synth
    if data is None:
        wl = synth.CONFIGS[wl_name](device="cpu", rows=rows)
        data, y, n_bins, params = wl.bins.numpy(), wl.labels.numpy(), wl.n_bins, wl.params
    prm = oracle.make_params(**dict(params, num_trees=1, seed=1))
    scores = np.zeros(rows, np.float32)
    rf, secs = 0, 0.0
    for k in range(warmup + steps):
        t0 = time.perf_counter()
        t = oracle.train_tree(data, n_bins, y, scores, prm, k)
        dt = time.perf_counter() - t0
        if k >= warmup:
            tree = dict(num_leaves=t.num_leaves, left=t.left, right=t.right, leaf_count=t.leaf_count)
            rf += needed_hist_rows(tree, rows) * data.shape[1]
            secs += dt
    return {"value": rf / secs, "unit": "row-features/s", "cores": 1, "kind": "oracle",
            "sample": "%d trees of %d leaves on all %d rows x %d features of workload '%s'"
                      % (steps, prm.num_leaves, rows, data.shape[1], wl_name),
            "ms_per_tree": 1e3 * secs / steps, "host_cores": os.cpu_count()}


def oracle_hist_all_cores(data, n_bins: int, max_rows: int = 4_000_000) -> dict:
    """The oracle's Algorithm 1 on every host core: the harness cuts the rows into one chunk per
    thread, every thread calls the unchanged single-threaded routine into arrays of its own (ctypes
    releases the interpreter lock), and the per-chunk histograms are added up afterwards."""
    import numpy as np
    import oracle
    from concurrent.futures import ThreadPoolExecutor
    cores = os.cpu_count() or 1
    n = min(len(data), max_rows)
    data = data[:n]
    r = np.random.default_rng(0)
    gq = r.integers(-7, 8, size=n).astype(np.int8)
    hq = np.ones(n, np.uint8)
    bounds = [n * i // cores for i in range(cores + 1)]

    def chunk(i):
        a, b = bounds[i], bounds[i + 1]
        return oracle.histogram(data[a:b], n_bins, gq[a:b], hq[a:b])

    best = None
    with ThreadPoolExecutor(max_workers=cores) as pool:
        for _ in range(3):
            t0 = time.perf_counter()
            parts = list(pool.map(chunk, range(cores)))
            hg = sum(p[0] for p in parts)
            dt = time.perf_counter() - t0
            best = dt if best is None else min(best, dt)
    assert int(hg.sum()) == int(gq.astype(np.int64).sum()) * data.shape[1]
    return {"value": n * data.shape[1] / best, "unit": "row-features/s", "cores": cores, "kind": "oracle",
            "scope": "root histogram build only (Algorithm 1), best of 3",
            "sample": "the first %d rows x %d features, one row chunk per thread" % (n, data.shape[1])}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    rows = min(args.rows or WORKLOAD_ROWS[args.workload], CPU_SAMPLE_ROWS[args.workload])
    steps, warmup = args.steps, args.warmup
    leg = oracle_leg(args.workload, rows, steps, warmup)
    line = {"impl": "reference", "metric": "hist_row_features_per_s", "value": leg["value"], "unit": "row-features/s",
            "n_gpus": args.gpus, "steps": steps, "warmup": warmup, "ms_per_step": leg["ms_per_tree"],
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int32", "data": "synthetic",
            "config": {"workload": args.workload, "rows": rows,
                       "note": "CPU oracle, one thread of %s host cores, whole boosting iterations" % os.cpu_count()},
            "cpu_baseline": {k: leg[k] for k in ("value", "unit", "cores", "kind", "sample", "host_cores")},
            "e2e": {"value": leg["value"], "unit": "row-features/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def time_hist_builds(ctx, torch, synth, n, features, n_bins, cbytes, reps=10, batch=10, fp32=None):
    """Stand-alone root and 50%-subset histogram builds on inputs larger than L2.

    `batch` builds are enqueued back to back between two CUDA events so that the GPU never waits
    for the host; the time per build is the median over `reps` such batches.  (Writing a buffer
    to flush L2 would leave it full of dirty lines whose write-back is then charged to the next
    build; the bin matrix itself is larger than L2, so nothing is reused between builds.)"""
    import numpy as np
    hist = ctx.new_hist()
    rows = synth.subset_rows(n, device="cuda")
    out = {}
    for name, r in (("root", None), ("subset50", rows)):
        ts = []
        for i in range(reps + 3):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(batch):
                if r is None:
                    ctx.build_histograms(0, hist)
                else:
                    ctx.build_histograms_rows(r, hist)
            e1.record()
            torch.cuda.synchronize()
            if i >= 3:
                ts.append(e0.elapsed_time(e1) / batch)
        nr = n if r is None else int(r.numel())
        ms = float(np.median(ts))
        nbytes = nr * (features + cbytes + (0 if r is None else 4)) + features * n_bins * 8
        out[name] = {"rows": nr, "us": 1e3 * ms, "row_features_per_s": nr * features / (ms * 1e-3),
                     "gbs": nbytes / (ms * 1e6), "note": "partial histograms and their merge in one cooperative kernel, %d builds per timing" % batch}
    if fp32 is not None:
        # the unquantized baseline on the same kernel design: Algorithm 1 with the original float gradients
        g, h = fp32
        ts = []
        for i in range(reps + 3):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(batch):
                ctx.build_histograms_fp32(g, h)
            e1.record()
            torch.cuda.synchronize()
            if i >= 3:
                ts.append(e0.elapsed_time(e1) / batch)
        ms = float(np.median(ts))
        out["root_fp32"] = {"rows": n, "us": 1e3 * ms, "row_features_per_s": n * features / (ms * 1e-3),
                            "slower_than_quantized": 1e3 * ms / out["root"]["us"],
                            "note": "floating-point histogram of the original gradients (Sec. 7.2's baseline; the paper reports "
                                    "quantized histograms 2.3x (Higgs) to 3.9x (Epsilon) faster on a V100)"}
    return out


def run_sweep(args):
    """Histogram-kernel sweep (rows x features x bins x gradient bits, root and 50 % subset builds);
    prints one text line per point.  Not a benchmark line: a table of the kernel over tile widths, bit widths and row fractions."""
    import torch
    from paper_2207_09682_b200 import binding, synth
    torch.cuda.set_device(0)
    peak, kind = measured_peak()
    print("# rows features bins bits | root us  GB/s  frac | subset50 us  GB/s  frac   (frac of %s %.0f GB/s)" % (kind, peak))
    for n in (1_000_000, 4_000_000, 16_000_000):
        for f in (28, 136, 1000):
            for nb in (16, 64, 255):
                bins = synth.sweep_bins(n, f, nb, device="cuda")
                g, h = synth.sweep_gradients(n, device="cuda")
                for bits in (2, 3, 4, 8):
                    ctx = binding.Context(binding.make_params(bits=bits))
                    ctx.load_binned(bins, nb)
                    ctx.quantize_gradients(g, h)
                    b = time_hist_builds(ctx, torch, synth, n, f, nb, code_bytes(bits), reps=3, batch=5)
                    print("%9d %5d %4d %2d | %9.1f %7.0f %5.3f | %9.1f %7.0f %5.3f" % (
                        n, f, nb, bits, b["root"]["us"], b["root"]["gbs"], b["root"]["gbs"] / peak,
                        b["subset50"]["us"], b["subset50"]["gbs"], b["subset50"]["gbs"] / peak), flush=True)
                    ctx.close()
                del bins


def aggregate_ranks(ms, row_features, launches, dist=None, device="cpu"):
    """Whole-job figures from per-rank ones: the step time is the maximum over the ranks, work and
    launch counts add up.  The ranks are independent replicas (no data-path collective): this is
    the only exchange of a multi-GPU run."""
    import torch
    if dist is None:
        return float(ms), float(row_features), float(launches)
    t = torch.tensor([ms, float(row_features), float(launches)], dtype=torch.float64, device=device)
    tmax = t.clone()
    dist.all_reduce(tmax, op=dist.ReduceOp.MAX)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(tmax[0]), float(t[1]), float(t[2])


def run_ours(args):
    import numpy as np
    import torch
    from paper_2207_09682_b200 import binding, synth

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    rows = args.rows or WORKLOAD_ROWS[args.workload]
    sharded = args.scaling == "strong" and world > 1
    if sharded:
        # data-distributed training (Sec. 7.3): one training set, every rank holds a contiguous row shard;
        # the ranks exchange integer histograms, counts and the two maxima through NCCL all-reduces
        from paper_2207_09682_b200 import dist as qdist
        wl = synth.CONFIGS[args.workload](device="cuda", rows=rows, seed=synth.MASTER_SEED + 100)
        lo, hi = rows * rank // world, rows * (rank + 1) // world
        wl.bins, wl.labels = wl.bins[lo:hi].contiguous(), wl.labels[lo:hi].contiguous()
        torch.cuda.empty_cache()
    else:
        wl = synth.CONFIGS[args.workload](device="cuda", rows=rows, seed=synth.MASTER_SEED + 100 + rank)
    n, features = wl.bins.shape
    n_bins = wl.n_bins
    kw = dict(wl.params, num_trees=1, seed=1 if sharded else 1 + rank)
    ctx = binding.Context(binding.make_params(**kw))
    ctx.load_binned(wl.bins, wl.n_bins)
    if sharded:
        reducer = qdist.TorchDistReducer()
        ctx.set_distributed(rank, world, lo, rows, reducer.callback)
    scores = torch.zeros(n, device="cuda")
    K, W = args.steps, args.warmup

    if args.stream_path:
        ctx.profile_histograms(True)
    ctx.train(wl.labels, scores, 0, W)                       # warm-up trees 0 .. W-1
    torch.cuda.synchronize()
    c0 = ctx.get_counters()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if dist:
        dist.barrier()
    torch.cuda.synchronize()
    with ClockSampler(local) as clocks:
        e0.record()
        model = ctx.train(wl.labels, scores, W, K)           # the timed K steps
        e1.record()
        torch.cuda.synchronize()
    if dist:
        dist.barrier()
    ms = e0.elapsed_time(e1)
    c1 = ctx.get_counters()
    # Roofline of the histogram kernels: the K boosting iterations that follow, with a pair of CUDA
    # events around every histogram build.  (The timed region above replays a tree's ~1000 launches
    # from a CUDA graph; event records between them would put the launches back on the stream, so
    # the per-build timing runs right after it, on the same data, trees W+K .. W+2K-1.)
    ctx.profile_histograms(True)
    e2, e3 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e2.record()
    ctx.train(wl.labels, scores, W + K, K)
    e3.record()
    torch.cuda.synchronize()
    phases = ctx.get_timings()
    prof = ctx.get_histogram_profile()
    ctx.profile_histograms(False)
    prof_ms = e2.elapsed_time(e3)
    rf = c1["hist_row_features"] - c0["hist_row_features"]
    launches = c1["kernel_launches"] - c0["kernel_launches"]
    leaves = [int(x) for x in model.num_leaves]

    ms, rf, launches = aggregate_ranks(ms, rf, launches, dist, "cuda")
    if rank != 0:
        dist.destroy_process_group()
        return

    peak, peak_kind = measured_peak()
    achieved = prof["total_bytes"] / (prof["total_ms"] * 1e6) if prof["total_ms"] > 0 else 0.0
    cbytes = code_bytes(kw["bits"])
    # the whole step against the bytes it has to move (this rank's trees; the ranks are replicas)
    step_bytes = tree_algorithmic_bytes([model.tree(k) for k in range(K)], n, features, n_bins, kw["bits"],
                                        kw["objective"] == 1)
    step_total = sum(step_bytes.values())
    line = {
        "metric": "hist_row_features_per_s", "value": rf / (ms * 1e-3), "unit": "row-features/s",
        "n_gpus": world, "steps": K, "warmup": W, "ms_per_step": ms / K, "higher_is_better": True,
        "scaling": "strong" if sharded else "weak", "vs_baseline": None, "dtype": "int32", "data": "synthetic",
        "config": {"workload": args.workload, "rows": rows if sharded else n, "features": features, "bins": wl.n_bins,
                   "bits": kw["bits"], "num_leaves": kw["num_leaves"], "objective": kw["objective"],
                   "l2_policy": "inputs larger than L2 (bin matrix %d MB)" % (n * ((features + 3) // 4 * 4) >> 20),
                   "multi_gpu": ("rows sharded over the ranks, integer all-reduces through NCCL (Sec. 7.3)" if sharded else
                                 "replicas: one independent training set per GPU, no data-path collective"),
                   "leaves_per_tree": [min(leaves), max(leaves)]},
        "gpu_launches": int(launches),
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "traffic": hist_traffic(args.workload, n), "peak_kind": peak_kind,
                     "kernel": "k_hist / k_hist_grow (+ merge): every histogram build of the timed trees",
                     "algorithmic_bytes_per_launch": prof["total_bytes"] / max(prof["builds"], 1),
                     "launches": prof["builds"], "total_ms": prof["total_ms"],
                     "share_of_step": prof["total_ms"] / prof_ms if prof_ms else None,
                     "region": "K more boosting iterations right after the timed ones, launches on the stream with "
                               "an event pair around every build (%.2f ms per tree there)" % (prof_ms / K)},
        "tree_roofline": {"bound": "hbm", "achieved": step_total / (ms * 1e6), "peak": peak, "unit": "GB/s",
                          "frac": step_total / (ms * 1e6) / peak, "peak_kind": peak_kind,
                          "algorithmic_bytes_per_tree": step_total / K,
                          "ms_per_tree_at_peak": step_total / K / (peak * 1e6),
                          "bytes_per_tree_by_step": {k: v / K for k, v in step_bytes.items()},
                          "note": "every kernel family of the timed trees: bytes the method has to move over the step time"},
        "phases_us_per_tree": {k: round(1e3 * v["ms"] / K, 1) for k, v in phases.items()},
        "clocks": clocks.summary(),
        "host_cores": os.cpu_count(),
    }
    line["phases_us_per_tree"]["note"] = ("CUDA events around every phase in the profiled pass (passes of tree growth on the "
                                          "stream, the host following): where a tree's time goes, not how long it takes")

    if sharded:
        line["exchanges"] = {"calls": reducer.calls, "words": reducer.words,
                             "note": "all-reduce calls and 32/64-bit words of rank 0 since the context was created"}
        print(json.dumps(line))
        dist.destroy_process_group()
        return

    # stand-alone histogram builds on the same data (root leaf and a 50 % subset)
    g = torch.empty(n, device="cuda")
    h = torch.empty(n, device="cuda") if kw["objective"] == 0 else None
    ctx.reset_leaves()
    ctx.compute_gradients(scores, wl.labels, g, h)
    ctx.quantize_gradients(g, h, tree=W + K)
    builds = time_hist_builds(ctx, torch, synth, n, features, n_bins, cbytes, fp32=(g, h))
    for b in builds.values():
        if "gbs" in b:
            b["frac"] = b["gbs"] / peak
    line["hist_builds"] = builds

    # end to end through the C ABI with host buffers: every step copies the bin matrix, labels and
    # scores from pinned host memory and reads the scores back
    host_data = None
    if not args.no_e2e:
        hb = wl.bins.cpu().pin_memory()
        hl = wl.labels.cpu().pin_memory()
        host_data = (hb.numpy(), hl.numpy())
        hs = torch.zeros(n).pin_memory()
        ctx.close()
        del wl, scores
        torch.cuda.empty_cache()
        ctx2 = binding.Context(binding.make_params(**kw))
        e_steps = max(1, min(K, 5))
        rf2, t_e2e = 0, 0.0
        for k in range(1 + e_steps):
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            ctx2.load_binned(hb, n_bins)
            m2 = ctx2.train(hl, hs, k, 1)
            torch.cuda.synchronize()
            dt = time.perf_counter() - t0
            if k >= 1:
                t_e2e += dt
                rf2 += needed_hist_rows(m2.tree(0), n) * features
        line["e2e"] = {"value": rf2 / t_e2e, "unit": "row-features/s", "h2d_bytes_per_step": int(hb.numel() + 8 * n),
                       "d2h_bytes_per_step": int(4 * n), "steps": e_steps, "ms_per_step": 1e3 * t_e2e / e_steps}
        ctx2.close()

    if not args.no_cpu_baseline:
        if host_data is None:
            leg = oracle_leg(args.workload, min(n, CPU_SAMPLE_ROWS[args.workload]), 1, 0)
        else:   # the very arrays the GPU path was timed on, all rows, one tree
            leg = oracle_leg(args.workload, n, 1, 0, host_data[0], host_data[1], n_bins, kw)
        line["cpu_baseline"] = {k: leg[k] for k in ("value", "unit", "cores", "kind", "sample", "host_cores")}
        if host_data is not None:
            line["cpu_baseline"]["all_cores"] = oracle_hist_all_cores(host_data[0], n_bins)
    print(json.dumps(line))
    if dist:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="large", choices=sorted(WORKLOAD_ROWS))
    ap.add_argument("--rows", type=int, default=0, help="override the workload's row count (profiling captures)")
    ap.add_argument("--stream-path", action="store_true",
                    help="launch every kernel of tree growth on the stream (the host follows the passes) instead of "
                         "replaying the growth graph: for per-kernel launch lists, not for timing")
    ap.add_argument("--scaling", default="weak", choices=["weak", "strong"],
                    help="with --gpus N > 1: weak = N independent replicas of the workload (default); strong = one "
                         "training set sharded by rows over the ranks (data-distributed training, NCCL all-reduces)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--sweep", action="store_true", help="print the histogram-kernel sweep table instead")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # started by hand: start the N ranks (one per GPU) the way the driver does
        import socket
        with socket.socket() as sk:
            sk.bind(("127.0.0.1", 0))
            port = sk.getsockname()[1]
        cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(args.gpus),
               "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
        sys.exit(subprocess.call(cmd))
    if args.sweep:
        run_sweep(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
