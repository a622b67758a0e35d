#!/usr/bin/env python
"""Benchmark of the example-retrieval hot path (one JSON line on stdout).

A step is one pass of the whole path over one query batch, as a serving loop would issue
it: register the previous batch's requests (insert), then prepare, score, select and merge
the new batch (query).  The clustered workload instead appends its 10,000 new rows per step.  The default workload is the "online" configuration: 1,000,000 cached
bf16 embeddings of dimension 768, batch of 64 queries, k = 10.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload online] [--nq 64]
  python bench.py --impl reference ...     # times the CPU oracle on the same configuration

With N > 1 (under torchrun, one rank per GPU) every rank runs an independent replica of the
same workload: the path has no cross-GPU step.
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

METRIC = "retrieval_queries_per_sec"
UNIT = "queries/s"

# dram__bytes_read.sum + dram__bytes_write.sum of the dominant kernel, per launch, from the ncu
# captures summarised under profiles/ (key: workload, rows, nq).  An entry is removed (the JSON
# then says null) whenever that kernel changes after its capture.
NCU_TRAFFIC_BYTES_PER_LAUNCH = {
    ("online", 1_000_000, 64): 1_540_728_528,   # profiles/umma_online_q64.md, main pass
    ("online", 1_000_000, 1): 1_540_006_832,    # profiles/scan_online_q1.md
}


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="online")
    ap.add_argument("--nq", type=int, default=None, help="query batch size (default: largest of the workload's sweep)")
    ap.add_argument("--path", default="auto", choices=["auto", "generic", "scan", "umma"])
    ap.add_argument("--rows", type=int, default=None, help="scale the workload's cache to this many rows (profiling aid)")
    ap.add_argument("--no-sweep", action="store_true", help="skip the secondary batch sizes")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--two-level", type=int, default=0, metavar="NPROBE",
                    help="also build the K-Means index (K = sqrt(N), 5 iterations) and time the two-level search "
                         "with this many probed clusters, with its recall against the exhaustive result")
    ap.add_argument("--self-similarity-rows", type=int, default=0,
                    help="also time the all-pairs top-1 self-similarity over this many cached rows")
    return ap.parse_args()


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """nvidia-smi clock/throttle samples taken in the background while the timed regions run."""
    FIELDS = ("timestamp,index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.tmp = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.proc = None
        self.windows = []
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={gpu_index}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "50"], stdout=self.tmp, stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def window(self, t0: float, t1: float):
        self.windows.append((t0, t1))

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.12)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        self.tmp.flush()
        self.tmp.seek(0)
        import datetime
        sm, smax, reasons, all_sm = [], [], set(), []
        for line in self.tmp.read().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 10:
                continue
            try:
                ts = datetime.datetime.strptime(f[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                clk, cmax = float(f[2]), float(f[3])
            except ValueError:
                continue
            all_sm.append(clk)
            smax.append(cmax)
            if any(a - 0.05 <= ts <= b + 0.05 for a, b in self.windows):
                sm.append(clk)
                for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"),
                                     f[6:10]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
        os.unlink(self.tmp.name)
        use = sm or all_sm
        return {"sm_mhz": statistics.median(use) if use else None,
                "sm_max_mhz": max(smax) if smax else None,
                "reasons": sorted(reasons), "samples_in_timed_regions": len(sm)}


def dist_setup(n_gpus: int):
    import torch
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        torch.cuda.set_device(local)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
        return dist, rank, world, local
    if n_gpus > 1:
        raise SystemExit("--gpus N > 1 must be launched with torch.distributed.run, one rank per GPU")
    torch.cuda.set_device(0)
    return None, 0, 1, 0


def aggregate_ranks(dist, local_ms: float, local_units: float, device="cuda"):
    """Whole-job figures: time is the maximum over ranks, work is the sum over ranks."""
    import torch
    if dist is None:
        return local_ms, local_units
    t = torch.tensor([local_ms], dtype=torch.float64, device=device)
    u = torch.tensor([local_units], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


def barrier(dist):
    import torch
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()


def timed_steps(cache, batches, ins_batches, ids_batches, k, steps, out_ids, out_scores, dist, first_step,
                time_inserts=False):
    """K steps of [insert; query batch] timed with CUDA events on the stream the library launches
    on (the current torch stream).  The inserted rows are the previous query batch (a served
    request is registered afterwards) or, for a workload with streaming inserts, that step's own
    batch of new rows (ins_batches).  Returns (ms, wall window, ms spent in the inserts or None)."""
    import torch
    nb = len(batches)
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    marks = []
    barrier(dist)
    w0 = time.time()
    start.record()
    for i in range(first_step, first_step + steps):
        rows = ins_batches[i] if ins_batches is not None else batches[(i - 1) % nb]
        if time_inserts:
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            cache.insert(rows, ids_batches[i])
            e1.record()
            marks.append((e0, e1))
        else:
            cache.insert(rows, ids_batches[i])
        cache.query(batches[i % nb], k, out_ids, out_scores)
    stop.record()
    torch.cuda.synchronize()
    w1 = time.time()
    barrier(dist)
    ins_ms = sum(a.elapsed_time(b) for a, b in marks) if marks else None
    return start.elapsed_time(stop), (w0, w1), ins_ms


def run_ours(args):
    import torch
    from paper_2501_12689_b200 import ICCache, ic_cache_plan, workloads as wl
    from paper_2501_12689_b200 import binding

    dist, rank, world, local = dist_setup(args.gpus)
    dev = torch.device("cuda", local)
    w = wl.WORKLOADS[args.workload]
    if args.rows:
        w = w.scaled(args.rows)
    nq = args.nq or max(w.q_sweep)
    # a workload with streaming inserts appends insert_rows new rows per step: 20 steps by default
    steps = args.steps if args.steps is not None else (20 if w.insert_rows else 500)
    warmup = max(args.warmup if args.warmup is not None else (3 if w.insert_rows else 10), 3)
    path = {"auto": 0, "generic": 1, "scan": 2, "umma": 3}[args.path]
    peaks = load_peaks()
    props = torch.cuda.get_device_properties(dev)

    n_batches = 8
    max_nq = max(max(w.q_sweep), nq)
    ins_rows = w.insert_rows if w.insert_rows else None      # rows appended per step (None: the previous batch)
    per_step = max(max_nq, w.insert_rows)
    capacity = w.n + ((steps + warmup) * (3 + len(w.q_sweep)) + 64) * per_step   # regions: value, profiled, e2e, sweeps
    cache = ICCache(w.dim, capacity, input_dtype=wl.torch_dtype(w))
    cache.set_path(path)
    x = wl.cache_rows(w, dev)
    cache.insert(x, wl.labels(w.n, dev))
    del x
    torch.cuda.synchronize()

    sampler = ClockSampler(local) if rank == 0 else None
    step_counter = [0]

    def measure(q, n_steps, n_warm, profiled):
        batches = [wl.queries(w, q, dev, round_idx=r) for r in range(n_batches)]
        first = step_counter[0] + 1
        tot = n_warm + n_steps
        ins = ins_rows or q
        all_ids = wl.labels(tot * ins, dev, first_slot=cache.size)   # labels follow slots
        ids_batches = {first + j: all_ids[j * ins:(j + 1) * ins] for j in range(tot)}
        ins_batches = {first + j: wl.insert_batch(w, first + j, dev) for j in range(tot)} if ins_rows else None
        out_ids = torch.empty(q, w.k, dtype=torch.int64, device=dev)
        out_scores = torch.empty(q, w.k, dtype=torch.float32, device=dev)
        timed_steps(cache, batches, ins_batches, ids_batches, w.k, n_warm, out_ids, out_scores, dist, first)
        launches0 = cache.launch_count
        cache.set_profiling(profiled)
        if profiled:
            cache.read_profile()
        n_start = cache.size
        ms, win, ins_ms = timed_steps(cache, batches, ins_batches, ids_batches, w.k, n_steps, out_ids, out_scores, dist,
                                      first + n_warm, time_inserts=profiled)
        prof = cache.read_profile() if profiled else None
        if prof is not None:
            prof["insert_ms"] = ins_ms
        cache.set_profiling(False)
        launches = cache.launch_count - launches0
        cache.sync()
        step_counter[0] += tot
        # the cache grows by `ins` rows per step: step j scans n_start + (j + 1) ins rows
        rows_scanned = n_steps * n_start + ins * n_steps * (n_steps + 1) // 2
        if sampler:
            sampler.window(*win)
        return {"ms": ms, "steps": n_steps, "nq": q, "launches": launches, "profile": prof,
                "rows_scanned": rows_scanned, "n_start": n_start, "n_end": cache.size}

    main = measure(nq, steps, warmup, profiled=False)
    prof = measure(nq, steps, warmup, profiled=True)

    # end to end through the host-buffer entry points (pinned host memory)
    e2e_steps = min(steps, 200)
    e2e_ms = None
    if not args.no_e2e:
        hb = [wl.queries(w, nq, dev, round_idx=r).cpu().pin_memory() for r in range(n_batches)]
        ins = ins_rows or nq
        h_ids = wl.labels((e2e_steps + warmup) * ins, "cpu", first_slot=cache.size).pin_memory()
        # new rows of a streaming-insert workload: a few pinned batches, cycled
        h_ins = [wl.insert_batch(w, 10_000 + r, dev).cpu().pin_memory() for r in range(4)] if ins_rows else None
        ho_ids = torch.empty(nq, w.k, dtype=torch.int64).pin_memory()
        ho_sc = torch.empty(nq, w.k, dtype=torch.float32).pin_memory()

        def e2e_rows(i):
            return h_ins[i % 4] if h_ins is not None else hb[(i - 1) % n_batches]

        for i in range(warmup):
            cache.insert_host(e2e_rows(i), h_ids[i * ins:(i + 1) * ins])
            cache.query_host(hb[i % n_batches], w.k, ho_ids, ho_sc)
        barrier(dist)
        t0w = time.time()
        t0 = time.perf_counter()
        for i in range(warmup, warmup + e2e_steps):
            cache.insert_host(e2e_rows(i), h_ids[i * ins:(i + 1) * ins])
            cache.query_host(hb[i % n_batches], w.k, ho_ids, ho_sc)
        torch.cuda.synchronize()
        e2e_ms = (time.perf_counter() - t0) * 1e3
        if sampler:
            sampler.window(t0w, time.time())
        barrier(dist)
    elem = 2 if w.input_dtype == "bf16" else 4
    n_ins = ins_rows or nq
    h2d = nq * w.dim * elem + n_ins * w.dim * elem + n_ins * 8   # query batch + inserted rows + their ids
    d2h = nq * w.k * 12

    sweep = []
    if not args.no_sweep:
        for q in w.q_sweep:
            if q != nq:
                sweep.append(measure(q, min(steps, 200), max(3, min(warmup, 5)), profiled=True))

    self_sim = None
    if args.self_similarity_rows > 0:
        rows = min(args.self_similarity_rows, cache.size)
        cache.self_similarity(0, min(rows, 2048))            # warm-up (grows scratch)
        cache.sync()
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        n_now = cache.size
        ev0.record()
        cache.self_similarity(0, rows)
        ev1.record()
        torch.cuda.synchronize()
        ms = ev0.elapsed_time(ev1)
        self_sim = {"rows": rows, "cache_rows": n_now, "ms": ms, "rows_per_sec": rows / (ms * 1e-3),
                    "tflops": 2.0 * rows * n_now * w.dim / (ms * 1e-3) / 1e12}

    two_level = None
    if args.two_level > 0:
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        cache.build_index(0, 5)
        cache.sync()
        build_s = time.perf_counter() - t0
        k_clusters, n_indexed = cache.index_info()
        rows = []
        for q in sorted(set(w.q_sweep) | {nq}):
            qb = wl.queries(w, q, dev, round_idx=99)
            exact_ids, _ = cache.query(qb, w.k)
            for _ in range(3):
                cache.query_clustered(qb, w.k, args.two_level)
            ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            reps = 50
            ev0.record()
            for _ in range(reps):
                got_ids, _ = cache.query_clustered(qb, w.k, args.two_level)
            ev1.record()
            torch.cuda.synchronize()
            ms = ev0.elapsed_time(ev1) / reps
            e, g = exact_ids.cpu().numpy(), got_ids.cpu().numpy()
            recall = sum(len(set(e[i]) & set(g[i])) for i in range(q)) / float(q * w.k)
            rows.append({"nq": q, "ms_per_call": ms, "queries_per_sec": q / (ms * 1e-3), "recall_at_k": recall})
        two_level = {"n_clusters": k_clusters, "n_indexed": n_indexed, "rows_outside_index": cache.size - n_indexed,
                     "nprobe": args.two_level, "build_s": build_s, "kmeans_iters": 5, "calls": rows}

    # context for the HBM denominator: a pure read stream (torch sum-reduction over 4 GiB), since the
    # measured copy peak mixes reads and writes
    read_stream = None
    if rank == 0:
        try:
            buf = torch.ones(1 << 29, dtype=torch.int64, device=dev)   # int64 sum: the fastest of torch's reductions here
            for _ in range(2):
                buf.sum()
            ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            ev0.record()
            for _ in range(5):
                buf.sum()
            ev1.record()
            torch.cuda.synchronize()
            read_stream = 5 * buf.numel() * 8 / (ev0.elapsed_time(ev1) * 1e-3) / 1e9
            del buf
        except RuntimeError:
            read_stream = None

    clocks = sampler.stop() if sampler else None

    ms_all, q_all = aggregate_ranks(dist, main["ms"], float(nq * steps))
    value = q_all / (ms_all * 1e-3)
    if e2e_ms is not None:
        e2e_ms_all, e2e_q_all = aggregate_ranks(dist, e2e_ms, float(nq * e2e_steps))
        e2e = {"value": e2e_q_all / (e2e_ms_all * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "steps": e2e_steps, "ms_per_step": e2e_ms_all / e2e_steps}
    else:
        e2e = None

    if rank != 0:
        cache.close()
        if dist is not None:
            dist.destroy_process_group()
        return

    def roofline_of(r):
        """Roofline of the dominant kernel: the main scoring launch (fused score + partial top-k;
        on the tensor-core path the launch that reads every row outside the seeding samples).
        Algorithmic bytes per launch = 2*dim per row it scans, flops = 2*dim per (query, row);
        the bound is whichever takes longer at the measured peaks."""
        pr = r["profile"]
        if not pr or pr["scoring_launches"] == 0:
            return None
        rows = r["rows_scanned"] / r["steps"]                     # mean cache rows per step
        pl = ic_cache_plan(w.dim, int(rows), r["nq"], w.k, path, props.multi_processor_count,
                           props.shared_memory_per_block_optin)
        launches_per_step = pr["scoring_launches"] / r["steps"]
        rows_main = rows - min(rows, pl["seed_tiles"] * 256)       # rows the dominant launch reads
        bytes_per_launch = rows_main * w.dim * 2
        flops_per_launch = bytes_per_launch * min(r["nq"], pl["query_tile"] * pl["n_query_tiles"])
        t_launch = pr["scoring_ms"] * 1e-3 / pr["scoring_launches"]
        t_hbm = bytes_per_launch / (peaks["hbm_gbs"] * 1e9)
        t_tensor = flops_per_launch / (peaks["bf16_tflops_sustained"] * 1e12)
        if t_hbm >= t_tensor:
            ach = bytes_per_launch / t_launch / 1e9
            out = {"bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                   "frac": ach / peaks["hbm_gbs"]}
        else:
            ach = flops_per_launch / t_launch / 1e12
            out = {"bound": "tensor", "achieved": ach, "peak": peaks["bf16_tflops_sustained"], "unit": "TFLOP/s",
                   "frac": ach / peaks["bf16_tflops_sustained"]}
        # the same achieved figure against the nominal peaks (8 TB/s HBM3e, 2250 TFLOP/s dense bf16)
        out["frac_of_nominal"] = out["achieved"] / (8000.0 if out["bound"] == "hbm" else 2250.0)
        traffic = NCU_TRAFFIC_BYTES_PER_LAUNCH.get((w.name, w.n, r["nq"]))
        out.update({"traffic": traffic, "peak_source": peaks["source"] + " (sustained figure for tensor)",
                    "kernel": {2: "scan_score_topk_kernel", 3: "umma_score_topk_kernel (main pass)",
                               1: "generic_score_topk_kernel"}[pl["path"]],
                    "kernel_us_per_launch": t_launch * 1e6,
                    "launches_per_step": launches_per_step,
                    "algorithmic_bytes_per_launch": bytes_per_launch,
                    "rows_per_launch": rows_main,
                    "insert_us_per_step": (pr["insert_ms"] * 1e3 / r["steps"]) if pr.get("insert_ms") is not None else None,
                    "seed_passes_us_per_step": pr["seed_ms"] * 1e3 / r["steps"],
                    "final_merge_us_per_step": pr["merge_ms"] * 1e3 / r["steps"]})
        return out

    plan = ic_cache_plan(w.dim, w.n, nq, w.k, path, props.multi_processor_count,
                         props.shared_memory_per_block_optin)
    roof = roofline_of(prof) or {"bound": "hbm", "achieved": None, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                                 "frac": None, "traffic": None}
    mean_rows = main["rows_scanned"] / steps
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps, "warmup": warmup,
        "ms_per_step": ms_all / steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": f"{w.name}: N={w.n} d={w.dim} {w.input_dtype} unit {w.kind}, nq={nq}, k={w.k}",
                   "step": (f"insert {w.insert_rows} new rows + query batch (prep, score, partial top-k, merge)" if w.insert_rows
                            else "insert previous batch (nq rows) + query batch (prep, score, partial top-k, merge)"),
                   "n_start": main["n_start"], "n_end": main["n_end"], "path": binding.PATH_NAMES[plan["path"]],
                   "plan": plan, "l2": "slab is many times larger than L2 (126 MB): no flush between steps",
                   "replicas": world},
        "cache_entries_per_sec": mean_rows * nq * world / (ms_all / steps * 1e-3),
        "read_stream_gb_per_sec": read_stream,
        "slab_gb_per_sec_whole_step": mean_rows * w.dim * 2 / (ms_all / steps * 1e-3) / 1e9,
        "gpu_launches": main["launches"],
        "e2e": e2e,
        "roofline": roof,
        "profiled_region": {"ms_per_step": prof["ms"] / steps},
        "clocks": clocks,
        "self_similarity": self_sim,
        "two_level": two_level,
        "sweep": [{"nq": r["nq"], "queries_per_sec": r["nq"] * r["steps"] / (r["ms"] * 1e-3),
                   "ms_per_step": r["ms"] / r["steps"], "roofline": roofline_of(r)} for r in sweep],
    }
    cache.close()
    torch.cuda.empty_cache()
    if not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline(w, nq)
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def oracle_seconds(w, n_rows, nq_sample, x_bits, q_bits, threads):
    import oracle
    t0 = time.perf_counter()
    oracle.search(x_bits[:n_rows], q_bits[:nq_sample], w.k, threads=threads)
    return time.perf_counter() - t0


def cpu_baseline(w, nq):
    """The oracle as it stands, timed on this host's cores on a bounded sample of the same
    workload: a few queries of the batch against the workload's initial cache rows."""
    import torch
    from oracle.ic_oracle import default_threads
    from paper_2501_12689_b200 import workloads as wl
    threads = default_threads()
    x_bits = wl.as_bits(wl.cache_rows(w, "cuda" if torch.cuda.is_available() else "cpu"))
    q_bits = wl.as_bits(wl.queries(w, nq, "cpu"))
    n_probe = min(w.n, 100_000)
    per_query = oracle_seconds(w, n_probe, 1, x_bits, q_bits, threads) * w.n / n_probe
    n_sample = int(max(1, min(nq, 15.0 / max(per_query, 1e-6))))
    dt = oracle_seconds(w, w.n, n_sample, x_bits, q_bits, threads)
    return {"value": n_sample / dt, "unit": UNIT, "cores": threads, "kind": "oracle",
            "sample": f"{n_sample} of the batch's {nq} queries against all {w.n} rows (scores + full sort), {dt:.1f} s"}


def run_reference(args):
    """The reference arm: the CPU oracle, unmodified, on the same configuration and metric.
    Each step scores a bounded sample of the batch; rank 0 alone works."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    import torch
    import oracle
    from oracle.ic_oracle import default_threads
    from paper_2501_12689_b200 import workloads as wl
    w = wl.WORKLOADS[args.workload]
    if args.rows:
        w = w.scaled(args.rows)
    nq = args.nq or max(w.q_sweep)
    steps = args.steps if args.steps is not None else 8
    warmup = args.warmup if args.warmup is not None else 1
    threads = default_threads()
    dev = "cuda" if torch.cuda.is_available() else "cpu"
    x_bits = wl.as_bits(wl.cache_rows(w, dev))
    batches = [wl.as_bits(wl.queries(w, nq, "cpu", round_idx=r)) for r in range(4)]
    # size the per-step sample so that the whole run stays within about two minutes
    n_probe = min(w.n, 100_000)
    per_query = oracle_seconds(w, n_probe, 1, x_bits, batches[0], threads) * w.n / n_probe
    budget = 120.0 / max(1, steps + warmup)
    n_rows = w.n
    q_per_step = int(min(nq, budget / per_query))
    if q_per_step < 1:
        q_per_step = 1
        n_rows = int(max(min(w.n, 10_000), min(w.n, w.n * budget / per_query)))
    for i in range(warmup):
        oracle.search(x_bits[:n_rows], batches[i % 4][:q_per_step], w.k, threads=threads)
    t0 = time.perf_counter()
    for i in range(steps):
        oracle.search(x_bits[:n_rows], batches[i % 4][:q_per_step], w.k, threads=threads)
    dt = time.perf_counter() - t0
    # queries/s against the full cache: a sample of n_rows rows is scaled by n_rows / N
    value = q_per_step * steps / dt * (n_rows / w.n)
    sample = f"{q_per_step} of {nq} queries per step against {n_rows} of {w.n} rows"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": steps,
        "warmup": warmup, "ms_per_step": dt / steps * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": f"{w.name}: N={w.n} d={w.dim} {w.input_dtype} unit {w.kind}, nq={nq}, k={w.k}",
                   "step": "CPU oracle: brute-force fp32 scores + full sort, " + sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
