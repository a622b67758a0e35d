#!/usr/bin/env python
"""Benchmark of the example-retrieval hot path (one JSON line on stdout).

A step is one pass of the whole path over one query batch, as a serving loop would issue
it: register the previous batch's requests (insert), then prepare, score, select and merge
the new batch (query).  The clustered workload instead appends its 10,000 new rows per step.

The default workload is the largest single-GPU configuration, "stress": 16,000,000 cached bf16
embeddings of dimension 768 (24.6 GB), k = 64, headline batch of 1024 queries, with the batch
sizes 1 and 64 in `sweep`, a forced-path sweep over the batch size in `crossover` (CUDA-core scan
against the tensor-core path), one compact entry per other configuration in `configs`, and the
two widening workloads (`two_level`, `self_similarity`).

Every timed region is exactly --steps steps between CUDA events; a region is repeated --repeats
times (the cache is brought back to its starting size in between, untimed) and the line reports
the median and the best region with the SM clock sampled during each.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--repeats R] [--workload stress] [--nq 1024]
  python bench.py --impl reference ...     # times the CPU oracle on the same configuration

With N > 1 (under torchrun, one rank per GPU) every rank runs an independent replica of the
same workload: the path has no cross-GPU step.
"""
from __future__ import annotations

import argparse
import datetime
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
NOMINAL_HBM_GBS = 8000.0
NOMINAL_BF16_TFLOPS = 2250.0

# DRAM traffic of the dominant kernel (dram__bytes_read.sum + dram__bytes_write.sum per launch) from
# the ncu captures summarised under profiles/, as bytes per cache row the launch scans: the
# captures run on a scaled-down cache, and the traffic of this kernel grows in proportion to the
# rows scanned.  Key: (kernel, dim).  An entry is removed (the line then says null) whenever that
# kernel changes after its capture.
NCU_TRAFFIC_BYTES_PER_ROW = {
    # profiles/umma_stress_2m_q1024.md: main pass, CTA pairs, 2,890,656,256 B over 1,877,632 scanned rows
    ("umma_score_topk_kernel<2,streamed> (main pass)", 768): 2_890_656_256 / 1_877_632,
    # profiles/umma_dense_1m_q256.md: CTA pairs, 2,095,586,048 B over 1,000,512 rows (incl. the re-read first tiles)
    ("umma_score_topk_kernel<2,streamed> (main pass)", 1024): 2_095_586_048 / 1_000_512,
    # profiles/umma_online_q64.md: resident query tile, 1,542,629,632 B over 1,000,128 rows
    ("umma_score_topk_kernel<1,resident> (main pass)", 768): 1_542_629_632 / 1_000_128,
    # profiles/scan_online_q1.md: CUDA-core scan, 1,540,525,312 B over 1,000,002 rows
    ("scan_score_topk_kernel", 768): 1_540_525_312 / 1_000_002,
}


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--repeats", type=int, default=None, help="timed regions of --steps steps per measurement (default 20)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="stress")
    ap.add_argument("--nq", type=int, default=None, help="query batch size (default: largest of the workload's sweep)")
    ap.add_argument("--path", default="auto", choices=["auto", "generic", "scan", "umma"])
    ap.add_argument("--rows", type=int, default=None, help="scale the workload's cache to this many rows (profiling aid)")
    ap.add_argument("--no-sweep", action="store_true", help="skip the secondary batch sizes")
    ap.add_argument("--no-crossover", action="store_true", help="skip the forced-path sweep over the batch size")
    ap.add_argument("--no-configs", action="store_true", help="skip the compact entries of the other configurations")
    ap.add_argument("--no-widening", action="store_true", help="skip the two-level and self-similarity workloads")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--minimal", action="store_true",
                    help="headline measurement only (profiling aid): implies every --no-* switch")
    ap.add_argument("--only-widening", action="store_true",
                    help="with --minimal: keep the widening workload of the chosen configuration (profiling aid)")
    ap.add_argument("--two-level-nprobe", type=int, default=4)
    ap.add_argument("--self-similarity-rows", type=int, default=65536)
    a = ap.parse_args()
    if a.minimal:
        a.no_sweep = a.no_crossover = a.no_configs = a.no_cpu_baseline = a.no_e2e = True
        a.no_widening = not a.only_widening
    return a


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
    REASONS = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")

    def __init__(self, gpu_index: int):
        self.tmp = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.proc = None
        self.samples = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={gpu_index}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "20"], stdout=self.tmp, stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def stop(self) -> None:
        self.samples = []
        if self.proc is None:
            return
        time.sleep(0.1)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        self.tmp.flush()
        self.tmp.seek(0)
        for line in self.tmp.read().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 10:
                continue
            try:
                ts = datetime.datetime.strptime(f[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                clk, cmax, watts = float(f[2]), float(f[3]), float(f[4])
            except ValueError:
                continue
            active = [name for name, val in zip(self.REASONS, f[6:10]) if val.lower().startswith("active")]
            self.samples.append((ts, clk, cmax, watts, active))
        os.unlink(self.tmp.name)

    def stats(self, windows, pad: float = 0.02) -> dict:
        """Median SM clock and the throttle reasons seen inside the given wall-clock windows."""
        if self.samples is None:
            raise RuntimeError("stop() the sampler before reading it")
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"], "samples": 0}
        inside = [s for s in self.samples if any(a - pad <= s[0] <= b + pad for a, b in windows)]
        # a region shorter than the sampling period may hold no sample: take the nearest one
        if not inside and windows and self.samples:
            mid = 0.5 * (windows[0][0] + windows[-1][1])
            inside = [min(self.samples, key=lambda s: abs(s[0] - mid))]
        reasons = sorted({r for s in inside for r in s[4]})
        return {"sm_mhz": statistics.median(s[1] for s in inside) if inside else None,
                "sm_max_mhz": max((s[2] for s in self.samples), default=None),
                "power_w": statistics.median(s[3] for s in inside) if inside else None,
                "reasons": reasons, "samples": len(inside)}


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


def median_index(values):
    """Index of the median element (the lower one of the two middle elements for an even count)."""
    order = sorted(range(len(values)), key=lambda i: values[i])
    return order[(len(values) - 1) // 2]


class Bench:
    """One workload's cache on the GPU and the timed regions run against it."""

    def __init__(self, w, args, dist, world, dev, peaks, props, steps, warmup, repeats, max_nq):
        import torch
        from paper_2501_12689_b200 import ICCache, workloads as wl
        self.torch, self.wl = torch, wl
        self.w, self.args, self.dist, self.world, self.dev = w, args, dist, world, dev
        self.peaks, self.props = peaks, props
        self.steps, self.warmup, self.repeats = steps, warmup, repeats
        self.path = {"auto": 0, "generic": 1, "scan": 2, "umma": 3}[args.path]
        per_step = max(max_nq, w.insert_rows)
        self.capacity = w.n + (max(steps, warmup) + 2) * per_step
        self.cache = ICCache(w.dim, self.capacity, input_dtype=wl.torch_dtype(w))
        self.cache.set_path(self.path)
        x = wl.cache_rows(w, dev)
        self.cache.insert(x, wl.labels(w.n, dev))
        del x
        torch.cuda.synchronize()
        self.n0 = self.cache.size
        self.n_batches = 8
        self.round = 0           # distinct insert batches per region of a streaming-insert workload

    def close(self):
        self.cache.close()
        self.torch.cuda.empty_cache()

    def reset(self):
        """Drop the rows the last region appended (untimed), so that every region scans the same cache."""
        grown = self.cache.size - self.n0
        if grown > 0:
            self.cache.remove(self.wl.labels(grown, "cpu", first_slot=self.n0))
            assert self.cache.size == self.n0
        self.cache.sync()

    def region(self, batches, q, n_steps, out_ids, out_scores, profiled=False):
        """n_steps steps of [insert; query batch] timed with CUDA events on the stream the library
        launches on (the current torch stream).  The inserted rows are the previous query batch (a
        served request is registered afterwards) or, for a workload with streaming inserts, that
        step's own batch of new rows."""
        torch, wl, w, cache = self.torch, self.wl, self.w, self.cache
        ins = w.insert_rows or q
        all_ids = wl.labels(n_steps * ins, self.dev, first_slot=cache.size)   # labels follow slots
        if w.insert_rows:
            ins_batches = [wl.insert_batch(w, self.round * 64 + j, self.dev) for j in range(n_steps)]
            self.round += 1
        launches0 = cache.launch_count
        cache.set_profiling(profiled)
        if profiled:
            cache.read_profile()
        start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        marks = []
        nb = len(batches)
        barrier(self.dist)
        w0 = time.time()
        start.record()
        for i in range(n_steps):
            rows = ins_batches[i] if w.insert_rows else batches[(i - 1) % nb]
            ids = all_ids[i * ins:(i + 1) * ins]
            if profiled:
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                cache.insert(rows, ids)
                e1.record()
                marks.append((e0, e1))
            else:
                cache.insert(rows, ids)
            cache.query(batches[i % nb], w.k, out_ids, out_scores)
        stop.record()
        torch.cuda.synchronize()
        w1 = time.time()
        barrier(self.dist)
        prof = cache.read_profile() if profiled else None
        if prof is not None:
            prof["insert_ms"] = sum(a.elapsed_time(b) for a, b in marks)
        cache.set_profiling(False)
        out = {"ms": start.elapsed_time(stop), "window": (w0, w1), "launches": cache.launch_count - launches0,
               "profile": prof, "rows_scanned": n_steps * self.n0 + ins * n_steps * (n_steps + 1) // 2}
        self.reset()
        return out

    def measure(self, q, repeats=None, steps=None, warmup=None, forced_path=None):
        """`repeats` timed regions plus one with the library's per-kernel event brackets."""
        torch, wl, w = self.torch, self.wl, self.w
        steps = steps or self.steps
        warmup = warmup or self.warmup
        repeats = repeats or self.repeats
        if forced_path is not None:
            self.cache.set_path(forced_path)
        batches = [wl.queries(w, q, self.dev, round_idx=r) for r in range(self.n_batches)]
        out_ids = torch.empty(q, w.k, dtype=torch.int64, device=self.dev)
        out_scores = torch.empty(q, w.k, dtype=torch.float32, device=self.dev)
        self.region(batches, q, warmup, out_ids, out_scores)
        regions = [self.region(batches, q, steps, out_ids, out_scores) for _ in range(repeats)]
        prof = self.region(batches, q, steps, out_ids, out_scores, profiled=True)
        if forced_path is not None:
            self.cache.set_path(self.path)
        return {"nq": q, "steps": steps, "warmup": warmup, "regions": regions, "profiled": prof,
                "path": self.path if forced_path is None else forced_path}

    def e2e(self, q):
        """The same step through the host-buffer entry points: pinned host inputs and outputs, the
        copies inside the timed region (wall clock around a synchronising call sequence)."""
        torch, wl, w, cache = self.torch, self.wl, self.w, self.cache
        steps, warmup = self.steps, self.warmup
        hb = [wl.queries(w, q, self.dev, round_idx=r).cpu().pin_memory() for r in range(self.n_batches)]
        ins = w.insert_rows or q
        h_ins = [wl.insert_batch(w, 10_000 + r, self.dev).cpu().pin_memory() for r in range(4)] if w.insert_rows else None
        ho_ids = torch.empty(q, w.k, dtype=torch.int64).pin_memory()
        ho_sc = torch.empty(q, w.k, dtype=torch.float32).pin_memory()

        def run(n_steps):
            h_ids = wl.labels(n_steps * ins, "cpu", first_slot=cache.size).pin_memory()
            barrier(self.dist)
            w0 = time.time()
            t0 = time.perf_counter()
            for i in range(n_steps):
                rows = h_ins[i % 4] if h_ins is not None else hb[(i - 1) % self.n_batches]
                cache.insert_host(rows, h_ids[i * ins:(i + 1) * ins])
                cache.query_host(hb[i % self.n_batches], w.k, ho_ids, ho_sc)
            torch.cuda.synchronize()
            ms = (time.perf_counter() - t0) * 1e3
            w1 = time.time()
            barrier(self.dist)
            self.reset()
            return ms, (w0, w1)

        run(warmup)
        runs = [run(steps) for _ in range(min(self.repeats, 5))]
        elem = 2 if w.input_dtype == "bf16" else 4
        return {"runs": runs, "steps": steps,
                "h2d": q * w.dim * elem + ins * w.dim * elem + ins * 8,   # query batch + inserted rows + their ids
                "d2h": q * w.k * 12}

    # ---- derived figures
    def roofline(self, m):
        """Roofline of the dominant kernel: the main scoring launch (fused score + partial top-k;
        on the tensor-core path the launch that reads every row outside the seeding sample).
        Algorithmic bytes per launch = 2*dim per row it scans, flops = 2*dim per (query, row);
        the bound is whichever takes longer at the measured peaks."""
        from paper_2501_12689_b200 import ic_cache_plan
        w, peaks = self.w, self.peaks
        r = m["profiled"]
        pr = r["profile"]
        if not pr or pr["scoring_launches"] == 0:
            return None
        steps = m["steps"]
        rows = r["rows_scanned"] / steps                     # mean cache rows per step
        pl = ic_cache_plan(w.dim, int(rows), m["nq"], w.k, m["path"], self.props.multi_processor_count,
                           self.props.shared_memory_per_block_optin)
        rows_main = rows - min(rows, pl["seed_tiles"] * 256)       # rows the dominant launch reads
        bytes_per_launch = rows_main * w.dim * 2
        flops_per_launch = bytes_per_launch * m["nq"]
        t_launch = pr["scoring_ms"] * 1e-3 / pr["scoring_launches"]
        t_hbm = bytes_per_launch / (peaks["hbm_gbs"] * 1e9)
        t_tensor = flops_per_launch / (peaks["bf16_tflops_sustained"] * 1e12)
        if t_hbm >= t_tensor:
            ach = bytes_per_launch / t_launch / 1e9
            out = {"bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                   "frac": ach / peaks["hbm_gbs"], "frac_of_nominal": ach / NOMINAL_HBM_GBS}
        else:
            ach = flops_per_launch / t_launch / 1e12
            out = {"bound": "tensor", "achieved": ach, "peak": peaks["bf16_tflops_sustained"], "unit": "TFLOP/s",
                   "frac": ach / peaks["bf16_tflops_sustained"], "frac_of_nominal": ach / NOMINAL_BF16_TFLOPS,
                   "frac_of_burst_peak": ach / peaks["bf16_tflops"]}
        variant = "<1,resident>" if pl["query_resident"] else f"<{pl['cta_group']},streamed>"
        kernel = {2: "scan_score_topk_kernel", 3: f"umma_score_topk_kernel{variant} (main pass)",
                  1: "generic_score_topk_kernel"}[pl["path"]]
        per_row = NCU_TRAFFIC_BYTES_PER_ROW.get((kernel, w.dim))
        out.update({"traffic": per_row * rows_main if per_row else None,
                    "traffic_source": ("ncu capture on a scaled-down cache, bytes per scanned row x rows of this launch"
                                       if per_row else "no ncu capture of this kernel build"),
                    "peak_source": peaks["source"] + (" (sustained bf16 figure)" if out["bound"] == "tensor" else " (copy)"),
                    "kernel": kernel, "kernel_us_per_launch": t_launch * 1e6,
                    "launches_per_step": pr["scoring_launches"] / steps,
                    "algorithmic_bytes_per_launch": bytes_per_launch, "rows_per_launch": rows_main,
                    "insert_us_per_step": pr["insert_ms"] * 1e3 / steps,
                    "seed_passes_us_per_step": pr["seed_ms"] * 1e3 / steps,
                    "final_merge_us_per_step": pr["merge_ms"] * 1e3 / steps})
        return out

    def whole_step(self, m, ms_per_step):
        """Roofline fraction of the whole step: every launch of the step (insert, seeding, main pass,
        merges) counts as time, the work is one read of all rows / all (query, row) products."""
        w, peaks = self.w, self.peaks
        rows = m["regions"][0]["rows_scanned"] / m["steps"]
        t_hbm = rows * w.dim * 2 / (peaks["hbm_gbs"] * 1e9)
        t_tensor = rows * w.dim * 2 * m["nq"] / (peaks["bf16_tflops_sustained"] * 1e12)
        t_hbm_nom = rows * w.dim * 2 / (NOMINAL_HBM_GBS * 1e9)
        t_tensor_nom = rows * w.dim * 2 * m["nq"] / (NOMINAL_BF16_TFLOPS * 1e12)
        return {"bound": "hbm" if t_hbm >= t_tensor else "tensor",
                "frac": max(t_hbm, t_tensor) / (ms_per_step * 1e-3),
                "frac_of_nominal": max(t_hbm_nom, t_tensor_nom) / (ms_per_step * 1e-3)}

    def entry(self, m, sampler, compact=False):
        """Median and best region of a measurement, with the clocks sampled during each region."""
        steps, q = m["steps"], m["nq"]
        ms = [r["ms"] for r in m["regions"]]
        mi = median_index(ms)
        med, best = ms[mi], min(ms)
        rows = m["regions"][0]["rows_scanned"] / steps
        out = {"nq": q, "queries_per_sec": q * steps / (med * 1e-3) * self.world,
               "queries_per_sec_best": q * steps / (best * 1e-3) * self.world,
               "ms_per_step": med / steps, "ms_per_step_best": best / steps,
               "cache_entries_per_sec": rows * q * self.world / (med / steps * 1e-3),
               "slab_gb_per_sec_whole_step": rows * self.w.dim * 2 / (med / steps * 1e-3) / 1e9,
               "repeats": len(ms), "steps": steps,
               "whole_step": self.whole_step(m, med / steps), "roofline": self.roofline(m),
               "gpu_launches": m["regions"][mi]["launches"]}
        if sampler is not None:
            out["clocks"] = sampler.stats([r["window"] for r in m["regions"]])
            if not compact:
                per = [sampler.stats([r["window"]]) for r in m["regions"]]
                out["regions"] = [{"ms_per_step": r["ms"] / steps, "sm_mhz": c["sm_mhz"], "reasons": c["reasons"]}
                                  for r, c in zip(m["regions"], per)]
        return out


def run_widening_two_level(b, nprobe):
    """Two-level search (K-Means index, K = sqrt(N)) on the current cache: build time, time per call
    and recall against the exhaustive result, for the workload's batch size and two smaller ones."""
    torch, wl, w, cache = b.torch, b.wl, b.w, b.cache
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    cache.build_index(0, 5)
    cache.sync()
    build_s = time.perf_counter() - t0
    k_clusters, n_indexed = cache.index_info()
    calls = []
    for q in sorted({1, 16, max(w.q_sweep)}):
        qb = wl.queries(w, q, b.dev, round_idx=99)
        exact_ids, _ = cache.query(qb, w.k)
        times = {}
        for name, fn in (("two_level", lambda: cache.query_clustered(qb, w.k, nprobe)),
                         ("exhaustive", lambda: cache.query(qb, w.k))):
            for _ in range(3):
                got = fn()
            ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            reps = 50
            ev0.record()
            for _ in range(reps):
                got = fn()
            ev1.record()
            torch.cuda.synchronize()
            times[name] = ev0.elapsed_time(ev1) / reps
            if name == "two_level":
                got_ids = got[0]
        e, g = exact_ids.cpu().numpy(), got_ids.cpu().numpy()
        recall = sum(len(set(e[i]) & set(g[i])) for i in range(q)) / float(q * w.k)
        # rows a two-level query has to read: the centroids and its probed clusters (average size)
        rows_touched = k_clusters + nprobe * n_indexed / max(1, k_clusters)
        calls.append({"nq": q, "ms_per_call": times["two_level"], "queries_per_sec": q / (times["two_level"] * 1e-3),
                      "exhaustive_ms_per_call": times["exhaustive"], "recall_at_k": recall,
                      "rows_touched_per_query": rows_touched})
    return {"workload": w.name, "n_clusters": k_clusters, "n_indexed": n_indexed, "nprobe": nprobe,
            "build_s": build_s, "kmeans_iters": 5, "calls": calls}


def run_widening_self_similarity(b, rows):
    """All-pairs top-1 self-similarity of the first `rows` cached rows against the whole cache: a
    purely tensor-bound use of the same kernels (2 * rows * N * dim flops)."""
    torch, w, cache, peaks = b.torch, b.w, b.cache, b.peaks
    rows = min(rows, cache.size)
    cache.self_similarity(0, min(rows, 2048))            # warm-up (grows scratch)
    cache.sync()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    n_now = cache.size
    ev0.record()
    cache.self_similarity(0, rows)
    ev1.record()
    torch.cuda.synchronize()
    ms = ev0.elapsed_time(ev1)
    tflops = 2.0 * rows * n_now * w.dim / (ms * 1e-3) / 1e12
    return {"workload": w.name, "rows": rows, "cache_rows": n_now, "ms": ms, "rows_per_sec": rows / (ms * 1e-3),
            "roofline": {"bound": "tensor", "achieved": tflops, "peak": peaks["bf16_tflops_sustained"], "unit": "TFLOP/s",
                         "frac": tflops / peaks["bf16_tflops_sustained"], "frac_of_nominal": tflops / NOMINAL_BF16_TFLOPS,
                         "peak_source": peaks["source"] + " (sustained bf16 figure)", "what": "whole call"}}


def run_ours(args):
    import torch
    from paper_2501_12689_b200 import ic_cache_plan, workloads as wl
    from paper_2501_12689_b200 import binding

    dist, rank, world, local = dist_setup(args.gpus)
    dev = torch.device("cuda", local)
    w = wl.WORKLOADS[args.workload]
    if args.rows:
        w = w.scaled(args.rows)
    nq = args.nq or max(w.q_sweep)
    steps = args.steps if args.steps is not None else 20
    warmup = max(args.warmup if args.warmup is not None else 3, 3)
    repeats = max(1, args.repeats if args.repeats is not None else 20)
    peaks = load_peaks()
    props = torch.cuda.get_device_properties(dev)
    sampler = ClockSampler(local) if rank == 0 else None
    mk = lambda wk, max_nq: Bench(wk, args, dist, world, dev, peaks, props, steps, warmup, repeats, max_nq)

    others, two_level, self_sim = [], None, None
    # ---- the other configurations, compactly, and the two widening workloads (before the 16 M-row entries)
    if not args.no_configs or not args.no_widening:
        for name in ("online", "clustered", "dense"):
            if name == w.name:
                continue
            need_cfg = not args.no_configs
            need_wide = not args.no_widening and name in ("online", "clustered")
            if not (need_cfg or need_wide):
                continue
            wk = wl.WORKLOADS[name]
            bk = mk(wk, max(wk.q_sweep))
            if need_cfg:
                others.append((wk, bk, bk.measure(max(wk.q_sweep))))
            if need_wide and name == "clustered":
                two_level = run_widening_two_level(bk, args.two_level_nprobe)
            if need_wide and name == "online":
                self_sim = run_widening_self_similarity(bk, args.self_similarity_rows)
            bk.close()

    # ---- the headline workload
    b = mk(w, max(max(w.q_sweep), nq, 512))
    main = b.measure(nq)
    e2e_raw = None if args.no_e2e else b.e2e(nq)
    sweep = []
    if not args.no_sweep:
        sweep = [b.measure(q) for q in w.q_sweep if q != nq]
    crossover = []
    if not args.no_crossover and args.path == "auto":
        # forced paths over the batch size: where the CUDA-core scan stops keeping up with HBM and
        # where the tensor-core path turns from HBM-bound to tensor-bound (few short regions each)
        cross_plan = [("scan", 2, q) for q in (1, 2, 4) if w.dim <= 1024] + \
                     [("umma", 3, q) for q in (1, 2, 4, 8, 16, 32, 64, 128, 256, 512)]
        for name, code, q in cross_plan:
            crossover.append((name, b.measure(q, repeats=3, steps=min(steps, 5), warmup=3, forced_path=code)))
    plan = ic_cache_plan(w.dim, w.n, nq, w.k, b.path, props.multi_processor_count, props.shared_memory_per_block_optin)
    n_start = b.n0
    if not args.no_widening and w.name == "clustered":
        two_level = run_widening_two_level(b, args.two_level_nprobe)
    if not args.no_widening and w.name == "online":
        self_sim = run_widening_self_similarity(b, args.self_similarity_rows)
    b.close()

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
            torch.cuda.empty_cache()
        except RuntimeError:
            read_stream = None

    if sampler:
        sampler.stop()

    # ---- whole-job figures: per region the maximum over ranks, work summed over ranks
    ms_regions = [aggregate_ranks(dist, r["ms"], float(nq * steps))[0] for r in main["regions"]]
    for r, ms in zip(main["regions"], ms_regions):
        r["ms"] = ms
    e2e = None
    if e2e_raw is not None:
        e_ms = [aggregate_ranks(dist, ms, float(nq * steps))[0] for ms, _ in e2e_raw["runs"]]
        mi = median_index(e_ms)
        e2e = {"value": nq * steps * world / (e_ms[mi] * 1e-3), "unit": UNIT, "h2d_bytes_per_step": e2e_raw["h2d"],
               "d2h_bytes_per_step": e2e_raw["d2h"], "steps": steps, "ms_per_step": e_ms[mi] / steps,
               "best_value": nq * steps * world / (min(e_ms) * 1e-3), "repeats": len(e_ms)}
    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    head = b.entry(main, sampler)
    roof = head.pop("roofline") or {"bound": "hbm", "achieved": None, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                                    "frac": None, "traffic": None}
    if roof.get("bound") == "hbm" and read_stream and roof.get("achieved"):
        roof["frac_of_read_stream"] = roof["achieved"] / read_stream
    clocks = sampler.stats([r["window"] for r in main["regions"]]) if sampler else None
    line = {
        "metric": METRIC, "value": head["queries_per_sec"], "unit": UNIT, "n_gpus": world, "steps": steps, "warmup": warmup,
        "ms_per_step": head["ms_per_step"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": f"{w.name}: N={w.n} d={w.dim} {w.input_dtype} unit {w.kind}, nq={nq}, k={w.k}",
                   "step": (f"insert {w.insert_rows} new rows + query batch (prep, score, partial top-k, merge)" if w.insert_rows
                            else "insert previous batch (nq rows) + query batch (prep, score, partial top-k, merge)"),
                   "n_start": n_start, "path": binding.PATH_NAMES[plan["path"]], "plan": plan,
                   "l2": "slab is many times larger than L2 (126 MB): no flush between steps",
                   "timing": f"value = median of {len(ms_regions)} regions of {steps} steps; the rows a region appends "
                             "are removed again (untimed) before the next one",
                   "replicas": world},
        "repeats": len(ms_regions), "value_best": head["queries_per_sec_best"], "ms_per_step_best": head["ms_per_step_best"],
        "regions": head.get("regions"),
        "cache_entries_per_sec": head["cache_entries_per_sec"],
        "slab_gb_per_sec_whole_step": head["slab_gb_per_sec_whole_step"],
        "read_stream_gb_per_sec": read_stream,
        "gpu_launches": head["gpu_launches"],
        "e2e": e2e,
        "roofline": roof,
        "whole_step": head["whole_step"],
        "clocks": clocks,
        "sweep": [b.entry(m, sampler, compact=True) for m in sweep],
        "crossover": [{"path": name, **{k: v for k, v in b.entry(m, sampler, compact=True).items()
                                        if k in ("nq", "ms_per_step", "ms_per_step_best", "queries_per_sec", "whole_step")},
                       "main_pass_us": (m["profiled"]["profile"]["scoring_ms"] * 1e3 / max(1, m["profiled"]["profile"]["scoring_launches"])),
                       "scoring_launches_per_step": m["profiled"]["profile"]["scoring_launches"] / m["steps"]}
                      for name, m in crossover],
        "configs": [{"workload": f"{wk.name}: N={wk.n} d={wk.dim}, k={wk.k}", **bk.entry(m, sampler, compact=True)}
                    for wk, bk, m in others],
        "two_level": two_level,
        "self_similarity": self_sim,
    }
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
    batches = [wl.as_bits(wl.queries(w, nq, "cpu", round_idx=r)) for r in range(4)]
    # size the per-step sample so that the whole run stays within about two minutes: first the cost
    # of one query per row on 100,000 rows of the same recipe, then either a few queries per step
    # against all rows or one query against as many rows as the budget allows
    n_probe = min(w.n, 100_000)
    probe_bits = wl.as_bits(wl.cache_rows(w.scaled(n_probe), dev))
    per_query = oracle_seconds(w, n_probe, 1, probe_bits, batches[0], threads) * w.n / n_probe
    budget = 120.0 / max(1, steps + warmup)
    n_rows = w.n
    q_per_step = int(min(nq, budget / per_query))
    if q_per_step < 1:
        q_per_step = 1
        n_rows = int(max(min(w.n, 10_000), min(w.n, w.n * budget / per_query)))
    x_bits = probe_bits if n_rows <= n_probe else wl.as_bits(wl.cache_rows(w.scaled(n_rows), dev))
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
