"""ctypes front-end of the CPU oracle (oracle/ic_oracle.c).  Test infrastructure only.

The arithmetic lives in the C file; this module only compiles it with gcc,
marshals numpy arrays and returns numpy arrays.  bf16 data travels as uint16
bit patterns.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ic_oracle.c")
_LIB = os.path.join(_HERE, "libic_oracle.so")
_lock = threading.Lock()
_lib = None

BF16 = 0
F32 = 1


def build_oracle(force: bool = False) -> str:
    """Compile the C oracle into oracle/libic_oracle.so (if stale) and return its path."""
    with _lock:
        stale = (
            force
            or not os.path.exists(_LIB)
            or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
        )
        if stale:
            tmp = _LIB + ".tmp.%d" % os.getpid()
            cmd = [
                "gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp",
                "-ffp-contract=off", "-fno-fast-math", "-Wall", "-Wextra",
                "-o", tmp, _SRC, "-lm",
            ]
            subprocess.run(cmd, check=True)
            os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build_oracle())
        lib.ic_oracle_bf16_to_f32.restype = ctypes.c_float
        lib.ic_oracle_bf16_to_f32.argtypes = [ctypes.c_uint16]
        lib.ic_oracle_f32_to_bf16.restype = ctypes.c_uint16
        lib.ic_oracle_f32_to_bf16.argtypes = [ctypes.c_float]
        lib.ic_oracle_search.restype = ctypes.c_int
        lib.ic_oracle_search.argtypes = [
            ctypes.c_void_p, ctypes.c_int, ctypes.c_void_p, ctypes.c_int64, ctypes.c_int32,
            ctypes.c_void_p, ctypes.c_int, ctypes.c_int32, ctypes.c_int32, ctypes.c_int,
            ctypes.c_int, ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
            ctypes.c_void_p,
        ]
        lib.ic_oracle_apply_min_score.restype = None
        lib.ic_oracle_apply_min_score.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int32,
                                                  ctypes.c_int32, ctypes.c_float, ctypes.c_void_p]
        lib.ic_oracle_self_similarity.restype = ctypes.c_int
        lib.ic_oracle_self_similarity.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_void_p, ctypes.c_int64,
                                                  ctypes.c_int32, ctypes.c_int64, ctypes.c_int64, ctypes.c_int,
                                                  ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]
        lib.ic_oracle_kmeans_assign.restype = ctypes.c_int
        lib.ic_oracle_kmeans_assign.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, ctypes.c_int32,
                                                ctypes.c_void_p, ctypes.c_int32, ctypes.c_int, ctypes.c_void_p,
                                                ctypes.c_void_p]
        lib.ic_oracle_kmeans_update.restype = ctypes.c_int
        lib.ic_oracle_kmeans_update.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, ctypes.c_int32,
                                                ctypes.c_void_p, ctypes.c_int32, ctypes.c_void_p, ctypes.c_void_p,
                                                ctypes.c_void_p, ctypes.c_void_p]
        lib.ic_oracle_search_clustered.restype = ctypes.c_int
        lib.ic_oracle_search_clustered.argtypes = [
            ctypes.c_void_p, ctypes.c_int, ctypes.c_void_p, ctypes.c_int64, ctypes.c_int32, ctypes.c_void_p,
            ctypes.c_int, ctypes.c_int32, ctypes.c_int32, ctypes.c_void_p, ctypes.c_int32, ctypes.c_void_p,
            ctypes.c_int64, ctypes.c_int32, ctypes.c_void_p, ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p,
            ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]
        _lib = lib
    return _lib


def bf16_bits_to_f32(bits) -> np.ndarray:
    """Widen bf16 bit patterns (uint16) to fp32, element by element, through the C helper."""
    lib = _load()
    b = np.asarray(bits, dtype=np.uint16)
    out = np.empty(b.shape, dtype=np.float32)
    flat_in, flat_out = b.reshape(-1), out.reshape(-1)
    for i in range(flat_in.size):
        flat_out[i] = lib.ic_oracle_bf16_to_f32(int(flat_in[i]))
    return out


def f32_to_bf16_bits(x) -> np.ndarray:
    """Round fp32 values to bf16 (nearest, ties to even) through the C helper; returns uint16."""
    lib = _load()
    a = np.asarray(x, dtype=np.float32)
    out = np.empty(a.shape, dtype=np.uint16)
    flat_in, flat_out = a.reshape(-1), out.reshape(-1)
    for i in range(flat_in.size):
        flat_out[i] = lib.ic_oracle_f32_to_bf16(float(flat_in[i]))
    return out


def _as_matrix(a, what: str):
    a = np.ascontiguousarray(a)
    if a.dtype == np.uint16:
        return a, BF16
    if a.dtype == np.float32:
        return a, F32
    raise TypeError(f"{what}: expected float32 values or uint16 bf16 bit patterns, got {a.dtype}")


def default_threads() -> int:
    try:
        return max(1, len(os.sched_getaffinity(0)))
    except AttributeError:  # pragma: no cover
        return max(1, os.cpu_count() or 1)


def search(x, q, k: int, ids=None, normalize: bool = False, round_bf16: bool = False,
           threads: int | None = None, want_all_scores: bool = False, min_score: float | None = None):
    """Exhaustive cosine/inner-product top-k of every query row against every cache row.

    x: [n, d] float32, or uint16 holding bf16 bits.  q: [nq, d] likewise.
    ids: optional int64 [n] labels (default: the slot number).
    round_bf16: round float32 inputs to bf16 first (what a bf16 store keeps).
    min_score: if given, entries scoring below it are reported as absent and the result also
    carries counts [nq] int32 (entries kept per query).
    Returns dict(ids [nq,k] int64, scores [nq,k] float32, slots [nq,k] int64,
    all_scores [nq,n] float32 or None).  Rows past min(k, n) are (-1, -inf, -1).
    """
    lib = _load()
    x, xdt = _as_matrix(x, "x")
    q, qdt = _as_matrix(q, "q")
    if x.ndim != 2 or q.ndim != 2:
        raise ValueError("x and q must be 2-D")
    n, d = x.shape
    nq = q.shape[0]
    if nq and n and q.shape[1] != d:
        raise ValueError("dimension mismatch")
    if n == 0:
        d = q.shape[1]
    if ids is not None:
        ids = np.ascontiguousarray(ids, dtype=np.int64)
        if ids.shape != (n,):
            raise ValueError("ids must have shape [n]")
    out_ids = np.empty((nq, k), dtype=np.int64)
    out_scores = np.empty((nq, k), dtype=np.float32)
    out_slots = np.empty((nq, k), dtype=np.int64)
    all_scores = np.empty((nq, n), dtype=np.float32) if want_all_scores else None
    rc = lib.ic_oracle_search(
        x.ctypes.data, xdt, ids.ctypes.data if ids is not None else None, n, d,
        q.ctypes.data, qdt, nq, k, int(bool(normalize)), int(bool(round_bf16)),
        int(threads or default_threads()),
        out_ids.ctypes.data, out_scores.ctypes.data, out_slots.ctypes.data,
        all_scores.ctypes.data if all_scores is not None else None,
    )
    if rc != 0:
        raise RuntimeError(f"ic_oracle_search failed with code {rc}")
    res = {"ids": out_ids, "scores": out_scores, "slots": out_slots, "all_scores": all_scores}
    if min_score is not None:
        counts = np.empty((nq,), dtype=np.int32)
        lib.ic_oracle_apply_min_score(out_ids.ctypes.data, out_scores.ctypes.data, out_slots.ctypes.data, nq, k,
                                      float(min_score), counts.ctypes.data)
        res["counts"] = counts
    return res


def self_similarity(x, first: int = 0, count: int | None = None, ids=None, threads: int | None = None):
    """For rows first .. first+count-1 of x: the most similar OTHER row (fp32 dot product, ties to
    the lower slot).  Returns dict(ids, scores, slots), each of length count."""
    lib = _load()
    x, xdt = _as_matrix(x, "x")
    n, d = x.shape
    count = n - first if count is None else count
    if ids is not None:
        ids = np.ascontiguousarray(ids, dtype=np.int64)
    out_ids = np.empty((count,), dtype=np.int64)
    out_scores = np.empty((count,), dtype=np.float32)
    out_slots = np.empty((count,), dtype=np.int64)
    rc = lib.ic_oracle_self_similarity(x.ctypes.data, xdt, ids.ctypes.data if ids is not None else None, n, d,
                                       first, count, int(threads or default_threads()), out_ids.ctypes.data,
                                       out_scores.ctypes.data, out_slots.ctypes.data)
    if rc != 0:
        raise RuntimeError(f"ic_oracle_self_similarity failed with code {rc}")
    return {"ids": out_ids, "scores": out_scores, "slots": out_slots}


def kmeans_assign(x, centroids, threads: int | None = None):
    """Assignment step of K-Means under the cosine metric: for every row of x the centroid (bf16
    bits, [K,d] uint16) with the largest fp32 dot product, ties to the lower index.
    Returns (assign int32 [n], best float32 [n])."""
    lib = _load()
    x, xdt = _as_matrix(x, "x")
    c = np.ascontiguousarray(centroids, dtype=np.uint16)
    n, d = x.shape
    assign = np.empty((n,), dtype=np.int32)
    best = np.empty((n,), dtype=np.float32)
    rc = lib.ic_oracle_kmeans_assign(x.ctypes.data, xdt, n, d, c.ctypes.data, c.shape[0],
                                     int(threads or default_threads()), assign.ctypes.data, best.ctypes.data)
    if rc != 0:
        raise RuntimeError(f"ic_oracle_kmeans_assign failed with code {rc}")
    return assign, best


def kmeans_update(x, assign, centroids_prev):
    """Update step: every centroid becomes the unit-length mean of its rows (fp64 sums in slot order),
    rounded to bf16; a centroid without rows keeps its previous value.
    Returns (centroids uint16 [K,d], exact float64 [K,d], counts int64 [K])."""
    lib = _load()
    x, xdt = _as_matrix(x, "x")
    prev = np.ascontiguousarray(centroids_prev, dtype=np.uint16)
    a = np.ascontiguousarray(assign, dtype=np.int32)
    n, d = x.shape
    k_clusters = prev.shape[0]
    out = np.empty_like(prev)
    exact = np.empty((k_clusters, d), dtype=np.float64)
    counts = np.empty((k_clusters,), dtype=np.int64)
    rc = lib.ic_oracle_kmeans_update(x.ctypes.data, xdt, n, d, a.ctypes.data, k_clusters, prev.ctypes.data,
                                     out.ctypes.data, exact.ctypes.data, counts.ctypes.data)
    if rc != 0:
        raise RuntimeError(f"ic_oracle_kmeans_update failed with code {rc}")
    return out, exact, counts


def kmeans(x_bits, init_slots, n_iters: int, threads: int | None = None):
    """Lloyd iteration from the rows at init_slots: n_iters times (assign, update), then one last
    assignment to the final centroids.  x_bits: bf16 bits [n,d] (what the cache stores).
    Returns dict(centroids uint16 [K,d], assign int32 [n], best float32 [n])."""
    x_bits = np.ascontiguousarray(x_bits, dtype=np.uint16)
    cent = x_bits[np.asarray(init_slots, dtype=np.int64)].copy()
    for _ in range(n_iters):
        assign, _best = kmeans_assign(x_bits, cent, threads)
        cent, _exact, _counts = kmeans_update(x_bits, assign, cent)
    assign, best = kmeans_assign(x_bits, cent, threads)
    return {"centroids": cent, "assign": assign, "best": best}


def search_clustered(x, q, k: int, centroids, assign, nprobe: int, n_indexed: int | None = None, ids=None,
                     probes=None, threads: int | None = None, want_all_scores: bool = False):
    """Two-level retrieval: probe the nprobe closest centroids, search their rows and every row
    past n_indexed exhaustively.  probes: optional int64 [nq,nprobe] centroid indices to use
    instead of the centroid step.  Returns dict(ids, scores, slots [nq,k], probes [nq,nprobe],
    centroid_scores [nq,K], all_scores [nq,n] with -inf for rows not searched, or None)."""
    lib = _load()
    x, xdt = _as_matrix(x, "x")
    q, qdt = _as_matrix(q, "q")
    c = np.ascontiguousarray(centroids, dtype=np.uint16)
    n, d = x.shape
    nq = q.shape[0]
    n_indexed = n if n_indexed is None else int(n_indexed)
    a = np.ascontiguousarray(assign, dtype=np.int32)
    if a.shape[0] < n_indexed:
        raise ValueError("assign must cover the indexed rows")
    if ids is not None:
        ids = np.ascontiguousarray(ids, dtype=np.int64)
    if probes is not None:
        probes = np.ascontiguousarray(probes, dtype=np.int64)
        if probes.shape != (nq, nprobe):
            raise ValueError("probes must have shape [nq, nprobe]")
    out_ids = np.empty((nq, k), dtype=np.int64)
    out_scores = np.empty((nq, k), dtype=np.float32)
    out_slots = np.empty((nq, k), dtype=np.int64)
    out_probes = np.empty((nq, nprobe), dtype=np.int64)
    cscores = np.empty((nq, c.shape[0]), dtype=np.float32)
    all_scores = np.empty((nq, n), dtype=np.float32) if want_all_scores else None
    rc = lib.ic_oracle_search_clustered(
        x.ctypes.data, xdt, ids.ctypes.data if ids is not None else None, n, d, q.ctypes.data, qdt, nq, k,
        c.ctypes.data, c.shape[0], a.ctypes.data, n_indexed, nprobe,
        probes.ctypes.data if probes is not None else None, int(threads or default_threads()),
        out_ids.ctypes.data, out_scores.ctypes.data, out_slots.ctypes.data, out_probes.ctypes.data,
        cscores.ctypes.data, all_scores.ctypes.data if all_scores is not None else None)
    if rc != 0:
        raise RuntimeError(f"ic_oracle_search_clustered failed with code {rc}")
    return {"ids": out_ids, "scores": out_scores, "slots": out_slots, "probes": out_probes,
            "centroid_scores": cscores, "all_scores": all_scores}


def utility_add(entry_ids, utility, add_ids, gains):
    """Per-entry utility bookkeeping of the cache manager (paper Sec. 4.3, "Example Manager": an
    example's value is the efficiency gain it enabled, kept as a moving average).  For every pair
    (add_ids[i], gains[i]), in order, the gain is added (one fp32 addition) to the utility of every
    entry carrying that id.  Plain loops; returns a new float32 array."""
    ids = np.asarray(entry_ids, dtype=np.int64)
    out = np.array(utility, dtype=np.float32, copy=True)
    for wanted, gain in zip(np.asarray(add_ids, dtype=np.int64).tolist(), np.asarray(gains, dtype=np.float32)):
        for slot in range(ids.shape[0]):
            if ids[slot] == wanted:
                out[slot] = np.float32(out[slot] + gain)
    return out


def utility_decay(utility, factor):
    """The moving average's decay step (paper Sec. 4.3: a factor of 0.9 every hour): every utility
    is multiplied by the factor, one fp32 multiplication each."""
    f = np.float32(factor)
    return np.array([np.float32(u * f) for u in np.asarray(utility, dtype=np.float32)], dtype=np.float32)
