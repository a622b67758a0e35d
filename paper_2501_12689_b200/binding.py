"""Thin ctypes binding of the C ABI in include/ic_cache.h.

Argument marshalling only: every step of the retrieval path runs in the CUDA library.
The functions carry the names of the C entry points; `ICCache` is a small convenience
wrapper that owns a handle.  torch is used for device memory and streams, nothing else.
If the shared library is missing this module raises at import of the first call; there is
no fallback implementation.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Tuple

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
# IC_CACHE_LIB names another build of the same library (the debug build with index checks,
# libic_cache_debug.so); there is still no fallback if it is missing
LIB_PATH = os.environ.get("IC_CACHE_LIB") or os.path.join(_PKG, "libic_cache.so")

IC_OK, IC_ERR_INVALID, IC_ERR_NOMEM, IC_ERR_FULL = 0, -1, -2, -3
IC_ERR_CUDA, IC_ERR_UNSUPPORTED, IC_ERR_TIMEOUT = -4, -5, -6
IC_BF16, IC_F32 = 0, 1
IC_PATH_AUTO, IC_PATH_GENERIC, IC_PATH_SCAN, IC_PATH_UMMA = 0, 1, 2, 3
IC_MAX_K, IC_MAX_DIM = 128, 4096
IC_STATIC_SCRATCH_BYTES = 8 << 20
PATH_NAMES = {IC_PATH_AUTO: "auto", IC_PATH_GENERIC: "generic", IC_PATH_SCAN: "scan", IC_PATH_UMMA: "umma"}


class ic_cache_opts_t(ctypes.Structure):
    _fields_ = [
        ("struct_size", ctypes.c_uint32),
        ("device", ctypes.c_int32),
        ("input_dtype", ctypes.c_int32),
        ("normalize", ctypes.c_int32),
        ("slab", ctypes.c_void_p),
        ("ids", ctypes.c_void_p),
        ("stream", ctypes.c_void_p),
        ("workspace", ctypes.c_void_p),
        ("workspace_bytes", ctypes.c_size_t),
    ]


class ic_cache_plan_t(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in (
        "path", "query_tile", "n_query_tiles", "n_partitions", "n_ctas", "n_stages", "smem_bytes",
        "n_launches", "queue_cap", "seed_tiles", "seed0_tiles", "cta_group", "query_resident")]

    def as_dict(self):
        return {n: getattr(self, n) for n, _ in self._fields_}


class ICCacheError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"ic_cache status {status}: {message}")
        self.status = status


_lib = None

# name -> (restype, argtypes); also the list the symbol test checks against the header
SIGNATURES = {
    "ic_cache_create": (ctypes.c_void_p, [ctypes.c_int32, ctypes.c_int64]),
    "ic_cache_create_ex": (ctypes.c_void_p, [ctypes.c_int32, ctypes.c_int64, ctypes.POINTER(ic_cache_opts_t)]),
    "ic_cache_insert": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64]),
    "ic_cache_query": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32,
                                      ctypes.c_void_p, ctypes.c_void_p]),
    "ic_cache_workspace_bytes": (ctypes.c_size_t, [ctypes.c_int32, ctypes.c_int64, ctypes.c_int32, ctypes.c_int32]),
    "ic_cache_query_min_score": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32,
                                                ctypes.c_float, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]),
    "ic_cache_query_static": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32,
                                             ctypes.c_void_p, ctypes.c_void_p]),
    "ic_cache_query_host": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32,
                                           ctypes.c_void_p, ctypes.c_void_p]),
    "ic_cache_insert_host": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64]),
    "ic_cache_self_similarity": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_int64, ctypes.c_int64, ctypes.c_void_p,
                                                ctypes.c_void_p]),
    "ic_cache_remove": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64, ctypes.POINTER(ctypes.c_int64)]),
    "ic_cache_save": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_char_p]),
    "ic_cache_load": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_char_p]),
    "ic_cache_utility_add": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64]),
    "ic_cache_utility_decay": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_float]),
    "ic_cache_utility_read": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]),
    "ic_cache_build_index": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32, ctypes.c_void_p]),
    "ic_cache_index_info": (ctypes.c_int, [ctypes.c_void_p, ctypes.POINTER(ctypes.c_int32), ctypes.POINTER(ctypes.c_int64)]),
    "ic_cache_read_index": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]),
    "ic_cache_query_clustered": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32,
                                                ctypes.c_int32, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]),
    "ic_cache_destroy": (None, [ctypes.c_void_p]),
    "ic_cache_set_stream": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_void_p]),
    "ic_cache_set_path": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_int32]),
    "ic_cache_size": (ctypes.c_int64, [ctypes.c_void_p]),
    "ic_cache_clear": (ctypes.c_int, [ctypes.c_void_p]),
    "ic_cache_sync": (ctypes.c_int, [ctypes.c_void_p]),
    "ic_cache_probe_wait_limit": (ctypes.c_int, [ctypes.c_void_p]),
    "ic_cache_launch_count": (ctypes.c_int64, [ctypes.c_void_p]),
    "ic_cache_set_profiling": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_int32]),
    "ic_cache_read_profile": (ctypes.c_int, [ctypes.c_void_p, ctypes.POINTER(ctypes.c_double),
                                             ctypes.POINTER(ctypes.c_int64), ctypes.POINTER(ctypes.c_double),
                                             ctypes.POINTER(ctypes.c_int64), ctypes.POINTER(ctypes.c_double),
                                             ctypes.POINTER(ctypes.c_int64)]),
    "ic_cache_plan": (ctypes.c_int, [ctypes.c_int32, ctypes.c_int64, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32,
                                     ctypes.c_int32, ctypes.c_int32, ctypes.POINTER(ic_cache_plan_t)]),
    "ic_cache_last_error": (ctypes.c_char_p, []),
    "ic_cache_version": (ctypes.c_int32, []),
}


def load_library():
    """dlopen the in-tree CUDA library.  Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2501_12689_b200.build` "
                "(there is no CPU or PyTorch fallback)")
        lib = ctypes.CDLL(LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(lib, name)
            fn.restype = res
            fn.argtypes = args
        _lib = lib
    return _lib


def ic_cache_last_error() -> str:
    return load_library().ic_cache_last_error().decode("utf-8", "replace")


def _check(status: int) -> None:
    if status != IC_OK:
        raise ICCacheError(status, ic_cache_last_error())


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def ic_cache_create(dim: int, capacity: int):
    h = load_library().ic_cache_create(dim, capacity)
    if not h:
        raise ICCacheError(IC_ERR_INVALID, ic_cache_last_error())
    return h


def ic_cache_create_ex(dim: int, capacity: int, *, device: int = -1, input_dtype: int = IC_BF16,
                       normalize: bool = False, slab: Optional[torch.Tensor] = None,
                       ids: Optional[torch.Tensor] = None, stream: int = 0,
                       workspace: Optional[torch.Tensor] = None):
    o = ic_cache_opts_t()
    o.struct_size = ctypes.sizeof(ic_cache_opts_t)
    o.device = device
    o.input_dtype = input_dtype
    o.normalize = int(bool(normalize))
    o.slab = slab.data_ptr() if slab is not None else None
    o.ids = ids.data_ptr() if ids is not None else None
    o.stream = stream or None
    o.workspace = workspace.data_ptr() if workspace is not None else None
    o.workspace_bytes = workspace.numel() * workspace.element_size() if workspace is not None else 0
    h = load_library().ic_cache_create_ex(dim, capacity, ctypes.byref(o))
    if not h:
        raise ICCacheError(IC_ERR_INVALID, ic_cache_last_error())
    return h


def ic_cache_workspace_bytes(dim: int, capacity: int, max_nq: int, max_k: int) -> int:
    return int(load_library().ic_cache_workspace_bytes(dim, capacity, max_nq, max_k))


def ic_cache_insert(h, emb: torch.Tensor, ids: torch.Tensor, n: Optional[int] = None) -> None:
    n = emb.shape[0] if n is None else n
    _check(load_library().ic_cache_insert(h, _ptr(emb), _ptr(ids), n))


def ic_cache_query(h, q: torch.Tensor, nq: int, k: int, out_ids: torch.Tensor, out_scores: torch.Tensor) -> None:
    _check(load_library().ic_cache_query(h, _ptr(q), nq, k, _ptr(out_ids), _ptr(out_scores)))


def ic_cache_query_min_score(h, q: torch.Tensor, nq: int, k: int, min_score: float, out_ids: torch.Tensor,
                             out_scores: torch.Tensor, out_counts: Optional[torch.Tensor]) -> None:
    _check(load_library().ic_cache_query_min_score(h, _ptr(q), nq, k, min_score, _ptr(out_ids), _ptr(out_scores),
                                                   _ptr(out_counts)))


def ic_cache_query_static(h, q: torch.Tensor, nq: int, k: int, out_ids: torch.Tensor, out_scores: torch.Tensor) -> None:
    """ic_cache_query with all scratch in the library's fixed static array: for callers that
    must not allocate device memory at query time.  The caller supplies every buffer."""
    _check(load_library().ic_cache_query_static(h, _ptr(q), nq, k, _ptr(out_ids), _ptr(out_scores)))


def ic_cache_query_host(h, q: torch.Tensor, nq: int, k: int, out_ids: torch.Tensor, out_scores: torch.Tensor) -> None:
    _check(load_library().ic_cache_query_host(h, _ptr(q), nq, k, _ptr(out_ids), _ptr(out_scores)))


def ic_cache_insert_host(h, emb: torch.Tensor, ids: torch.Tensor, n: Optional[int] = None) -> None:
    n = emb.shape[0] if n is None else n
    _check(load_library().ic_cache_insert_host(h, _ptr(emb), _ptr(ids), n))


def ic_cache_destroy(h) -> None:
    load_library().ic_cache_destroy(h)


def ic_cache_plan(dim: int, n: int, nq: int, k: int, path: int = IC_PATH_AUTO, sm_count: int = 148,
                  smem_optin: int = 232448) -> dict:
    p = ic_cache_plan_t()
    _check(load_library().ic_cache_plan(dim, n, nq, k, path, sm_count, smem_optin, ctypes.byref(p)))
    return p.as_dict()


class ICCache:
    """Owns one ic_cache_t handle.  Tensors passed to insert/query must live on the handle's
    device (or, for the *_host variants, in host memory), be contiguous and have the dtype
    chosen at construction."""

    def __init__(self, dim: int, capacity: int, *, input_dtype: torch.dtype = torch.bfloat16,
                 normalize: bool = False, device: Optional[int] = None, stream: Optional[torch.cuda.Stream] = None,
                 workspace: Optional[torch.Tensor] = None):
        if input_dtype not in (torch.bfloat16, torch.float32):
            raise TypeError("input_dtype must be torch.bfloat16 or torch.float32")
        self.dim, self.capacity, self.input_dtype = dim, capacity, input_dtype
        dev = torch.cuda.current_device() if device is None else device
        self.device = torch.device("cuda", dev)
        st = stream if stream is not None else torch.cuda.current_stream(self.device)
        self._h = ic_cache_create_ex(
            dim, capacity, device=dev, input_dtype=IC_F32 if input_dtype == torch.float32 else IC_BF16,
            normalize=normalize, stream=st.cuda_stream, workspace=workspace)
        self._workspace = workspace     # borrowed by the handle: keep it alive

    # -- lifetime
    def close(self) -> None:
        if getattr(self, "_h", None):
            ic_cache_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    # -- calls
    def _check_rows(self, t: torch.Tensor, on_device: bool, what: str) -> None:
        if t.dtype != self.input_dtype or t.dim() != 2 or t.shape[1] != self.dim or not t.is_contiguous():
            raise ValueError(f"{what} must be a contiguous [*, {self.dim}] tensor of {self.input_dtype}")
        if on_device != t.is_cuda:
            raise ValueError(f"{what} must live in {'device' if on_device else 'host'} memory")

    def insert(self, emb: torch.Tensor, ids: torch.Tensor) -> None:
        self._check_rows(emb, True, "emb")
        if ids.dtype != torch.int64 or ids.shape != (emb.shape[0],) or not ids.is_cuda or not ids.is_contiguous():
            raise ValueError("ids must be a contiguous int64 device tensor with one entry per row")
        ic_cache_insert(self._h, emb, ids, emb.shape[0])

    def insert_host(self, emb: torch.Tensor, ids: torch.Tensor) -> None:
        self._check_rows(emb, False, "emb")
        if ids.dtype != torch.int64 or ids.shape != (emb.shape[0],) or ids.is_cuda or not ids.is_contiguous():
            raise ValueError("ids must be a contiguous int64 host tensor with one entry per row")
        ic_cache_insert_host(self._h, emb, ids, emb.shape[0])

    def query(self, q: torch.Tensor, k: int, out_ids: Optional[torch.Tensor] = None,
              out_scores: Optional[torch.Tensor] = None) -> Tuple[torch.Tensor, torch.Tensor]:
        self._check_rows(q, True, "q")
        nq = q.shape[0]
        if out_ids is None:
            out_ids = torch.empty(nq, k, dtype=torch.int64, device=self.device)
        if out_scores is None:
            out_scores = torch.empty(nq, k, dtype=torch.float32, device=self.device)
        ic_cache_query(self._h, q, nq, k, out_ids, out_scores)
        return out_ids, out_scores

    def query_min_score(self, q: torch.Tensor, k: int, min_score: float):
        """Top-k restricted to entries scoring at least min_score; returns (ids, scores, counts)."""
        self._check_rows(q, True, "q")
        nq = q.shape[0]
        out_ids = torch.empty(nq, k, dtype=torch.int64, device=self.device)
        out_scores = torch.empty(nq, k, dtype=torch.float32, device=self.device)
        counts = torch.empty(nq, dtype=torch.int32, device=self.device)
        ic_cache_query_min_score(self._h, q, nq, k, float(min_score), out_ids, out_scores, counts)
        return out_ids, out_scores, counts

    def query_static(self, q: torch.Tensor, k: int, out_ids: torch.Tensor, out_scores: torch.Tensor) -> None:
        """Allocation-free query: results go into the caller's preallocated device tensors and
        the library's scratch comes from its fixed static array (shared by all handles on the
        GPU; keep calls ordered).  Raises ICCacheError(IC_ERR_NOMEM) if the shape needs more
        scratch than the array holds."""
        self._check_rows(q, True, "q")
        nq = q.shape[0]
        if out_ids.shape != (nq, k) or out_ids.dtype != torch.int64 or not out_ids.is_cuda or not out_ids.is_contiguous():
            raise ValueError("out_ids must be a contiguous int64 device tensor of shape [nq, k]")
        if out_scores.shape != (nq, k) or out_scores.dtype != torch.float32 or not out_scores.is_cuda \
                or not out_scores.is_contiguous():
            raise ValueError("out_scores must be a contiguous float32 device tensor of shape [nq, k]")
        ic_cache_query_static(self._h, q, nq, k, out_ids, out_scores)

    def query_host(self, q: torch.Tensor, k: int, out_ids: Optional[torch.Tensor] = None,
                   out_scores: Optional[torch.Tensor] = None) -> Tuple[torch.Tensor, torch.Tensor]:
        self._check_rows(q, False, "q")
        nq = q.shape[0]
        if out_ids is None:
            out_ids = torch.empty(nq, k, dtype=torch.int64).pin_memory()
        if out_scores is None:
            out_scores = torch.empty(nq, k, dtype=torch.float32).pin_memory()
        ic_cache_query_host(self._h, q, nq, k, out_ids, out_scores)
        return out_ids, out_scores

    def self_similarity(self, first: int = 0, count: Optional[int] = None):
        """Best other entry (id, score) for the entries in slots [first, first+count)."""
        count = self.size - first if count is None else count
        out_ids = torch.empty(count, dtype=torch.int64, device=self.device)
        out_scores = torch.empty(count, dtype=torch.float32, device=self.device)
        _check(load_library().ic_cache_self_similarity(self._h, first, count, _ptr(out_ids), _ptr(out_scores)))
        return out_ids, out_scores

    def save(self, path: str) -> None:
        """Write the entries (rows, ids, utilities) to a checkpoint file."""
        _check(load_library().ic_cache_save(self._h, os.fsencode(path)))

    def load(self, path: str) -> None:
        """Replace the contents with a checkpoint written by save() for the same dimension."""
        _check(load_library().ic_cache_load(self._h, os.fsencode(path)))

    def utility_add(self, ids: torch.Tensor, gains: torch.Tensor) -> None:
        """Add gains[i] to the utility of every entry whose id is ids[i] (host int64 / float32 tensors)."""
        if ids.dtype != torch.int64 or ids.is_cuda or not ids.is_contiguous() or gains.dtype != torch.float32 \
                or gains.is_cuda or not gains.is_contiguous() or gains.numel() != ids.numel():
            raise ValueError("ids (int64) and gains (float32) must be contiguous host tensors of equal length")
        _check(load_library().ic_cache_utility_add(self._h, _ptr(ids), _ptr(gains), ids.numel()))

    def utility_decay(self, factor: float) -> None:
        _check(load_library().ic_cache_utility_decay(self._h, float(factor)))

    def utility_read(self) -> Tuple[torch.Tensor, torch.Tensor]:
        """Host copies (ids int64 [size], utility float32 [size]) in slot order."""
        n = self.size
        ids = torch.empty(n, dtype=torch.int64)
        util = torch.empty(n, dtype=torch.float32)
        _check(load_library().ic_cache_utility_read(self._h, _ptr(ids), _ptr(util)))
        return ids, util

    def build_index(self, n_clusters: int = 0, n_iters: int = 10, init_slots: Optional[torch.Tensor] = None) -> None:
        """Cluster the current entries (ic_cache_build_index).  init_slots: optional host int64
        tensor of n_clusters distinct slots whose rows are the initial centroids."""
        ptr = None
        if init_slots is not None:
            if init_slots.dtype != torch.int64 or init_slots.is_cuda or not init_slots.is_contiguous() \
                    or init_slots.numel() != n_clusters:
                raise ValueError("init_slots must be a contiguous int64 host tensor with n_clusters entries")
            ptr = _ptr(init_slots)
        _check(load_library().ic_cache_build_index(self._h, int(n_clusters), int(n_iters), ptr))

    def index_info(self) -> Tuple[int, int]:
        """(number of clusters, number of entries the index covers); (0, 0) without an index."""
        k, n = ctypes.c_int32(0), ctypes.c_int64(0)
        _check(load_library().ic_cache_index_info(self._h, ctypes.byref(k), ctypes.byref(n)))
        return int(k.value), int(n.value)

    def read_index(self) -> Tuple[torch.Tensor, torch.Tensor]:
        """Host copies of the index: (centroids [K, dim] bfloat16, assign [n_indexed] int64)."""
        k, n = self.index_info()
        cent = torch.empty(k, self.dim, dtype=torch.bfloat16)
        assign = torch.empty(n, dtype=torch.int64)
        _check(load_library().ic_cache_read_index(self._h, _ptr(cent), _ptr(assign)))
        return cent, assign

    def query_clustered(self, q: torch.Tensor, k: int, nprobe: int, return_probes: bool = False):
        """Two-level search (ic_cache_query_clustered): (ids, scores) or (ids, scores, probes)."""
        self._check_rows(q, True, "q")
        nq = q.shape[0]
        out_ids = torch.empty(nq, k, dtype=torch.int64, device=self.device)
        out_scores = torch.empty(nq, k, dtype=torch.float32, device=self.device)
        probes = torch.empty(nq, nprobe, dtype=torch.int64, device=self.device) if return_probes else None
        _check(load_library().ic_cache_query_clustered(self._h, _ptr(q), nq, int(k), int(nprobe), _ptr(out_ids),
                                                       _ptr(out_scores), _ptr(probes) if return_probes else None))
        return (out_ids, out_scores, probes) if return_probes else (out_ids, out_scores)

    def remove(self, ids: torch.Tensor) -> int:
        """Remove every entry whose id is in `ids` (a host int64 tensor); returns how many went."""
        if ids.dtype != torch.int64 or ids.is_cuda or not ids.is_contiguous():
            raise ValueError("ids must be a contiguous int64 host tensor")
        removed = ctypes.c_int64(0)
        _check(load_library().ic_cache_remove(self._h, _ptr(ids), ids.numel(), ctypes.byref(removed)))
        return int(removed.value)

    def set_path(self, path: int) -> None:
        _check(load_library().ic_cache_set_path(self._h, path))

    def set_stream(self, stream: torch.cuda.Stream) -> None:
        _check(load_library().ic_cache_set_stream(self._h, ctypes.c_void_p(stream.cuda_stream)))

    def probe_wait_limit(self) -> None:
        """Enqueue the diagnostic kernel whose bounded wait expires (see ic_cache_probe_wait_limit)."""
        _check(load_library().ic_cache_probe_wait_limit(self._h))

    def clear(self) -> None:
        _check(load_library().ic_cache_clear(self._h))

    def sync(self) -> None:
        _check(load_library().ic_cache_sync(self._h))

    def set_profiling(self, enable: bool) -> None:
        _check(load_library().ic_cache_set_profiling(self._h, int(bool(enable))))

    def read_profile(self) -> dict:
        """Device time of the main scoring launches, the seeding passes (each with its merge) and
        the final merges recorded since the last read."""
        s_ms, m_ms, d_ms = ctypes.c_double(), ctypes.c_double(), ctypes.c_double()
        s_n, m_n, d_n = ctypes.c_int64(), ctypes.c_int64(), ctypes.c_int64()
        _check(load_library().ic_cache_read_profile(self._h, ctypes.byref(s_ms), ctypes.byref(s_n),
                                                    ctypes.byref(m_ms), ctypes.byref(m_n),
                                                    ctypes.byref(d_ms), ctypes.byref(d_n)))
        return {"scoring_ms": s_ms.value, "scoring_launches": s_n.value,
                "merge_ms": m_ms.value, "merge_launches": m_n.value,
                "seed_ms": d_ms.value, "seed_passes": d_n.value}

    @property
    def size(self) -> int:
        return int(load_library().ic_cache_size(self._h))

    @property
    def launch_count(self) -> int:
        return int(load_library().ic_cache_launch_count(self._h))
