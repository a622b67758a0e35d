"""Seeded synthetic inputs shaped like the paper's request workloads.

This module only draws inputs (embeddings, ids, query batches, insert batches);
it holds none of the retrieval arithmetic and is the one module both the CUDA
path's callers and the CPU oracle's callers use, so that both see the same bits.

The paper's pools are text requests embedded by a trained encoder (Table 1:
7,500 - 808,731 examples; Sec. 2.2: ~1 M-request similarity study).  Neither
the datasets nor an encoder are available offline, so each workload below
borrows only sizes and similarity structure:

  tiny       10 k fp32 unit Gaussian rows, d=384   (size of a saturated cache, Sec. 6.4)
  online     1 M bf16 unit Gaussian rows, d=768    ("1 million requests" pools)
  clustered  2 M rows from 1,000 Gaussian clusters (sigma 0.3 => in-cluster
             cosine ~ 0.917, echoing ">70 % of requests have a neighbour with
             cosine > 0.8"), 1 % bit-exact duplicates, streaming inserts
  dense      4 M rows, d=1024, 256-query bursts    (25x load peaks)
  stress     16 M rows, d=768                      ("millions of daily requests")

Every tensor is drawn from a torch.Generator seeded from (workload seed, stream
number), on whichever device the caller names; parity checks always copy the
drawn bits to the other side rather than re-drawing them.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Optional, Tuple

import torch

_CHUNK_ROWS = 1 << 18

# stream numbers: one independent random stream per kind of draw
_S_CENTRES, _S_ROWS, _S_DUPS, _S_QUERIES, _S_INSERTS = 1, 2, 3, 4, 5


@dataclass(frozen=True)
class Workload:
    name: str
    n: int                      # cache entries before any streaming insert
    dim: int
    input_dtype: str            # "f32" or "bf16": dtype handed to insert/query
    q_sweep: Tuple[int, ...]    # query batch sizes
    k: int
    seed: int
    kind: str = "gaussian"      # "gaussian" or "clustered"
    n_clusters: int = 0
    sigma: float = 0.0
    dup_frac: float = 0.0       # fraction of rows overwritten by exact copies of other rows
    insert_rows: int = 0        # rows appended between consecutive query batches
    planted_queries: int = 0    # queries that are bit-exact copies of cached rows

    def scaled(self, n: int) -> "Workload":
        """Same recipe at a smaller cache size (for parity cases the oracle can finish)."""
        return replace(self, n=int(n))


WORKLOADS = {
    "tiny": Workload("tiny", 10_000, 384, "f32", (16,), 8, seed=0),
    "online": Workload("online", 1_000_000, 768, "bf16", (1, 4, 16, 64), 10, seed=1),
    "clustered": Workload("clustered", 2_000_000, 768, "bf16", (128,), 16, seed=2,
                          kind="clustered", n_clusters=1000, sigma=0.3, dup_frac=0.01,
                          insert_rows=10_000, planted_queries=8),
    "dense": Workload("dense", 4_000_000, 1024, "bf16", (256,), 32, seed=3),
    "stress": Workload("stress", 16_000_000, 768, "bf16", (1, 64, 1024), 64, seed=4),
}


def _generator(w: Workload, stream: int, device, sub: int = 0) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed((w.seed * 1_000_003 + stream) * 1_000_003 + sub)
    return g


def torch_dtype(w: Workload) -> torch.dtype:
    return torch.float32 if w.input_dtype == "f32" else torch.bfloat16


def _unit(x: torch.Tensor) -> torch.Tensor:
    return x / x.norm(dim=1, keepdim=True).clamp_min(1e-30)


def centres(w: Workload, device) -> Optional[torch.Tensor]:
    if w.kind != "clustered":
        return None
    g = _generator(w, _S_CENTRES, device)
    return torch.randn(w.n_clusters, w.dim, generator=g, device=device, dtype=torch.float32)


def _draw_rows(w: Workload, rows: int, g: torch.Generator, device, c: Optional[torch.Tensor]):
    x = torch.randn(rows, w.dim, generator=g, device=device, dtype=torch.float32)
    if w.kind == "clustered":
        z = torch.randint(0, w.n_clusters, (rows,), generator=g, device=device)
        x = c[z] + w.sigma * x
    return _unit(x).to(torch_dtype(w))


def cache_rows(w: Workload, device="cpu", out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """The initial cache contents [n, dim] in the workload's input dtype, drawn in row chunks."""
    if out is None:
        out = torch.empty(w.n, w.dim, dtype=torch_dtype(w), device=device)
    c = centres(w, device)
    g = _generator(w, _S_ROWS, device)
    for r0 in range(0, w.n, _CHUNK_ROWS):
        rows = min(_CHUNK_ROWS, w.n - r0)
        out[r0:r0 + rows] = _draw_rows(w, rows, g, device, c)
    if w.dup_frac > 0 and w.n > 1:
        gd = _generator(w, _S_DUPS, device)
        m = int(w.n * w.dup_frac)
        dst = torch.randperm(w.n, generator=gd, device=device)[:m]
        src = torch.randint(0, w.n, (m,), generator=gd, device=device)
        keep = ~torch.isin(src, dst)   # a copied row must itself be an original
        out[dst[keep]] = out[src[keep]]
    return out


def labels(n: int, device="cpu", first_slot: int = 0) -> torch.Tensor:
    """Unique int64 labels for slots first_slot .. first_slot+n-1 (an odd-multiplier bijection
    on 32-bit slots, offset so that a label never equals its slot)."""
    s = torch.arange(first_slot, first_slot + n, device=device, dtype=torch.int64)
    return ((s * 2654435761) & 0xFFFFFFFF) + (1 << 33)


def queries(w: Workload, nq: int, device="cpu", round_idx: int = 0,
            cache: Optional[torch.Tensor] = None) -> torch.Tensor:
    """One query batch [nq, dim]; drawn by the same law as the cache rows.  When the workload
    plants exact copies and `cache` is given, the first few queries are copies of cached rows
    (taken from the end of the cache, i.e. from the most recently inserted entries)."""
    g = _generator(w, _S_QUERIES, device, sub=round_idx * 4096 + nq)
    q = _draw_rows(w, nq, g, device, centres(w, device))
    if w.planted_queries and cache is not None and cache.shape[0] > 0:
        m = min(w.planted_queries, nq, cache.shape[0])
        pick = torch.randint(max(0, cache.shape[0] - max(w.insert_rows, m)), cache.shape[0], (m,),
                             generator=g, device=device)
        q[:m] = cache[pick].to(q.dtype)
    return q


def insert_batch(w: Workload, round_idx: int, device="cpu") -> torch.Tensor:
    """Rows appended before query round `round_idx` (same law as the cache rows)."""
    g = _generator(w, _S_INSERTS, device, sub=round_idx)
    return _draw_rows(w, w.insert_rows, g, device, centres(w, device))


def as_bits(t: torch.Tensor):
    """numpy view of a tensor for the oracle: float32 stays float32, bf16 becomes its uint16 bits."""
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.uint16).numpy()
    return t.numpy()
