"""Shared helpers of the GPU parity tests: run the CUDA path through the C ABI binding and
check it against the CPU oracle on the same bits."""
from __future__ import annotations

import numpy as np
import torch

import oracle
from oracle import accept
from paper_2501_12689_b200 import ICCache, workloads as wl

TOL = 2e-2          # binding tolerance: |score - oracle fp32 score| for bf16-stored embeddings
TOL_STRICT = 1e-4   # diagnostic tolerance against the oracle on the exact stored bf16 bits


def run_and_check(x: torch.Tensor, q: torch.Tensor, k: int, *, path: int = 0, normalize: bool = False,
                  ids: torch.Tensor | None = None, sample_queries=None, capacity: int | None = None,
                  insert_splits=None, what: str = ""):
    """Insert x (device tensor, fp32 or bf16), query q, compare with the oracle.

    sample_queries: indices of the queries the oracle checks (default: all).
    insert_splits: row counts of successive insert calls (default: one call).
    Returns (out_ids, out_scores) as CPU tensors.
    """
    n, dim = x.shape
    nq = q.shape[0]
    dev = x.device
    if ids is None:
        ids = wl.labels(n, dev)
    with ICCache(dim, capacity or max(n, 1), input_dtype=x.dtype, normalize=normalize) as cache:
        cache.set_path(path)
        r0 = 0
        for rows in (insert_splits or [n]):
            cache.insert(x[r0:r0 + rows], ids[r0:r0 + rows])
            r0 += rows
        assert r0 == n and cache.size == n
        out_ids, out_scores = cache.query(q, k)
        cache.sync()
        again_ids, again_scores = cache.query(q, k)
        cache.sync()
    assert torch.equal(out_ids, again_ids) and torch.equal(out_scores, again_scores), \
        f"{what}: two identical queries gave different results"
    out_ids, out_scores = out_ids.cpu(), out_scores.cpu()
    sel = list(range(nq)) if sample_queries is None else list(sample_queries)
    if not sel:
        return out_ids, out_scores
    xb, qb = wl.as_bits(x), wl.as_bits(q[sel])
    ids_np = ids.cpu().numpy()
    # binding check: oracle on the data as the caller supplied it
    ref = oracle.search(xb, qb, k, ids=ids_np, normalize=normalize, want_all_scores=True)
    accept(out_ids[sel].numpy(), out_scores[sel].numpy(), ref["all_scores"], k, ids=ids_np, tol=TOL,
           what=what + " [binding]")
    # strict diagnostic: oracle on the bf16 bits the slab holds (differs from the above only
    # when the caller's data is fp32 or gets normalised)
    if x.dtype == torch.float32 or normalize:
        xs, qs = x.float(), q[sel].float()
        if normalize:
            xs = xs / xs.norm(dim=1, keepdim=True).clamp_min(1e-30)
            qs = qs / qs.norm(dim=1, keepdim=True).clamp_min(1e-30)
        ref = oracle.search(wl.as_bits(xs.to(torch.bfloat16)), wl.as_bits(qs.to(torch.bfloat16)), k,
                            ids=ids_np, want_all_scores=True)
        strict = 5e-4 if normalize else TOL_STRICT   # the two fp32 norms may round one bf16 ulp apart
    else:
        strict = TOL_STRICT
    rep = accept(out_ids[sel].numpy(), out_scores[sel].numpy(), ref["all_scores"], k, ids=ids_np,
                 tol=strict, what=what + " [strict]")
    return out_ids, out_scores, rep
