"""ic_cache_query_static: the query entry point for callers that must not allocate device
memory while serving (the GPU is fully reserved by their framework's memory pool, or their
loop may not make calls that can synchronise the device).  Its scratch is a fixed array inside
the library, so the test checks that it returns what ic_cache_query returns, twice in a row
(the array keeps the previous call's contents), through the C ABI, with every buffer supplied
by the caller.  Collected last on purpose: a run that stops at the first failure has then
already run every other test."""
import pytest
import torch

import oracle
from paper_2501_12689_b200 import (ICCache, ICCacheError, IC_ERR_NOMEM, IC_ERR_INVALID, IC_PATH_AUTO,
                                   IC_PATH_GENERIC, workloads as wl)
from parity_util import TOL_STRICT

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _case(n, dim, nq, k, seed, path=IC_PATH_AUTO):
    w = wl.Workload("z", n, dim, "bf16", (nq,), k, seed=seed)
    x = wl.cache_rows(w, DEV)
    with ICCache(dim, n) as c:
        c.set_path(path)
        c.insert(x, wl.labels(n, DEV))
        q1, q2 = wl.queries(w, nq, DEV, round_idx=0), wl.queries(w, nq, DEV, round_idx=1)
        want = [c.query(q, k) for q in (q1, q2)]
        c.sync()
        # caller-owned outputs, allocated before the calls under test
        outs = [(torch.empty(nq, k, dtype=torch.int64, device=DEV),
                 torch.empty(nq, k, dtype=torch.float32, device=DEV)) for _ in range(2)]
        c.query_static(q1, k, *outs[0])      # first use on this GPU looks the array's address up
        c.sync()
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        c.query_static(q1, k, *outs[0])      # two calls in a row share the static scratch
        c.query_static(q2, k, *outs[1])
        c.sync()
        # nothing was allocated on the device by the two calls (torch allocated nothing either:
        # every tensor above exists already)
        assert torch.cuda.mem_get_info()[0] == free_before
        for (wi, ws), (gi, gs) in zip(want, outs):
            assert torch.equal(wi, gi)
            assert torch.allclose(ws, gs, atol=TOL_STRICT, rtol=0)
        # and against the CPU oracle, strictly
        lab = wl.labels(n).numpy()
        for q, (gi, gs) in zip((q1, q2), outs):
            ref = oracle.search(wl.as_bits(x), wl.as_bits(q), k, ids=lab, want_all_scores=True)
            oracle.accept(gi.cpu().numpy(), gs.cpu().numpy(), ref["all_scores"], k, ids=lab, tol=TOL_STRICT,
                          what=f"static scratch n {n} dim {dim} nq {nq} k {k}")


def test_static_query_matches_query_scan_path():
    _case(50_001, 384, 3, 10, seed=201)


def test_static_query_matches_query_tensor_core_path():
    _case(70_001, 768, 64, 10, seed=202)


def test_static_query_matches_query_with_threshold_seeding():
    _case(400_003, 64, 40, 16, seed=203)


def test_static_query_matches_query_generic_path():
    _case(9_000, 128, 5, 4, seed=204, path=IC_PATH_GENERIC)


def test_static_query_rejects_shapes_beyond_its_scratch():
    with ICCache(64, 1000) as c:
        c.insert(torch.zeros(1000, 64, device=DEV, dtype=torch.bfloat16), wl.labels(1000, DEV))
        nq, k = 512, 64                                   # ~20 MB of partial lists
        q = torch.zeros(nq, 64, device=DEV, dtype=torch.bfloat16)
        oi = torch.empty(nq, k, dtype=torch.int64, device=DEV)
        os_ = torch.empty(nq, k, dtype=torch.float32, device=DEV)
        with pytest.raises(ICCacheError) as e:
            c.query_static(q, k, oi, os_)
        assert e.value.status == IC_ERR_NOMEM and "static scratch" in str(e.value)
        nq = 1025                                         # more than one window
        q = torch.zeros(nq, 64, device=DEV, dtype=torch.bfloat16)
        oi = torch.empty(nq, 1, dtype=torch.int64, device=DEV)
        os_ = torch.empty(nq, 1, dtype=torch.float32, device=DEV)
        with pytest.raises(ICCacheError) as e:
            c.query_static(q, 1, oi, os_)
        assert e.value.status == IC_ERR_INVALID
        assert c.size == 1000
