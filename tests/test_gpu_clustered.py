"""GPU parity of the two-level search: K-Means index build (assignment step, update step, the
whole Lloyd loop) and the clustered query, through the C ABI, against the CPU oracle on the
same seeded inputs."""
import numpy as np
import pytest
import torch

import oracle
from oracle import accept
from paper_2501_12689_b200 import ICCache, ICCacheError, IC_ERR_INVALID, workloads as wl
from parity_util import TOL_STRICT

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _blob_workload(n, dim, n_blobs, sigma, seed, nq=8):
    return wl.Workload("blobs", n, dim, "bf16", (nq,), 8, seed=seed, kind="clustered", n_clusters=n_blobs, sigma=sigma)


def _bits(t):
    return wl.as_bits(t)


def _cache_with(x, extra_capacity=0, **kw):
    c = ICCache(x.shape[1], x.shape[0] + extra_capacity, input_dtype=x.dtype, **kw)
    c.insert(x, wl.labels(x.shape[0], DEV))
    return c


def _check_choice(chosen, scores, tol, what):
    """chosen [n] indices into the columns of scores [n, K]: each must be the row's best column,
    or score within tol of it; returns the fraction that is the exact argmax."""
    best = scores.max(axis=1)
    got = scores[np.arange(scores.shape[0]), chosen]
    bad = np.flatnonzero(got < best - tol)
    assert bad.size == 0, f"{what}: row {bad[:5]} assigned to a centroid scoring {got[bad[:5]]} against best {best[bad[:5]]}"
    return float((chosen == scores.argmax(axis=1)).mean())


@pytest.mark.parametrize("n,dim,k_clusters", [(20_003, 128, 141), (5_000, 768, 70), (1_500, 64, 1), (3_000, 40, 300)])
def test_assignment_step(n, dim, k_clusters):
    w = wl.Workload("g", n, dim, "bf16", (4,), 8, seed=301)
    x = wl.cache_rows(w, DEV)
    init = torch.randperm(n, generator=torch.Generator().manual_seed(5))[:k_clusters].contiguous()
    with _cache_with(x) as c:
        c.build_index(k_clusters, 0, init)
        assert c.index_info() == (k_clusters, n)
        cent, assign = c.read_index()
    xb = _bits(x)
    # without update steps the centroids are the chosen rows, bit for bit
    assert np.array_equal(_bits(cent), xb[init.numpy()])
    assign = assign.numpy()
    assert assign.min() >= 0 and assign.max() < k_clusters
    # oracle scores of every row against every centroid (the centroids are the cache here)
    ref = oracle.search(_bits(cent), xb, 1, want_all_scores=True)
    exact = _check_choice(assign, ref["all_scores"], TOL_STRICT, "assignment")
    assert exact > 0.999
    o_assign, _ = oracle.kmeans_assign(xb, _bits(cent))
    gap_ok = np.sort(ref["all_scores"], axis=1)[:, -1] - (np.sort(ref["all_scores"], axis=1)[:, -2] if k_clusters > 1 else -1.0) > TOL_STRICT
    assert np.array_equal(assign[gap_ok], o_assign[gap_ok])


def _init_inside_blobs(w, x, n_blobs):
    """One initial slot per blob: the first row closest to each centre."""
    cen = wl.centres(w, DEV)
    z = (x.float() @ wl._unit(cen).T).argmax(dim=1)
    init = torch.stack([torch.nonzero(z == b)[0, 0] for b in range(n_blobs)]).cpu().contiguous()
    return init, z.cpu().numpy()


@pytest.mark.parametrize("n,dim,n_blobs", [(12_000, 128, 24), (6_001, 768, 9)])
def test_update_step_and_lloyd_loop(n, dim, n_blobs):
    w = _blob_workload(n, dim, n_blobs, 0.25, seed=302)
    x = wl.cache_rows(w, DEV)
    init, _ = _init_inside_blobs(w, x, n_blobs)
    xb = _bits(x)
    cent0 = xb[init.numpy()]
    o_assign0, _ = oracle.kmeans_assign(xb, cent0)
    with _cache_with(x) as c:
        c.build_index(n_blobs, 0, init)
        _, g_assign0 = c.read_index()
        # well-separated blobs: the first assignment has no near-ties, so both sides agree on it
        assert np.array_equal(g_assign0.numpy(), o_assign0)
        # one update step from that assignment: fp64 sums in slot order on both sides
        c.build_index(n_blobs, 1, init)
        g_cent1, g_assign1 = c.read_index()
        o_cent1, o_exact, counts = oracle.kmeans_update(xb, o_assign0, cent0)
        assert counts.min() > 0
        diff = np.flatnonzero(_bits(g_cent1).reshape(-1) != o_cent1.reshape(-1))
        assert diff.size <= 1e-4 * o_cent1.size, f"{diff.size} centroid components differ"
        g_w = g_cent1.float().numpy().reshape(-1)
        np.testing.assert_allclose(g_w[diff], o_exact.reshape(-1)[diff], rtol=2 ** -8)   # at most one bf16 step
        # the whole loop
        c.build_index(n_blobs, 3, init)
        g_cent3, g_assign3 = c.read_index()
    km = oracle.kmeans(xb, init.numpy(), 3)
    same = (_bits(g_cent3) == km["centroids"]).mean()
    assert same > 0.999
    assert (g_assign3.numpy() == km["assign"]).mean() > 0.9999


def _check_probes(probes, centroid_scores, nprobe, tol, what):
    """probes [nq, nprobe] against oracle centroid scores [nq, K]: the set must hold every centroid
    beating the nprobe-th score by more than tol and nothing more than tol below it, best first."""
    nq, k_clusters = centroid_scores.shape
    real = min(nprobe, k_clusters)
    for iq in range(nq):
        p = probes[iq]
        assert np.all(p[real:] == -1), f"{what} q{iq}: padding"
        p = p[:real]
        assert len(set(p.tolist())) == real and p.min() >= 0 and p.max() < k_clusters, f"{what} q{iq}: bad probe list {p}"
        s = centroid_scores[iq]
        t = np.sort(s)[::-1][real - 1]
        assert np.all(s[p] >= t - tol), f"{what} q{iq}: probed a centroid below the cut"
        must = np.flatnonzero(s > t + tol)
        assert set(must.tolist()) <= set(p.tolist()), f"{what} q{iq}: missed a centroid above the cut"
        assert np.all(np.diff(s[p]) <= tol), f"{what} q{iq}: probes not ordered best first"


def _clustered_case(x, q, k, k_clusters, n_iters, nprobe, extra=None, what=""):
    n = x.shape[0]
    ids = wl.labels(n + (0 if extra is None else extra.shape[0]), DEV)
    with ICCache(x.shape[1], n + (0 if extra is None else extra.shape[0]), input_dtype=x.dtype) as c:
        c.insert(x, ids[:n])
        c.build_index(k_clusters, n_iters)
        if extra is not None:
            c.insert(extra, ids[n:])
        kc, n_indexed = c.index_info()
        assert n_indexed == n
        out_ids, out_scores, probes = c.query_clustered(q, k, nprobe, return_probes=True)
        again = c.query_clustered(q, k, nprobe)
        c.sync()
        cent, assign = c.read_index()
        full_ids, full_scores = c.query(q, k)
        c.sync()
    assert torch.equal(out_ids, again[0]) and torch.equal(out_scores, again[1]), f"{what}: not repeatable"
    x_all = x if extra is None else torch.cat([x, extra])
    xb, qb = _bits(x_all.to(torch.bfloat16)), _bits(q.to(torch.bfloat16))
    ids_np = ids.cpu().numpy()
    # the centroid step
    ref_c = oracle.search_clustered(xb, qb, k, _bits(cent), assign.numpy().astype(np.int32), nprobe, n_indexed=n)
    _check_probes(probes.cpu().numpy(), ref_c["centroid_scores"], nprobe, TOL_STRICT, what)
    # the search inside the clusters the library probed
    ref = oracle.search_clustered(xb, qb, k, _bits(cent), assign.numpy().astype(np.int32), nprobe, n_indexed=n,
                                  probes=probes.cpu().numpy(), ids=ids_np, want_all_scores=True)
    searched = np.isfinite(ref["all_scores"]).sum(axis=1)
    assert searched.min() >= k, "test case too small: fewer searched rows than k"
    rep = accept(out_ids.cpu().numpy(), out_scores.cpu().numpy(), ref["all_scores"], k, ids=ids_np, tol=TOL_STRICT,
                 what=what + " [clustered]")
    return out_ids.cpu(), full_ids.cpu(), rep, kc


@pytest.mark.parametrize("nq,nprobe,k", [(1, 4, 10), (16, 8, 10), (130, 3, 16), (5, 64, 5)])
def test_clustered_query_on_blobs(nq, nprobe, k):
    w = _blob_workload(60_000, 256, 300, 0.3, seed=303, nq=nq)
    x, q = wl.cache_rows(w, DEV), wl.queries(w, nq, DEV)
    got, full, rep, kc = _clustered_case(x, q, k, 0, 4, nprobe, what=f"blobs/nq{nq}/p{nprobe}")
    assert kc == round(60_000 ** 0.5)
    # queries sit near blob centres, so probing a few clusters finds most of the exact top-k
    recall = np.mean([len(set(got[i].tolist()) & set(full[i].tolist())) / k for i in range(nq)])
    assert recall > 0.8, recall


def test_clustered_query_on_gaussian_rows():
    w = wl.WORKLOADS["online"].scaled(40_000)
    x, q = wl.cache_rows(w, DEV), wl.queries(w, 9, DEV)
    _clustered_case(x, q, 10, 64, 2, 16, what="gauss")


def test_probing_every_cluster_gives_the_exhaustive_result():
    # with every cluster probed the oracle's candidate set is the whole cache, so the acceptance
    # check inside _clustered_case is the one of the exhaustive search: a row missing from the
    # member lists, or listed twice, would fail it
    w = _blob_workload(30_011, 128, 40, 0.5, seed=304)
    x, q = wl.cache_rows(w, DEV), wl.queries(w, 33, DEV)
    got, full, _, _ = _clustered_case(x, q, 12, 48, 3, 48, what="all-probes")
    same = np.mean([len(set(got[i].tolist()) & set(full[i].tolist())) / 12 for i in range(33)])
    assert same > 0.99      # the two kernels may order near-ties at the 12th place differently


def test_rows_inserted_after_the_build_are_always_searched():
    w = _blob_workload(20_000, 128, 100, 0.3, seed=305)
    x = wl.cache_rows(w, DEV)
    extra = wl.cache_rows(_blob_workload(5_003, 128, 100, 0.3, seed=306), DEV)
    q = torch.cat([extra[[0, 17, 5_002]], wl.queries(w, 6, DEV)])
    got, _, _, _ = _clustered_case(x, q, 8, 0, 3, 2, extra=extra, what="tail")
    ids = wl.labels(25_003, "cpu")
    # a query equal to a row inserted after the build finds that row first
    assert got[0, 0] == ids[20_000] and got[1, 0] == ids[20_017] and got[2, 0] == ids[25_002]


@pytest.mark.parametrize("nq,k", [(130, 8), (40, 64)])
def test_long_tail_of_unindexed_rows(nq, k):
    # 40,003 rows inserted after the build under a batch of queries: the tiles wholly past the
    # index (from row 20,224 on) are scored by the tensor-core kernel, rows 20,000 .. 20,223 by
    # the cluster scan; every row must be searched exactly once
    w = _blob_workload(20_000, 128, 100, 0.3, seed=309)
    x = wl.cache_rows(w, DEV)
    extra = wl.cache_rows(_blob_workload(40_003, 128, 100, 0.3, seed=310), DEV)
    q = torch.cat([extra[[0, 100, 223, 224, 300, 40_002]], wl.queries(w, nq - 6, DEV)])
    got, _, _, _ = _clustered_case(x, q, k, 0, 2, 3, extra=extra, what=f"long-tail/nq{nq}")
    ids = wl.labels(60_003, "cpu")
    for i, row in enumerate([0, 100, 223, 224, 300, 40_002]):
        assert got[i, 0] == ids[20_000 + row]


def test_fp32_input_and_few_clusters():
    w = wl.WORKLOADS["tiny"]
    x, q = wl.cache_rows(w, DEV), wl.queries(w, 16, DEV)
    _clustered_case(x, q, 8, 3, 2, 8, what="tiny-fp32")        # nprobe above the number of clusters


def test_index_lifecycle_and_errors():
    w = _blob_workload(4_000, 64, 10, 0.3, seed=307)
    x, q = wl.cache_rows(w, DEV), wl.queries(w, 3, DEV)
    with ICCache(64, 8) as empty:
        with pytest.raises(ICCacheError):
            empty.build_index(0, 1)                              # nothing to cluster
        assert empty.index_info() == (0, 0)
        assert empty.utility_read()[0].numel() == 0
    with _cache_with(x, extra_capacity=16) as c:
        with pytest.raises(ICCacheError) as e:
            c.query_clustered(q, 4, 2)
        assert e.value.status == IC_ERR_INVALID
        for bad in [dict(n_clusters=-1), dict(n_clusters=4_001), dict(n_clusters=3, n_iters=-1)]:
            with pytest.raises(ICCacheError):
                c.build_index(**bad)
        with pytest.raises(ICCacheError):
            c.build_index(2, 1, torch.tensor([5, 5]))            # repeated slot
        with pytest.raises(ICCacheError):
            c.build_index(2, 1, torch.tensor([5, 4_000]))        # slot outside the cache
        c.build_index(10, 2)
        assert c.index_info() == (10, 4_000)
        with pytest.raises(ICCacheError):
            c.query_clustered(q, 4, 0)
        with pytest.raises(ICCacheError):
            c.query_clustered(q, 4, 65)
        c.query_clustered(q, 4, 2)
        none_ids, none_scores = c.query_clustered(q[:0], 4, 2)   # no queries: nothing to do
        assert none_ids.shape == (0, 4) and none_scores.shape == (0, 4)
        before = c.query(q, 4)
        assert c.remove(wl.labels(1, "cpu")) == 1                # moving rows drops the index
        assert c.index_info() == (0, 0)
        c.build_index(0, 1)
        assert c.index_info()[0] == round(3_999 ** 0.5)
        c.clear()
        assert c.index_info() == (0, 0)
        del before


def test_more_queries_than_one_window():
    # 1030 queries: two windows of the query loop, the second with six queries
    w = _blob_workload(9_000, 64, 30, 0.3, seed=308, nq=1030)
    x, q = wl.cache_rows(w, DEV), wl.queries(w, 1030, DEV)
    _clustered_case(x, q, 6, 30, 2, 3, what="two-windows")
