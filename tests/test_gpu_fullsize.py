"""GPU parity at the full benchmark sizes, in the launch configuration bench.py times (automatic
path choice, same plan).  The oracle cannot score every query against 16 M rows in seconds, so
it checks a sample of the batch's queries one by one (first, last, and a few in between, which
covers every query tile of the launch); each sampled query is compared element by element."""
import gc

import numpy as np
import pytest
import torch

import oracle
from paper_2501_12689_b200 import ICCache, ic_cache_plan, IC_PATH_AUTO, workloads as wl
from parity_util import TOL, TOL_STRICT

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


class _Loaded:
    """One workload's cache on the GPU plus its rows on the host (for the oracle)."""

    def __init__(self, name):
        self.w = wl.WORKLOADS[name]
        w = self.w
        rounds = 19 if w.insert_rows else 0
        self.x = wl.cache_rows(w, DEV)
        self.cache = ICCache(w.dim, w.n + rounds * w.insert_rows, input_dtype=wl.torch_dtype(w))
        self.cache.insert(self.x, wl.labels(w.n, DEV))
        self.host_rows = [wl.as_bits(self.x)]
        self.n = w.n
        if not w.planted_queries:
            self.x = None            # device copy only needed to plant queries
            gc.collect()
            torch.cuda.empty_cache()

    def append_round(self, rnd):
        new = wl.insert_batch(self.w, rnd, DEV)
        self.cache.insert(new, wl.labels(new.shape[0], DEV, first_slot=self.n))
        self.host_rows.append(wl.as_bits(new))
        self.x = torch.cat([self.x, new])
        self.n += new.shape[0]

    def check(self, nq, sample, rnd=0):
        w = self.w
        q = wl.queries(w, nq, DEV, round_idx=rnd, cache=self.x)
        ids, sc = self.cache.query(q, w.k)
        self.cache.sync()
        ids2, sc2 = self.cache.query(q, w.k)
        self.cache.sync()
        assert torch.equal(ids, ids2) and torch.equal(sc, sc2), "two identical queries differ"
        sample = sorted(set(min(nq - 1, s) for s in sample))
        xb = np.concatenate(self.host_rows) if len(self.host_rows) > 1 else self.host_rows[0]
        lab = wl.labels(self.n).numpy()
        ref = oracle.search(xb, wl.as_bits(q[sample]), w.k, ids=lab, want_all_scores=True)
        got_ids, got_sc = ids[sample].cpu().numpy(), sc[sample].cpu().numpy()
        what = f"{w.name} nq={nq}"
        oracle.accept(got_ids, got_sc, ref["all_scores"], w.k, ids=lab, tol=TOL, what=what + " [binding]")
        rep = oracle.accept(got_ids, got_sc, ref["all_scores"], w.k, ids=lab, tol=TOL_STRICT, what=what + " [strict]")
        assert rep["max_abs_err"] < TOL_STRICT
        return ids, sc

    def close(self):
        self.cache.close()
        self.x = None
        self.host_rows = None
        gc.collect()
        torch.cuda.empty_cache()


@pytest.fixture(scope="module", params=["online", "clustered", "dense", "stress"])
def loaded(request):
    import psutil
    w = wl.WORKLOADS[request.param]
    need = 2.5 * w.n * w.dim * 2
    if psutil.virtual_memory().available < need + (8 << 30):
        pytest.skip("not enough host memory to hold this workload for the oracle")
    if torch.cuda.mem_get_info()[0] < need:
        pytest.skip("not enough free device memory for this workload")
    item = _Loaded(request.param)
    yield item
    item.close()


def test_full_size_workloads_match_the_oracle_on_sampled_queries(loaded):
    w = loaded.w
    for nq in w.q_sweep:
        plan = ic_cache_plan(w.dim, w.n, nq, w.k, IC_PATH_AUTO)
        assert plan["n_ctas"] >= 140
        # first, last and two inner queries: with several query tiles this touches the first
        # and the last tile and a tile boundary
        if w.n <= 4_000_000:
            sample = [0, nq - 1, nq // 2, max(0, min(nq - 1, 128))]
        else:
            # 16 M rows: one query of every 128-query tile (eight oracle queries for the batch of 1024)
            sample = sorted({min(nq - 1, t * 128 + (37 * t) % 128) for t in range((nq + 127) // 128)} | {0, nq - 1})
        loaded.check(nq, sample)
    if w.n > 4_000_000:
        # a batch size between the sweep's: two CTA pairs per row partition, and a sampling launch
        # whose first floor comes from a different number of tiles per CTA
        loaded.check(512, [t * 128 + (53 * t) % 128 for t in range(4)])
    if w.insert_rows:
        # streaming inserts between query batches; planted queries copy rows of the newest batch.
        # The oracle re-checks the first rounds and the last of the 20-round timed loop (round 19).
        for rnd in range(1, 20):
            loaded.append_round(rnd)
            if rnd not in (1, 2, 19):
                continue
            ids, sc = loaded.check(w.q_sweep[0], [0, 1, w.planted_queries, w.q_sweep[0] - 1], rnd=rnd)
            m = w.planted_queries
            newest = wl.labels(w.insert_rows, "cpu", first_slot=loaded.n - w.insert_rows)
            assert torch.all(sc[:m, 0] > 0.99)
            assert all(int(i) in set(newest.tolist()) for i in ids[:m, 0].cpu())


def test_two_level_search_at_full_size():
    """The two-level search on the clustered workload at its full size: index build with
    K = sqrt(N), then sampled queries against the oracle's two-level definition on the library's
    own centroids, assignment and probes."""
    loaded = _Loaded("clustered")
    try:
        _two_level_at_full_size(loaded)
    finally:
        loaded.close()


def _two_level_at_full_size(loaded):
    w = loaded.w
    c = loaded.cache
    c.build_index(0, 3)
    k_clusters, n_indexed = c.index_info()
    assert k_clusters == round(n_indexed ** 0.5) and n_indexed == loaded.n
    nq, nprobe = w.q_sweep[0], 4
    q = wl.queries(w, nq, DEV, round_idx=7, cache=loaded.x)
    ids, sc, probes = c.query_clustered(q, w.k, nprobe, return_probes=True)
    exact_ids, _ = c.query(q, w.k)
    c.sync()
    cent, assign = c.read_index()
    sample = [0, 1, nq // 2, nq - 1]
    xb = np.concatenate(loaded.host_rows)
    lab = wl.labels(loaded.n).numpy()
    ref = oracle.search_clustered(xb, wl.as_bits(q[sample]), w.k, wl.as_bits(cent), assign.numpy().astype(np.int32), nprobe,
                                  probes=probes[sample].cpu().numpy(), ids=lab, want_all_scores=True)
    # the probes themselves: each must be within tolerance of the oracle's nprobe best centroids
    cs = ref["centroid_scores"]
    for j in range(len(sample)):
        cut = np.sort(cs[j])[::-1][nprobe - 1]
        assert np.all(cs[j][probes[sample[j]].cpu().numpy()] >= cut - TOL_STRICT)
    oracle.accept(ids[sample].cpu().numpy(), sc[sample].cpu().numpy(), ref["all_scores"], w.k, ids=lab, tol=TOL_STRICT,
                  what="clustered two-level [strict]")
    # queries sit near cluster centres: a few probes recover the exhaustive result
    e, g = exact_ids.cpu().numpy(), ids.cpu().numpy()
    recall = np.mean([len(set(e[i]) & set(g[i])) / w.k for i in range(nq)])
    assert recall > 0.95, recall


@pytest.mark.parametrize("name,rows", [("dense", 160_003), ("stress", 70_000)])
def test_every_query_of_the_large_batches_on_a_truncated_cache(name, rows):
    """The full-size checks above sample a few queries per batch.  Here every query of the two
    large-batch workloads (256 and 1024 queries: two and eight query tiles, CTA pairs, seeding)
    is checked against the oracle, on a cache cut down to 160,003 / 70,000 rows of the same
    recipe (still enough tiles per CTA for the seeding launch) so that the oracle finishes soon."""
    from parity_util import run_and_check
    w = wl.WORKLOADS[name].scaled(rows)
    nq = max(w.q_sweep)
    plan = ic_cache_plan(w.dim, w.n, nq, w.k, IC_PATH_AUTO)
    assert plan["n_query_tiles"] == nq // 128 and plan["cta_group"] == 2 and plan["seed0_tiles"] > 0
    x, q = wl.cache_rows(w, DEV), wl.queries(w, nq, DEV)
    run_and_check(x, q, w.k, path=IC_PATH_AUTO, what=f"{name}/truncated/all-queries")
