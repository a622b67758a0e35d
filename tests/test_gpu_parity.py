"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle element by
element on the same seeded inputs.  Sizes span several tiles and ragged tails of every
kernel path (scan pieces of 32 rows, tensor-core tiles of 256 rows x 128 queries x 64 dims)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2501_12689_b200 import (ICCache, ICCacheError, IC_PATH_AUTO, IC_PATH_GENERIC, IC_PATH_SCAN,
                                   IC_PATH_UMMA, IC_ERR_FULL, IC_ERR_INVALID, workloads as wl)
from parity_util import run_and_check, TOL

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
PATHS = {"auto": IC_PATH_AUTO, "generic": IC_PATH_GENERIC, "scan": IC_PATH_SCAN, "umma": IC_PATH_UMMA}


def _gauss(n, dim, nq, seed, dtype="bf16"):
    w = wl.Workload("g", n, dim, dtype, (nq,), 8, seed=seed)
    return wl.cache_rows(w, DEV), wl.queries(w, nq, DEV)


@pytest.mark.parametrize("path", ["generic", "scan", "umma", "auto"])
def test_tiny_config(path):
    w = wl.WORKLOADS["tiny"]
    x, q = wl.cache_rows(w, DEV), wl.queries(w, 16, DEV)
    run_and_check(x, q, w.k, path=PATHS[path], what=f"tiny/{path}")


@pytest.mark.parametrize("path", ["generic", "scan", "umma", "auto"])
@pytest.mark.parametrize("nq", [1, 4, 16, 64])
def test_online_config_scaled(path, nq):
    if path == "generic" and nq > 16:
        pytest.skip("generic path is a slow cross-check; covered at nq <= 16")
    w = wl.WORKLOADS["online"].scaled(70_001)      # 273.4 tensor-core tiles, 2187.5 scan pieces
    x, q = wl.cache_rows(w, DEV), wl.queries(w, nq, DEV)
    run_and_check(x, q, w.k, path=PATHS[path], what=f"online/{path}/nq{nq}")


@pytest.mark.parametrize("path", ["scan", "umma"])
@pytest.mark.parametrize("dim", [8, 40, 264, 520, 1024])
def test_ragged_dims(path, dim):
    x, q = _gauss(5_003, dim, 3, seed=20 + dim)
    run_and_check(x, q, 5, path=PATHS[path], what=f"dim{dim}/{path}")


@pytest.mark.parametrize("dim", [1032, 2048, 4096])
def test_large_dims_take_the_tensor_core_path(dim):
    x, q = _gauss(3_000, dim, 2, seed=30)
    run_and_check(x, q, 4, path=IC_PATH_AUTO, what=f"dim{dim}/auto")
    with ICCache(dim, 16) as c:
        c.set_path(IC_PATH_SCAN)
        c.insert(x[:16], wl.labels(16, DEV))
        with pytest.raises(ICCacheError):
            c.query(q, 2)


@pytest.mark.parametrize("path", ["generic", "scan", "umma"])
@pytest.mark.parametrize("n,k", [(1, 1), (5, 8), (31, 31), (300, 128), (4097, 64), (9, 128)])
def test_small_caches_and_k_edges(path, n, k):
    x, q = _gauss(n, 64, 3, seed=40 + n)
    out_ids, out_scores, _ = run_and_check(x, q, k, path=PATHS[path], what=f"n{n}k{k}/{path}")
    if k > n:
        assert torch.all(out_ids[:, n:] == -1) and torch.all(torch.isneginf(out_scores[:, n:]))


@pytest.mark.parametrize("path", ["generic", "scan", "umma"])
def test_empty_cache(path):
    with ICCache(64, 10) as c:
        c.set_path(PATHS[path])
        q = torch.randn(2, 64, device=DEV).to(torch.bfloat16)
        ids, sc = c.query(q, 3)
        c.sync()
        assert torch.all(ids == -1) and torch.all(torch.isneginf(sc))
        ids, sc = c.query(q[:0], 3)       # nq == 0 is a no-op
        assert ids.shape == (0, 3)


@pytest.mark.parametrize("path", ["scan", "umma"])
@pytest.mark.parametrize("nq,k", [(2, 16), (130, 16), (257, 7)])
def test_query_tiling(path, nq, k):
    if path == "scan" and nq > 4:
        nq = 7                                         # several scan passes with a ragged last one
    x, q = _gauss(20_011, 128, nq, seed=50 + nq)
    run_and_check(x, q, k, path=PATHS[path], what=f"qtile/{path}/nq{nq}")


@pytest.mark.parametrize("path", ["umma", "auto"])
@pytest.mark.parametrize("nq", [96, 100, 127, 224, 250, 1000])
def test_bf16_queries_read_in_place_with_a_partly_filled_last_tile(path, nq):
    """bf16 queries that need no normalisation are read by the tensor-core kernel straight from the
    caller's rows when the last 128-query tile is nearly full: the query tensor map then covers
    fewer rows than its box and the rows past nq must read as zero.  Covers single CTAs (one
    tile), CTA pairs with a ragged second tile (224, 250) and eight tiles (1000), every query
    checked against the oracle."""
    x, q = _gauss(40_003, 256, nq, seed=300 + nq)
    run_and_check(x, q, 12, path=PATHS[path], what=f"in-place/{path}/nq{nq}")


def test_bf16_queries_read_in_place_from_a_16_byte_aligned_pointer():
    """Same path with a query pointer that is 16-byte but not 128-byte aligned (a view that starts
    one row into a larger tensor whose rows are 48 bytes long)."""
    nq, dim = 100, 24
    x, qq = _gauss(30_001, dim, nq + 1, seed=311)
    q = qq[1:]
    assert q.data_ptr() % 16 == 0 and q.data_ptr() % 128 != 0 and q.is_contiguous()
    run_and_check(x, q, 9, path=IC_PATH_UMMA, what="in-place/offset-pointer")


@pytest.mark.parametrize("order", ["random", "best_first", "best_last"])
@pytest.mark.parametrize("nq,k", [(9, 10), (130, 64), (130, 128), (5, 128)])
def test_threshold_seeding_pass(order, nq, k):
    _seeding_case(order, nq, k, 400_003, levels=1)


@pytest.mark.parametrize("order", ["random", "best_first", "best_last"])
def test_two_level_threshold_seeding(order):
    # enough tiles that a sample of them is scored into lists, by a launch of its own, ahead of the main pass
    _seeding_case(order, 40, 16, 2_600_011, levels=2)


@pytest.mark.parametrize("order", ["best_first", "best_last"])
def test_long_sampling_launch_takes_its_first_floor_from_more_tiles(order):
    """A batch of several query tiles against a cache large enough that the sampling launch runs
    over dozens of tiles per CTA: it then exchanges the group maxima of more than the usual one
    tile per SM.  The best rows sit all inside, or all outside, what is sampled."""
    from paper_2501_12689_b200 import ic_cache_plan
    dim, n, nq, k = 64, 12_000_517, 512, 10
    plan = ic_cache_plan(dim, n, nq, k, IC_PATH_UMMA)
    per_cta = plan["seed0_tiles"] // plan["n_partitions"]
    assert plan["seed_tiles"] > 0 and plan["cta_group"] == 2 and per_cta > (148 + plan["n_partitions"] - 1) // plan["n_partitions"]
    x, q = _gauss(n, dim, nq, seed=77)
    s0 = (x.float() @ q[300].float())
    x = x[torch.argsort(s0, descending=(order == "best_first"))].contiguous()
    del s0
    run_and_check(x, q, k, path=IC_PATH_UMMA, sample_queries=[0, 129, 300, 511], what=f"long sample/{order}")


@pytest.mark.parametrize("nq,k", [(40, 10), (130, 64)])
def test_seeding_falls_back_to_local_floors_when_the_siblings_are_not_waited_for(nq, k, monkeypatch):
    """The exchange of group maxima inside a launch is a bounded look, never a condition for
    progress.  With the look cut to nothing, CTAs that do not find all their siblings' maxima at the
    first glance score their first tile with a local floor instead: the results must not change."""
    monkeypatch.setenv("IC_CACHE_SEED_LOOK_CYCLES", "0")
    _seeding_case("random", nq, k, 400_003, levels=1)


def _seeding_case(order, nq, k, n, levels):
    # enough row tiles per CTA that the tensor-core path takes a floor from a sample first and
    # starts the main pass from it; with the best rows all inside (or all outside) the sample,
    # the final merge must still return the exact top-k
    from paper_2501_12689_b200 import ic_cache_plan
    dim = 64
    plan = ic_cache_plan(dim, n, nq, k, IC_PATH_UMMA)
    # level 0: group maxima exchanged inside the scoring launch; level 1: a sample scored into lists
    assert plan["seed0_tiles"] > 0 and (plan["seed_tiles"] > 0) == (levels == 2)
    x, q = _gauss(n, dim, nq, seed=55)
    if order != "random":
        s0 = (x.float() @ q[0].float())
        idx = torch.argsort(s0, descending=(order == "best_first"))
        x = x[idx].contiguous()
    run_and_check(x, q, k, path=IC_PATH_UMMA, sample_queries=[0, 1, nq // 2, nq - 1], what=f"seed/{order}/nq{nq}")


def test_more_queries_than_one_window():
    x, q = _gauss(3_001, 64, 1030, seed=60)
    run_and_check(x, q, 4, path=IC_PATH_UMMA, sample_queries=[0, 1, 127, 128, 1023, 1024, 1029], what="window")


@pytest.mark.parametrize("path", ["generic", "scan", "umma"])
def test_adversarial_orders(path):
    # rows arrive in ascending order of their score against query 0: every row is a new best
    dim, n = 64, 6_000
    g = torch.Generator(device=DEV).manual_seed(70)
    qv = torch.nn.functional.normalize(torch.randn(1, dim, generator=g, device=DEV), dim=1)
    x = torch.nn.functional.normalize(torch.randn(n, dim, generator=g, device=DEV), dim=1).to(torch.bfloat16)
    order = torch.argsort((x.float() @ qv.T).squeeze(1))
    q = torch.cat([qv, -qv]).to(torch.bfloat16)       # second query sees descending order
    run_and_check(x[order].contiguous(), q, 32, path=PATHS[path], what=f"ascending/{path}")
    # all rows identical: every score ties, so the answer is the first k slots in order
    same = x[:1].repeat(1000, 1).contiguous()
    ids = wl.labels(1000, DEV)
    out_ids, out_scores, _ = run_and_check(same, q[:1], 16, path=PATHS[path], ids=ids, what=f"ties/{path}")
    assert torch.equal(out_ids[0], ids[:16].cpu())
    assert torch.all(out_scores[0] == out_scores[0, 0])


@pytest.mark.parametrize("path", ["scan", "umma"])
def test_clustered_config_scaled_with_streaming_inserts(path):
    w = wl.WORKLOADS["clustered"].scaled(60_000)
    w = wl.Workload(**{**w.__dict__, "insert_rows": 1_000})
    nq = 128 if path == "umma" else 4
    x0 = wl.cache_rows(w, DEV)
    cap = w.n + 3 * w.insert_rows
    with ICCache(w.dim, cap) as c:
        c.set_path(PATHS[path])
        c.insert(x0, wl.labels(w.n, DEV))
        allx = x0
        for rnd in range(3):
            new = wl.insert_batch(w, rnd, DEV)
            c.insert(new, wl.labels(w.insert_rows, DEV, first_slot=allx.shape[0]))
            allx = torch.cat([allx, new])
            q = wl.queries(w, nq, DEV, round_idx=rnd, cache=allx)
            ids, sc = c.query(q, w.k)
            c.sync()
            ref = oracle.search(wl.as_bits(allx), wl.as_bits(q), w.k, ids=wl.labels(allx.shape[0]).numpy(),
                                want_all_scores=True)
            lab = wl.labels(allx.shape[0]).numpy()
            oracle.accept(ids.cpu().numpy(), sc.cpu().numpy(), ref["all_scores"], w.k, ids=lab, tol=1e-4,
                          what=f"clustered/{path}/round{rnd}")
            # planted queries copy rows inserted this round: they must come back first, score ~1
            m = min(w.planted_queries, nq)
            assert torch.all(sc[:m, 0] > 0.99)
            assert torch.all(ids[:m, 0].cpu() >= 0)
            # exact duplicates tie bit for bit: equal returned scores come back in slot order
            sorter = np.argsort(lab)
            slots = sorter[np.searchsorted(lab[sorter], ids.cpu().numpy())]
            scn = sc.cpu().numpy()
            tie = scn[:, 1:] == scn[:, :-1]
            if nq >= 64:
                assert tie.any(), "the workload should force exact score ties"
            assert np.all(slots[:, 1:][tie] > slots[:, :-1][tie])


@pytest.mark.parametrize("path", ["generic", "scan", "umma"])
def test_split_inserts_equal_one_insert(path):
    x, q = _gauss(10_000, 96, 4, seed=80)
    a = run_and_check(x, q, 9, path=PATHS[path], what="one insert")
    b = run_and_check(x, q, 9, path=PATHS[path], insert_splits=[1, 4_999, 5_000], what="three inserts")
    assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1])


@pytest.mark.parametrize("path", ["generic", "scan", "umma"])
def test_fp32_input_with_normalisation(path):
    g = torch.Generator(device=DEV).manual_seed(90)
    x = torch.randn(8_000, 200, generator=g, device=DEV) * 3.0
    x[17] = 0.0                                                   # a zero row stays zero
    q = torch.randn(4, 200, generator=g, device=DEV) * 0.2
    q[3] = x[4321] * 5.0                                          # same direction as a cached row
    out_ids, out_scores, _ = run_and_check(x, q, 6, path=PATHS[path], normalize=True, what=f"normalize/{path}")
    assert out_ids[3, 0].item() == wl.labels(8_000)[4321].item()
    assert abs(out_scores[3, 0].item() - 1.0) < 5e-3


def test_paths_agree_bit_for_bit_on_ids():
    x, q = _gauss(40_000, 384, 4, seed=100)
    res = {p: run_and_check(x, q, 10, path=PATHS[p], what=p)[:2] for p in ("generic", "scan", "umma")}
    assert torch.equal(res["generic"][0], res["scan"][0])
    assert torch.equal(res["generic"][0], res["umma"][0])
    assert torch.allclose(res["generic"][1], res["umma"][1], atol=1e-5)


def test_host_buffers_end_to_end():
    x, q = _gauss(12_345, 128, 5, seed=110)
    with ICCache(128, 12_345) as c:
        c.insert_host(x.cpu(), wl.labels(12_345))
        assert c.size == 12_345
        ids_h, sc_h = c.query_host(q.cpu().pin_memory(), 7)
        ids_d, sc_d = c.query(q, 7)
        c.sync()
        assert torch.equal(ids_h, ids_d.cpu()) and torch.equal(sc_h, sc_d.cpu())
        assert c.launch_count > 0


def test_error_returns_leave_the_cache_unchanged():
    with ICCache(64, 100) as c:
        x = torch.zeros(60, 64, device=DEV, dtype=torch.bfloat16)
        ids = wl.labels(60, DEV)
        c.insert(x, ids)
        with pytest.raises(ICCacheError) as e:
            c.insert(x, ids)
        assert e.value.status == IC_ERR_FULL and c.size == 60
        q = torch.zeros(1, 64, device=DEV, dtype=torch.bfloat16)
        for bad_k in (0, 129):
            with pytest.raises(ICCacheError) as e:
                c.query(q, bad_k)
            assert e.value.status == IC_ERR_INVALID
        import paper_2501_12689_b200.binding as b
        host_q = torch.zeros(1, 64, dtype=torch.bfloat16)
        out_i = torch.empty(1, 4, dtype=torch.int64, device=DEV)
        out_s = torch.empty(1, 4, dtype=torch.float32, device=DEV)
        with pytest.raises(ICCacheError) as e:     # host pointer handed to the device entry point
            b.ic_cache_query(c._h, host_q, 1, 4, out_i, out_s)
        assert e.value.status == IC_ERR_INVALID
    for dim, cap in ((0, 10), (12, 10), (8192, 10), (64, 0)):
        with pytest.raises(ICCacheError):
            ICCache(dim, cap)


@pytest.mark.parametrize("path", ["generic", "scan", "umma"])
def test_min_score_filter_and_counts(path):
    w = wl.WORKLOADS["clustered"].scaled(50_000)
    x = wl.cache_rows(w, DEV)
    nq = 4 if path != "umma" else 40
    q = wl.queries(w, nq, DEV, cache=x)
    lab = wl.labels(w.n, DEV)
    with ICCache(w.dim, w.n) as c:
        c.set_path(PATHS[path])
        c.insert(x, lab)
        for tau in (0.85, 0.999, 2.0, float("-inf")):
            ids, sc, counts = c.query_min_score(q, w.k, tau)
            c.sync()
            ref = oracle.search(wl.as_bits(x), wl.as_bits(q), w.k, ids=lab.cpu().numpy(), min_score=tau,
                                want_all_scores=True)
            got_counts = counts.cpu().numpy()
            # a score within rounding distance of the threshold may fall on either side
            near = np.abs(ref["all_scores"] - tau).min(axis=1) < 1e-5 if np.isfinite(tau) else np.zeros(nq, bool)
            assert np.array_equal(got_counts[~near], ref["counts"][~near])
            scn, idn = sc.cpu().numpy(), ids.cpu().numpy()
            for i in range(nq):
                kept = int(got_counts[i])
                assert np.all(scn[i, :kept] >= tau) and np.all(np.isneginf(scn[i, kept:])) and np.all(idn[i, kept:] == -1)
                if not near[i]:
                    assert np.array_equal(idn[i, :kept], ref["ids"][i, :kept]) or \
                        np.allclose(scn[i, :kept], ref["scores"][i, :kept], atol=1e-5)
        assert counts.max().item() <= w.k
    with ICCache(w.dim, 10) as c:
        with pytest.raises(ICCacheError):
            c.query_min_score(q, 3, float("nan"))


@pytest.mark.parametrize("path", ["scan", "umma"])
def test_remove_closes_gaps_and_frees_capacity(path):
    n, dim, k = 30_000, 128, 12
    nq = 2 if path == "scan" else 33
    x, q = _gauss(n, dim, nq, seed=120)
    lab = wl.labels(n, DEV)
    g = torch.Generator().manual_seed(121)
    with ICCache(dim, n) as c:
        c.set_path(PATHS[path])
        c.insert(x, lab)
        # victims: the best match of every query, the first and last rows, a random 10 %, an id
        # that does not exist and a repeated id
        ids0, _ = c.query(q, 1)
        victims = torch.cat([ids0.flatten().cpu(), lab[:3].cpu(), lab[-5:].cpu(),
                             lab.cpu()[torch.randperm(n, generator=g)[: n // 10]],
                             torch.tensor([12345, int(lab[7])])])
        removed = c.remove(victims.contiguous())
        keep = ~torch.isin(lab.cpu(), victims)
        assert removed == int((~keep).sum()) and c.size == int(keep.sum())
        xr, lr = x.cpu()[keep], lab.cpu()[keep]

        def check(rows, labels, what):
            ids, sc = c.query(q, k)
            c.sync()
            ref = oracle.search(wl.as_bits(rows), wl.as_bits(q), k, ids=labels.numpy(), want_all_scores=True)
            oracle.accept(ids.cpu().numpy(), sc.cpu().numpy(), ref["all_scores"], k, ids=labels.numpy(), tol=1e-4, what=what)
            return ids
        ids1 = check(xr, lr, f"after remove/{path}")
        assert not torch.isin(ids1.cpu(), victims).any()
        # the freed capacity takes new rows
        extra = wl.queries(wl.Workload("g", n, dim, "bf16", (1,), 8, seed=122), removed, DEV)
        extra_lab = wl.labels(removed, DEV, first_slot=n)
        c.insert(extra, extra_lab)
        assert c.size == n
        check(torch.cat([xr, extra.cpu()]), torch.cat([lr, extra_lab.cpu()]), f"after refill/{path}")
        with pytest.raises(ICCacheError):
            c.insert(extra[:1], extra_lab[:1])
        # removing ids that are not there changes nothing; removing everything empties the cache
        assert c.remove(torch.tensor([1, 2, 3])) == 0 and c.size == n
        everything = torch.cat([lr, extra_lab.cpu()])
        assert c.remove(everything) == n and c.size == 0
        ids, sc = c.query(q, 3)
        c.sync()
        assert torch.all(ids == -1)


@pytest.mark.parametrize("n,dim", [(5, 64), (1, 64), (6_000, 128), (2_500, 768)])
def test_self_similarity_matches_oracle(n, dim):
    x, _ = _gauss(n, dim, 1, seed=130 + n)
    if n > 100:
        x[17] = x[n - 3]                       # an exact duplicate pair: each is the other's best
        x[40] = x[41] = x[42]                  # a triple
    lab = wl.labels(n, DEV)
    with ICCache(dim, n) as c:
        c.insert(x, lab)
        ids, sc = c.self_similarity()
        c.sync()
        ref = oracle.self_similarity(wl.as_bits(x), ids=lab.cpu().numpy())
        got_ids, got_sc = ids.cpu().numpy(), sc.cpu().numpy()
        if n == 1:
            assert got_ids.tolist() == [-1] and np.isneginf(got_sc[0])
            return
        assert np.allclose(got_sc, ref["scores"], atol=1e-4)
        # the partner may differ only where two candidates score within rounding distance
        differ = np.flatnonzero(got_ids != ref["ids"])
        xb = x.float().cpu()
        labc = lab.cpu().numpy()
        for i in differ:
            j = int(np.flatnonzero(labc == got_ids[i])[0])
            assert j != i and abs(float(xb[i] @ xb[j]) - float(ref["scores"][i])) < 1e-4
        assert differ.size <= max(2, n // 200)
        if n > 100:
            assert got_ids[17] == labc[n - 3] and got_ids[n - 3] == labc[17] and abs(got_sc[17] - 1.0) < 5e-3
            assert got_ids[40] == labc[41] and got_ids[41] == labc[40] and got_ids[42] == labc[40]
        # a sub-range gives the same answers
        ids2, sc2 = c.self_similarity(first=n // 2, count=min(n - n // 2, 1500))
        c.sync()
        assert torch.equal(ids2, ids[n // 2: n // 2 + ids2.numel()])
        with pytest.raises(ICCacheError):
            c.self_similarity(first=n - 1, count=5)


def test_expired_device_wait_is_reported_and_the_handle_recovers():
    # failure detection without a fault: a bounded wait runs out (nothing completes the barrier),
    # the kernel reports it, the host surfaces IC_ERR_TIMEOUT, and the cache keeps working
    from paper_2501_12689_b200 import IC_ERR_TIMEOUT
    x, q = _gauss(5_000, 64, 3, seed=140)
    with ICCache(64, 5_010) as c:
        c.insert(x, wl.labels(5_000, DEV))
        before = c.query(q, 4)
        c.sync()
        c.probe_wait_limit()
        torch.cuda.synchronize()
        with pytest.raises(ICCacheError) as e:      # the bypass signal: serve without examples
            c.query(q, 4)
        assert e.value.status == IC_ERR_TIMEOUT
        with pytest.raises(ICCacheError) as e:
            c.insert(x[:1], wl.labels(1, DEV))
        assert e.value.status == IC_ERR_TIMEOUT and c.size == 5_000
        with pytest.raises(ICCacheError) as e:      # sync reports it once and clears it
            c.sync()
        assert e.value.status == IC_ERR_TIMEOUT
        c.sync()
        after = c.query(q, 4)
        c.sync()
        assert torch.equal(before[0], after[0]) and torch.equal(before[1], after[1])


@pytest.mark.parametrize("seed", [1, 2, 3])
def test_random_shapes_tensor_core_path_agrees_with_the_plain_kernel(seed):
    """Seeded random shapes, large enough to reach the seeding launches and CTA pairs, where the
    oracle would take too long: the tensor-core path and the automatic choice must agree with the
    plain CUDA-core kernel (itself checked against the oracle above) up to ties at the k-th place."""
    import random
    rng = random.Random(seed)
    for case in range(12):
        dim = rng.choice([8, 64, 128, 384, 520, 768, 1024, 1536])
        n = rng.choice([rng.randint(1, 3000), rng.randint(3000, 80_000), rng.randint(80_000, 700_000)])
        n = min(n, 400_000_000 // dim)
        nq = rng.choice([1, 2, 3, 7, 9, 33, 64, 65, 128, 129, 257])
        k = rng.choice([1, 2, 8, 10, 16, 17, 32, 64, 100, 128])
        kind = rng.choice(["gaussian", "clustered", "sorted"])
        w = wl.Workload("f", n, dim, "bf16", (nq,), k, seed=7000 + 100 * seed + case,
                        kind="clustered" if kind == "clustered" else "gaussian", n_clusters=50, sigma=0.3,
                        dup_frac=0.01 if kind == "clustered" else 0.0)
        x, q = wl.cache_rows(w, DEV), wl.queries(w, nq, DEV)
        if kind == "sorted":
            x = x[torch.argsort(x.float() @ q[0].float(), descending=rng.random() < 0.5)].contiguous()
        got = {}
        with ICCache(dim, n) as c:
            c.insert(x, wl.labels(n, DEV))
            for name, path in (("umma", IC_PATH_UMMA), ("auto", IC_PATH_AUTO), ("plain", IC_PATH_GENERIC)):
                c.set_path(path)
                ids, sc = c.query(q, k)
                c.sync()
                got[name] = (ids.cpu(), sc.cpu())
        p_ids, p_sc = got["plain"]
        fin = torch.isfinite(p_sc)
        what = f"seed {seed} case {case}: dim {dim} n {n} nq {nq} k {k} {kind}"
        if n <= 80_000:      # small enough for the oracle: all three paths against it, strictly
            lab = wl.labels(n).numpy()
            ref = oracle.search(wl.as_bits(x), wl.as_bits(q), k, ids=lab, want_all_scores=True)
            for name in ("umma", "auto", "plain"):
                oracle.accept(got[name][0].numpy(), got[name][1].numpy(), ref["all_scores"], k, ids=lab, tol=1e-4,
                              what=what + f" [{name} vs oracle]")
        for name in ("umma", "auto"):
            a_ids, a_sc = got[name]
            assert torch.equal(torch.isfinite(a_sc), fin), what
            if fin.any():
                assert (a_sc[fin] - p_sc[fin]).abs().max().item() <= 1e-4, what
            for i in range(nq):
                sa, sp = set(a_ids[i].tolist()), set(p_ids[i].tolist())
                if sa != sp:     # only entries tied with the k-th score may differ
                    kth = p_sc[i][fin[i]].min().item()
                    for arr_ids, arr_sc in ((a_ids[i], a_sc[i]), (p_ids[i], p_sc[i])):
                        for j, idv in enumerate(arr_ids.tolist()):
                            assert idv not in (sa ^ sp) or abs(arr_sc[j].item() - kth) <= 2e-4, what


def test_caller_owned_workspace_serves_queries_without_allocation():
    """A handle created with a workspace of ic_cache_workspace_bytes takes the scratch of its
    queries from it: same results as a handle that grows its own buffers, for every kernel path
    the automatic choice reaches; a workspace that is too small is an error, not an allocation."""
    from paper_2501_12689_b200 import ic_cache_workspace_bytes, IC_ERR_NOMEM
    w = wl.WORKLOADS["online"].scaled(400_003)         # enough tiles for the seeding launches
    x = wl.cache_rows(w, DEV)
    ids = wl.labels(w.n, DEV)
    need = ic_cache_workspace_bytes(w.dim, w.n, 300, 16)
    ws = torch.empty(need, dtype=torch.uint8, device=DEV)
    xb, lab = wl.as_bits(x), wl.labels(w.n).numpy()
    with ICCache(w.dim, w.n) as plain, ICCache(w.dim, w.n, workspace=ws) as fixed:
        plain.insert(x, ids)
        fixed.insert(x, ids)
        for nq, k in ((1, 10), (2, 16), (5, 3), (64, 10), (130, 16), (300, 8)):
            q = wl.queries(w, nq, DEV, round_idx=nq)
            a_ids, a_sc = plain.query(q, k)
            b_ids, b_sc = fixed.query(q, k)
            plain.sync()
            fixed.sync()
            assert torch.equal(a_ids, b_ids) and torch.equal(a_sc, b_sc), f"nq {nq} k {k}"
            sel = sorted({0, nq // 2, nq - 1})
            ref = oracle.search(xb, wl.as_bits(q[sel]), k, ids=lab, want_all_scores=True)
            oracle.accept(b_ids[sel].cpu().numpy(), b_sc[sel].cpu().numpy(), ref["all_scores"], k, ids=lab, tol=1e-4,
                          what=f"workspace handle nq {nq} k {k}")
        c_ids, c_sc, c_cnt = fixed.query_min_score(wl.queries(w, 7, DEV), 5, 0.12)
        d_ids, d_sc, d_cnt = plain.query_min_score(wl.queries(w, 7, DEV), 5, 0.12)
        assert torch.equal(c_ids, d_ids) and torch.equal(c_cnt, d_cnt)
        with pytest.raises(ICCacheError) as e:                 # beyond what the workspace was sized for
            fixed.query(wl.queries(w, 1024, DEV), 64)
        assert e.value.status == IC_ERR_NOMEM
        fixed.query(wl.queries(w, 3, DEV), 4)                  # the handle stays usable
    tiny = torch.empty(4096, dtype=torch.uint8, device=DEV)
    with ICCache(w.dim, 1000, workspace=tiny) as c:
        c.insert(x[:1000], ids[:1000])
        with pytest.raises(ICCacheError) as e:
            c.query(wl.queries(w, 1, DEV), 1)
        assert e.value.status == IC_ERR_NOMEM
