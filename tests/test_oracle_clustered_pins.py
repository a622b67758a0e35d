"""Pins for the K-Means / two-level search part of the CPU oracle: hand-computed values,
library cross-checks and invariants, none of them computed by the oracle itself."""
import os

import numpy as np
import pytest
import torch

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "hand_kmeans.txt")


def _golden():
    g = {"x": [], "search": []}
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        tok = line.split()
        if tok[0] == "x":
            g["x"].append([float(v) for v in tok[2:]])
        elif tok[0] in ("init", "assign", "count"):
            g[tok[0]] = [int(v) for v in tok[1:]]
        elif tok[0] == "best":
            g["best"] = [float(v) for v in tok[1:]]
        elif tok[0] == "centroid":
            g.setdefault("centroid", {})[int(tok[1])] = [float(v) for v in tok[2:]]
        elif tok[0] == "search":
            arrow, bar = tok.index("->"), tok.index("|")
            g["search"].append({"n_indexed": int(tok[1]), "nprobe": int(tok[2]), "k": int(tok[3]),
                                "probes": [int(v) for v in tok[arrow + 1:bar]],
                                "ranked": [(int(t.split(":")[0]), float(t.split(":")[1])) for t in tok[bar + 1:]]})
    return g


def _bits(a):
    return torch.tensor(np.asarray(a, dtype=np.float32)).to(torch.bfloat16).view(torch.uint16).numpy()


def _widen(bits):
    return torch.tensor(np.asarray(bits, dtype=np.uint16)).view(torch.bfloat16).float().numpy()


# ---------------------------------------------------------------- hand-computed values

def test_hand_computed_assignment_and_tie():
    g = _golden()
    x = np.array(g["x"], dtype=np.float32)
    cent = _bits(x[g["init"]])               # (1,0) and (-1,0) are exact in bf16
    assign, best = oracle.kmeans_assign(x, cent)
    assert assign.tolist() == g["assign"]
    np.testing.assert_allclose(best, g["best"], atol=1e-6)


def test_hand_computed_update():
    g = _golden()
    x = np.array(g["x"], dtype=np.float32)
    cent0 = _bits(x[g["init"]])
    cent, exact, counts = oracle.kmeans_update(x, np.array(g["assign"], dtype=np.int32), cent0)
    assert counts.tolist() == g["count"]
    for c, want in g["centroid"].items():
        np.testing.assert_allclose(exact[c], want, atol=1e-7)   # fp32 inputs 0.6 / 0.8 are not exact
    # the stored centroid is the nearest-even bf16 rounding of the exact one (library cast)
    assert np.array_equal(cent, _bits(exact.astype(np.float32)))


def test_empty_cluster_keeps_its_centroid():
    g = _golden()
    x = np.array(g["x"], dtype=np.float32)
    cent0 = _bits([[1, 0], [-1, 0], [0.5, -0.5]])
    cent, exact, counts = oracle.kmeans_update(x, np.array(g["assign"], dtype=np.int32), cent0)
    assert counts.tolist() == g["count"] + [0]
    assert np.array_equal(cent[2], cent0[2])
    np.testing.assert_allclose(exact[2], [0.5, -0.5])


@pytest.mark.parametrize("case", range(4))
def test_hand_computed_two_level_search(case):
    g = _golden()
    s = g["search"][case]
    x = np.array(g["x"], dtype=np.float32)
    cent = _bits([[1, 0], [-1, 0]])
    q = np.array([[-0.6, 0.8]], dtype=np.float32)
    r = oracle.search_clustered(x, q, s["k"], cent, np.array(g["assign"], dtype=np.int32), s["nprobe"],
                                n_indexed=s["n_indexed"], want_all_scores=True)
    assert r["probes"][0].tolist() == s["probes"]
    np.testing.assert_allclose(r["centroid_scores"][0], [-0.6, 0.6], atol=1e-6)
    assert r["slots"][0].tolist() == [slot for slot, _ in s["ranked"]]
    want = [v for _, v in s["ranked"]]
    np.testing.assert_allclose(r["scores"][0], want, atol=1e-6)
    # rows that were not searched carry -inf in the full score row
    searched = np.isfinite(r["all_scores"][0])
    expect = np.array([(i >= s["n_indexed"]) or (g["assign"][i] in s["probes"]) for i in range(5)])
    assert np.array_equal(searched, expect)


def test_given_probes_replace_the_centroid_step():
    g = _golden()
    x = np.array(g["x"], dtype=np.float32)
    cent = _bits([[1, 0], [-1, 0]])
    q = np.array([[-0.6, 0.8]], dtype=np.float32)
    r = oracle.search_clustered(x, q, 2, cent, np.array(g["assign"], dtype=np.int32), 1,
                                probes=np.array([[0]], dtype=np.int64))
    assert r["slots"][0].tolist() == [2, 1]        # cluster 0 holds slots 0, 1, 2: scores -0.6, 0.28, 0.8


# ---------------------------------------------------------------- reductions to pinned / library routines

def _blobs(n, d, n_blobs, sigma, seed):
    rng = np.random.default_rng(seed)
    centres = rng.standard_normal((n_blobs, d))
    z = rng.integers(0, n_blobs, n)
    x = centres[z] + sigma * rng.standard_normal((n, d))
    x /= np.linalg.norm(x, axis=1, keepdims=True)
    return x.astype(np.float32), z


def test_probing_every_cluster_is_the_exhaustive_search():
    x, _ = _blobs(3000, 24, 12, 0.4, seed=1)
    xb = _bits(x)
    q = _bits(_blobs(7, 24, 12, 0.4, seed=2)[0])
    km = oracle.kmeans(xb, np.arange(0, 3000, 250), 2)
    full = oracle.search(xb, q, 9)
    two = oracle.search_clustered(xb, q, 9, km["centroids"], km["assign"], nprobe=12)
    assert np.array_equal(full["slots"], two["slots"])
    assert np.array_equal(full["scores"], two["scores"])
    # with fewer probes every returned row belongs to a probed cluster and carries its exhaustive score
    part = oracle.search_clustered(xb, q, 9, km["centroids"], km["assign"], nprobe=3, want_all_scores=True)
    exh = oracle.search(xb, q, 9, want_all_scores=True)["all_scores"]
    for iq in range(7):
        slots = part["slots"][iq][part["slots"][iq] >= 0]
        assert set(km["assign"][slots].tolist()) <= set(part["probes"][iq].tolist())
        assert np.array_equal(part["scores"][iq][:len(slots)], exh[iq][slots])
        # and nothing better was left behind inside the probed clusters
        inside = np.isin(km["assign"], part["probes"][iq])
        assert np.array_equal(np.sort(exh[iq][inside])[::-1][:len(slots)], part["scores"][iq][:len(slots)])


def test_assignment_against_numpy_argmax():
    x, _ = _blobs(2000, 32, 10, 0.5, seed=3)
    xb = _bits(x)
    cent = xb[np.arange(0, 2000, 200)]
    assign, best = oracle.kmeans_assign(xb, cent)
    s = _widen(xb).astype(np.float64) @ _widen(cent).astype(np.float64).T
    top2 = np.sort(s, axis=1)[:, -2:]
    clear = (top2[:, 1] - top2[:, 0]) > 1e-5          # leave out near-ties that fp32 may order differently
    assert clear.mean() > 0.99
    assert np.array_equal(assign[clear], np.argmax(s, axis=1)[clear])
    np.testing.assert_allclose(best, s.max(axis=1), atol=1e-5)


def test_update_against_sklearn_one_lloyd_step():
    from sklearn.cluster import KMeans
    x, _ = _blobs(1500, 16, 6, 0.15, seed=4)          # well separated: Euclidean and cosine assignments agree
    xb = _bits(x)
    xw = _widen(xb).astype(np.float64)
    init = np.array([int(np.flatnonzero(_blobs(1500, 16, 6, 0.15, seed=4)[1] == b)[0]) for b in range(6)])
    cent0 = xb[init]
    assign, _ = oracle.kmeans_assign(xb, cent0)
    cent, exact, counts = oracle.kmeans_update(xb, assign, cent0)
    km = KMeans(n_clusters=6, init=_widen(cent0).astype(np.float64), n_init=1, max_iter=1, algorithm="lloyd", tol=0.0).fit(xw)
    want = km.cluster_centers_ / np.linalg.norm(km.cluster_centers_, axis=1, keepdims=True)
    np.testing.assert_allclose(exact, want, atol=1e-9)
    assert counts.sum() == 1500 and np.array_equal(counts, np.bincount(assign, minlength=6))


# ---------------------------------------------------------------- invariants

def test_lloyd_iterations_do_not_lower_the_objective():
    x, _ = _blobs(4000, 32, 20, 0.6, seed=5)
    xb = _bits(x)
    init = np.arange(0, 4000, 200)
    prev = -1.0
    for iters in range(4):
        km = oracle.kmeans(xb, init, iters)
        obj = float(km["best"].astype(np.float64).mean())
        assert obj >= prev - 1e-4        # bf16 rounding of the centroids may cost a little
        prev = obj
        norms = np.linalg.norm(_widen(km["centroids"]).astype(np.float64), axis=1)
        np.testing.assert_allclose(norms, 1.0, atol=4e-3)
        assert km["assign"].min() >= 0 and km["assign"].max() < 20
    assert prev > 0.5


def test_well_separated_blobs_are_recovered():
    x, z = _blobs(1200, 16, 4, 0.1, seed=6)
    xb = _bits(x)
    init = np.array([int(np.flatnonzero(z == b)[0]) for b in range(4)])
    km = oracle.kmeans(xb, init, 3)
    assert np.array_equal(km["assign"], z)           # centroid b starts inside blob b and keeps it


# ---------------------------------------------------------------- utility bookkeeping (Sec. 4.3)

def test_utility_hand_computed_sequence():
    ids = np.array([7, 8, 7, 9], dtype=np.int64)          # id 7 is carried by two entries
    u = np.zeros(4, dtype=np.float32)
    u = oracle.utility_add(ids, u, [7, 9, 5], [1.0, 2.0, 4.0])   # id 5 matches nothing
    assert u.tolist() == [1.0, 0.0, 1.0, 2.0]
    u = oracle.utility_decay(u, 0.5)
    assert u.tolist() == [0.5, 0.0, 0.5, 1.0]
    u = oracle.utility_add(ids, u, [9, 9], [0.25, 0.25])          # the same id twice in one call
    assert u.tolist() == [0.5, 0.0, 0.5, 1.5]
    # the paper's decay: 0.9 per hour; after one gain of 1 and two hours 0.81 remains
    v = oracle.utility_decay(oracle.utility_decay(np.array([1.0], dtype=np.float32), 0.9), 0.9)
    np.testing.assert_allclose(v, [0.81], rtol=1e-6)


def test_utility_moving_average_closed_form():
    # a gain of g every hour, decayed by 0.9 per hour, is the geometric series g (1 - 0.9^h) / 0.1
    ids = np.array([1], dtype=np.int64)
    u = np.zeros(1, dtype=np.float32)
    for h in range(1, 41):
        u = oracle.utility_decay(u, 0.9)
        u = oracle.utility_add(ids, u, [1], [3.0])
        np.testing.assert_allclose(u[0], 3.0 * (1.0 - 0.9 ** h) / 0.1, rtol=1e-5)
