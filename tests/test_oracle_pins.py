"""Pins for the CPU oracle: things the paper's definition and mathematics fix, none of which
is computed by the oracle itself.  A dropped term, wrong sign, transposed operand, wrong sort
direction or wrong tie-break in oracle/ic_oracle.c fails at least one test here."""
import math
import os
import statistics

import numpy as np
import pytest
import torch

import oracle
from oracle import accept, AcceptanceError
from paper_2501_12689_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "hand_cosine.txt")


def _parse_golden():
    caches, cur = {}, None
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        tok = line.split()
        if tok[0] == "cache":
            cur = {"d": int(tok[2].split("=")[1]), "x": [], "q": []}
            caches[tok[1]] = cur
        elif tok[0] == "x":
            assert int(tok[1]) == len(cur["x"])
            cur["x"].append([float(v) for v in tok[2:]])
        elif tok[0] == "self":
            caches[tok[1]].setdefault("self", {})[int(tok[2])] = (int(tok[4].split(":")[0]), float(tok[4].split(":")[1]))
        elif tok[0] == "q":
            arrow = tok.index("->")
            vec = [float(v) for v in tok[1:arrow]]
            ranked = [(int(t.split(":")[0]), float(t.split(":")[1])) for t in tok[arrow + 1:]]
            cur["q"].append((vec, ranked))
    return caches


# ---------------------------------------------------------------- hand-computed values

@pytest.mark.parametrize("name", ["axes", "onehot"])
def test_hand_computed_rankings_fp32(name):
    c = _parse_golden()[name]
    x = np.array(c["x"], dtype=np.float32)
    for vec, ranked in c["q"]:
        q = np.array([vec], dtype=np.float32)
        r = oracle.search(x, q, k=len(ranked))
        assert r["slots"][0].tolist() == [s for s, _ in ranked]
        np.testing.assert_allclose(r["scores"][0], [v for _, v in ranked], atol=1e-6)
        # default labels are the slots
        assert r["ids"][0].tolist() == r["slots"][0].tolist()


def test_hand_computed_onehot_bf16_exact():
    c = _parse_golden()["onehot"]
    xb = torch.tensor(c["x"], dtype=torch.float32).to(torch.bfloat16).view(torch.uint16).numpy()
    for vec, ranked in c["q"]:
        qb = torch.tensor([vec], dtype=torch.float32).to(torch.bfloat16).view(torch.uint16).numpy()
        r = oracle.search(xb, qb, k=len(ranked))
        assert r["slots"][0].tolist() == [s for s, _ in ranked]
        assert r["scores"][0].tolist() == [v for _, v in ranked]


def test_normalize_divides_by_both_norms():
    # (3,4) against (5,12): dot 63, norms 5 and 13 -> 63/65; against (-4,3): orthogonal.
    x = np.array([[5, 12], [-4, 3], [6, 8]], dtype=np.float32)
    q = np.array([[3, 4]], dtype=np.float32)
    r = oracle.search(x, q, k=3, normalize=True)
    assert r["slots"][0].tolist() == [2, 0, 1]
    np.testing.assert_allclose(r["scores"][0], [1.0, 63.0 / 65.0, 0.0], atol=1e-6)
    # without normalisation the raw inner products come back
    r = oracle.search(x, q, k=3, normalize=False)
    assert r["slots"][0].tolist() == [0, 2, 1]
    assert r["scores"][0].tolist() == [63.0, 50.0, 0.0]
    # a zero row scores 0 under normalisation instead of dividing by zero
    r = oracle.search(np.zeros((1, 2), np.float32), q, k=1, normalize=True)
    assert r["scores"][0, 0] == 0.0


def test_labels_padding_and_ties():
    x = np.array([[1, 0], [1, 0], [0, 1]], dtype=np.float32)
    ids = np.array([70, 50, 60], dtype=np.int64)
    r = oracle.search(x, np.array([[1, 0]], np.float32), k=5, ids=ids)
    # equal scores: earlier slot first, whatever the labels; tail padded
    assert r["ids"][0].tolist() == [70, 50, 60, -1, -1]
    assert r["slots"][0].tolist() == [0, 1, 2, -1, -1]
    assert r["scores"][0, :3].tolist() == [1.0, 1.0, 0.0]
    assert np.all(np.isneginf(r["scores"][0, 3:]))
    # empty cache
    r = oracle.search(np.zeros((0, 2), np.float32), np.array([[1, 0]], np.float32), k=2)
    assert r["ids"][0].tolist() == [-1, -1]


# ---------------------------------------------------------------- bf16 format

def test_bf16_rounding_known_bit_patterns():
    cases = [
        (1.0, 0x3F80), (-2.5, 0xC020), (0.0, 0x0000),
        (1.0 + 2.0 ** -8, 0x3F80),              # exact tie -> even (down)
        (1.0 + 3 * 2.0 ** -8, 0x3F82),          # exact tie -> even (up)
        (1.0 + 2.0 ** -8 + 2.0 ** -20, 0x3F81),  # just above a tie -> up
        (1.0 + 2.0 ** -8 - 2.0 ** -20, 0x3F80),  # just below a tie -> down
        (float("inf"), 0x7F80), (3.3895313892515355e38, 0x7F7F),   # largest bf16
        (3.4028234663852886e38, 0x7F80),        # fp32 max rounds up to inf
    ]
    vals = np.array([c[0] for c in cases], dtype=np.float32)
    assert oracle.f32_to_bf16_bits(vals).tolist() == [c[1] for c in cases]
    assert oracle.bf16_bits_to_f32(np.array([0x3F80, 0xC020, 0x3F81], np.uint16)).tolist() == \
        [1.0, -2.5, 1.0078125]


def test_bf16_rounding_matches_library_cast():
    g = torch.Generator().manual_seed(5)
    v = torch.randn(4096, generator=g) * torch.logspace(-20, 20, 4096)
    want = v.to(torch.bfloat16).view(torch.uint16).numpy()
    got = oracle.f32_to_bf16_bits(v.numpy())
    assert np.array_equal(got, want)
    back = oracle.bf16_bits_to_f32(got)
    assert np.array_equal(back, v.to(torch.bfloat16).float().numpy())


def test_round_bf16_flag_equals_presupplied_bf16_bits():
    g = torch.Generator().manual_seed(6)
    x = torch.randn(300, 40, generator=g)
    q = torch.randn(3, 40, generator=g)
    a = oracle.search(x.numpy(), q.numpy(), k=7, round_bf16=True, want_all_scores=True)
    b = oracle.search(wl.as_bits(x.to(torch.bfloat16)), wl.as_bits(q.to(torch.bfloat16)), k=7,
                      want_all_scores=True)
    assert np.array_equal(a["all_scores"], b["all_scores"])
    assert np.array_equal(a["slots"], b["slots"])


# ---------------------------------------------------------------- invariants

def _tiny(n=2000, d=96, nq=5, seed=11):
    w = wl.Workload("t", n, d, "f32", (nq,), 8, seed=seed)
    return wl.cache_rows(w).numpy(), wl.queries(w, nq).numpy()


def test_scores_are_cosine_and_sorted():
    x, q = _tiny()
    r = oracle.search(x, q, k=20, want_all_scores=True)
    xd, qd = x.astype(np.float64), q.astype(np.float64)
    cos = (qd @ xd.T) / (np.linalg.norm(qd, axis=1)[:, None] * np.linalg.norm(xd, axis=1)[None, :])
    np.testing.assert_allclose(r["all_scores"], cos, atol=2e-6)
    assert np.all(r["scores"][:, 1:] <= r["scores"][:, :-1])
    assert np.all(np.abs(r["all_scores"]) <= 1.0 + 1e-5)
    # returned scores are the scores of the returned slots
    for i in range(q.shape[0]):
        assert np.array_equal(r["scores"][i], r["all_scores"][i, r["slots"][i]])


def test_duplicate_query_returns_itself_with_score_one():
    x, _ = _tiny()
    picks = [0, 17, 1999]
    r = oracle.search(x, x[picks], k=3)
    assert r["slots"][:, 0].tolist() == picks
    np.testing.assert_allclose(r["scores"][:, 0], 1.0, atol=1e-6)
    assert np.all(r["scores"][:, 1] < 0.9)


def test_k_equals_n_is_a_permutation_and_prefix_property():
    x, q = _tiny(n=257)
    full = oracle.search(x, q, k=257)
    for row in full["slots"]:
        assert sorted(row.tolist()) == list(range(257))
    for k in (1, 2, 31, 256):
        part = oracle.search(x, q, k=k)
        assert np.array_equal(part["slots"], full["slots"][:, :k])
        assert np.array_equal(part["scores"], full["scores"][:, :k])


def test_row_permutation_and_query_scaling():
    x, q = _tiny(n=500)
    base = oracle.search(x, q, k=10)
    perm = np.random.default_rng(3).permutation(500)
    ids = np.arange(500, dtype=np.int64)
    shuffled = oracle.search(x[perm], q, k=10, ids=ids[perm])
    assert np.array_equal(shuffled["ids"], base["ids"])       # labels follow their rows
    assert np.array_equal(shuffled["scores"], base["scores"])
    scaled = oracle.search(x, (q * 4.0).astype(np.float32), k=10, normalize=True)
    normed = oracle.search(x, q, k=10, normalize=True)
    assert np.array_equal(scaled["slots"], normed["slots"])
    np.testing.assert_allclose(scaled["scores"], normed["scores"], atol=1e-6)
    plain = oracle.search(x, (q * 4.0).astype(np.float32), k=10)
    np.testing.assert_allclose(plain["scores"], base["scores"] * 4.0, rtol=1e-6)


def test_merge_identity():
    # top-k(A u B) == top-k(top-k(A) u top-k(B)): what partial lists plus a merge rely on.
    x, q = _tiny(n=1200)
    k = 12
    whole = oracle.search(x, q, k=k)
    a = oracle.search(x[:700], q, k=k)
    b = oracle.search(x[700:], q, k=k)
    for i in range(q.shape[0]):
        cand = [(-s, sl) for s, sl in zip(a["scores"][i], a["slots"][i])]
        cand += [(-s, sl + 700) for s, sl in zip(b["scores"][i], b["slots"][i])]
        cand.sort()
        assert [sl for _, sl in cand[:k]] == whole["slots"][i].tolist()


def test_threads_do_not_change_results():
    x, q = _tiny()
    a = oracle.search(x, q, k=9, threads=1, want_all_scores=True)
    b = oracle.search(x, q, k=9, threads=5, want_all_scores=True)
    assert np.array_equal(a["all_scores"], b["all_scores"])
    assert np.array_equal(a["slots"], b["slots"])


# ---------------------------------------------------------------- library cross-check

def test_tiny_config_against_library_matmul_and_argsort():
    w = wl.WORKLOADS["tiny"]
    x = wl.cache_rows(w).numpy()
    q = wl.queries(w, 16).numpy()
    r = oracle.search(x, q, k=w.k, want_all_scores=True)
    s64 = q.astype(np.float64) @ x.astype(np.float64).T
    np.testing.assert_allclose(r["all_scores"], s64, atol=2e-6)
    lib = np.argsort(-s64, axis=1, kind="stable")[:, :w.k]
    for i in range(16):
        top = np.sort(s64[i])[::-1]
        if np.min(top[:w.k] - top[1:w.k + 1]) > 1e-5:   # no near-tie that fp32 could reorder
            assert lib[i].tolist() == r["slots"][i].tolist()
        assert set(lib[i].tolist()) == set(r["slots"][i].tolist()) or \
            abs(top[w.k - 1] - top[w.k]) <= 1e-5


# ---------------------------------------------------------------- closed-form statistics

def _phi_inv(p):
    return statistics.NormalDist().inv_cdf(p)


def test_gaussian_workload_statistics():
    w = wl.WORKLOADS["tiny"]
    x = wl.cache_rows(w).numpy()
    q = wl.queries(w, 16).numpy()
    np.testing.assert_allclose(np.linalg.norm(x, axis=1), 1.0, atol=1e-5)
    r = oracle.search(x, q, k=w.k, want_all_scores=True)
    s = r["all_scores"]
    assert abs(float(s.mean())) < 3.0 / math.sqrt(w.dim * s.size)
    assert abs(float(s.var()) * w.dim - 1.0) < 0.05
    expect_kth = _phi_inv(1.0 - w.k / w.n) / math.sqrt(w.dim)      # ~0.161
    assert abs(float(np.median(r["scores"][:, -1])) - expect_kth) < 0.02


def test_clustered_workload_structure():
    w = wl.WORKLOADS["clustered"].scaled(20_000)
    x = wl.cache_rows(w)
    q = wl.queries(w, 32, cache=x)
    r = oracle.search(wl.as_bits(x), wl.as_bits(q), k=w.k, want_all_scores=True)
    # planted queries are bit-exact copies of cached rows: best score ~1 (bf16 unit norm)
    np.testing.assert_allclose(r["scores"][:w.planted_queries, 0], 1.0, atol=4e-3)
    # in-cluster cosine ~ 1/(1+sigma^2) for the others
    inc = r["scores"][w.planted_queries:, 0]
    assert abs(float(np.median(inc)) - 1.0 / (1.0 + w.sigma ** 2)) < 0.02
    # exact duplicates exist and score identically
    xb = wl.as_bits(x)
    _, counts = np.unique(xb, axis=0, return_counts=True)
    assert counts.max() >= 2 and abs((counts - 1).sum() - 0.01 * w.n) < 0.003 * w.n


# ---------------------------------------------------------------- the acceptance rule itself

def test_acceptance_rule_catches_planted_mistakes():
    x, q = _tiny(n=3000, d=64)
    k = 8
    r = oracle.search(x, q, k=k, want_all_scores=True)
    ok = accept(r["ids"], r["scores"], r["all_scores"], k, tol=1e-4)
    assert ok["max_abs_err"] == 0.0
    bad = r["scores"].copy(); bad[0, 3] += 0.05
    with pytest.raises(AcceptanceError):
        accept(r["ids"], bad, r["all_scores"], k)
    # an id far below the k-th place
    worst = int(np.argmin(r["all_scores"][1]))
    ids2 = r["ids"].copy(); sc2 = r["scores"].copy()
    ids2[1, -1] = worst; sc2[1, -1] = r["all_scores"][1, worst]
    with pytest.raises(AcceptanceError):
        accept(ids2, sc2, r["all_scores"], k)
    # a repeated entry
    ids3 = r["ids"].copy(); ids3[2, 1] = ids3[2, 0]
    sc3 = r["scores"].copy(); sc3[2, 1] = sc3[2, 0]
    with pytest.raises(AcceptanceError):
        accept(ids3, sc3, r["all_scores"], k)
    # ascending instead of descending
    with pytest.raises(AcceptanceError):
        accept(r["ids"][:, ::-1], r["scores"][:, ::-1], r["all_scores"], k)
    # scores computed with the last 8 of 64 dimensions dropped pass a loose tolerance at
    # most, never the strict one
    trunc = oracle.search(np.ascontiguousarray(x[:, :56]), np.ascontiguousarray(q[:, :56]), k=k)
    with pytest.raises(AcceptanceError):
        accept(trunc["ids"], trunc["scores"], r["all_scores"], k, tol=1e-4)
    # labels
    lab = wl.labels(3000).numpy()
    rl = oracle.search(x, q, k=k, ids=lab)
    accept(rl["ids"], rl["scores"], r["all_scores"], k, ids=lab, tol=1e-4)
    with pytest.raises(AcceptanceError):
        accept(r["ids"], r["scores"], r["all_scores"], k, ids=lab, tol=1e-4)


# ---------------------------------------------------------------- similarity threshold

def test_min_score_filter_hand_computed():
    c = _parse_golden()["axes"]
    x = np.array(c["x"], dtype=np.float32)
    q = np.array([[1, 0], [0, 1], [0.6, 0.8]], dtype=np.float32)
    r = oracle.search(x, q, k=4, min_score=0.7)
    # from the golden file: q0 -> 0:1, 4:0.8 | q1 -> 1:1, 3:0.8 | q2 -> 3:1, 1:0.8 (0.6 and below drop)
    assert r["counts"].tolist() == [2, 2, 2]
    assert r["slots"].tolist() == [[0, 4, -1, -1], [1, 3, -1, -1], [3, 1, -1, -1]]
    assert np.all(np.isneginf(r["scores"][:, 2:]))
    np.testing.assert_allclose(r["scores"][:, :2], [[1, 0.8], [1, 0.8], [1, 0.8]], atol=1e-6)
    # a threshold exactly at a score keeps it; above every score keeps nothing; -inf keeps all
    assert oracle.search(x, q[:1], k=5, min_score=1.0)["counts"].tolist() == [1]
    assert oracle.search(x, q[:1], k=5, min_score=1.5)["counts"].tolist() == [0]
    assert oracle.search(x, q[:1], k=7, min_score=-np.inf)["counts"].tolist() == [5]


# ---------------------------------------------------------------- similarity to the other entries

def test_self_similarity_hand_computed_and_against_search():
    c = _parse_golden()["axes"]
    x = np.array(c["x"], dtype=np.float32)
    r = oracle.self_similarity(x)
    assert r["slots"].tolist() == [c["self"][i][0] for i in range(5)]
    np.testing.assert_allclose(r["scores"], [c["self"][i][1] for i in range(5)], atol=1e-6)
    # a row's best other row is the first entry of its own top-2 that is not the row itself
    xs, _ = _tiny(n=700, d=48)
    xs[13] = xs[400]                      # an exact duplicate pair: each is the other's best
    full = oracle.search(xs, xs, k=2)
    want = [row[0] if row[0] != i else row[1] for i, row in enumerate(full["slots"])]
    got = oracle.self_similarity(xs, threads=3)
    assert got["slots"].tolist() == want and got["slots"][13] == 400 and got["slots"][400] == 13
    part = oracle.self_similarity(xs, first=100, count=50, ids=np.arange(700, dtype=np.int64) + 7)
    assert part["ids"].tolist() == [w + 7 for w in want[100:150]]
    one = oracle.self_similarity(xs[:1])
    assert one["slots"].tolist() == [-1] and np.isneginf(one["scores"][0])
