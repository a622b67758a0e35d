"""Checkpoint and restore through the C ABI: a restored cache answers exactly as the saved one."""
import pytest
import torch

from paper_2501_12689_b200 import ICCache, ICCacheError, IC_ERR_INVALID, workloads as wl

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def test_save_and_load_round_trip(tmp_path):
    w = wl.Workload("g", 30_011, 128, "bf16", (9,), 12, seed=501)
    x, q = wl.cache_rows(w, DEV), wl.queries(w, 9, DEV)
    ids = wl.labels(w.n, DEV)
    path = str(tmp_path / "cache.ckpt")
    with ICCache(w.dim, w.n) as a:
        a.insert(x, ids)
        a.utility_add(ids[:5].cpu(), torch.tensor([1.0, 2.0, 3.0, 4.0, 5.0]))
        a.utility_decay(0.9)
        want_ids, want_sc = a.query(q, w.k)
        want_util = a.utility_read()
        a.save(path)
    with ICCache(w.dim, w.n + 100) as b:                       # a larger capacity is fine
        b.insert(x[:7], ids[:7])                               # previous contents are replaced
        b.build_index(2, 1)
        b.load(path)
        assert b.size == w.n and b.index_info() == (0, 0)
        got_ids, got_sc = b.query(q, w.k)
        b.sync()
        assert torch.equal(got_ids, want_ids) and torch.equal(got_sc, want_sc)
        got_util = b.utility_read()
        assert torch.equal(got_util[0], want_util[0]) and torch.equal(got_util[1], want_util[1])
        b.insert(x[:50], wl.labels(50, DEV, first_slot=w.n))   # and it keeps working as a cache
        assert b.size == w.n + 50
    # a checkpoint without utilities clears the ones the handle had
    with ICCache(w.dim, 64) as c:
        c.insert(x[:64], ids[:64])
        c.save(path)
        c.utility_add(ids[:1].cpu(), torch.tensor([7.0]))
        c.load(path)
        assert not c.utility_read()[1].any()


def test_load_rejects_foreign_and_mismatching_files(tmp_path):
    path = str(tmp_path / "cache.ckpt")
    x = torch.zeros(20, 64, dtype=torch.bfloat16, device=DEV)
    with ICCache(64, 20) as a:
        a.insert(x, torch.arange(20, device=DEV))
        a.save(path)
    for dim, cap in ((128, 20), (64, 19)):                     # other dimension, too little room
        with ICCache(dim, cap) as b:
            with pytest.raises(ICCacheError) as e:
                b.load(path)
            assert e.value.status == IC_ERR_INVALID
    junk = str(tmp_path / "junk.bin")
    open(junk, "wb").write(b"not a checkpoint at all" * 10)
    with ICCache(64, 20) as b:
        for bad in (junk, str(tmp_path / "missing.ckpt")):
            with pytest.raises(ICCacheError):
                b.load(bad)
        assert b.size == 0
    # a truncated file leaves the handle empty
    data = open(path, "rb").read()
    open(path, "wb").write(data[: len(data) // 2])
    with ICCache(64, 20) as b:
        b.insert(x[:3], torch.arange(3, device=DEV))
        with pytest.raises(ICCacheError):
            b.load(path)
        assert b.size == 0
