"""GPU parity of the per-entry utility side array (the cache manager's moving average of each
example's gain) against the plain CPU definition, through the C ABI: bit-exact fp32."""
import numpy as np
import pytest
import torch

import oracle
from paper_2501_12689_b200 import ICCache, ICCacheError, workloads as wl

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def test_utility_add_decay_read_and_removal():
    n, dim = 5_000, 64
    w = wl.Workload("g", n, dim, "bf16", (4,), 8, seed=401)
    x = wl.cache_rows(w, DEV)
    ids = wl.labels(n, "cpu")
    ids[77] = ids[11]                                   # two entries share an id: both are credited
    rng = np.random.default_rng(7)
    with ICCache(dim, n + 100) as c:
        c.insert(x[:4_000], ids[:4_000].to(DEV))
        got_ids, got_u = c.utility_read()               # before any update everything is zero
        assert torch.equal(got_ids, ids[:4_000]) and not got_u.any()
        c.utility_decay(0.9)                            # no-op on zeros
        ref = np.zeros(4_000, dtype=np.float32)
        for step in range(6):
            pick = rng.integers(0, 4_000, 300)
            pick[:3] = [11, 11, 77]                     # the same id several times in one call
            add_ids = ids[pick].clone()
            add_ids[5] = 123                            # an id nobody carries
            gains = torch.tensor(rng.random(300).astype(np.float32) * 3)
            c.utility_add(add_ids, gains)
            ref = oracle.utility_add(ids[:4_000].numpy(), ref, add_ids.numpy(), gains.numpy())
            if step % 2:
                c.utility_decay(0.9)
                ref = oracle.utility_decay(ref, 0.9)
        _, got_u = c.utility_read()
        assert np.array_equal(got_u.numpy(), ref)       # one fp32 operation per update on both sides
        # entries inserted later start at zero
        c.insert(x[4_000:], ids[4_000:].to(DEV))
        _, got_u = c.utility_read()
        assert np.array_equal(got_u.numpy()[:4_000], ref) and not got_u[4_000:].any()
        ref = np.concatenate([ref, np.zeros(1_000, dtype=np.float32)])
        # utilities travel with their entries when a removal closes gaps
        gone = ids[[3, 500, 501, 4_999]].clone()
        assert c.remove(gone) == 4
        left_ids, left_u = c.utility_read()
        keep = ~np.isin(ids.numpy(), gone.numpy())
        assert sorted(left_ids.tolist()) == sorted(ids.numpy()[keep].tolist())
        by_id = {}
        for i, u in zip(ids.numpy()[keep].tolist(), ref[keep].tolist()):
            by_id.setdefault(i, []).append(u)
        got = {}
        for i, u in zip(left_ids.tolist(), left_u.tolist()):
            got.setdefault(i, []).append(u)
        assert {k: sorted(v) for k, v in got.items()} == {k: sorted(v) for k, v in by_id.items()}


def test_utility_argument_errors():
    with ICCache(64, 16) as c:
        c.insert(torch.zeros(4, 64, dtype=torch.bfloat16, device=DEV), torch.arange(4, device=DEV))
        with pytest.raises(ICCacheError):
            c.utility_decay(-0.1)
        with pytest.raises(ICCacheError):
            c.utility_decay(float("nan"))
        with pytest.raises(ICCacheError):
            c.utility_add(torch.tensor([1]), torch.tensor([float("inf")]))
        c.utility_add(torch.tensor([], dtype=torch.int64), torch.tensor([], dtype=torch.float32))
        c.utility_add(torch.tensor([2]), torch.tensor([1.5]))
        assert c.utility_read()[1].tolist() == [0.0, 0.0, 1.5, 0.0]
