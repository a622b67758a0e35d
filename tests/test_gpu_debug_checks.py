"""The debug build of the library (libic_cache_debug.so: the same kernels compiled with
-DIC_CACHE_DEBUG_CHECKS) checks tile, list and slot indices on the device and reports a failed check
through the status word instead of trapping.  This test runs every kernel path through it, in a child
process (the binding loads one library per process), and requires that no check fires and that the
results are bit-identical to the normal build's."""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r"""
import hashlib, json, sys
sys.path.insert(0, %(root)r)
import torch
from paper_2501_12689_b200 import ICCache, IC_PATH_AUTO, IC_PATH_SCAN, IC_PATH_UMMA, workloads as wl
dev = "cuda:0"
out = {}
def digest(*tensors):
    h = hashlib.sha256()
    for t in tensors:
        h.update(t.cpu().contiguous().numpy().tobytes())
    return h.hexdigest()
cases = [("scan", 50_001, 384, 2, 10, IC_PATH_SCAN), ("resident", 70_001, 768, 33, 10, IC_PATH_UMMA),
         ("streamed", 70_001, 768, 100, 16, IC_PATH_UMMA), ("pairs-seeded", 400_003, 64, 250, 64, IC_PATH_AUTO),
         ("ragged-small", 4_097, 40, 5, 128, IC_PATH_UMMA)]
for name, n, dim, nq, k, path in cases:
    w = wl.Workload("d", n, dim, "bf16", (nq,), k, seed=900 + n %% 97)
    with ICCache(dim, n) as c:
        c.set_path(path)
        c.insert(wl.cache_rows(w, dev), wl.labels(n, dev))
        ids, sc = c.query(wl.queries(w, nq, dev), k)
        c.sync()            # raises if a kernel wrote the status word
        out[name] = digest(ids, sc)
w = wl.WORKLOADS["clustered"].scaled(120_000)
with ICCache(w.dim, w.n) as c:
    c.insert(wl.cache_rows(w, dev), wl.labels(w.n, dev))
    c.build_index(0, 2)
    ids, sc = c.query_clustered(wl.queries(w, 40, dev), w.k, 4)
    c.sync()
    out["two-level"] = digest(ids, sc)
    ids, sc = c.self_similarity(0, 3000)
    c.sync()
    out["self-similarity"] = digest(ids, sc)
print("RESULT " + json.dumps(out))
"""


def _run(lib):
    env = dict(os.environ)
    if lib:
        env["IC_CACHE_LIB"] = lib
    else:
        env.pop("IC_CACHE_LIB", None)
    r = subprocess.run([sys.executable, "-c", CHILD % {"root": ROOT}], env=env, capture_output=True, text=True, timeout=900)
    assert r.returncode == 0, r.stdout[-2000:] + r.stderr[-4000:]
    line = [ln for ln in r.stdout.splitlines() if ln.startswith("RESULT ")][-1]
    return json.loads(line[len("RESULT "):])


def test_debug_build_checks_stay_silent_and_results_match():
    from paper_2501_12689_b200.build import LIB_DEBUG, build
    if not os.path.exists(LIB_DEBUG):
        build(debug_checks=True)
    checked = _run(LIB_DEBUG)
    plain = _run(None)
    assert checked == plain
