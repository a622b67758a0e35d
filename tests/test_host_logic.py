"""CPU-only checks: the shared library loads and exports every symbol the header declares,
argument validation and launch planning work without a GPU, and the benchmark's cross-rank
aggregation is right on a two-process gloo group."""
import json
import os
import re
import subprocess
import sys

import pytest

import paper_2501_12689_b200 as pkg
from paper_2501_12689_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "ic_cache.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ic_cache_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    from paper_2501_12689_b200.build import build
    build()
    lib = pkg.load_library()
    names = _declared_symbols()
    assert "ic_cache_create" in names and "ic_cache_query" in names and len(names) >= 15
    for name in names:
        assert hasattr(lib, name), f"{name} is declared in ic_cache.h but not exported"
        assert name in binding.SIGNATURES, f"{name} has no Python binding signature"
    assert lib.ic_cache_version() >= 100


def test_debug_build_exports_the_same_symbols():
    """The debug build (index checks compiled in) is the same ABI: it builds without a GPU and
    exports every declared symbol."""
    import ctypes
    from paper_2501_12689_b200.build import build
    lib = ctypes.CDLL(build(debug_checks=True))
    for name in _declared_symbols():
        assert hasattr(lib, name), f"{name} is missing from the debug build"


def test_header_constants_match_binding():
    text = open(os.path.join(ROOT, "include", "ic_cache.h")).read()
    assert int(re.search(r"#define IC_MAX_K (\d+)", text).group(1)) == binding.IC_MAX_K
    assert int(re.search(r"#define IC_MAX_DIM (\d+)", text).group(1)) == binding.IC_MAX_DIM
    for name in ("IC_ERR_INVALID", "IC_ERR_NOMEM", "IC_ERR_FULL", "IC_ERR_CUDA", "IC_ERR_UNSUPPORTED", "IC_ERR_TIMEOUT"):
        assert int(re.search(name + r" = (-\d+)", text).group(1)) == getattr(binding, name)


def test_plan_paths_and_shapes():
    p = pkg.ic_cache_plan(768, 1_000_000, 1, 10)
    assert p["path"] == pkg.IC_PATH_SCAN and p["query_tile"] == 1 and p["n_ctas"] == 148 and p["n_stages"] >= 2
    p = pkg.ic_cache_plan(768, 1_000_000, 2, 10)
    assert p["path"] == pkg.IC_PATH_SCAN and p["query_tile"] == 2 and p["n_launches"] == 1
    p = pkg.ic_cache_plan(768, 1_000_000, 4, 10, path=pkg.IC_PATH_SCAN)
    assert p["query_tile"] == 4 and p["n_launches"] == 1
    assert pkg.ic_cache_plan(768, 1_000_000, 4, 10)["path"] == pkg.IC_PATH_UMMA
    p = pkg.ic_cache_plan(768, 1_000_000, 64, 10)
    assert p["path"] == pkg.IC_PATH_UMMA and p["n_query_tiles"] == 1 and p["n_partitions"] == 148
    p = pkg.ic_cache_plan(1024, 4_000_000, 256, 32)
    assert p["n_query_tiles"] == 2 and p["n_partitions"] == 74 and p["n_ctas"] == 148
    p = pkg.ic_cache_plan(768, 16_000_000, 1024, 64)
    assert p["n_query_tiles"] == 8 and p["n_partitions"] == 18 and p["n_ctas"] == 144 and p["n_launches"] == 2
    # 24 tiles (a ninth of the sampling launch's 217 per CTA pair) for each of 18 partitions
    assert p["cta_group"] == 2 and p["seed0_tiles"] == 432 < p["seed_tiles"] and p["query_resident"] == 0
    assert p["smem_bytes"] <= 232448
    assert p["seed_tiles"] > 0 and p["seed_tiles"] % 18 == 0 and p["seed_tiles"] * 256 * 15 < 16_000_000
    assert pkg.ic_cache_plan(768, 70_001, 64, 10)["seed_tiles"] == 0      # too few tiles per CTA
    assert pkg.ic_cache_plan(768, 70_001, 64, 10)["seed0_tiles"] == 0
    # threshold seeding: inside the scoring launch, from the first tile of every partition; a
    # list-level sample of 1/16 of the tiles, in a launch of its own, only on large caches
    p = pkg.ic_cache_plan(768, 1_000_000, 64, 10)
    assert (p["seed0_tiles"], p["seed_tiles"], p["n_launches"]) == (148, 0, 1)
    p = pkg.ic_cache_plan(768, 16_000_000, 64, 64)
    assert p["seed0_tiles"] == 148 and p["seed_tiles"] == 16_000_000 // 256 // 16 // 148 * 148
    p = pkg.ic_cache_plan(1024, 4_000_000, 256, 32)
    assert p["seed0_tiles"] == 148 and p["seed_tiles"] % 74 == 0 and p["seed_tiles"] > 148
    # the exchanged sample stays at about one tile per SM however few partitions there are
    assert pkg.ic_cache_plan(768, 40_000, 1024, 128)["seed0_tiles"] == 144      # 8 tiles for each of 18 partitions
    # batches of at most 64 queries keep the query tile in shared memory (M = 64) while a ring of
    # four 16 KiB stages still fits beside it
    p = pkg.ic_cache_plan(768, 1_000_000, 64, 10)
    assert p["query_resident"] == 1 and p["query_tile"] == 64 and p["n_stages"] >= 6 and p["smem_bytes"] <= 232448
    assert pkg.ic_cache_plan(768, 1_000_000, 65, 10)["query_resident"] == 0
    assert pkg.ic_cache_plan(768, 16_000_000, 64, 64)["query_resident"] == 1
    assert pkg.ic_cache_plan(2048, 1_000_000, 8, 10)["query_resident"] == 0      # 256 KiB of queries do not fit
    for dim in (8, 384, 768, 1024, 1536, 4096):
        for nq in (1, 64, 128, 1024):
            for k in (1, 10, 64, 128):
                p = pkg.ic_cache_plan(dim, 1_000_000, nq, k, path=pkg.IC_PATH_UMMA)
                assert p["smem_bytes"] <= 232448 and p["n_stages"] >= 2 and p["queue_cap"] >= 1
    p = pkg.ic_cache_plan(768, 16_000_000, 3000, 64)
    assert p["n_launches"] == 6
    assert pkg.ic_cache_plan(768, 1_000_000, 300, 10)["cta_group"] == 1    # odd number of query tiles
    p = pkg.ic_cache_plan(2048, 1000, 2, 5)          # too wide for the scan path
    assert p["path"] == pkg.IC_PATH_UMMA
    p = pkg.ic_cache_plan(64, 1000, 6, 128, path=pkg.IC_PATH_GENERIC)
    assert p["n_launches"] == 2 and p["n_partitions"] * 128 * 8 < 232448
    for k in (1, 10, 64, 128):                       # every k leaves at least two ring stages
        assert pkg.ic_cache_plan(4096, 10, 128, k)["n_stages"] >= 2


def test_workspace_bytes_covers_every_batch_shape_up_to_the_limits():
    # pure host arithmetic (B200 figures without a device): enough for the largest batch of every
    # query-tile count, growing with the limits, zero for bad arguments
    small = pkg.ic_cache_workspace_bytes(768, 1_000_000, 64, 10)
    big = pkg.ic_cache_workspace_bytes(768, 1_000_000, 1024, 64)
    assert 0 < small < big < (1 << 30)
    assert pkg.ic_cache_workspace_bytes(768, 1_000_000, 5000, 64) == big       # windows of 1024 queries
    assert pkg.ic_cache_workspace_bytes(768, 16_000_000, 64, 10) >= small      # more seeding tiles at most
    # query staging alone: bf16 padded to 128 rows plus fp32
    assert small >= 128 * 768 * 2 + 64 * 768 * 4
    for bad in [(12, 10, 1, 1), (768, 0, 1, 1), (768, 10, 0, 1), (768, 10, 1, 0), (768, 10, 1, 129)]:
        assert pkg.ic_cache_workspace_bytes(*bad) == 0


@pytest.mark.parametrize("args", [
    dict(dim=12, n=10, nq=1, k=1), dict(dim=0, n=10, nq=1, k=1), dict(dim=8192, n=10, nq=1, k=1),
    dict(dim=64, n=10, nq=0, k=1), dict(dim=64, n=10, nq=1, k=0), dict(dim=64, n=10, nq=1, k=129),
    dict(dim=64, n=-1, nq=1, k=1), dict(dim=64, n=10, nq=1, k=1, path=9),
])
def test_plan_rejects_bad_arguments(args):
    with pytest.raises(pkg.ICCacheError) as e:
        pkg.ic_cache_plan(**args)
    assert e.value.status == pkg.IC_ERR_INVALID and str(e.value)


def test_forced_scan_path_rejects_wide_rows():
    with pytest.raises(pkg.ICCacheError) as e:
        pkg.ic_cache_plan(2048, 10, 1, 1, path=pkg.IC_PATH_SCAN)
    assert e.value.status == pkg.IC_ERR_UNSUPPORTED


def test_create_fails_loudly_without_a_gpu_or_with_bad_arguments():
    import torch
    lib = pkg.load_library()
    assert not lib.ic_cache_create(12, 10) and b"multiple of 8" in lib.ic_cache_last_error()
    assert not lib.ic_cache_create(64, 0) and b"capacity" in lib.ic_cache_last_error()
    if not torch.cuda.is_available():
        assert not lib.ic_cache_create(64, 10)
        assert b"no CPU fallback" in lib.ic_cache_last_error()
    # NULL handles are rejected, destroy(NULL) is a no-op
    assert lib.ic_cache_size(None) == pkg.IC_ERR_INVALID
    assert lib.ic_cache_insert(None, None, None, 1) == pkg.IC_ERR_INVALID
    assert lib.ic_cache_query(None, None, 1, 1, None, None) == pkg.IC_ERR_INVALID
    lib.ic_cache_destroy(None)


def test_two_rank_gloo_aggregation():
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
           "--master-addr", "127.0.0.1", "--master-port", "29531", os.path.join(ROOT, "tests", "_gloo_worker.py")]
    r = subprocess.run(cmd, capture_output=True, text=True, timeout=240, cwd=ROOT)
    assert r.returncode == 0, r.stdout + r.stderr
    assert "AGGREGATE_OK 15.0 3000.0" in r.stdout


def test_reference_arm_runs_the_oracle_and_prints_the_contract_line():
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "tiny",
                        "--steps", "2", "--warmup", "1"], capture_output=True, text=True, timeout=240, cwd=ROOT)
    assert r.returncode == 0, r.stderr
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["unit"] == "queries/s" and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0
