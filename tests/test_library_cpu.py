"""Host-side checks that need no GPU: the C-ABI library builds, loads and exports every symbol the
header declares; size helpers; loud failure without a device; multi-rank aggregation (gloo)."""
import ctypes
import os
import re
import subprocess
import sys

import pytest
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    from paper_2605_26632_b200 import binding

    lib = binding.load_library()
    header = open(os.path.join(ROOT, "include", "lynx.h")).read()
    declared = set(re.findall(r"LYNX_API\s+[\w\s\*]+?\b(lynx_\w+)\s*\(", header))
    assert declared, "no declarations parsed"
    assert declared == set(binding.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


def test_size_helpers():
    from paper_2605_26632_b200 import binding

    assert binding.values_bytes(4096, 12288) == 4096 * 6144 * 2
    assert binding.meta_bytes(4096, 12288) == 4096 * 12288 // 8
    assert binding.meta_bytes(200, 384) == 2 * 3 * 2048  # padded to 128 rows
    assert binding.meta_bytes(1, 128) == 2048
    lib = binding.load_library()
    assert lib.lynx_workspace_bytes(256, 512, 512) >= 256 * 256 * 2 + 2 * 4 * 2048 + 256 * 4


def test_two_row_tile_schedule_covers_every_tile_exactly_once():
    """Host logic of the GEMM's work distribution: for any number of row tiles, column tiles,
    CTA pairs and 512-row items, every 256 x 240 tile is computed exactly once, doubles pair the
    row tiles 2d / 2d + 1, consecutive single-tile items of a pair alternate accumulators, and
    the pairs' loads differ by at most one item of each kind."""
    from paper_2605_26632_b200 import binding

    import itertools
    import random

    rng = random.Random(0)
    cases = [(16, 13, 74, 74), (16, 13, 74, 0), (16, 13, 74, 104), (17, 13, 74, 80), (3, 5, 74, 5), (3, 5, 4, 2),
             (1, 7, 74, 0), (64, 13, 74, 300), (19, 5, 74, 45), (47, 5, 74, 115), (2, 1, 74, 1)]
    cases += [(rng.randint(1, 40), rng.randint(1, 30), rng.randint(1, 74), rng.randint(0, 700)) for _ in range(60)]
    for tm, tn, pairs, doubles in cases:
        dmax = (tm // 2) * tn
        d_eff = min(doubles, dmax)
        clusters = max(1, min(pairs, tm * tn - d_eff))
        seen = {}
        nd, ns = [], []
        for c in range(clusters):
            items = binding.gemm_schedule_items(tm, tn, clusters, doubles, c)
            singles = [it for it in items if it[2] == 1]
            assert [it[3] for it in singles] == list(range(len(singles)))  # ordinals 0, 1, 2, ...
            assert all(it[2] == 2 for it in items[:len(items) - len(singles)])  # doubles first
            for (m0, n, rows, _) in items:
                assert rows in (1, 2) and 0 <= n < tn
                if rows == 2:
                    assert m0 % 2 == 0 and m0 + 1 < tm
                for r in range(rows):
                    assert 0 <= m0 + r < tm
                    seen[(m0 + r, n)] = seen.get((m0 + r, n), 0) + 1
            nd.append(len(items) - len(singles))
            ns.append(len(singles))
        assert len(seen) == tm * tn and set(seen.values()) == {1}, (tm, tn, pairs, doubles)
        assert sum(nd) == d_eff
        assert max(nd) - min(nd) <= 1
        # a pair with one double fewer never has fewer singles than a pair with one double more
        light = [s_ for d_, s_ in zip(nd, ns) if d_ == min(nd)]
        heavy = [s_ for d_, s_ in zip(nd, ns) if d_ == max(nd)]
        if max(nd) != min(nd):
            assert min(light) >= max(heavy)
        assert max(light) - min(light) <= 1 and max(heavy) - min(heavy) <= 1


def test_gemm_plan_prefers_single_tiles_for_small_problems():
    from paper_2605_26632_b200 import binding

    use, d, c = binding.gemm_plan(148, 1024, 3072, 3072)
    assert d == 0 or not use  # 52 tiles on 74 pairs: pairing row tiles would only serialise them
    use, d, c = binding.gemm_plan(148, 4096, 3072, 12288)
    assert c == 74 and 0 <= d <= 8 * 13


def test_status_strings():
    from paper_2605_26632_b200 import binding

    assert binding.status_string(0) == "ok"
    assert "128" in binding.status_string(2)
    assert "sm_100" in binding.status_string(7)


@pytest.mark.skipif(torch.cuda.is_available(), reason="checks the no-GPU failure path")
def test_no_gpu_means_loud_failure_not_fallback():
    from paper_2605_26632_b200 import binding

    with pytest.raises(binding.LynxError):
        binding.Lynx(0)


def test_product_never_imports_the_oracle():
    pkg = os.path.join(ROOT, "paper_2605_26632_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                for needle in ("import oracle", "from oracle", "liblynx_oracle", "lynx_oracle.c", "oracle_"):
                    assert needle not in text, f"{f} reaches into the oracle ({needle})"
    for f in os.listdir(os.path.join(ROOT, "oracle")):
        if f.endswith((".py", ".c")):
            text = open(os.path.join(ROOT, "oracle", f)).read()
            assert "paper_2605_26632_b200" not in text and "liblynx.so" not in text


_WORKER = r"""
import os, sys
sys.path.insert(0, {root!r})
import torch.distributed as dist
import bench
rank = int(os.environ["RANK"]); world = int(os.environ["WORLD_SIZE"])
dist.init_process_group("gloo")
ms = bench.max_over_ranks(10.0 + 5.0 * rank, world, device="cpu")
assert ms == 15.0, ms
v = bench.aggregate_tflops(1e12, 10, ms, world)
assert abs(v - 1e12 * 10 * 2 / 15e-3 / 1e12) < 1e-9, v
dist.barrier(); dist.destroy_process_group()
print("ok", rank)
"""


def test_replica_aggregation_two_ranks_gloo(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(_WORKER.format(root=ROOT))
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT="29611", WORLD_SIZE="2")
    procs = [subprocess.Popen([sys.executable, str(script)], env=dict(env, RANK=str(r)),
                              stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True) for r in range(2)]
    outs = [p.communicate(timeout=120)[0] for p in procs]
    for p, o in zip(procs, outs):
        assert p.returncode == 0, o


def test_bench_launches_its_own_ranks_when_started_plainly():
    """``python bench.py --gpus 2`` without torchrun starts two ranks itself (127.0.0.1 rendezvous);
    checked through the GPU-free launch check: gloo ranks, max-over-ranks and aggregation."""
    import json

    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK")}
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--launch-check"],
                         env=env, capture_output=True, text=True, timeout=300)
    assert res.returncode == 0, res.stderr[-2000:]
    line = [l for l in res.stdout.splitlines() if l.startswith("{")][-1]
    d = json.loads(line)
    assert d["launch_check"] and d["n_gpus"] == 2 and d["slowest_rank_ms"] == 15.0
    assert abs(d["aggregate_tflops"] - 1e12 * 10 * 2 / 15e-3 / 1e12) < 1e-6
