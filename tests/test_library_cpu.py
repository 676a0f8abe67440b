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
