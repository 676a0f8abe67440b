#!/usr/bin/env python
"""Benchmark of the 2:4 activation-sparse linear layer (prune/compress + sparse GEMM + epilogue).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

One "step" is one pass of the whole hot path over one batch of synthetic activations: one call of
``lynx_act_sparse_linear`` in its two-kernel mode = the prune/compress launch (Top-2-of-4
selection, compression, row sums of the norm-compensation scale) followed by the tcgen05 sparse
GEMM launch (scale + bias epilogue).  Prints ONE JSON line.

* ``value``   dense-equivalent TFLOP/s (2*M*N*K per step) with inputs resident in HBM.
* ``e2e``     same metric through ``lynx_act_sparse_linear_host`` (pinned host X in, host Y out).
* ``roofline`` for the dominant kernel (the sparse GEMM), timed live with CUDA events around each
  launch in a second loop of the same steps issued as two calls; ``roofline_prune`` for the
  HBM-bound prune/compress kernel.
* ``cpu_baseline`` the CPU oracle, as it stands, on a bounded sample of rows of the same workload.
* ``sustained`` the same step, the sparse GEMM alone and the dense linear again in interleaved blocks
  of >= 0.5 s each (seconds of tensor-core work: the GPU settles at its power-capped clocks), with
  the clocks seen in each leg (``--no-sustained`` skips it).
* ``sweep``   every other configuration the metric names (attention projections, mlp.up with the
  one-kernel variant beside it, the 16 shapes of the token sweep): prune, GEMM, layer and dense
  linear, a few milliseconds each (``--no-sweep`` skips it).
* ``--impl reference`` times the CPU oracle only (there is no other reference implementation).

Multi-GPU (``--gpus N``): the path does not shard; every rank runs an independent replica on its
own GPU and the aggregate is reported ("replicas only", weak scaling).  Under torchrun the ranks
come from the environment; started plainly with ``--gpus N`` (N > 1) the script launches its own N
ranks through ``torch.distributed.run`` on 127.0.0.1.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "2:4-act linear TFLOP/s (dense-equiv) and speedup vs dense bf16 GEMM, 1xB200"
UNIT = "TFLOP/s"



def ncu_traffic_bytes(wl, num_sms: int):
    """dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel on this
    workload, as recorded from its profiler capture in ncu_traffic.json next to the capture
    summaries.  None when no capture is recorded, or when the library would now run the GEMM
    differently (other kernel or schedule) than it did when the capture was taken."""
    from paper_2605_26632_b200 import binding

    path = os.path.join(ROOT, "profiles", "ncu_traffic.json")
    try:
        with open(path) as f:
            rec = json.load(f).get("sparse_gemm", {}).get(wl.name)
        if not rec:
            return None
        use, doubles, clusters = binding.gemm_plan(num_sms, wl.M, wl.N, wl.K)
        now = {"two_row_tile_kernel": bool(use), "doubles": int(doubles), "clusters": int(clusters)}
        return int(rec["bytes"]) if rec.get("plan") == now else None
    except (OSError, ValueError, KeyError):
        return None


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="mlp_down")
    ap.add_argument("--comp", default="row", choices=["none", "row", "tensor"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-lora", action="store_true", help="skip the extra measurement of the layer with the low-rank branch")
    ap.add_argument("--no-fp8", action="store_true", help="skip the extra measurement of the layer on FP8 operands")
    ap.add_argument("--no-sustained", action="store_true", help="skip the seconds-long interleaved legs")
    ap.add_argument("--no-sweep", action="store_true", help="skip the other configurations (attention projections, mlp.up, token sweep)")
    ap.add_argument("--launch-check", action="store_true",
                    help="only check the multi-rank launch and aggregation on the CPU (gloo): no GPU work")
    return ap.parse_args()


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"],
                "bf16_tflops_sustained": p.get("bf16_tflops_sustained", p["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clock, power and throttle reasons through NVML every few milliseconds while the
    timed region runs (nvidia-smi's 100 ms loop is too coarse for a region of a few milliseconds)."""

    # nvmlClocksEventReasons bits
    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown"}

    def __init__(self, index: int, period_s: float = 0.002):
        self.index = index
        self.period = period_s
        self.samples = []  # (time, sm_mhz, power_w, reasons_mask)
        self.max_mhz = None
        self._stop = threading.Event()
        self._thread = threading.Thread(target=self._run, daemon=True)

    def _run(self):
        try:
            import pynvml

            pynvml.nvmlInit()
            # NVML enumerates physical devices; honour CUDA_VISIBLE_DEVICES when it lists indices
            phys = self.index
            vis = os.environ.get("CUDA_VISIBLE_DEVICES")
            if vis:
                ids = [v for v in vis.split(",") if v.strip() != ""]
                if self.index < len(ids) and ids[self.index].strip().isdigit():
                    phys = int(ids[self.index])
            h = pynvml.nvmlDeviceGetHandleByIndex(phys)
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(h, pynvml.NVML_CLOCK_SM))
            while not self._stop.is_set():
                mhz = float(pynvml.nvmlDeviceGetClockInfo(h, pynvml.NVML_CLOCK_SM))
                try:
                    pw = pynvml.nvmlDeviceGetPowerUsage(h) / 1000.0
                except Exception:
                    pw = float("nan")
                try:
                    mask = int(pynvml.nvmlDeviceGetCurrentClocksEventReasons(h))
                except Exception:
                    try:
                        mask = int(pynvml.nvmlDeviceGetCurrentClocksThrottleReasons(h))
                    except Exception:
                        mask = 0
                self.samples.append((time.time(), mhz, pw, mask))
                time.sleep(self.period)
        except Exception:
            return

    def start(self):
        self._thread.start()

    def stop(self):
        self._stop.set()
        self._thread.join(timeout=3)

    def summary(self, t0: float, t1: float):
        rows = [s for s in self.samples if t0 <= s[0] <= t1]
        if not rows:  # region shorter than one sampling period: take the nearest samples
            rows = sorted(self.samples, key=lambda s: abs(s[0] - 0.5 * (t0 + t1)))[:3]
        if not rows:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0}
        reasons = set()
        for r in rows:
            for bit, name in self.REASONS.items():
                if r[3] & bit:
                    reasons.add(name)
        pw = [r[2] for r in rows if r[2] == r[2]]
        return {"sm_mhz": statistics.median(r[1] for r in rows), "sm_max_mhz": self.max_mhz,
                "power_w_max": max(pw) if pw else None, "reasons": sorted(reasons), "samples": len(rows)}


def max_over_ranks(ms: float, world: int, device: str = "cuda") -> float:
    """Slowest rank's time: replicas run independently, the job is as slow as its slowest rank."""
    if world <= 1:
        return ms
    import torch
    import torch.distributed as dist

    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_tflops(flops_per_step: float, steps: int, total_ms: float, world: int) -> float:
    """Whole-job dense-equivalent TFLOP/s of `world` independent replicas."""
    return flops_per_step * steps * world / (total_ms * 1e-3) / 1e12


NSETS = 3  # rotating copies of every per-step buffer


def workload_config(wl, comp: str, world: int) -> dict:
    """The `config` object of the JSON line: the same for our arm and for the reference arm (which
    times a bounded sample of this workload; the sample is described in its `cpu_baseline`)."""
    M, K, N = wl.M, wl.K, wl.N
    return {"workload": wl.name, "M": M, "K": K, "N": N, "comp": comp, "fuse": "separate",
            "parallelism": "replicas only" if world > 1 else "single gpu",
            "l2": f"inputs larger than L2: {NSETS} rotating copies of X/W/values/metadata/Y, "
                  f"{(M*K*2 + N*K*2 + M*K + M*K//8 + M*N*2)/1e6:.0f} MB touched per step"}


def oracle_sample_rate(wl, comp_mode, target_seconds=15.0):
    """Times the CPU oracle on a bounded sample of rows of the workload.  -> dict for the JSON."""
    import numpy as np

    import oracle
    from paper_2605_26632_b200 import inputs

    cores = oracle.num_threads()
    rows_small = max(8, cores)
    # generate only as many rows of X as the largest sample can use; W in full
    max_rows = wl.M
    d = inputs.make_workload(wl, with_bias=True, M=max_rows)
    X, W, b = inputs.as_u16(d["X"]), inputs.as_u16(d["W"]), inputs.as_u16(d["bias"])
    t0 = time.perf_counter()
    oracle.act_sparse_linear(X[:rows_small], W, bias=b, comp_mode=comp_mode)
    dt = time.perf_counter() - t0
    n_rows = int(min(max_rows, max(rows_small, rows_small * target_seconds / max(dt, 1e-3))))
    n_rows = max(rows_small, (n_rows // cores) * cores)
    t0 = time.perf_counter()
    oracle.act_sparse_linear(X[:n_rows], W, bias=b, comp_mode=comp_mode)
    dt = time.perf_counter() - t0
    tflops = 2.0 * n_rows * wl.N * wl.K / dt / 1e12
    return {"value": tflops, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"first {n_rows} of {wl.M} rows of {wl.name} (all N={wl.N} outputs, full K={wl.K}), "
                      f"{dt:.1f} s wall", "seconds": dt, "rows": n_rows}


def run_reference(args):
    """--impl reference: the CPU oracle, as it stands, on bounded samples (rank 0 only)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2605_26632_b200 import inputs

    import oracle

    wl = inputs.WORKLOADS[args.workload]
    comp_mode = {"none": 0, "row": 1, "tensor": 2}[args.comp]
    oracle.build()
    budget = 120.0  # seconds for the whole run
    per_step = max(0.5, budget / max(1, args.steps + args.warmup))
    cal = oracle_sample_rate(wl, comp_mode, target_seconds=min(per_step, 10.0))
    rows = cal["rows"]
    import numpy as np

    d = inputs.make_workload(wl, with_bias=True, M=rows)
    X, W, b = inputs.as_u16(d["X"]), inputs.as_u16(d["W"]), inputs.as_u16(d["bias"])
    for _ in range(min(args.warmup, 2)):
        oracle.act_sparse_linear(X, W, bias=b, comp_mode=comp_mode)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle.act_sparse_linear(X, W, bias=b, comp_mode=comp_mode)
    dt = time.perf_counter() - t0
    tflops = 2.0 * rows * wl.N * wl.K * args.steps / dt / 1e12
    cpu = {"value": tflops, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
           "sample": f"each step = first {rows} of {wl.M} rows of {wl.name} (all N, full K)"}
    out = {"impl": "reference", "metric": METRIC, "value": tflops, "unit": UNIT, "n_gpus": args.gpus,
           "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
           "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
           "data": "synthetic", "config": workload_config(wl, args.comp, max(1, args.gpus)),
           "cpu_baseline": cpu,
           "e2e": {"value": tflops, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
           "gpu_launches": 0}
    print(json.dumps(out), flush=True)


def self_launch(args) -> int:
    """``python bench.py --gpus N`` without torchrun: start the N ranks ourselves (one process per
    GPU, rendezvous on 127.0.0.1) and return their exit code."""
    import socket

    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def launch_check(args):
    """The multi-rank plumbing without a GPU: gloo ranks, the two aggregation helpers, one JSON line."""
    import torch.distributed as dist

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    if world > 1:
        dist.init_process_group("gloo")
    ms = max_over_ranks(10.0 + 5.0 * rank, world, device="cpu")
    value = aggregate_tflops(1e12, 10, ms, world)
    if rank == 0:
        print(json.dumps({"launch_check": True, "n_gpus": world, "requested_gpus": args.gpus,
                          "slowest_rank_ms": ms, "aggregate_tflops": value}), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def sustained_legs(legs, ms_guess, sampler, block_s=0.5, rounds=4):
    """Runs the named legs (name -> callable(i)) in interleaved blocks of >= block_s seconds each,
    `rounds` times round-robin, so that every leg sees the same thermal / power state.  One CUDA-event
    pair and one synchronisation per block.  -> name -> dict(ms_per_step, blocks, clocks)."""
    import torch

    stream = torch.cuda.current_stream()
    out = {name: {"ms": [], "windows": []} for name in legs}
    for _ in range(rounds):
        for name, fn in legs.items():
            n = max(8, int(block_s * 1e3 / max(ms_guess[name], 1e-3)) + 1)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            t0 = time.time()
            e0.record(stream)
            for i in range(n):
                fn(i)
            e1.record(stream)
            torch.cuda.synchronize()
            t1 = time.time()
            out[name]["ms"].append(e0.elapsed_time(e1) / n)
            out[name]["windows"].append((t0, t1))
    res = {}
    for name, d in out.items():
        rows = [smp for (t0, t1) in d["windows"] for smp in sampler.samples if t0 <= smp[0] <= t1]
        reasons = sorted({nm for r in rows for bit, nm in ClockSampler.REASONS.items() if r[3] & bit})
        pw = [r[2] for r in rows if r[2] == r[2]]
        res[name] = {"ms_per_step": statistics.median(d["ms"]), "ms_per_step_blocks": d["ms"],
                     "sm_mhz_median": statistics.median(r[1] for r in rows) if rows else None,
                     "power_w_max": max(pw) if pw else None, "reasons": reasons, "clock_samples": len(rows)}
    return res


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
        return
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(self_launch(args))
    if args.launch_check:
        launch_check(args)
        return

    import torch
    import torch.distributed as dist

    from paper_2605_26632_b200 import binding, inputs

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    wl = inputs.WORKLOADS[args.workload]
    comp_mode = {"none": 0, "row": 1, "tensor": 2}[args.comp]
    M, K, N = wl.M, wl.K, wl.N
    peaks = load_peaks()
    lx = binding.Lynx(local_rank)
    lx.reserve(M, N, K)

    d = inputs.make_workload(wl, with_bias=True)
    # Device-resident inputs, rotated over NSETS distinct copies so that, together with W, values,
    # metadata and Y (>= 246 MB per step for mlp_down), nothing a step reads is left in the 126 MB L2
    # by the previous step.
    Xs = [d["X"].cuda() if i == 0 else None for i in range(NSETS)]
    for i in range(1, NSETS):
        Xs[i] = torch.roll(Xs[0], shifts=i * 4, dims=0).contiguous()
    Ws = [d["W"].cuda() for _ in range(NSETS)]
    bias = d["bias"].cuda()
    vals = [torch.empty((M, K // 2), dtype=torch.bfloat16, device="cuda") for _ in range(NSETS)]
    metas = [torch.empty(binding.meta_bytes(M, K), dtype=torch.uint8, device="cuda") for _ in range(NSETS)]
    scales = [torch.empty(M, dtype=torch.float32, device="cuda") for _ in range(NSETS)]
    Ys = [torch.empty((M, N), dtype=torch.bfloat16, device="cuda") for _ in range(NSETS)]
    stream = torch.cuda.current_stream()

    def step(i):
        # the call a user makes: one layer = prune/compress launch + sparse GEMM launch
        j = i % NSETS
        lx.act_sparse_linear(Xs[j], Ws[j], bias, comp_mode, None, Ys[j], binding.FUSE_SEPARATE)

    def probe_scale(j):
        # ROW mode: the deferred form, i.e. exactly the two launches the layer call makes
        if comp_mode == 1:
            return binding.ROW_SCALE_DEFERRED
        return scales[j] if comp_mode else None

    def probe_step(i, ev):
        # the same two kernels as separate calls with an event between them (per-kernel times)
        j = i % NSETS
        ev[0].record(stream)
        lx.prune_compress(Xs[j], comp_mode, vals[j], metas[j], probe_scale(j))
        ev[1].record(stream)
        lx.sparse_linear(vals[j], metas[j], Ws[j], bias, probe_scale(j), None, Ys[j])
        ev[2].record(stream)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(max(args.warmup, 3)):
        step(i)
    barrier()
    if lx.last_error() != 0:
        raise SystemExit("device-side timeout during warm-up")

    sampler = ClockSampler(local_rank)
    sampler.start()
    time.sleep(0.3)
    launches0 = lx.launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    t_wall0 = time.time()
    e0.record(stream)
    for i in range(args.steps):
        step(i)
    e1.record(stream)
    barrier()
    launches = lx.launch_count() - launches0
    total_ms = e0.elapsed_time(e1)
    total_ms = max_over_ranks(total_ms, world)

    # per-kernel times: the same number of steps again, as two calls with CUDA events around each
    # kernel (an event between two launches keeps the second kernel from starting early as a
    # programmatic dependent, so these steps are a little slower than the timed ones; in ROW mode the
    # two calls use the deferred row scale, i.e. they are the launches the layer call makes)
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    probed = list(range(args.steps))
    for i in probed:
        probe_step(i, evs[i])
    barrier()
    t_wall1 = time.time()
    prune_ms = [evs[i][0].elapsed_time(evs[i][1]) for i in probed]
    gemm_ms = [evs[i][1].elapsed_time(evs[i][2]) for i in probed]

    # prune/compress (row scale finalized in the same launch) alone, back to back over the rotating sets: the
    # per-launch time that the HBM roofline of that kernel is computed from
    def prune_loop(scale_of):
        p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        for i in range(3):
            lx.prune_compress(Xs[i % NSETS], comp_mode, vals[i % NSETS], metas[i % NSETS], scale_of(i % NSETS))
        torch.cuda.synchronize()
        p0.record(stream)
        for i in range(args.steps):
            j = i % NSETS
            lx.prune_compress(Xs[j], comp_mode, vals[j], metas[j], scale_of(j))
        p1.record(stream)
        torch.cuda.synchronize()
        return p0.elapsed_time(p1) / args.steps

    # as launched by the layer call (ROW mode: the scale is finished by the GEMM epilogue), and the
    # stand-alone form that finishes the scale in the same launch
    prune_loop_ms = prune_loop(probe_scale)
    prune_alone_ms = prune_loop(lambda j: scales[j] if comp_mode else None)

    # dense bf16 GEMM of the same shape on the same GPU (same rotation, same event timing)
    dense_out = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    for i in range(3):
        torch.nn.functional.linear(Xs[i % NSETS], Ws[i % NSETS], bias, out=None)
    torch.cuda.synchronize()
    d0, d1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    d0.record(stream)
    for i in range(args.steps):
        dense_out = torch.nn.functional.linear(Xs[i % NSETS], Ws[i % NSETS], bias)
    d1.record(stream)
    torch.cuda.synchronize()
    dense_ms = d0.elapsed_time(d1) / args.steps
    t_wall2 = time.time()

    # the same layer with the rank-64 low-rank branch (Y = Y_s + X (L_A L_B)^T), outside the headline
    # number: its cost on top of the step, same rotation and event timing
    lora = None
    if not args.no_lora:
        R = 64
        LA, LB = inputs.make_lora(N, K, R, wl.seed)
        LA, LB = LA.cuda(), LB.cuda()
        lx.reserve_lora(M, K, R)
        for i in range(3):
            lx.act_sparse_linear_lora(Xs[i % NSETS], Ws[i % NSETS], LA, LB, bias, comp_mode, None, Ys[i % NSETS])
        torch.cuda.synchronize()
        l0, l1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        l0.record(stream)
        for i in range(args.steps):
            j = i % NSETS
            lx.act_sparse_linear_lora(Xs[j], Ws[j], LA, LB, bias, comp_mode, None, Ys[j])
        l1.record(stream)
        torch.cuda.synchronize()
        lora_ms = l0.elapsed_time(l1) / args.steps
        lora = {"rank": R, "ms_per_step": lora_ms, "overhead_vs_step": lora_ms / (total_ms / args.steps) - 1.0,
                "speedup_vs_dense_bf16_without_lora": dense_ms / lora_ms,
                "how": "lynx_act_sparse_linear_lora: one launch that prunes / compresses X and computes "
                       "T = (X L_B^T) / s from the same read of X, then the sparse GEMM that adds T L_A^T in its accumulator"}

    # the same layer on FP8 (E4M3) operands, outside the headline number: weights quantised once
    # (symmetric per output channel), activations pruned and quantised (per-row scale found in the
    # data) inside every step; same rotation and event timing
    fp8 = None
    if not args.no_fp8 and comp_mode in (0, 1):
        Wqs = [lx.quantize_weights_fp8(w, True) for w in Ws]
        for i in range(3):
            lx.act_sparse_linear_fp8(Xs[i % NSETS], Wqs[i % NSETS][0], Wqs[i % NSETS][1], bias, comp_mode, None,
                                     Ys[i % NSETS])
        torch.cuda.synchronize()
        f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        f0.record(stream)
        for i in range(args.steps):
            j = i % NSETS
            lx.act_sparse_linear_fp8(Xs[j], Wqs[j][0], Wqs[j][1], bias, comp_mode, None, Ys[j])
        f1.record(stream)
        torch.cuda.synchronize()
        fp8_ms = f0.elapsed_time(f1) / args.steps
        fp8 = {"ms_per_step": fp8_ms, "tflops_dense_equivalent": 2.0 * M * N * K / (fp8_ms * 1e-3) / 1e12,
               "speedup_vs_step": (total_ms / args.steps) / fp8_ms, "speedup_vs_dense_bf16": dense_ms / fp8_ms,
               "dtype": "e4m3 operands, f32 accumulation, bf16 output",
               "how": "lynx_act_sparse_linear_fp8: single-read quantising prune/compress + kind::f8f6f4 sparse GEMM"}
        del Wqs

    # ---- sustained regime: seconds of back-to-back work, interleaved A/B/C so that all legs see the same
    # power state; the GPU leaves its burst clocks and settles where the power cap puts it
    sustained = None
    if not args.no_sustained:
        for j in range(NSETS):  # finished row scales for the GEMM-alone leg
            lx.prune_compress(Xs[j], comp_mode, vals[j], metas[j], scales[j] if comp_mode else None)
        legs = {
            "layer": lambda i: step(i),
            "sparse_gemm": lambda i: lx.sparse_linear(vals[i % NSETS], metas[i % NSETS], Ws[i % NSETS], bias,
                                                      scales[i % NSETS] if comp_mode else None, None, Ys[i % NSETS]),
            "dense_bf16": lambda i: torch.nn.functional.linear(Xs[i % NSETS], Ws[i % NSETS], bias),
        }
        guess = {"layer": total_ms / args.steps, "sparse_gemm": sum(gemm_ms) / len(gemm_ms), "dense_bf16": dense_ms}
        sl = sustained_legs(legs, guess, sampler)
        flops_ = 2.0 * M * N * K
        for name in sl:
            sl[name]["tflops"] = flops_ / (sl[name]["ms_per_step"] * 1e-3) / 1e12
            mhz = sl[name]["sm_mhz_median"]
            # time x clock: what the leg would cost in SM cycles (shows how much of a slowdown is the clock)
            sl[name]["mcycles_per_step"] = sl[name]["ms_per_step"] * mhz * 1e-3 if mhz else None
        sustained = {
            "how": "each leg in blocks of >= 0.5 s, four rounds interleaved layer / sparse GEMM alone / dense linear, "
                   "same rotating buffers as the timed loop, CUDA events per block, median block; clocks = NVML samples "
                   "inside the leg's blocks",
            "layer": sl["layer"], "sparse_gemm": sl["sparse_gemm"], "dense_bf16": sl["dense_bf16"],
            "speedup_vs_dense_bf16": sl["dense_bf16"]["ms_per_step"] / sl["layer"]["ms_per_step"],
            "gemm_frac_of_2x_bf16_tflops_sustained": sl["sparse_gemm"]["tflops"] / (2.0 * peaks["bf16_tflops_sustained"]),
            "layer_frac_of_2x_bf16_tflops_sustained": sl["layer"]["tflops"] / (2.0 * peaks["bf16_tflops_sustained"]),
            "dense_frac_of_bf16_tflops_sustained": sl["dense_bf16"]["tflops"] / peaks["bf16_tflops_sustained"],
        }

    # ---- the other configurations the metric names: attention projections, mlp.up (with the one-kernel
    # variant beside it), the 16 shapes of the token sweep; a few milliseconds per stage and shape
    sweep = None
    if not args.no_sweep and world == 1:
        from paper_2605_26632_b200 import sweep as sweep_mod

        rows = []
        named = [("attn_qkv", inputs.WORKLOADS["attn_qkv"]), ("attn_out", inputs.WORKLOADS["attn_out"]),
                 ("mlp_up", inputs.WORKLOADS["mlp_up"])]
        shapes = [(nm, w.M, w.K, w.N, w.x_dist) for nm, w in named]
        for Ms in inputs.SWEEP_M:
            for (Kk, Nn) in inputs.SWEEP_KN:
                w = inputs.sweep_workload(Ms, Kk, Nn)
                shapes.append(("sweep", w.M, w.K, w.N, w.x_dist))
        for (nm, Ms, Kk, Nn, dist_) in shapes:
            r = sweep_mod.time_shape(lx, Ms, Kk, Nn, iters=30, fused=(nm == "mlp_up"), x_dist=dist_)
            fl = 2.0 * Ms * Nn * Kk
            row = {"config": nm, "M": Ms, "K": Kk, "N": Nn,
                   "prune_us": r["prune_ms"] * 1e3, "gemm_us": r["gemm_ms"] * 1e3, "layer_us": r["layer_ms"] * 1e3,
                   "dense_us": r["dense_ms"] * 1e3, "layer_over_dense": r["dense_ms"] / r["layer_ms"],
                   "gemm_over_dense": r["dense_ms"] / r["gemm_ms"], "layer_tflops": fl / r["layer_ms"] / 1e9,
                   "gemm_frac": fl / r["gemm_ms"] / 1e9 / (2.0 * peaks["bf16_tflops"]),
                   "prune_frac_of_hbm": Ms * Kk * 3.125 / r["prune_ms"] / 1e6 / peaks["hbm_gbs"]}
            if nm == "mlp_up":
                row["fused_us"] = r["fused_ms"] * 1e3
                row["fused_over_separate"] = r["layer_ms"] / r["fused_ms"]
            rows.append(row)
        sweep = {"how": "per shape: prune/compress alone (ROW mode, scale finished in the launch), sparse GEMM alone, the "
                        "two-kernel layer, torch's dense bf16 linear; inputs drawn on the device by the workload's recipe, "
                        "rotating over enough copies to exceed the L2; each stage replayed from a CUDA graph for ~6 ms, "
                        "median of three replays (burst clocks)",
                 "rows": rows,
                 "layer_over_dense_min": min(r["layer_over_dense"] for r in rows),
                 "shapes_where_layer_beats_dense": sum(1 for r in rows if r["layer_over_dense"] > 1.0), "shapes": len(rows)}

    # end to end through the host-buffer entry point: pinned X in, pinned Y out, every step
    e2e = None
    if not args.no_e2e:
        xh = [d["X"].pin_memory(), torch.roll(d["X"], 4, 0).contiguous().pin_memory()]
        yh = torch.empty((M, N), dtype=torch.bfloat16).pin_memory()
        for i in range(2):
            lx.act_sparse_linear_host(xh[i % 2], Ws[0], bias, comp_mode, yh)
        e2e_steps = max(3, min(args.steps, 20))
        barrier()
        h0, h1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        h0.record(stream)
        for i in range(e2e_steps):
            lx.act_sparse_linear_host(xh[i % 2], Ws[i % NSETS], bias, comp_mode, yh)
        h1.record(stream)
        barrier()
        e2e_ms = h0.elapsed_time(h1)
        e2e_ms = max_over_ranks(e2e_ms, world)
        e2e = {"value": aggregate_tflops(2.0 * M * N * K, e2e_steps, e2e_ms, world), "unit": UNIT,
               "h2d_bytes_per_step": M * K * 2, "d2h_bytes_per_step": M * N * 2, "steps": e2e_steps,
               "ms_per_step": e2e_ms / e2e_steps}
    sampler.stop()
    if lx.last_error() != 0:
        raise SystemExit("device-side timeout during the timed region")

    flops = 2.0 * M * N * K
    ms_per_step = total_ms / args.steps
    value = aggregate_tflops(flops, args.steps, total_ms, world)
    gemm_avg_ms = sum(gemm_ms) / len(gemm_ms)
    prune_avg_ms = sum(prune_ms) / len(prune_ms)
    # the timed region lasts milliseconds: the GPU stays at its burst clocks (see "clocks"), so the
    # burst cuBLAS figure is the fair denominator; the sustained one applies to seconds-long loops
    long_run = total_ms > 2000.0
    dense_peak = peaks["bf16_tflops_sustained"] if long_run else peaks["bf16_tflops"]
    sparse_peak = 2.0 * dense_peak
    gemm_tf = flops / (gemm_avg_ms * 1e-3) / 1e12
    prune_bytes = M * K * 3.125 + (4 * M if comp_mode else 0)
    prune_gbs = prune_bytes / (prune_loop_ms * 1e-3) / 1e9
    prune_alone_gbs = prune_bytes / (prune_alone_ms * 1e-3) / 1e9
    clocks = sampler.summary(t_wall0, t_wall1)
    clocks_dense = sampler.summary(t_wall1, t_wall2)

    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": workload_config(wl, args.comp, world),
        "speedup_vs_dense_bf16": dense_ms / ms_per_step,
        "dense_bf16": {"ms": dense_ms, "tflops": flops / (dense_ms * 1e-3) / 1e12, "impl": "torch F.linear (cuBLASLt)",
                       "sm_mhz": clocks_dense.get("sm_mhz")},
        "kernels": {"prune_compress_ms": prune_avg_ms, "sparse_gemm_ms": gemm_avg_ms,
                    "probed_steps": len(probed),
                    "how": "CUDA events around each kernel in a second loop of the same steps issued as two calls "
                           "(lynx_prune_compress + lynx_sparse_linear), right after the timed loop"},
        "roofline": {"bound": "tensor", "kernel": "sparse_gemm_kernel", "achieved": gemm_tf, "peak": sparse_peak,
                     "unit": "TFLOP/s", "frac": gemm_tf / sparse_peak,
                     "traffic": ncu_traffic_bytes(wl, torch.cuda.get_device_properties(local_rank).multi_processor_count),
                     "peak_kind": f"2 x {'bf16_tflops_sustained' if long_run else 'bf16_tflops (burst)'} of "
                                  f"{peaks['source']} peaks; 2:4 sparse bf16 = 2 x dense bf16 (nominal ratio); "
                                  "dense-equivalent flops; the seconds-long regime is under `sustained`"},
        "roofline_prune": {"bound": "hbm", "kernel": "prune_compress_kernel", "achieved": prune_alone_gbs,
                           "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": prune_alone_gbs / peaks["hbm_gbs"],
                           "frac_of_8TBs_nominal": prune_alone_gbs / 8000.0, "bytes_per_launch": prune_bytes,
                           "ms_per_launch": prune_alone_ms,
                           "deferred_ms_per_launch": prune_loop_ms, "deferred_frac": prune_gbs / peaks["hbm_gbs"],
                           "deferred_frac_of_8TBs_nominal": prune_gbs / 8000.0, "in_step_ms": prune_avg_ms,
                           "how": "back-to-back loop of lynx_prune_compress over rotating buffers, CUDA events: achieved / frac = "
                                  "the stand-alone public form (select, compress, row sums and the finished row scale from the "
                                  "one call); deferred_* = the form the layer call launches (the GEMM epilogue finishes the "
                                  "scale); in_step_ms = kernels.prune_compress_ms",
                           "peak_kind": f"hbm_gbs ({peaks['source']})"},
        "clocks": clocks,
        "sustained": sustained,
        "sweep": sweep,
        "e2e": e2e,
        "lora": lora,
        "fp8": fp8,
        "gpu_launches": int(launches),
    }

    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        import oracle

        oracle.build()
        out["cpu_baseline"] = {k: v for k, v in oracle_sample_rate(wl, comp_mode).items() if k not in ("seconds", "rows")}
    elif rank == 0:
        out["cpu_baseline"] = None

    if rank == 0:
        print(json.dumps(out), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
