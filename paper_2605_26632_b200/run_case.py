"""Runs a few launches of one kernel of the path on a named synthetic workload.

    python -m paper_2605_26632_b200.run_case --kernel prune|gemm|layer|fused|lora_down|prune_lora|lora_layer|fp8_prune|fp8_gemm|fp8_layer --workload mlp_down [--iters 3]

Meant as the small, self-terminating command to put under a profiler (one kernel, a few launches,
well under a GB on the device), and as a minimal usage example of the binding.
"""
from __future__ import annotations

import argparse

import torch

from . import binding, inputs


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--kernel", default="layer", choices=["prune", "gemm", "layer", "fused", "lora_down", "prune_lora", "lora_layer", "fp8_prune", "fp8_gemm",
                             "fp8_layer"])
    ap.add_argument("--rank", type=int, default=64, help="rank R of the low-rank branch")
    ap.add_argument("--workload", default="mlp_down")
    ap.add_argument("--M", type=int, default=0, help="override the number of token rows")
    ap.add_argument("--iters", type=int, default=3)
    ap.add_argument("--comp", type=int, default=1)
    args = ap.parse_args()
    wl = inputs.WORKLOADS[args.workload]
    M = args.M or wl.M
    g = torch.Generator(device="cuda").manual_seed(wl.seed)
    # device-side random inputs: this command is about timing/counters, not parity
    X = torch.randn(M, wl.K, device="cuda", generator=g).to(torch.bfloat16)
    W = (torch.randn(wl.N, wl.K, device="cuda", generator=g) * wl.K ** -0.5).to(torch.bfloat16)
    b = torch.zeros(wl.N, device="cuda", dtype=torch.bfloat16)
    lx = binding.Lynx(0)
    lx.reserve(M, wl.N, wl.K)
    values, meta, scale = lx.prune_compress(X, args.comp)
    Y = torch.empty(M, wl.N, device="cuda", dtype=torch.bfloat16)
    R = args.rank
    LB = (torch.randn(R, wl.K, device="cuda", generator=g) * wl.K ** -0.5).to(torch.bfloat16)
    LA = (torch.randn(wl.N, R, device="cuda", generator=g) * 0.3 * R ** -0.5).to(torch.bfloat16)
    T = torch.empty(M, R, device="cuda", dtype=torch.bfloat16)
    if "lora" in args.kernel:
        lx.reserve_lora(M, wl.K, R)
    if args.kernel.startswith("fp8"):
        Wq, ws = lx.quantize_weights_fp8(W, per_channel=True)
        vq, meta8, rs = lx.prune_compress_fp8(X, args.comp)
    for _ in range(args.iters):
        if args.kernel == "fp8_prune":
            lx.prune_compress_fp8(X, args.comp, vq, meta8, rs)
        if args.kernel == "fp8_gemm":
            lx.sparse_linear_fp8(vq, meta8, Wq, ws, b, rs, None, Y)
        if args.kernel == "fp8_layer":
            lx.act_sparse_linear_fp8(X, Wq, ws, b, args.comp, None, Y)
        if args.kernel in ("prune", "layer"):
            lx.prune_compress(X, args.comp, values, meta, scale)
        if args.kernel in ("gemm", "layer"):
            lx.sparse_linear(values, meta, W, b, scale, None, Y)
        if args.kernel == "lora_down":
            lx.lora_down(X, LB, scale, T)
        if args.kernel == "prune_lora":
            lx.prune_compress_lora(X, LB, args.comp, values, meta, T)
        if args.kernel == "lora_layer":
            lx.act_sparse_linear_lora(X, W, LA, LB, b, args.comp, None, Y)
        if args.kernel == "fused":
            lx.act_sparse_linear(X, W, b, args.comp, None, Y, binding.FUSE_FUSED)
    torch.cuda.synchronize()
    assert lx.last_error() == 0
    print(f"ran {args.iters} x {args.kernel} on {args.workload} (M={M}, K={wl.K}, N={wl.N}); "
          f"{lx.launch_count()} launches")


if __name__ == "__main__":
    main()
