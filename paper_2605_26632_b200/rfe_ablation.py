"""Relative Frobenius error of the sparse layer against the dense one, per norm-compensation mode.

    python -m paper_2605_26632_b200.rfe_ablation

RFE = |X W^T - Y_mode|_F / |X W^T|_F (the error metric of the paper's layer-wise analysis) on the
seeded synthetic workloads, for Y_mode = the 2:4 activation-sparse layer with no compensation, one
factor per token row, one for the whole tensor, and one per group of four; plus the time of the
prune/compress launch in each mode.  The dense product is torch's fp32 matmul of the same bf16
operands.  Prints a markdown table.
"""
from __future__ import annotations

import torch

from . import binding, inputs

MODES = (("none", binding.COMP_NONE), ("row", binding.COMP_ROW), ("tensor", binding.COMP_TENSOR),
         ("group", binding.COMP_GROUP))


def main():
    lx = binding.Lynx(0)
    print("| workload | M x K x N | input | RFE none | RFE row | RFE tensor | RFE group | "
          "prune us none / row / tensor / group |")
    print("|---|---|---|---|---|---|---|---|")
    cases = [inputs.WORKLOADS[n] for n in ("tiny", "mlp_down", "attn_qkv", "attn_out", "mlp_up")]
    cases.append(inputs.Workload("mlp_down_normal", 4096, 12288, 3072, "normal", 11))
    for wl in cases:
        d = inputs.make_workload(wl, with_bias=False)
        X, W = d["X"].cuda(), d["W"].cuda()
        ref = X.float() @ W.float().T
        rfes, times = [], []
        for _, mode in MODES:
            Y = lx.act_sparse_linear(X, W, None, mode)
            rfes.append(((Y.float() - ref).norm() / ref.norm()).item())
            v, m, s = lx.prune_compress(X, mode)
            torch.cuda.synchronize()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            for _ in range(20):
                lx.prune_compress(X, mode, v, m, s)
            b.record()
            torch.cuda.synchronize()
            times.append(a.elapsed_time(b) / 20 * 1e3)
        print(f"| {wl.name} | {wl.M} x {wl.K} x {wl.N} | {wl.x_dist} | " + " | ".join(f"{r:.4f}" for r in rfes) +
              " | " + " / ".join(f"{t:.1f}" for t in times) + " |", flush=True)
    assert lx.last_error() == 0


if __name__ == "__main__":
    main()
