"""Times every stage of the path over the DiT shape sweep and prints a markdown table.

    python -m paper_2605_26632_b200.sweep [--quick] [--iters 30]

For each (M, K, N): prune/compress alone (GB/s of its 3.125 B/element), sparse GEMM alone, the
two-kernel layer, the fused one-kernel layer, and the dense bf16 linear (torch / cuBLASLt) on the
same GPU with the same timing loop.  Inputs rotate over enough copies that nothing a launch reads
is left in the L2 by the previous launch; times are CUDA-event averages over `iters` launches
replayed from a CUDA graph (`--no-graph`: eager launches, host-bound below ~15 us per call).
"""
from __future__ import annotations

import argparse
import math

import torch

from . import binding, inputs


USE_GRAPH = True


def timeloop(fn, nsets, iters, warm=5):
    """Average device time of one call of fn (ms).  The calls are captured into one CUDA graph and
    the graph is replayed, so that launches shorter than the host's per-call cost (tensor-map
    encoding + launch, ~10 us from Python) are timed at the GPU's pace, not the host's.  The
    number of calls is cut so that one replay lasts about 6 ms: seconds of back-to-back tensor-core
    work run into the power cap and would time the sustained clocks, not the kernel."""
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    a.record()
    for i in range(warm):
        fn(i % nsets)
    b.record()
    torch.cuda.synchronize()
    est_ms = a.elapsed_time(b) / warm
    iters = max(4, min(iters, int(6.0 / max(est_ms, 1e-3))))
    if not USE_GRAPH:
        a.record()
        for i in range(iters):
            fn(i % nsets)
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) / iters
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        for i in range(iters):
            fn(i % nsets)
    torch.cuda.synchronize()
    best = None
    for _ in range(3):  # three separate replays with an idle gap; the median is reported
        torch.cuda.synchronize()
        a.record()
        g.replay()
        b.record()
        torch.cuda.synchronize()
        t = a.elapsed_time(b) / iters
        best = [t] if best is None else best + [t]
    return sorted(best)[1]


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--quick", action="store_true", help="M = 4096 only")
    ap.add_argument("--iters", type=int, default=30)
    ap.add_argument("--no-fused", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="time eager launches instead of a CUDA graph replay")
    ap.add_argument("--fp8", action="store_true",
                    help="time the FP8 (E4M3) composition instead: quantising prune, FP8 sparse GEMM, the FP8 layer, "
                         "next to the bf16 sparse layer, the dense bf16 linear and torch's dense FP8 GEMM")
    ap.add_argument("--lora", type=int, default=0, metavar="R",
                    help="time the low-rank branch of rank R instead: down projection alone, layer with it, "
                         "and the dense linear followed by the two dense low-rank GEMMs of torch")
    args = ap.parse_args()
    global USE_GRAPH
    USE_GRAPH = not args.no_graph
    lx = binding.Lynx(0)
    Ms = (4096,) if args.quick else inputs.SWEEP_M
    shapes = [(M, K, N) for M in Ms for (K, N) in inputs.SWEEP_KN]
    shapes += [(4352, 3072, 9216), (4352, 3072, 3072)]
    shapes += [(inputs.OTHER_FAMILY_M, K, N) for (K, N) in inputs.OTHER_FAMILY_KN]
    if not args.quick:
        shapes += [(M, K, M) for M in (2048, 4096, 8192) for K in (3072, 12288)]  # the paper's kernel grid
    if args.fp8:
        return fp8_sweep(lx, shapes, args.iters)
    if args.lora:
        return lora_sweep(lx, shapes, args.lora, args.iters)
    print("| M | K | N | prune us | prune GB/s | GEMM us | GEMM TF | layer us | layer TF | fused us | fused TF | "
          "dense us | dense TF | GEMM/dense | layer/dense |")
    print("|---|---|---|---|---|---|---|---|---|---|---|---|---|---|---|")
    for (M, K, N) in shapes:
        r = time_shape(lx, M, K, N, args.iters, fused=not args.no_fused)
        tp, tg, tl, tf, td = r["prune_ms"], r["gemm_ms"], r["layer_ms"], r["fused_ms"], r["dense_ms"]
        fl = 2.0 * M * N * K
        tf_s = lambda t: fl / t / 1e9
        print(f"| {M} | {K} | {N} | {tp*1e3:.1f} | {M*K*3.125/tp/1e6:.0f} | {tg*1e3:.1f} | {tf_s(tg):.0f} | "
              f"{tl*1e3:.1f} | {tf_s(tl):.0f} | {tf*1e3:.1f} | {tf_s(tf):.0f} | {td*1e3:.1f} | {tf_s(td):.0f} | "
              f"{td/tg:.2f} | {td/tl:.2f} |", flush=True)


def device_x(M, K, x_dist, g):
    """Activations drawn on the device by the recipe of inputs.make_x (same distributions, other
    random numbers: these tensors are for timing, the parity tests use the CPU generator)."""
    x = torch.randn(M, K, device="cuda", generator=g)
    if x_dist in ("gelu", "gelu_chan"):
        x = torch.nn.functional.gelu(x)
        if x_dist == "gelu_chan":
            x = x * torch.exp(0.5 * torch.randn(K, device="cuda", generator=g))
    elif x_dist == "outlier":
        idx = torch.randperm(K, device="cuda", generator=g)[:K // 100]
        x[:, idx] *= 20.0
    return x.to(torch.bfloat16)


def time_shape(lx, M, K, N, iters=30, fused=False, with_prune_forms=False, x_dist="normal"):
    """Device times (ms) of the stages of one layer shape, each over rotating inputs larger than the
    L2: prune/compress alone (ROW mode, scale finished in the launch), sparse GEMM alone, the
    two-kernel layer, optionally the one-kernel layer, and torch's dense bf16 linear."""
    per_set = M * K * 2 + M * K + M * K // 8 + N * K * 2 + M * N * 2
    nsets = max(2, math.ceil(400e6 / per_set))
    g = torch.Generator(device="cuda").manual_seed(M + K + N)
    Xs = [device_x(M, K, x_dist, g) for _ in range(nsets)]
    Ws = [(torch.randn(N, K, device="cuda", generator=g) * K ** -0.5).to(torch.bfloat16) for _ in range(nsets)]
    b = torch.zeros(N, device="cuda", dtype=torch.bfloat16)
    vs = [torch.empty(M, K // 2, device="cuda", dtype=torch.bfloat16) for _ in range(nsets)]
    ms = [torch.empty(binding.meta_bytes(M, K), device="cuda", dtype=torch.uint8) for _ in range(nsets)]
    ss = [torch.empty(M, device="cuda", dtype=torch.float32) for _ in range(nsets)]
    Ys = [torch.empty(M, N, device="cuda", dtype=torch.bfloat16) for _ in range(nsets)]
    lx.reserve(M, N, K)
    for j in range(nsets):
        lx.prune_compress(Xs[j], 1, vs[j], ms[j], ss[j])
    out = {"M": M, "K": K, "N": N, "nsets": nsets}
    out["prune_ms"] = timeloop(lambda j: lx.prune_compress(Xs[j], 1, vs[j], ms[j], ss[j]), nsets, iters)
    if with_prune_forms:
        out["prune_deferred_ms"] = timeloop(
            lambda j: lx.prune_compress(Xs[j], 1, vs[j], ms[j], binding.ROW_SCALE_DEFERRED), nsets, iters)
        for j in range(nsets):  # leave finished scales behind for the GEMM loop
            lx.prune_compress(Xs[j], 1, vs[j], ms[j], ss[j])
    out["gemm_ms"] = timeloop(lambda j: lx.sparse_linear(vs[j], ms[j], Ws[j], b, ss[j], None, Ys[j]), nsets, iters)
    out["layer_ms"] = timeloop(lambda j: lx.act_sparse_linear(Xs[j], Ws[j], b, 1, None, Ys[j], binding.FUSE_SEPARATE),
                               nsets, iters)
    out["fused_ms"] = float("nan")
    if fused:
        out["fused_ms"] = timeloop(lambda j: lx.act_sparse_linear(Xs[j], Ws[j], b, 1, None, Ys[j], binding.FUSE_FUSED),
                                   nsets, iters)
    out["dense_ms"] = timeloop(lambda j: torch.nn.functional.linear(Xs[j], Ws[j], b), nsets, iters)
    if lx.last_error() != 0:
        raise RuntimeError("device-side timeout")
    del Xs, Ws, vs, ms, ss, Ys
    torch.cuda.empty_cache()
    return out


def fp8_sweep(lx, shapes, iters):
    print("| M | K | N | prune fp8 us | prune fp8 (given amax) us | GEMM fp8 us | GEMM fp8 TF | layer fp8 us | "
          "layer fp8 (given amax) us | layer bf16 us | dense bf16 us | dense fp8 (torch) us | fp8 layer / bf16 layer | "
          "fp8 layer / dense bf16 | fp8 layer / dense fp8 |")
    print("|---|---|---|---|---|---|---|---|---|---|---|---|---|---|---|")
    for (M, K, N) in shapes:
        if K % 256:
            continue
        per_set = M * K * 2 + M * K + M * K // 8 + N * K * 2 + M * N * 2
        nsets = max(2, math.ceil(400e6 / per_set))
        g = torch.Generator(device="cuda").manual_seed(M + K + N)
        Xs = [torch.randn(M, K, device="cuda", generator=g).to(torch.bfloat16) for _ in range(nsets)]
        Ws = [(torch.randn(N, K, device="cuda", generator=g) * K ** -0.5).to(torch.bfloat16) for _ in range(nsets)]
        b = torch.zeros(N, device="cuda", dtype=torch.bfloat16)
        Ys = [torch.empty(M, N, device="cuda", dtype=torch.bfloat16) for _ in range(nsets)]
        lx.reserve(M, N, K)
        Wqs = [lx.quantize_weights_fp8(W, True) for W in Ws]
        cs = [lx.prune_compress_fp8(X, 1) for X in Xs]
        tp = timeloop(lambda j: lx.prune_compress_fp8(Xs[j], 1, *cs[j]), nsets, iters)
        tg = timeloop(lambda j: lx.sparse_linear_fp8(cs[j][0], cs[j][1], Wqs[j][0], Wqs[j][1], b, cs[j][2], None, Ys[j]),
                      nsets, iters)
        tl = timeloop(lambda j: lx.act_sparse_linear_fp8(Xs[j], Wqs[j][0], Wqs[j][1], b, 1, None, Ys[j]), nsets, iters)
        am = [X.float().abs().amax(dim=1).contiguous() for X in Xs]
        tpg = timeloop(lambda j: lx.prune_compress_fp8(Xs[j], 1, *cs[j], row_amax=am[j]), nsets, iters)
        tlg = timeloop(lambda j: lx.act_sparse_linear_fp8(Xs[j], Wqs[j][0], Wqs[j][1], b, 1, None, Ys[j], row_amax=am[j]),
                       nsets, iters)
        tb = timeloop(lambda j: lx.act_sparse_linear(Xs[j], Ws[j], b, 1, None, Ys[j], binding.FUSE_SEPARATE), nsets, iters)
        td = timeloop(lambda j: torch.nn.functional.linear(Xs[j], Ws[j], b), nsets, iters)
        # torch's dense FP8 GEMM (cuBLASLt) on pre-quantised operands, per-tensor scales
        Xq = [X.to(torch.float8_e4m3fn) for X in Xs]
        Wt = [W.to(torch.float8_e4m3fn) for W in Ws]
        one = torch.ones((), device="cuda", dtype=torch.float32)
        try:
            t8 = timeloop(lambda j: torch._scaled_mm(Xq[j], Wt[j].t(), scale_a=one, scale_b=one, bias=b,
                                                     out_dtype=torch.bfloat16), nsets, iters)
        except Exception:
            t8 = float("nan")
        fl = 2.0 * M * N * K
        print(f"| {M} | {K} | {N} | {tp*1e3:.1f} | {tpg*1e3:.1f} | {tg*1e3:.1f} | {fl/tg/1e9:.0f} | {tl*1e3:.1f} | "
              f"{tlg*1e3:.1f} | {tb*1e3:.1f} | {td*1e3:.1f} | {t8*1e3:.1f} | {tb/tl:.2f} | {td/tl:.2f} | {t8/tl:.2f} |",
              flush=True)
        assert lx.last_error() == 0
        del Xs, Ws, Ys, Wqs, cs, Xq, Wt
        torch.cuda.empty_cache()


def lora_sweep(lx, shapes, R, iters):
    print("| M | K | N | R | prune us | prune+down us | lora_down us | layer us | layer+LoRA us | overhead | "
          "dense+LoRA (torch) us | speedup with LoRA |")
    print("|---|---|---|---|---|---|---|---|---|---|---|---|")
    for (M, K, N) in shapes:
        per_set = M * K * 2 + M * K + M * K // 8 + N * K * 2 + M * N * 2
        nsets = max(2, math.ceil(400e6 / per_set))
        g = torch.Generator(device="cuda").manual_seed(M + K + N)
        Xs = [torch.randn(M, K, device="cuda", generator=g).to(torch.bfloat16) for _ in range(nsets)]
        Ws = [(torch.randn(N, K, device="cuda", generator=g) * K ** -0.5).to(torch.bfloat16) for _ in range(nsets)]
        LB = (torch.randn(R, K, device="cuda", generator=g) * K ** -0.5).to(torch.bfloat16)
        LA = (torch.randn(N, R, device="cuda", generator=g) * 0.3 * R ** -0.5).to(torch.bfloat16)
        b = torch.zeros(N, device="cuda", dtype=torch.bfloat16)
        Ys = [torch.empty(M, N, device="cuda", dtype=torch.bfloat16) for _ in range(nsets)]
        Ts = [torch.empty(M, R, device="cuda", dtype=torch.bfloat16) for _ in range(nsets)]
        ss = [torch.ones(M, device="cuda", dtype=torch.float32) for _ in range(nsets)]
        lx.reserve(M, N, K)
        lx.reserve_lora(M, K, R)
        vs = [torch.empty(M, K // 2, device="cuda", dtype=torch.bfloat16) for _ in range(nsets)]
        ms = [torch.empty(binding.meta_bytes(M, K), device="cuda", dtype=torch.uint8) for _ in range(nsets)]
        tp = timeloop(lambda j: lx.prune_compress(Xs[j], 1, vs[j], ms[j], binding.ROW_SCALE_DEFERRED), nsets, iters)
        tpd = timeloop(lambda j: lx.prune_compress_lora(Xs[j], LB, 1, vs[j], ms[j], Ts[j]), nsets, iters)
        td = timeloop(lambda j: lx.lora_down(Xs[j], LB, ss[j], Ts[j]), nsets, iters)
        tl = timeloop(lambda j: lx.act_sparse_linear(Xs[j], Ws[j], b, 1, None, Ys[j], binding.FUSE_SEPARATE), nsets, iters)
        tll = timeloop(lambda j: lx.act_sparse_linear_lora(Xs[j], Ws[j], LA, LB, b, 1, None, Ys[j]), nsets, iters)

        def dense_lora(j):
            y = torch.nn.functional.linear(Xs[j], Ws[j], b)
            y.addmm_(torch.nn.functional.linear(Xs[j], LB), LA.t())

        tdl = timeloop(dense_lora, nsets, iters)
        print(f"| {M} | {K} | {N} | {R} | {tp*1e3:.1f} | {tpd*1e3:.1f} | {td*1e3:.1f} | {tl*1e3:.1f} | {tll*1e3:.1f} | "
              f"{100*(tll/tl-1):.1f} % | {tdl*1e3:.1f} | {tdl/tll:.2f} |", flush=True)
        assert lx.last_error() == 0
        del Xs, Ws, Ys, Ts, ss, vs, ms
        torch.cuda.empty_cache()


if __name__ == "__main__":
    main()
