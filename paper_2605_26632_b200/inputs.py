"""Seeded synthetic inputs shaped like the DiT linear layers the paper measures.

This module holds NO arithmetic of the method (no selection, compression, scaling or product):
it only draws random tensors.  It is the one module both the CPU oracle's tests and the CUDA
path's tests/bench read, so that both sides see the same bytes.

The paper measured on activations captured from Qwen-Image / FLUX.1-dev / Z-Image runs; those
models and prompts are not available offline, so these tensors stand in for them: same shapes
(Qwen-Image image-branch linears: (K, N) = (3072, 3072) Q/K/V/Out, (3072, 9216) fused QKV,
(3072, 12288) MLP up, (12288, 3072) MLP down; M = image tokens), activations concentrated near
zero after GELU for the MLP-down input, and a few high-magnitude outlier channels elsewhere.

Everything is generated on the CPU with ``torch.Generator().manual_seed(seed)`` in fp32 and
rounded once (nearest-even) to bf16.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Optional

import torch


@dataclass(frozen=True)
class Workload:
    name: str
    M: int
    K: int
    N: int
    x_dist: str  # "gelu", "gelu_chan", "outlier"
    seed: int


# The named configurations.  "tiny" is the full-oracle case; the others are DiT shaped.
WORKLOADS = {
    "tiny": Workload("tiny", 256, 512, 512, "gelu", 0),
    "mlp_down": Workload("mlp_down", 4096, 12288, 3072, "gelu_chan", 2),
    "attn_qkv": Workload("attn_qkv", 4352, 3072, 9216, "outlier", 3),
    "attn_out": Workload("attn_out", 4352, 3072, 3072, "outlier", 3),
    "mlp_up": Workload("mlp_up", 4096, 3072, 12288, "outlier", 4),
}

SWEEP_M = (1024, 4096, 8192, 16384)
SWEEP_KN = ((3072, 9216), (3072, 3072), (3072, 12288), (12288, 3072))
# Linear shapes that only the other two DiT families have: FLUX.1-dev single-stream blocks
# ((3072, 21504) fused QKV+MLP-up, (15360, 3072) fused Out+MLP-down) and Z-Image (hidden 3840,
# MLP 10240: N = 10240 is not a multiple of any tile width, so it exercises the column tail).
OTHER_FAMILY_KN = ((3072, 21504), (15360, 3072), (3840, 3840), (3840, 10240), (10240, 3840))
OTHER_FAMILY_M = 4096


def sweep_workload(M: int, K: int, N: int, index: int = 0) -> Workload:
    dist = "gelu_chan" if K >= 10240 else "outlier"
    return Workload(f"sweep_M{M}_K{K}_N{N}", M, K, N, dist, 5000 + index)


def _gen(seed: int) -> torch.Generator:
    g = torch.Generator(device="cpu")
    g.manual_seed(int(seed))
    return g


def make_x(M: int, K: int, dist: str, seed: int) -> torch.Tensor:
    """Activation matrix, bf16 [M, K] on the CPU."""
    g = _gen(seed)
    x = torch.randn(M, K, generator=g, dtype=torch.float32)
    if dist == "gelu":
        x = torch.nn.functional.gelu(x)  # exact (erf) GELU
    elif dist == "gelu_chan":
        x = torch.nn.functional.gelu(x)
        c = torch.exp(0.5 * torch.randn(K, generator=g, dtype=torch.float32))
        x = x * c
    elif dist == "outlier":
        n_out = K // 100
        idx = torch.randperm(K, generator=g)[:n_out]
        x[:, idx] *= 20.0
    elif dist == "normal":
        pass
    else:
        raise ValueError(dist)
    return x.to(torch.bfloat16).contiguous()


def make_w(N: int, K: int, seed: int) -> torch.Tensor:
    """Weight, bf16 [N, K], entries ~ N(0, 1/K)."""
    g = _gen(seed + 1_000_003)
    w = torch.randn(N, K, generator=g, dtype=torch.float32) * (K ** -0.5)
    return w.to(torch.bfloat16).contiguous()


def make_bias(N: int, seed: int) -> torch.Tensor:
    """Bias, bf16 [N], entries ~ N(0, 0.01^2)."""
    g = _gen(seed + 2_000_003)
    return (torch.randn(N, generator=g, dtype=torch.float32) * 0.01).to(torch.bfloat16).contiguous()


def make_residual(M: int, N: int, seed: int) -> torch.Tensor:
    """A stand-in for the low-rank branch output Y_r: bf16 [M, N], entries ~ N(0, 0.05^2)."""
    g = _gen(seed + 3_000_003)
    return (torch.randn(M, N, generator=g, dtype=torch.float32) * 0.05).to(torch.bfloat16).contiguous()


def make_lora(N: int, K: int, R: int, seed: int):
    """Low-rank factors -> (L_A [N, R], L_B [R, K]) bf16: L_B ~ N(0, 1/K), L_A ~ N(0, 0.3^2 / R),
    so that X (L_A L_B)^T is a correction of about a third of the main product's magnitude."""
    g = _gen(seed + 4_000_003)
    lb = torch.randn(R, K, generator=g, dtype=torch.float32) * (K ** -0.5)
    la = torch.randn(N, R, generator=g, dtype=torch.float32) * (0.3 * R ** -0.5)
    return la.to(torch.bfloat16).contiguous(), lb.to(torch.bfloat16).contiguous()


def make_workload(w: Workload, with_bias: bool = True, with_residual: bool = False,
                  M: Optional[int] = None):
    """-> dict(X, W, bias, residual) of CPU bf16 tensors (bias/residual may be None)."""
    m = w.M if M is None else M
    return {
        "X": make_x(m, w.K, w.x_dist, w.seed),
        "W": make_w(w.N, w.K, w.seed),
        "bias": make_bias(w.N, w.seed) if with_bias else None,
        "residual": make_residual(m, w.N, w.seed) if with_residual else None,
    }


def as_u16(t: torch.Tensor):
    """bf16 CPU tensor -> numpy uint16 view of the same bits."""
    import numpy as np

    return t.contiguous().view(torch.int16).numpy().view(np.uint16)


def from_u16(a) -> torch.Tensor:
    """numpy uint16 bit patterns -> bf16 CPU tensor."""
    import numpy as np

    return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).view(torch.bfloat16)
