"""B200 (sm_100a) 2:4 activation-sparse linear layer: Top-2-of-4 prune/compress, sparse tensor-core
GEMM and fused epilogue behind a C-ABI library, with a thin Python binding.

``inputs`` (seeded synthetic workloads) can be imported without a GPU; everything in ``binding``
needs the CUDA library and fails loudly without it.
"""
__all__ = ["inputs", "binding", "build"]
