"""Which rows of Y the full-size parity tests compare with the oracle.

Rule: every row when M <= 4608 (the oracle needs a few seconds for such a product on the host
cores); for taller problems at least 512 rows chosen so that every 128-row block (the rows one
CTA of the GEMM owns) contributes its first and its last row, the rest seeded at random.  All N
columns of a chosen row are compared, so every output tile of the GEMM is touched.
"""
import numpy as np

ALL_ROWS_UP_TO = 4608
MIN_SAMPLED_ROWS = 512


def parity_rows(M: int, seed: int, all_rows_up_to: int = ALL_ROWS_UP_TO, min_rows: int = MIN_SAMPLED_ROWS):
    """-> None (= all rows) or a sorted int64 array of distinct row indices."""
    if M <= all_rows_up_to:
        return None
    blocks = (M + 127) // 128
    first = np.arange(blocks, dtype=np.int64) * 128
    last = np.minimum(first + 127, M - 1)
    fixed = np.unique(np.concatenate([first, last]))
    want = min(M, max(min_rows, 2 * blocks + 128))
    rest = np.setdiff1d(np.arange(M, dtype=np.int64), fixed)
    extra = np.random.default_rng(seed).choice(rest, max(0, want - fixed.size), replace=False)
    rows = np.unique(np.concatenate([fixed, extra])).astype(np.int64)
    assert rows.size >= min(M, min_rows)
    return rows


def take(Y, rows):
    """Rows of a device tensor Y (all of it when rows is None)."""
    if rows is None:
        return Y
    import torch

    return Y[torch.from_numpy(rows).to(Y.device)]
