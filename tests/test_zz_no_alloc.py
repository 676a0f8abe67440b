"""`lynx_prune_compress_static`: the prune/compress entry point for callers that cannot allocate
device memory (their own pool owns the GPU, or an allocation's device-wide synchronisation is not
acceptable where they call from).  It keeps its partial row sums in a fixed array inside the
library instead of context scratch.

Checked here, through the C ABI, against the CPU oracle (values, hardware-order metadata and the
row scale) for every compensation mode, and against the ordinary entry point, always on two calls
in a row (the second finds the first call's leftovers in the shared array).  Shapes: several K
splits (the partial sums use the array), K = 128 (one split: no partial sums at all), a single
row, and ragged 16- and 128-row blocks.

Collected last on purpose: a run that stops at the first failure has then run every other test.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_26632_b200 import inputs

pytestmark = pytest.mark.gpu

SCALE_RTOL = 1e-5
GROUP = 3

# (M, K, distribution, seed): K = 3072 / 1024 split the row sums over several warps, K = 128 does not
CASES = [(1000, 3072, "outlier", 41), (384, 1024, "gelu", 42), (200, 128, "normal", 43), (1, 128, "gelu", 44),
         (200, 384, "gelu_chan", 45), (17, 256, "outlier", 46)]


def u16(t):
    return inputs.as_u16(t.detach().cpu())


@pytest.mark.parametrize("mode", [0, 1, 2, GROUP])
def test_static_scratch_entry_matches_the_oracle_twice_in_a_row(mode):
    from paper_2605_26632_b200 import binding

    lx = binding.Lynx(0)
    try:
        for (M, K, dist, seed) in CASES:
            Xc = inputs.make_x(M, K, dist, seed)
            Xu = u16(Xc)
            if mode == GROUP:
                ov, om = oracle.compress_group_scaled(Xu)
            else:
                ov, om = oracle.compress(Xu)
            hw = oracle.meta_canon_to_hw(om, M, K)
            X = Xc.cuda()
            for call in range(2):  # back to back on the shared array
                v, m, s = binding.prune_compress_static(X, mode)
                torch.cuda.synchronize()
                assert (u16(v) == ov).all(), f"values differ from the oracle (call {call})"
                assert (m.cpu().numpy() == hw).all(), f"metadata differs from the oracle (call {call})"
                if mode in (1, 2):
                    np.testing.assert_allclose(s.cpu().numpy(), oracle.row_scale(Xu, mode), rtol=SCALE_RTOL)
            # and the ordinary entry point gives the same bits (one work decomposition for both)
            v_ref, m_ref, s_ref = lx.prune_compress(X, mode)
            assert torch.equal(v, v_ref) and torch.equal(m, m_ref)
            if mode in (1, 2):
                assert torch.equal(s, s_ref), "row scale bits differ between the two entry points"
        torch.cuda.synchronize()
        assert lx.last_error() == 0
    finally:
        lx.close()


def test_static_scratch_entry_rejects_oversized_shapes_and_bad_arguments():
    from paper_2605_26632_b200 import binding

    lib = binding.load_library()
    from ctypes import c_void_p

    X = torch.zeros(16, 128, dtype=torch.bfloat16, device="cuda")
    v = torch.empty(16, 64, dtype=torch.bfloat16, device="cuda")
    m = torch.empty(2048, dtype=torch.uint8, device="cuda")
    s = torch.empty(16, dtype=torch.float32, device="cuda")
    p = lambda t: c_void_p(t.data_ptr())
    # M * K far beyond what the fixed array can hold partial sums for (no memory is touched:
    # the size check comes before any launch)
    st = lib.lynx_prune_compress_static(p(X), 1 << 22, 128 * 64, 128 * 64, p(v), p(m), p(s), 1, None)
    assert st == 4 and "scratch" in binding.status_string(st)
    assert lib.lynx_prune_compress_static(p(X), 16, 192, 192, p(v), p(m), p(s), 1, None) == 2
    assert lib.lynx_prune_compress_static(p(X), 16, 128, 128, p(v), p(m), None, 1, None) == 1
    torch.cuda.synchronize()
