"""`lynx_prune_compress_static`: the prune/compress entry point for callers that cannot allocate
device memory (their own pool owns the GPU, or an allocation's device-wide synchronisation is not
acceptable where they call from).  It keeps its partial row sums in a fixed array inside the
library instead of context scratch.  Checked here against the ordinary entry point, through the
C ABI, on two calls in a row (the second finds the first call's leftovers in the shared array).

Collected last on purpose: a run that stops at the first failure has then run every other test.
"""
import pytest
import torch

from paper_2605_26632_b200 import inputs

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("mode", [1, 2])
def test_static_scratch_entry_matches_context_entry_twice_in_a_row(mode):
    from paper_2605_26632_b200 import binding

    lx = binding.Lynx(0)
    try:
        # two different shapes and inputs, back to back: K splits > 1 so that the scratch is used
        cases = [(1000, 3072, "outlier", 41), (384, 1024, "gelu", 42)]
        for (M, K, dist, seed) in cases:
            X = inputs.make_x(M, K, dist, seed).cuda()
            v_ref, m_ref, s_ref = lx.prune_compress(X, mode)
            v, m, s = binding.prune_compress_static(X, mode)
            torch.cuda.synchronize()
            assert torch.equal(v, v_ref), "values differ"
            assert torch.equal(m, m_ref), "metadata differs"
            torch.testing.assert_close(s, s_ref, rtol=1e-5, atol=0.0)
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
