"""GPU parity tests of per-group norm compensation (LYNX_COMP_GROUP: the norm-compensation equation
read literally, one factor per group of four, folded into the stored values).

Bars: scaled values and metadata bit-exact against the oracle's fp32 reading (same IEEE operations
in the same order on both sides; NaN positions compare as NaN, their payload is not defined);
Y within relative Frobenius error 5e-3 and max |dY| <= 2e-2 * max |Y_ref|.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_26632_b200 import inputs
from row_sampling import parity_rows, take

pytestmark = pytest.mark.gpu

GROUP = 3


@pytest.fixture(scope="module")
def lx():
    from paper_2605_26632_b200 import binding

    ctx = binding.Lynx(0)
    yield ctx
    torch.cuda.synchronize()
    assert ctx.last_error() == 0
    ctx.close()


def u16(t):
    return inputs.as_u16(t.detach().cpu())


def check_y(Y, ref):
    yf = Y.float().cpu().numpy()
    rfe = np.linalg.norm(yf - ref) / max(np.linalg.norm(ref), 1e-30)
    mx = np.abs(yf - ref).max() / max(np.abs(ref).max(), 1e-30)
    assert rfe <= 5e-3, f"relative Frobenius error {rfe}"
    assert mx <= 2e-2, f"max abs error ratio {mx}"


@pytest.mark.parametrize("M,K,dist", [
    (256, 512, "gelu"), (300, 1024, "outlier"), (129, 128, "gelu_chan"), (1, 128, "outlier"),
    (4096, 3072, "outlier"), (2048, 12288, "gelu_chan"),
])
def test_group_scaled_values_and_metadata_are_bit_exact(lx, M, K, dist):
    X = inputs.make_x(M, K, dist, 900 + M)
    values, meta, scale = lx.prune_compress(X.cuda(), GROUP)
    assert scale is None
    ov, om = oracle.compress_group_scaled(u16(X))
    assert (u16(values) == ov).all(), "scaled values differ"
    assert (meta.cpu().numpy() == oracle.meta_canon_to_hw(om, M, K)).all(), "metadata differs"
    # the mask is the plain Top-2-of-4 one
    _, om0 = oracle.compress(u16(X))
    assert (om == om0).all()


def test_group_mode_strided_input_and_row_scale_written_as_one(lx):
    M, K = 200, 384
    X = inputs.make_x(M, 2 * K, "outlier", 31)
    Xc = X.cuda()[:, :K]
    scale = torch.full((M,), 7.0, dtype=torch.float32, device="cuda")
    values, meta, s = lx.prune_compress(Xc, GROUP, row_scale=scale)
    assert (s == 1.0).all()
    ov, om = oracle.compress_group_scaled(u16(X[:, :K].contiguous()))
    assert (u16(values) == ov).all()


def test_group_mode_special_values(lx):
    M, K = 32, 128
    g = torch.Generator().manual_seed(5)
    x = torch.randn(M, K, generator=g)
    x[0, 0:4] = 0.0
    x[1, 0:4] = torch.tensor([1e-40, -1e-40, 2e-40, 0.0])      # subnormals in bf16
    x[2, 0:4] = torch.tensor([float("inf"), 1.0, -2.0, 0.5])
    x[3, 0:4] = torch.tensor([float("nan"), 1.0, -2.0, 0.5])
    x[4, 0:4] = torch.tensor([-0.0, 0.0, -0.0, 0.0])
    x[5, 0:4] = torch.tensor([3e38, 3e38, 1.0, 1.0])            # squares overflow fp32
    X = x.to(torch.bfloat16)
    values, meta, _ = lx.prune_compress(X.cuda(), GROUP)
    ov, om = oracle.compress_group_scaled(u16(X))
    got = u16(values)
    gf, of = inputs.from_u16(got).float().numpy(), inputs.from_u16(ov).float().numpy()
    nan = np.isnan(of)
    assert (np.isnan(gf) == nan).all()
    assert (got[~nan] == ov[~nan]).all()
    assert (meta.cpu().numpy() == oracle.meta_canon_to_hw(om, M, K)).all()


@pytest.mark.parametrize("with_bias,with_res", [(False, False), (True, True)])
def test_tiny_config_group_mode_full_oracle(lx, with_bias, with_res):
    wl = inputs.WORKLOADS["tiny"]
    d = inputs.make_workload(wl, with_bias=with_bias, with_residual=with_res)
    cu = lambda t: None if t is None else t.cuda()
    ref = oracle.act_sparse_linear(u16(d["X"]), u16(d["W"]), bias=None if d["bias"] is None else u16(d["bias"]),
                                   comp_mode=GROUP, Yr=None if d["residual"] is None else u16(d["residual"]))
    Y = lx.act_sparse_linear(d["X"].cuda(), d["W"].cuda(), cu(d["bias"]), GROUP, cu(d["residual"]))
    check_y(Y, ref["Y"])
    # the two-call form: same bits
    values, meta, _ = lx.prune_compress(d["X"].cuda(), GROUP)
    Y2 = lx.sparse_linear(values, meta, d["W"].cuda(), cu(d["bias"]), None, cu(d["residual"]))
    assert torch.equal(Y, Y2)


def test_full_size_mlp_down_group_mode(lx):
    """Y of every row and column against the oracle."""
    wl = inputs.WORKLOADS["mlp_down"]
    d = inputs.make_workload(wl, with_bias=True)
    rows = parity_rows(wl.M, wl.seed)
    ref = oracle.act_sparse_linear(u16(d["X"]), u16(d["W"]), bias=u16(d["bias"]), comp_mode=GROUP, rows=rows)
    Y = lx.act_sparse_linear(d["X"].cuda(), d["W"].cuda(), d["bias"].cuda(), GROUP)
    check_y(take(Y, rows), ref["Y"])


def test_group_mode_with_low_rank_branch(lx):
    M, K, N, R = 520, 640, 1000, 64
    X = inputs.make_x(M, K, "outlier", 77)
    W = inputs.make_w(N, K, 77)
    b = inputs.make_bias(N, 77)
    LA, LB = inputs.make_lora(N, K, R, 77)
    ref = oracle.act_sparse_linear_lora(u16(X), u16(W), u16(LA), u16(LB), bias=u16(b), comp_mode=GROUP)
    Y = lx.act_sparse_linear_lora(X.cuda(), W.cuda(), LA.cuda(), LB.cuda(), b.cuda(), GROUP)
    check_y(Y, ref["Y"])


def test_group_mode_restores_the_norm_better_than_no_compensation(lx):
    """Sanity of the method, not of the kernel: on a GELU-like input the per-group factor brings
    |S(X)|_F back to |X|_F, which plain pruning does not."""
    X = inputs.make_x(512, 1024, "gelu", 3).cuda()
    v0, m0, _ = lx.prune_compress(X, 0)
    v3, m3, _ = lx.prune_compress(X, GROUP)
    n = X.float().norm().item()
    n0 = lx.decompress(v0, m0).float().norm().item()
    n3 = lx.decompress(v3, m3).float().norm().item()
    assert abs(n3 / n - 1.0) < 2e-3 < abs(n0 / n - 1.0)


def test_group_mode_static_entry_and_fused_rejection(lx):
    from paper_2605_26632_b200 import binding

    X = inputs.make_x(300, 512, "outlier", 12).cuda()
    v, m, _ = lx.prune_compress(X, GROUP)
    v2, m2, _ = binding.prune_compress_static(X, GROUP)
    assert torch.equal(v, v2) and torch.equal(m, m2)
    W = inputs.make_w(256, 512, 12).cuda()
    n0 = lx.launch_count()
    with pytest.raises(binding.LynxError) as e:
        lx.act_sparse_linear(X, W, None, GROUP, None, None, binding.FUSE_FUSED)
    assert e.value.status == 2
    assert lx.launch_count() == n0
