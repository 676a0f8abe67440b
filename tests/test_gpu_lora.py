"""GPU parity tests of the low-rank branch (Algorithm 1 lines 5-6, Y = Y_s + X (L_A L_B)^T):
down projection kernel, the dense accumulator steps inside the sparse GEMM, and the whole layer,
through the C ABI against the CPU oracle.

Bars: T = bf16((X L_B^T) / s) within one bf16 rounding (2^-8 relative) plus the fp32
summation-order slack of the oracle's fp32 result; Y within relative Frobenius error 5e-3 and
max |dY| <= 2e-2 * max |Y_ref| (the T rounding is of the same size as Y's own bf16 rounding).
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_26632_b200 import inputs
from row_sampling import parity_rows, take

pytestmark = pytest.mark.gpu

RFE_TOL = 5e-3
MAXABS_TOL = 2e-2


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
    assert rfe <= RFE_TOL, f"relative Frobenius error {rfe}"
    assert mx <= MAXABS_TOL, f"max abs error ratio {mx}"


def make_case(M, K, N, R, seed, dist="outlier", with_bias=True, with_res=False):
    X = inputs.make_x(M, K, dist, seed)
    W = inputs.make_w(N, K, seed)
    b = inputs.make_bias(N, seed) if with_bias else None
    res = inputs.make_residual(M, N, seed) if with_res else None
    LA, LB = inputs.make_lora(N, K, R, seed)
    return X, W, b, res, LA, LB


def oracle_t(X, LB, mode):
    """(X L_B^T) / s from the oracle: the residual through an identity L_A is the down projection."""
    R = LB.shape[0]
    eye = torch.eye(R, dtype=torch.bfloat16)
    t = oracle.lora_residual(u16(X), u16(LB), u16(eye))
    if mode:
        s = oracle.row_scale(u16(X), mode).astype(np.float32)
        with np.errstate(divide="ignore", invalid="ignore"):
            t = np.where(s[:, None] == 0, 0.0, t / s[:, None]).astype(np.float32)
    return t


@pytest.mark.parametrize("M,K,R,mode", [
    (256, 512, 64, 0), (256, 512, 64, 1), (300, 1024, 64, 1), (129, 128, 64, 2), (1000, 3072, 128, 1),
    (4096, 3072, 64, 1), (2048, 12288, 64, 1),
])
def test_lora_down_matches_oracle(lx, M, K, R, mode):
    X = inputs.make_x(M, K, "outlier", 40 + M)
    _, LB = inputs.make_lora(8, K, R, 41 + M)
    Xc = X.cuda()
    scale = None
    if mode:
        _, _, scale = lx.prune_compress(Xc, mode)
    T = lx.lora_down(Xc, LB.cuda(), scale)
    ref = oracle_t(X, LB, mode)
    got = T.float().cpu().numpy()
    tol = 2.0 ** -8 * np.abs(ref) + 1e-5 * np.abs(ref).max()
    assert (np.abs(got - ref) <= tol).all(), float(np.abs(got - ref).max())
    # reproducible whichever CTA finishes last
    T2 = lx.lora_down(Xc, LB.cuda(), scale)
    assert torch.equal(T, T2)


@pytest.mark.parametrize("M,K,R,mode", [
    (256, 512, 64, 0), (256, 512, 64, 1), (300, 1024, 64, 1), (129, 128, 64, 1), (1, 128, 64, 1),
    (1000, 3072, 128, 1), (700, 1664, 128, 0), (4096, 3072, 64, 1), (2048, 12288, 64, 1), (4352, 3072, 64, 0),
])
def test_prune_compress_lora_one_pass(lx, M, K, R, mode):
    """Prune / compress and the down projection in one launch (X read once): values and metadata
    bit for bit, T within a bf16 rounding, the row sums good for the GEMM that follows."""
    from paper_2605_26632_b200 import binding

    X = inputs.make_x(M, K, "outlier", 60 + M)
    N = 264
    W, b = inputs.make_w(N, K, 61 + M), inputs.make_bias(N, 61 + M)
    LA, LB = inputs.make_lora(N, K, R, 62 + M)
    Xc = X.cuda()
    values, meta, T = lx.prune_compress_lora(Xc, LB.cuda(), mode)
    ov, om = oracle.compress(u16(X))
    assert (u16(values) == ov).all(), "values differ"
    assert (meta.cpu().numpy() == oracle.meta_canon_to_hw(om, M, K)).all(), "metadata differs"
    ref = oracle_t(X, LB, mode)
    got = T.float().cpu().numpy()
    tol = 2.0 ** -8 * np.abs(ref) + 1e-5 * np.abs(ref).max()
    assert (np.abs(got - ref) <= tol).all(), float(np.abs(got - ref).max())
    # the GEMM that follows takes the row sums the launch left on the context
    Y = lx.sparse_linear_lora(values, meta, W.cuda(), T, LA.cuda(), b.cuda(),
                              binding.ROW_SCALE_DEFERRED if mode else None)
    yref = oracle.act_sparse_linear_lora(u16(X), u16(W), u16(LA), u16(LB), bias=u16(b), comp_mode=mode)
    check_y(Y, yref["Y"])
    # reproducible whichever CTA finishes a row block, and the layer call is these two launches
    values2, meta2, T2 = lx.prune_compress_lora(Xc, LB.cuda(), mode)
    assert torch.equal(T, T2) and torch.equal(values, values2) and torch.equal(meta, meta2)
    Y2 = lx.act_sparse_linear_lora(Xc, W.cuda(), LA.cuda(), LB.cuda(), b.cuda(), mode)
    assert torch.equal(Y, Y2)


@pytest.mark.parametrize("splits,K", [(1, 3584), (2, 3584), (3, 3584), (4, 3584), (5, 3584), (6, 3584), (7, 3584),
                                      (8, 4096)])
def test_prune_compress_lora_every_cluster_size(splits, K, monkeypatch):
    """The K splits of a row block form a cluster of 1..8 CTAs that add their partials through
    distributed shared memory; rows are shared out unevenly when the size does not divide 128."""
    from paper_2605_26632_b200 import binding

    monkeypatch.setenv("LYNX_PL_SPLITS", str(splits))
    ctx = binding.Lynx(0)
    try:
        M, R = 390, 64
        X = inputs.make_x(M, K, "outlier", 90 + splits)
        _, LB = inputs.make_lora(8, K, R, 91 + splits)
        values, meta, T = ctx.prune_compress_lora(X.cuda(), LB.cuda(), 1)
        ov, om = oracle.compress(u16(X))
        assert (u16(values) == ov).all()
        assert (meta.cpu().numpy() == oracle.meta_canon_to_hw(om, M, K)).all()
        ref = oracle_t(X, LB, 1)
        got = T.float().cpu().numpy()
        tol = 2.0 ** -8 * np.abs(ref) + 1e-5 * np.abs(ref).max()
        assert (np.abs(got - ref) <= tol).all(), float(np.abs(got - ref).max())
        torch.cuda.synchronize()
        assert ctx.last_error() == 0
    finally:
        ctx.close()


def test_prune_compress_lora_zero_rows_leading_dimensions_and_errors(lx):
    from paper_2605_26632_b200 import binding

    M, K, R = 200, 384, 64
    X = inputs.make_x(M, K, "outlier", 9)
    X[5] = 0
    X[199] = 0
    _, LB = inputs.make_lora(8, K, R, 9)
    wideX = torch.zeros((M, K + 64), dtype=torch.bfloat16)
    wideX[:, :K] = X
    wideLB = torch.zeros((R, K + 8), dtype=torch.bfloat16)
    wideLB[:, :K] = LB
    buf = torch.full((M, 2 * R), 7.0, dtype=torch.bfloat16, device="cuda")
    values, meta, T = lx.prune_compress_lora(wideX.cuda()[:, :K], wideLB.cuda()[:, :K], 1, T=buf[:, :R])
    assert (T[5] == 0).all() and (T[199] == 0).all()
    assert (buf[:, R:] == 7.0).all()
    ov, om = oracle.compress(u16(X))
    assert (u16(values) == ov).all()
    assert (meta.cpu().numpy() == oracle.meta_canon_to_hw(om, M, K)).all()
    ref = oracle_t(X, LB, 1)
    assert np.abs(T.float().cpu().numpy() - ref).max() <= 2.0 ** -8 * np.abs(ref).max() + 1e-6
    for bad_mode in (binding.COMP_TENSOR, binding.COMP_GROUP):
        with pytest.raises(binding.LynxError) as e:
            lx.prune_compress_lora(X.cuda(), LB.cuda(), bad_mode)
        assert e.value.status == 1
    with pytest.raises(binding.LynxError) as e:  # rank 32 is not built
        lx.prune_compress_lora(X.cuda(), LB.cuda()[:32], 1)
    assert e.value.status == 2


def test_lora_down_zero_rows_and_strided_output(lx):
    M, K, R = 200, 256, 64
    X = inputs.make_x(M, K, "outlier", 7)
    X[5] = 0
    X[199] = 0
    _, LB = inputs.make_lora(8, K, R, 7)
    Xc = X.cuda()
    _, _, scale = lx.prune_compress(Xc, 1)
    buf = torch.full((M, 2 * R), 7.0, dtype=torch.bfloat16, device="cuda")
    T = lx.lora_down(Xc, LB.cuda(), scale, out=buf[:, :R])
    assert (T[5] == 0).all() and (T[199] == 0).all()
    assert (buf[:, R:] == 7.0).all()
    ref = oracle_t(X, LB, 1)
    assert np.abs(T.float().cpu().numpy() - ref).max() <= 2.0 ** -8 * np.abs(ref).max() + 1e-6


@pytest.mark.parametrize("mode", [0, 1, 2])
@pytest.mark.parametrize("with_bias,with_res", [(False, False), (True, True)])
def test_tiny_config_with_lora_full_oracle(lx, mode, with_bias, with_res):
    wl = inputs.WORKLOADS["tiny"]
    X, W, b, res, LA, LB = make_case(wl.M, wl.K, wl.N, 64, wl.seed, wl.x_dist, with_bias, with_res)
    ref = oracle.act_sparse_linear_lora(u16(X), u16(W), u16(LA), u16(LB), bias=None if b is None else u16(b),
                                        comp_mode=mode, Yr=None if res is None else u16(res))
    cu = lambda t: None if t is None else t.cuda()
    Y = lx.act_sparse_linear_lora(X.cuda(), W.cuda(), LA.cuda(), LB.cuda(), cu(b), mode, cu(res))
    check_y(Y, ref["Y"])
    # the three-call form (own down-projection kernel; the layer call computes T in its prune launch
    # with another K split, so the two may differ in T's last bit)
    values, meta, scale = lx.prune_compress(X.cuda(), mode)
    T = lx.lora_down(X.cuda(), LB.cuda(), scale)
    Y2 = lx.sparse_linear_lora(values, meta, W.cuda(), T, LA.cuda(), cu(b), scale, cu(res))
    check_y(Y2, ref["Y"])
    # and the branch really contributes: without it the result is off by the residual's size
    Y0 = lx.act_sparse_linear(X.cuda(), W.cuda(), cu(b), mode, cu(res))
    assert (Y.float() - Y0.float()).abs().max().item() > 0.05


def test_zero_weight_leaves_the_dense_low_rank_product(lx):
    """W = 0: Y must equal X (L_A L_B)^T computed from the DENSE X (silicon check of the dense
    tensor-core steps: operand order, K advance, both halves of a CTA pair)."""
    M, K, N, R = 520, 384, 1000, 64
    X, _, _, _, LA, LB = make_case(M, K, N, R, 77)
    W = torch.zeros(N, K, dtype=torch.bfloat16)
    Y = lx.act_sparse_linear_lora(X.cuda(), W.cuda(), LA.cuda(), LB.cuda(), None, 1)
    ref = ((X.double() @ LB.double().T) @ LA.double().T).numpy()
    check_y(Y, ref)


def test_three_call_form_equals_unfused_layer_bit_for_bit(monkeypatch):
    from paper_2605_26632_b200 import binding

    monkeypatch.setenv("LYNX_LORA_FUSE", "0")
    ctx = binding.Lynx(0)
    try:
        X, W, b, res, LA, LB = make_case(520, 640, 1000, 64, 321, with_res=True)
        Y = ctx.act_sparse_linear_lora(X.cuda(), W.cuda(), LA.cuda(), LB.cuda(), b.cuda(), 1, res.cuda())
        values, meta, scale = ctx.prune_compress(X.cuda(), 1)
        T = ctx.lora_down(X.cuda(), LB.cuda(), scale)
        Y2 = ctx.sparse_linear_lora(values, meta, W.cuda(), T, LA.cuda(), b.cuda(), scale, res.cuda())
        assert torch.equal(Y, Y2)
    finally:
        ctx.close()


@pytest.mark.parametrize("fuse", [2, 1, 0])
@pytest.mark.parametrize("cfg", [1, 2, 3, 4, 5, 6, 7, 8])
@pytest.mark.parametrize("R", [64, 128])
def test_every_tile_configuration_with_lora(cfg, R, fuse, monkeypatch):
    """fuse = 2 (default): the down projection runs in the prune launch; fuse = 1: inside the GEMM
    launch where the tile has room for it (rank 64, every tile but the 256 x 128 pair tile);
    fuse = 0: always as its own kernel."""
    from paper_2605_26632_b200 import binding

    if fuse == 0 and R == 128:
        pytest.skip("rank 128 always uses the separate kernel; covered by fuse = 1")
    monkeypatch.setenv("LYNX_GEMM_CFG", str(cfg))
    monkeypatch.setenv("LYNX_LORA_FUSE", str(fuse))
    ctx = binding.Lynx(0)
    try:
        M, K, N = 700, 1664, 1096  # ragged in M and N for every tile width; 13 K blocks split unevenly
        X, W, b, res, LA, LB = make_case(M, K, N, R, 500 + cfg, with_res=True)
        ref = oracle.act_sparse_linear_lora(u16(X), u16(W), u16(LA), u16(LB), bias=u16(b), comp_mode=1, Yr=u16(res))
        Y = ctx.act_sparse_linear_lora(X.cuda(), W.cuda(), LA.cuda(), LB.cuda(), b.cuda(), 1, res.cuda())
        check_y(Y, ref["Y"])
        Y2 = ctx.act_sparse_linear_lora(X.cuda(), W.cuda(), LA.cuda(), LB.cuda(), b.cuda(), 1, res.cuda())
        assert torch.equal(Y, Y2)
        torch.cuda.synchronize()
        assert ctx.last_error() == 0
    finally:
        ctx.close()


@pytest.mark.parametrize("doubles", [-1, 0, 100000])
@pytest.mark.parametrize("R", [64, 128])
def test_two_row_tile_gemm_kernel_with_lora(R, doubles, monkeypatch):
    """The low-rank stages inside the GEMM kernel that runs two row tiles per W stage."""
    from paper_2605_26632_b200 import binding

    monkeypatch.setenv("LYNX_RT2", "1")
    monkeypatch.setenv("LYNX_RT2_D", str(doubles))
    ctx = binding.Lynx(0)
    try:
        M, K, N = 1100, 1664, 1096  # 5 row tiles (odd), ragged rows and columns
        X, W, b, res, LA, LB = make_case(M, K, N, R, 900 + R, with_res=True)
        ref = oracle.act_sparse_linear_lora(u16(X), u16(W), u16(LA), u16(LB), bias=u16(b), comp_mode=1, Yr=u16(res))
        Y = ctx.act_sparse_linear_lora(X.cuda(), W.cuda(), LA.cuda(), LB.cuda(), b.cuda(), 1, res.cuda())
        check_y(Y, ref["Y"])
        Y2 = ctx.act_sparse_linear_lora(X.cuda(), W.cuda(), LA.cuda(), LB.cuda(), b.cuda(), 1, res.cuda())
        assert torch.equal(Y, Y2)
        torch.cuda.synchronize()
        assert ctx.last_error() == 0
    finally:
        ctx.close()


@pytest.mark.parametrize("cfg", [4, 7])
def test_stream_k_with_lora(cfg, monkeypatch):
    from paper_2605_26632_b200 import binding

    monkeypatch.setenv("LYNX_GEMM_CFG", str(cfg))
    monkeypatch.setenv("LYNX_STREAMK", "1")
    ctx = binding.Lynx(0)
    try:
        M, K, N = 2304, 2048, 2880  # leaves a tail of tiles, long enough in K for the stream-K split
        X, W, b, _, LA, LB = make_case(M, K, N, 64, 600 + cfg)
        rows = np.arange(0, M, 37, dtype=np.int64)
        ref = oracle.act_sparse_linear_lora(u16(X), u16(W), u16(LA), u16(LB), bias=u16(b), comp_mode=1, rows=rows)
        Y = ctx.act_sparse_linear_lora(X.cuda(), W.cuda(), LA.cuda(), LB.cuda(), b.cuda(), 1)
        check_y(Y[torch.from_numpy(rows).cuda()], ref["Y"])
        torch.cuda.synchronize()
        assert ctx.last_error() == 0
    finally:
        ctx.close()


@pytest.mark.parametrize("name", ["mlp_down", "attn_out", "mlp_up"])
def test_dit_workloads_full_size_with_lora(lx, name):
    """Y of every row and column against the oracle (M <= 4608: row_sampling.parity_rows)."""
    wl = inputs.WORKLOADS[name]
    X, W, b, _, LA, LB = make_case(wl.M, wl.K, wl.N, 64, wl.seed, wl.x_dist)
    rows = parity_rows(wl.M, wl.seed)
    ref = oracle.act_sparse_linear_lora(u16(X), u16(W), u16(LA), u16(LB), bias=u16(b), comp_mode=1, rows=rows)
    Y = lx.act_sparse_linear_lora(X.cuda(), W.cuda(), LA.cuda(), LB.cuda(), b.cuda(), 1)
    check_y(take(Y, rows), ref["Y"])


def test_lora_argument_errors(lx):
    from paper_2605_26632_b200.binding import LynxError

    X = torch.zeros(128, 256, dtype=torch.bfloat16, device="cuda")
    W = torch.zeros(64, 256, dtype=torch.bfloat16, device="cuda")
    for R in (32, 96, 256):
        LA = torch.zeros(64, R, dtype=torch.bfloat16, device="cuda")
        LB = torch.zeros(R, 256, dtype=torch.bfloat16, device="cuda")
        n0 = lx.launch_count()
        with pytest.raises(LynxError) as e:
            lx.act_sparse_linear_lora(X, W, LA, LB)
        assert e.value.status == 2  # unsupported shape
        assert lx.launch_count() == n0
    LB = torch.zeros(64, 512, dtype=torch.bfloat16, device="cuda")[:, ::2]  # wrong inner stride
    with pytest.raises(TypeError):
        lx.lora_down(X, LB)
