"""GPU parity tests: the CUDA path (through the C ABI) against the CPU oracle.

Bars: selection masks, values and metadata bit-exact; row scale within 1e-5 relative (fp32 sums in
a different order than the oracle's fp64 sums); Y within relative Frobenius error 5e-3 and
max |dY| <= 2e-2 * max |Y_ref| of the oracle's fp32 result.
"""
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2605_26632_b200 import inputs
from row_sampling import parity_rows, take

pytestmark = pytest.mark.gpu

RFE_TOL = 5e-3
MAXABS_TOL = 2e-2
SCALE_RTOL = 1e-5


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
    return rfe, mx


def check_compressed(lx, X, values, meta, scale=None, mode=0):
    """values / metadata (hardware order and canonical) / decompression, all bit-exact."""
    M, K = X.shape
    Xu = u16(X)
    ov, om = oracle.compress(Xu)
    assert (u16(values) == ov).all(), "values differ"
    assert (meta.cpu().numpy() == oracle.meta_canon_to_hw(om, M, K)).all(), "hardware metadata differs"
    canon = lx.meta_to_canonical(meta, M, K).cpu().numpy().view(np.uint16)
    assert (canon == om).all(), "canonical metadata differs"
    dec = u16(lx.decompress(values, meta))
    assert (dec == Xu * oracle.topk24_mask(Xu)).all(), "decompress(compress(X)) != mask * X"
    if mode:
        np.testing.assert_allclose(scale.cpu().numpy(), oracle.row_scale(Xu, mode), rtol=SCALE_RTOL)
    return ov, om


# ------------------------------------------------------------------ prune / compress -----------

@pytest.mark.parametrize("M,K,dist,mode", [
    (256, 512, "gelu", 1),        # the tiny configuration
    (1, 128, "normal", 1),        # single row, single K block
    (17, 256, "outlier", 2),      # ragged 16-row block
    (200, 384, "gelu_chan", 1),   # ragged 128-row block, K not a multiple of 1024
    (300, 1024, "normal", 0),
    (1000, 3072, "outlier", 2),
])
def test_prune_compress_matches_oracle(lx, M, K, dist, mode):
    X = inputs.make_x(M, K, dist, 100 + M).cuda()
    values, meta, scale = lx.prune_compress(X, mode)
    check_compressed(lx, X, values, meta, scale, mode)


def test_prune_compress_strided_input(lx):
    M, K = 96, 256
    big = inputs.make_x(M, 512, "normal", 5).cuda()
    X = big[:, 128:128 + K]  # ldx = 512, 32-byte aligned start
    values, meta, scale = lx.prune_compress(X, 1)
    check_compressed(lx, X.contiguous(), values, meta, scale, 1)


def test_prune_compress_special_values(lx):
    """NaN, +-Inf, +-0 and subnormals rank by their 15 magnitude bits; ties go to the lower index."""
    rng = np.random.default_rng(1)
    pool = np.array([0x0000, 0x8000, 0x7FC0, 0xFFC1, 0x7F80, 0xFF80, 0x0001, 0x8001, 0x007F, 0x3F80, 0xBF80,
                     0x3F81, 0x4000, 0x7F7F], dtype=np.uint16)
    Xn = pool[rng.integers(0, len(pool), size=(64, 256))]
    X = inputs.from_u16(Xn).cuda()
    values, meta, _ = lx.prune_compress(X, 0)
    ov, om = oracle.compress(Xn)
    assert (u16(values) == ov).all()
    assert (meta.cpu().numpy() == oracle.meta_canon_to_hw(om, 64, 256)).all()


def test_prune_compress_all_bit_patterns(lx):
    rng = np.random.default_rng(2)
    Xn = rng.integers(0, 1 << 16, size=(128, 512), dtype=np.uint16)
    X = inputs.from_u16(Xn).cuda()
    values, meta, _ = lx.prune_compress(X, 0)
    ov, om = oracle.compress(Xn)
    assert (u16(values) == ov).all()
    assert (meta.cpu().numpy() == oracle.meta_canon_to_hw(om, 128, 512)).all()


def test_prune_compress_is_deterministic(lx):
    X = inputs.make_x(512, 1024, "gelu", 9).cuda()
    a = lx.prune_compress(X, 1)
    b = lx.prune_compress(X, 1)
    for s, t in zip(a, b):
        assert torch.equal(s, t)


@pytest.mark.parametrize("M,K", [(300, 8192), (200, 384), (1000, 12288)])
def test_row_scale_finalize_forms_agree_bit_for_bit(M, K, monkeypatch):
    """The per-row scale is finished either by the last CTA of a row block inside the prune kernel
    (ticket) or by a small dependent launch over the partial sums (the default for K >= 8192):
    the same additions in the same order, so the same bits; both within 1e-5 of the oracle."""
    from paper_2605_26632_b200 import binding

    X = inputs.make_x(M, K, "gelu_chan", 500 + M)
    want = oracle.row_scale(u16(X), 1)
    got = []
    for form in ("1", "2", "0"):
        monkeypatch.setenv("LYNX_PRUNE_FINALIZE", form)
        ctx = binding.Lynx(0)
        try:
            values, meta, scale = ctx.prune_compress(X.cuda(), 1)
            check_compressed(ctx, X.cuda(), values, meta, scale, 1)
            np.testing.assert_allclose(scale.cpu().numpy(), want, rtol=SCALE_RTOL)
            got.append(scale.clone())
            torch.cuda.synchronize()
            assert ctx.last_error() == 0
        finally:
            ctx.close()
    assert torch.equal(got[0], got[1]) and torch.equal(got[0], got[2])


# ------------------------------------------------------------------ silicon pins of the layout --

@pytest.mark.parametrize("M,K", [(128, 128), (256, 512), (300, 1024)])
def test_identity_weight_returns_masked_x_exactly(lx, M, K):
    """W = I: every product is x*1 and every other addend is 0, so Y must equal mask*X bit for bit
    (up to the sign of zero).  Any error in the metadata or value layout shows here."""
    X = inputs.make_x(M, K, "normal", 3).cuda()
    values, meta, _ = lx.prune_compress(X, 0)
    W = torch.eye(K, dtype=torch.bfloat16, device="cuda")
    Y = lx.sparse_linear(values, meta, W)
    Xu = u16(X)
    want = oracle.bf16_to_f32(Xu * oracle.topk24_mask(Xu))
    assert (Y.float().cpu().numpy() == want).all()


def test_one_hot_probes(lx):
    M, K = 128, 256
    W = torch.eye(K, dtype=torch.bfloat16, device="cuda")
    for (m, k) in [(0, 0), (7, 3), (8, 17), (15, 31), (16, 32), (64, 127), (127, 255), (33, 130)]:
        X = torch.zeros(M, K, dtype=torch.bfloat16)
        X[m, k] = 2.0
        values, meta, _ = lx.prune_compress(X.cuda(), 0)
        Y = lx.sparse_linear(values, meta, W).float().cpu()
        assert Y[m, k] == 2.0 and Y.abs().sum() == 2.0, (m, k)


# ------------------------------------------------------------------ product + epilogue ---------

@pytest.mark.parametrize("mode", [0, 1, 2])
@pytest.mark.parametrize("with_bias,with_res", [(False, False), (True, False), (True, True)])
def test_tiny_config_full_oracle(lx, mode, with_bias, with_res):
    wl = inputs.WORKLOADS["tiny"]
    d = inputs.make_workload(wl, with_bias=with_bias, with_residual=with_res)
    X, W = d["X"].cuda(), d["W"].cuda()
    b = d["bias"].cuda() if with_bias else None
    r = d["residual"].cuda() if with_res else None
    ref = oracle.act_sparse_linear(u16(X), u16(W), bias=None if b is None else u16(b), comp_mode=mode,
                                   Yr=None if r is None else u16(r))
    # separate calls
    values, meta, scale = lx.prune_compress(X, mode)
    check_compressed(lx, X, values, meta, scale, mode)
    Y = lx.sparse_linear(values, meta, W, b, scale, r)
    check_y(Y, ref["Y"])
    # one call
    Y2 = lx.act_sparse_linear(X, W, b, mode, r)
    check_y(Y2, ref["Y"])
    assert torch.equal(Y, Y2)


@pytest.mark.parametrize("cfg", [1, 2, 3, 4, 5, 6, 7, 8])
def test_every_tile_configuration(cfg, monkeypatch):
    """All compiled tile shapes (one- and two-CTA MMAs, 128/192/240/256 columns) give the same answer."""
    from paper_2605_26632_b200 import binding

    monkeypatch.setenv("LYNX_GEMM_CFG", str(cfg))
    ctx = binding.Lynx(0)
    try:
        wl = inputs.Workload("t", 300, 640, 456, "outlier", 77)  # ragged M, N not a tile multiple
        d = inputs.make_workload(wl, with_bias=True, with_residual=True)
        X, W, b, r = d["X"].cuda(), d["W"].cuda(), d["bias"].cuda(), d["residual"].cuda()
        ref = oracle.act_sparse_linear(u16(X), u16(W), bias=u16(b), comp_mode=1, Yr=u16(r))
        Y = ctx.act_sparse_linear(X, W, b, 1, r)
        check_y(Y, ref["Y"])
        torch.cuda.synchronize()
        assert ctx.last_error() == 0
    finally:
        ctx.close()


@pytest.mark.parametrize("cfg", [4, 5, 7])
def test_stream_k_tail_matches_oracle_and_is_deterministic(cfg, monkeypatch):
    """Optional stream-K tail (leftover tiles split along K, fp32 partial tiles added in fixed
    order): same answer within tolerance, bit-identical run to run."""
    from paper_2605_26632_b200 import binding

    monkeypatch.setenv("LYNX_GEMM_CFG", str(cfg))
    monkeypatch.setenv("LYNX_STREAMK", "1")
    ctx = binding.Lynx(0)
    try:
        wl = inputs.Workload("t", 2304, 2048, 2304, "outlier", 55)  # 81 / 108 tiles on 74 CTA pairs
        d = inputs.make_workload(wl, with_bias=True)
        X, W, b = d["X"].cuda(), d["W"].cuda(), d["bias"].cuda()
        rows = np.arange(0, wl.M, 37, dtype=np.int64)
        ref = oracle.act_sparse_linear(u16(X), u16(W), bias=u16(b), comp_mode=1, rows=rows)
        Y1 = ctx.act_sparse_linear(X, W, b, 1)
        Y2 = ctx.act_sparse_linear(X, W, b, 1)
        check_y(Y1[torch.from_numpy(rows).cuda()], ref["Y"])
        assert torch.equal(Y1, Y2)
        torch.cuda.synchronize()
        assert ctx.last_error() == 0
    finally:
        ctx.close()


@pytest.mark.parametrize("M,K,N", [(1, 128, 8), (5, 256, 72), (129, 384, 200), (257, 128, 1000)])
def test_ragged_shapes(lx, M, K, N):
    wl = inputs.Workload("t", M, K, N, "normal", 31)
    d = inputs.make_workload(wl, with_bias=True, with_residual=True)
    X, W, b, r = d["X"].cuda(), d["W"].cuda(), d["bias"].cuda(), d["residual"].cuda()
    ref = oracle.act_sparse_linear(u16(X), u16(W), bias=u16(b), comp_mode=1, Yr=u16(r))
    Y = lx.act_sparse_linear(X, W, b, 1, r)
    check_y(Y, ref["Y"])


def test_leading_dimensions_of_w_y_and_residual(lx):
    """W, Y and the residual as column slices of wider buffers (ld > extent); nothing outside the
    Y slice may be written."""
    M, K, N = 300, 384, 456
    X = inputs.make_x(M, K, "outlier", 91)
    Wbig = torch.zeros(N, K + 128, dtype=torch.bfloat16)
    Wbig[:, :K] = inputs.make_w(N, K, 91)
    Rbig = torch.zeros(M, N + 64, dtype=torch.bfloat16)
    Rbig[:, :N] = inputs.make_residual(M, N, 91)
    b = inputs.make_bias(N, 91)
    ref = oracle.act_sparse_linear(u16(X), u16(Wbig[:, :K].contiguous()), bias=u16(b), comp_mode=1,
                                   Yr=u16(Rbig[:, :N].contiguous()))
    Ybig = torch.full((M, N + 72), 3.0, dtype=torch.bfloat16, device="cuda")
    Y = lx.act_sparse_linear(X.cuda(), Wbig.cuda()[:, :K], b.cuda(), 1, Rbig.cuda()[:, :N], out=Ybig[:, :N])
    check_y(Y, ref["Y"])
    assert (Ybig[:, N:] == 3.0).all()


def test_deferred_row_scale_two_call_form(lx):
    """The prune call stops at its row sums, the GEMM epilogue finishes the scale: same bits as
    the form that finishes the scale inside the prune kernel, and as the layer call."""
    from paper_2605_26632_b200 import binding
    from paper_2605_26632_b200.binding import LynxError

    M, K, N = 700, 1664, 1096
    X = inputs.make_x(M, K, "outlier", 33).cuda()
    W, b = inputs.make_w(N, K, 33).cuda(), inputs.make_bias(N, 33).cuda()
    v, m, s = lx.prune_compress(X, 1)
    want = lx.sparse_linear(v, m, W, b, s)
    v2, m2, d = lx.prune_compress(X, 1, row_scale=binding.ROW_SCALE_DEFERRED)
    assert d is binding.ROW_SCALE_DEFERRED and torch.equal(v, v2) and torch.equal(m, m2)
    got = lx.sparse_linear(v2, m2, W, b, binding.ROW_SCALE_DEFERRED)
    assert torch.equal(got, want)
    assert torch.equal(lx.act_sparse_linear(X, W, b, 1), want)
    # the sums belong to the last prune call of that shape: another shape is refused, nothing is launched
    X2 = inputs.make_x(256, 512, "gelu", 1).cuda()
    v3, m3, _ = lx.prune_compress(X2, 1, row_scale=binding.ROW_SCALE_DEFERRED)
    n0 = lx.launch_count()
    with pytest.raises(LynxError) as e:
        lx.sparse_linear(v2, m2, W, b, binding.ROW_SCALE_DEFERRED)
    assert e.value.status == 1 and lx.launch_count() == n0


def test_deferred_row_sums_are_forgotten_when_the_scratch_is_reused_or_regrown():
    """The deferred sums live in the context's scratch.  Anything that reallocates the scratch
    (lynx_reserve of a larger shape) or writes other data into it (a layer call, the FP8 layer call)
    between the two calls must make the GEMM call that still asks for them fail with
    LYNX_ERR_INVALID_ARG before any launch -- never read freed or overwritten memory."""
    from paper_2605_26632_b200 import binding
    from paper_2605_26632_b200.binding import LynxError

    M, K, N = 512, 1024, 256
    X = inputs.make_x(M, K, "outlier", 61).cuda()
    W, b = inputs.make_w(N, K, 61).cuda(), inputs.make_bias(N, 61).cuda()
    X2 = inputs.make_x(256, 512, "gelu", 62).cuda()
    W2 = inputs.make_w(128, 512, 62).cuda()

    def refused(ctx, v, m):
        n0 = ctx.launch_count()
        with pytest.raises(LynxError) as e:
            ctx.sparse_linear(v, m, W, b, binding.ROW_SCALE_DEFERRED)
        return e.value.status == 1 and ctx.launch_count() == n0

    ctx = binding.Lynx(0)
    try:
        v, m, s = ctx.prune_compress(X, 1)
        want = ctx.sparse_linear(v, m, W, b, s)
        # (a) the scratch is regrown between the two calls
        v2, m2, _ = ctx.prune_compress(X, 1, row_scale=binding.ROW_SCALE_DEFERRED)
        ctx.reserve(8192, 1024, 4096)
        assert refused(ctx, v2, m2)
        # (b) a layer call of another shape writes its compressed operands over the scratch
        v2, m2, _ = ctx.prune_compress(X, 1, row_scale=binding.ROW_SCALE_DEFERRED)
        ctx.act_sparse_linear(X2, W2, None, 0)
        assert refused(ctx, v2, m2)
        # (c) the FP8 layer call does the same
        v2, m2, _ = ctx.prune_compress(X, 1, row_scale=binding.ROW_SCALE_DEFERRED)
        Wq, ws = ctx.quantize_weights_fp8(W2, True)
        ctx.act_sparse_linear_fp8(X2, Wq, ws, None, 1)
        assert refused(ctx, v2, m2)
        # (d) a layer call of the SAME shape leaves its own sums there: they are not the caller's
        v2, m2, _ = ctx.prune_compress(X, 1, row_scale=binding.ROW_SCALE_DEFERRED)
        ctx.act_sparse_linear(X, W, b, 1)
        assert refused(ctx, v2, m2)
        # and the undisturbed two-call form still works afterwards, same bits
        v2, m2, _ = ctx.prune_compress(X, 1, row_scale=binding.ROW_SCALE_DEFERRED)
        assert torch.equal(ctx.sparse_linear(v2, m2, W, b, binding.ROW_SCALE_DEFERRED), want)
        torch.cuda.synchronize()
        assert ctx.last_error() == 0
    finally:
        ctx.close()


def test_integer_valued_inputs_are_exact(lx):
    """Small integers: every partial sum is exact in fp32 and in bf16, so Y must equal the oracle."""
    rng = np.random.default_rng(4)
    M, K, N = 256, 512, 256
    X = torch.from_numpy(rng.integers(-4, 5, size=(M, K)).astype(np.float32)).to(torch.bfloat16)
    W = torch.from_numpy(rng.integers(-1, 2, size=(N, K)).astype(np.float32)).to(torch.bfloat16)
    ref = oracle.act_sparse_linear(u16(X), u16(W))
    assert np.abs(ref["Y"]).max() <= 256  # exactly representable in bf16
    Y = lx.act_sparse_linear(X.cuda(), W.cuda())
    assert (Y.float().cpu().numpy() == ref["Y"]).all()


def test_already_sparse_input_equals_dense_linear(lx):
    """X already 2:4 sparse: the layer is an ordinary linear layer (library reference, fp32)."""
    g = torch.Generator().manual_seed(8)
    M, K, N = 384, 1024, 320
    x = torch.randn(M, K, generator=g)
    keep = torch.zeros(M, K // 4, 4, dtype=torch.bool)
    pos = torch.rand(M, K // 4, 4, generator=g).argsort(-1)[..., :2]
    keep.scatter_(-1, pos, True)
    x = torch.where(keep.reshape(M, K), x + torch.sign(x), torch.zeros(())).to(torch.bfloat16)
    w = inputs.make_w(N, K, 8)
    b = inputs.make_bias(N, 8)
    Y = lx.act_sparse_linear(x.cuda(), w.cuda(), b.cuda(), 1)
    ref = torch.nn.functional.linear(x.float(), w.float(), b.float()).numpy()
    check_y(Y, ref)


def test_gemm_is_deterministic(lx):
    wl = inputs.Workload("t", 1024, 1024, 768, "gelu", 12)
    d = inputs.make_workload(wl)
    X, W, b = d["X"].cuda(), d["W"].cuda(), d["bias"].cuda()
    a = lx.act_sparse_linear(X, W, b, 1)
    c = lx.act_sparse_linear(X, W, b, 1)
    assert torch.equal(a, c)


def test_host_buffer_entry_point(lx):
    wl = inputs.WORKLOADS["tiny"]
    d = inputs.make_workload(wl)
    ref = oracle.act_sparse_linear(u16(d["X"]), u16(d["W"]), bias=u16(d["bias"]), comp_mode=1)
    Y = lx.act_sparse_linear_host(d["X"].pin_memory(), d["W"].cuda(), d["bias"].cuda(), 1)
    check_y(Y, ref["Y"])


@pytest.mark.parametrize("M,mode", [(2500, 1), (4096, 0), (2304, 2)])
def test_host_buffer_entry_point_pipelined_chunks(lx, M, mode):
    """From 2048 rows on the host entry point pipelines row chunks over copy streams (not under the
    whole-tensor scale): same bits as the device-buffer call, twice in a row."""
    K, N = 512, 776
    X = inputs.make_x(M, K, "outlier", 61)
    W, b = inputs.make_w(N, K, 61).cuda(), inputs.make_bias(N, 61).cuda()
    want = lx.act_sparse_linear(X.cuda(), W, b, mode).cpu()
    Xh = X.pin_memory()
    for _ in range(2):
        Y = lx.act_sparse_linear_host(Xh, W, b, mode)
        assert torch.equal(Y, want)


# ------------------------------------------------------------------ fused one-kernel path ------

@pytest.mark.parametrize("mode", [0, 1])
@pytest.mark.parametrize("with_bias,with_res", [(False, False), (True, True)])
def test_fused_tiny_config_full_oracle(lx, mode, with_bias, with_res):
    from paper_2605_26632_b200 import binding

    wl = inputs.WORKLOADS["tiny"]
    d = inputs.make_workload(wl, with_bias=with_bias, with_residual=with_res)
    X, W = d["X"].cuda(), d["W"].cuda()
    b = d["bias"].cuda() if with_bias else None
    r = d["residual"].cuda() if with_res else None
    ref = oracle.act_sparse_linear(u16(X), u16(W), bias=None if b is None else u16(b), comp_mode=mode,
                                   Yr=None if r is None else u16(r))
    Yf = lx.act_sparse_linear(X, W, b, mode, r, fuse=binding.FUSE_FUSED)
    check_y(Yf, ref["Y"])
    if mode == 0:
        # same products in the same order as the two-kernel path: identical bits
        Ys = lx.act_sparse_linear(X, W, b, mode, r, fuse=binding.FUSE_SEPARATE)
        assert torch.equal(Yf, Ys)


@pytest.mark.parametrize("M,K,N", [(1, 128, 8), (129, 384, 200), (300, 640, 456), (520, 1024, 1000)])
def test_fused_ragged_shapes(lx, M, K, N):
    from paper_2605_26632_b200 import binding

    wl = inputs.Workload("t", M, K, N, "outlier", 61)
    d = inputs.make_workload(wl, with_bias=True, with_residual=True)
    X, W, b, r = d["X"].cuda(), d["W"].cuda(), d["bias"].cuda(), d["residual"].cuda()
    ref = oracle.act_sparse_linear(u16(X), u16(W), bias=u16(b), comp_mode=1, Yr=u16(r))
    Y = lx.act_sparse_linear(X, W, b, 1, r, fuse=binding.FUSE_FUSED)
    check_y(Y, ref["Y"])
    Y2 = lx.act_sparse_linear(X, W, b, 1, r, fuse=binding.FUSE_FUSED)
    assert torch.equal(Y, Y2)


def test_fused_identity_weight_and_special_values(lx):
    """W = I through the fused kernel: its in-kernel selection, value packing and metadata must
    reproduce mask * X exactly, including NaN / Inf / subnormal ranking."""
    from paper_2605_26632_b200 import binding

    M, K = 200, 512
    X = inputs.make_x(M, K, "normal", 13).cuda()
    W = torch.eye(K, dtype=torch.bfloat16, device="cuda")
    Y = lx.act_sparse_linear(X, W, None, 0, None, fuse=binding.FUSE_FUSED)
    Xu = u16(X)
    want = oracle.bf16_to_f32(Xu * oracle.topk24_mask(Xu))
    assert (Y.float().cpu().numpy() == want).all()


def test_fused_full_size_mlp_up(lx):
    from paper_2605_26632_b200 import binding

    wl = inputs.WORKLOADS["mlp_up"]
    d = inputs.make_workload(wl, with_bias=True)
    X, W, b = d["X"].cuda(), d["W"].cuda(), d["bias"].cuda()
    Y = lx.act_sparse_linear(X, W, b, 1, None, fuse=binding.FUSE_FUSED)
    rows = np.sort(np.random.default_rng(4).choice(wl.M, 24, replace=False)).astype(np.int64)
    ref = oracle.act_sparse_linear(u16(d["X"]), u16(d["W"]), bias=u16(d["bias"]), comp_mode=1, rows=rows)
    check_y(Y[torch.from_numpy(rows).cuda()], ref["Y"])


def test_fused_rejects_whole_tensor_scale(lx):
    from paper_2605_26632_b200 import binding

    X = torch.zeros(16, 128, dtype=torch.bfloat16, device="cuda")
    W = torch.zeros(16, 128, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(binding.LynxError) as e:
        lx.act_sparse_linear(X, W, None, 2, None, fuse=binding.FUSE_FUSED)
    assert e.value.status == 2


# ------------------------------------------------------------------ two-row-tile GEMM kernel ----

@pytest.mark.parametrize("with_res", [True, False])
@pytest.mark.parametrize("doubles", [-1, 0, 1, 3, 100000])
@pytest.mark.parametrize("M,K,N", [
    (700, 1664, 1096),    # 3 row tiles (odd: the last one only forms single-tile items), ragged rows and columns
    (1024, 512, 2000),    # 4 x 9 tiles on 74 CTA pairs
    (4800, 1024, 1000),   # 19 x 5 tiles: more items than CTA pairs, several rounds, last row tile 192 rows
])
def test_two_row_tile_gemm_kernel(M, K, N, doubles, with_res, monkeypatch):
    """The GEMM kernel that runs two 256-row tiles per W stage, forced on, for several numbers of
    512-row items (-1 = the cost model's choice, 0 = single-tile items only, 100000 = as many as
    fit): Y of every row and column against the oracle with bias + row scale + residual, and bit
    for bit the single-tile kernel's result (same MMAs in the same order per tile, same epilogue
    arithmetic).  With a residual the epilogue works chunk by chunk; without, it converts the whole
    accumulator row in registers before the first store (two code paths)."""
    from paper_2605_26632_b200 import binding

    X = inputs.make_x(M, K, "outlier", 8100 + M)
    W, b = inputs.make_w(N, K, 8100 + M), inputs.make_bias(N, 8100 + M)
    res = inputs.make_residual(M, N, 8100 + M) if with_res else None
    ref = oracle.act_sparse_linear(u16(X), u16(W), bias=u16(b), comp_mode=1, Yr=None if res is None else u16(res))
    res = None if res is None else res.cuda()
    monkeypatch.setenv("LYNX_RT2", "1")
    monkeypatch.setenv("LYNX_RT2_D", str(doubles))
    ctx = binding.Lynx(0)
    try:
        Y = ctx.act_sparse_linear(X.cuda(), W.cuda(), b.cuda(), 1, res)
        check_y(Y, ref["Y"])
        v, m, s = ctx.prune_compress(X.cuda(), 1)
        assert torch.equal(ctx.sparse_linear(v, m, W.cuda(), b.cuda(), s, res), Y)
        torch.cuda.synchronize()
        assert ctx.last_error() == 0
    finally:
        ctx.close()
    monkeypatch.setenv("LYNX_RT2", "0")
    monkeypatch.setenv("LYNX_GEMM_CFG", "7")
    ctx = binding.Lynx(0)
    try:
        assert torch.equal(ctx.act_sparse_linear(X.cuda(), W.cuda(), b.cuda(), 1, res), Y)
    finally:
        ctx.close()


# ------------------------------------------------------------------ full-size workloads --------

def _full_size_case(lx, wl, mode=1):
    """Values, metadata and scale on every element; Y against the oracle on every row when
    M <= 4608, else on >= 512 rows that include the first and last row of every 128-row block
    (row_sampling.parity_rows), all N columns: every output tile of the launch is touched."""
    d = inputs.make_workload(wl, with_bias=True)
    X, W, b = d["X"].cuda(), d["W"].cuda(), d["bias"].cuda()
    values, meta, scale = lx.prune_compress(X, mode)
    Xu = u16(d["X"])
    ov, om = oracle.compress(Xu)
    assert (u16(values) == ov).all()
    assert (meta.cpu().numpy() == oracle.meta_canon_to_hw(om, wl.M, wl.K)).all()
    np.testing.assert_allclose(scale.cpu().numpy(), oracle.row_scale(Xu, mode), rtol=SCALE_RTOL)
    Y = lx.sparse_linear(values, meta, W, b, scale)
    rows = parity_rows(wl.M, wl.seed)
    ref = oracle.act_sparse_linear(Xu, u16(d["W"]), bias=u16(d["bias"]), comp_mode=mode, rows=rows)
    check_y(take(Y, rows), ref["Y"])
    # same launch configuration as the bench: the single-call path must agree bit for bit
    Y2 = lx.act_sparse_linear(X, W, b, mode)
    assert torch.equal(Y, Y2)
    torch.cuda.synchronize()
    assert lx.last_error() == 0


@pytest.mark.parametrize("name", ["mlp_down", "attn_qkv", "attn_out", "mlp_up"])
def test_dit_workloads_full_size(lx, name):
    """Values and metadata checked on every element, Y on every row and column."""
    _full_size_case(lx, inputs.WORKLOADS[name])


@pytest.mark.parametrize("M", inputs.SWEEP_M)
@pytest.mark.parametrize("K,N", inputs.SWEEP_KN)
def test_token_sweep(lx, M, K, N):
    """Y on every row for M <= 4096; for M = 8192 / 16384 on 512 rows covering every 128-row block."""
    idx = inputs.SWEEP_M.index(M) * 4 + inputs.SWEEP_KN.index((K, N))
    _full_size_case(lx, inputs.sweep_workload(M, K, N, idx))


@pytest.mark.parametrize("K,N", inputs.OTHER_FAMILY_KN)
def test_other_dit_family_shapes(lx, K, N):
    """FLUX.1-dev single-stream and Z-Image linear shapes (full size, M = 4096: Y on every row)."""
    idx = 100 + inputs.OTHER_FAMILY_KN.index((K, N))
    _full_size_case(lx, inputs.sweep_workload(inputs.OTHER_FAMILY_M, K, N, idx))


@pytest.mark.parametrize("M,K,N", [
    (4800, 1024, 1000),    # 19 row tiles of the CTA pair -> groups of 10 + 9, last row tile 192 rows, N tail
    (12000, 512, 1096),    # 47 row tiles -> three groups (16, 16, 15), 235 output tiles on 74 clusters
    (8448, 384, 2000),     # 33 row tiles -> 11 + 11 + 11, nine column tiles with a tail
])
def test_tile_order_with_several_row_groups_every_row(lx, M, K, N):
    """More output tiles than clusters, several row-tile groups of unequal size, ragged last row
    tile and column tail: Y of EVERY row and column against the oracle (a tile skipped, doubled or
    mapped to the wrong place would show), for bias + row scale + residual."""
    X = inputs.make_x(M, K, "outlier", 7000 + M)
    W, b = inputs.make_w(N, K, 7000 + M), inputs.make_bias(N, 7000 + M)
    res = inputs.make_residual(M, N, 7000 + M)
    ref = oracle.act_sparse_linear(u16(X), u16(W), bias=u16(b), comp_mode=1, Yr=u16(res))
    Y = lx.act_sparse_linear(X.cuda(), W.cuda(), b.cuda(), 1, res.cuda())
    check_y(Y, ref["Y"])
    # row by row as well: a misplaced tile of small norm must not hide in the Frobenius ratio
    yf = Y.float().cpu().numpy()
    err = np.linalg.norm(yf - ref["Y"], axis=1) / np.maximum(np.linalg.norm(ref["Y"], axis=1), 1e-30)
    assert err.max() <= 4 * RFE_TOL, f"row {int(err.argmax())}: relative error {err.max()}"
    torch.cuda.synchronize()
    assert lx.last_error() == 0


def test_more_than_2_to_the_31_elements(lx):
    """M x K = 176128 x 12288 > 2^31 elements (X alone is 4.3 GB): every offset in the prune kernels,
    the tensor maps and the GEMM has to be 64-bit.  The rows are 43 copies of one 4096-row matrix
    scaled by powers of two; the oracle sees the sampled rows as they sit on the device."""
    K, N, base_rows, copies = 12288, 256, 4096, 43
    M = base_rows * copies
    assert M * K > 2 ** 31 and M % 128 == 0
    base = inputs.make_x(base_rows, K, "outlier", 4242).cuda()
    X = torch.empty((M, K), dtype=torch.bfloat16, device="cuda")
    for c in range(copies):
        X[c * base_rows:(c + 1) * base_rows] = base * (2.0 ** ((c % 7) - 3))
    W, b = inputs.make_w(N, K, 4243), inputs.make_bias(N, 4243)
    edge = (2 ** 31) // K                     # the row in which element offset 2^31 falls
    rows = np.unique(np.concatenate([[0, 1, edge - 1, edge, edge + 1, M - 2, M - 1],
                                     np.random.default_rng(7).choice(M, 25, replace=False)])).astype(np.int64)
    ridx = torch.from_numpy(rows).cuda()
    Xs = u16(X[ridx].cpu())
    ov, om = oracle.compress(Xs)
    values, meta, scale = lx.prune_compress(X, 1)
    assert (u16(values[ridx].cpu()) == ov).all()
    canon = lx.meta_to_canonical(meta, M, K)
    assert (canon[ridx].cpu().numpy().view(np.uint16) == om.view(np.uint16)).all()
    np.testing.assert_allclose(scale[ridx].cpu().numpy(), oracle.row_scale(Xs, 1), rtol=SCALE_RTOL)
    Y = lx.sparse_linear(values, meta, W.cuda(), b.cuda(), scale)
    ref = oracle.act_sparse_linear(Xs, u16(W), bias=u16(b), comp_mode=1)
    check_y(Y[ridx], ref["Y"])
    Y2 = lx.act_sparse_linear(X, W.cuda(), b.cuda(), 1)
    assert torch.equal(Y, Y2)
    del values, meta, canon, Y2
    # the FP8 quantising prune on the same rows (single-read kernel, two warps per row)
    vq, meta8, rs8 = lx.prune_compress_fp8(X, 1)
    oq, om8, oact = oracle.compress_fp8(Xs)
    assert (vq[ridx].cpu().numpy() == oq).all()
    hw = oracle.meta_canon_to_hw_fp8(om8, len(rows), K)          # rows 0.. of one 128-row block
    kb = torch.arange(K // 128, device="cuda").view(1, -1, 1)
    byte = torch.arange(16, device="cuda").view(1, 1, -1)
    r = ridx.view(-1, 1, 1)
    got = meta8[((r // 128) * (K // 128) + kb) * 2048 + (r % 128) * 16 + byte].cpu().numpy()
    i = np.arange(len(rows)).reshape(-1, 1, 1)
    want = hw[(kb.cpu().numpy()) * 2048 + i * 16 + byte.cpu().numpy()]
    assert (got == want).all()
    ref8 = oracle.row_scale(Xs, 1).astype(np.float64) * oact.astype(np.float64)
    np.testing.assert_allclose(rs8[ridx].cpu().numpy(), ref8, rtol=1e-5)
    torch.cuda.synchronize()
    assert lx.last_error() == 0


# ------------------------------------------------------------------ host-side error reporting ---

def test_argument_errors_are_reported_not_launched(lx):
    from paper_2605_26632_b200 import binding

    X = torch.zeros(16, 192, dtype=torch.bfloat16, device="cuda")  # K % 128 != 0
    with pytest.raises(binding.LynxError) as e:
        lx.prune_compress(X, 0, values=torch.empty(16, 96, dtype=torch.bfloat16, device="cuda"),
                          meta=torch.empty(4096, dtype=torch.uint8, device="cuda"))
    assert e.value.status == 2
    X = torch.zeros(16, 256 + 8, dtype=torch.bfloat16, device="cuda")[:, 8:]  # misaligned rows
    with pytest.raises(binding.LynxError) as e:
        lx.prune_compress(X, 0)
    assert e.value.status == 3
    values = torch.zeros(16, 64, dtype=torch.bfloat16, device="cuda")
    meta = torch.zeros(2048, dtype=torch.uint8, device="cuda")
    W = torch.zeros(12, 128, dtype=torch.bfloat16, device="cuda")  # N % 8 != 0
    with pytest.raises(binding.LynxError) as e:
        lx.sparse_linear(values, meta, W)
    assert e.value.status == 2
    with pytest.raises(binding.LynxError) as e:  # scale requested but no buffer
        lx._lib.lynx_prune_compress.restype = int
        from ctypes import c_void_p
        st = lx._lib.lynx_prune_compress(lx._h, c_void_p(values.data_ptr()), 16, 128, 128,
                                         c_void_p(values.data_ptr()), c_void_p(meta.data_ptr()), None, 1, None)
        binding._check(st, "prune")
    assert e.value.status == 1
    # an empty problem (M = 0) is refused by every entry point before anything is launched
    from ctypes import c_void_p
    n0 = lx.launch_count()
    vp, mp = c_void_p(values.data_ptr()), c_void_p(meta.data_ptr())
    Wk = torch.zeros(16, 128, dtype=torch.bfloat16, device="cuda")
    Y = torch.zeros(16, 16, dtype=torch.bfloat16, device="cuda")
    wp, yp = c_void_p(Wk.data_ptr()), c_void_p(Y.data_ptr())
    assert lx._lib.lynx_prune_compress(lx._h, vp, 0, 128, 128, vp, mp, None, 0, None) == 1
    assert lx._lib.lynx_sparse_linear(lx._h, vp, mp, 0, 128, wp, 16, 128, None, None, yp, 16, None) == 1
    assert lx._lib.lynx_act_sparse_linear(lx._h, vp, 0, 128, 128, wp, 16, 128, None, 0, None, 0, yp, 16, 0, None) == 1
    assert lx._lib.lynx_prune_compress_fp8(lx._h, vp, 0, 256, 256, None, vp, mp, c_void_p(Y.data_ptr()), 0, None) == 1
    assert lx.launch_count() == n0
    assert lx.last_error() == 0


def test_device_side_timeout_is_reported_and_cleared():
    """A bounded wait that runs out (one warp waiting 1 ms on a barrier nobody arrives at: nothing
    faults, the kernel returns) raises the context's error word: the next call on the context is
    refused with LYNX_ERR_TIMEOUT before launching, lynx_last_error reports it once and clears it,
    and the context is fully usable afterwards."""
    from paper_2605_26632_b200 import binding
    from paper_2605_26632_b200.binding import LynxError

    ctx = binding.Lynx(0)
    try:
        X = inputs.make_x(256, 512, "gelu", 1).cuda()
        W = inputs.make_w(256, 512, 1).cuda()
        want = ctx.act_sparse_linear(X, W, None, 1)
        torch.cuda.synchronize()
        assert ctx.last_error() == 0
        ctx.selftest_wait_timeout(1000)
        torch.cuda.synchronize()
        n0 = ctx.launch_count()
        with pytest.raises(LynxError) as e:
            ctx.act_sparse_linear(X, W, None, 1)
        assert e.value.status == 6 and ctx.launch_count() == n0
        assert ctx.last_error() == 6      # reported ...
        assert ctx.last_error() == 0      # ... once, then cleared
        assert torch.equal(ctx.act_sparse_linear(X, W, None, 1), want)
        torch.cuda.synchronize()
        assert ctx.last_error() == 0
    finally:
        ctx.close()
