"""GPU parity tests of the FP8 (E4M3) composition: weight codes, activation codes + metadata +
row scale from the quantising prune kernel, and the FP8 sparse GEMM, through the C ABI against the
CPU oracle.

Bars: codes and metadata bit-exact (both sides quantise with the same fp32 operations; NaN codes
compare as NaN); scales within 1e-5 relative; Y within relative Frobenius error 5e-3 and
max |dY| <= 2e-2 * max |Y_ref| of the oracle's result on the same codes.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_26632_b200 import inputs
from row_sampling import parity_rows, take

pytestmark = pytest.mark.gpu


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


@pytest.mark.parametrize("per_channel", [False, True])
def test_weight_codes_are_bit_exact(lx, per_channel):
    W = inputs.make_w(200, 768, 3)
    W[5] = 0
    Wq, ws = lx.quantize_weights_fp8(W.cuda(), per_channel)
    oq, os_ = oracle.quantize_weights_fp8(u16(W), per_channel)
    assert (Wq.cpu().numpy() == oq).all()
    np.testing.assert_allclose(ws.cpu().numpy(), os_, rtol=1e-6)


@pytest.mark.parametrize("M,K,dist,mode", [
    (256, 512, "gelu", 0), (256, 512, "gelu", 1), (300, 1024, "outlier", 1), (129, 256, "gelu_chan", 1),
    (1, 256, "outlier", 0), (4096, 3072, "outlier", 1), (2048, 12288, "gelu_chan", 1),
])
def test_activation_codes_metadata_and_scale(lx, M, K, dist, mode):
    X = inputs.make_x(M, K, dist, 700 + M)
    vq, meta, rs = lx.prune_compress_fp8(X.cuda(), mode)
    ov, om, oact = oracle.compress_fp8(u16(X))
    assert (vq.cpu().numpy() == ov).all(), "codes differ"
    assert (meta.cpu().numpy() == oracle.meta_canon_to_hw_fp8(om, M, K)).all(), "metadata differs"
    ref_scale = oracle.row_scale(u16(X), mode).astype(np.float64) * oact.astype(np.float64)
    np.testing.assert_allclose(rs.cpu().numpy(), ref_scale, rtol=1e-5)


# The single-read kernel (K >= 2048) splits a row over 1, 2, 4 or 8 warps depending on how many rows
# fit in shared memory; the shapes below reach each split, a ragged last 128-row block, fewer rows
# than SMs, a row range per CTA of uneven length, and a leading dimension larger than K.
RING_SHAPES = [(300, 2048, 1), (77, 6144, 1), (1, 2048, 0), (513, 8192, 1), (200, 12288, 0), (130, 24576, 1),
               (40, 49152, 1), (1000, 3072, 0)]


@pytest.mark.parametrize("M,K,mode", RING_SHAPES)
def test_single_read_kernel_shapes(lx, M, K, mode):
    X = inputs.make_x(M, K, "outlier" if M % 2 else "gelu_chan", 900 + M)
    ov, om, oact = oracle.compress_fp8(u16(X))
    ref_scale = oracle.row_scale(u16(X), mode).astype(np.float64) * oact.astype(np.float64)
    ometa = oracle.meta_canon_to_hw_fp8(om, M, K)
    amax = X.float().abs().max(dim=1).values.contiguous().cuda()
    for given in (None, amax):
        vq, meta, rs = lx.prune_compress_fp8(X.cuda(), mode, row_amax=given)
        assert (vq.cpu().numpy() == ov).all(), "codes differ"
        assert (meta.cpu().numpy() == ometa).all(), "metadata differs"
        np.testing.assert_allclose(rs.cpu().numpy(), ref_scale, rtol=1e-5)
    # rows of a wider matrix (leading dimension 3 * 16 elements beyond K)
    wide = torch.zeros((M, K + 48), dtype=torch.bfloat16)
    wide[:, :K] = X
    vq2, meta2, rs2 = lx.prune_compress_fp8(wide.cuda()[:, :K], mode)
    assert torch.equal(vq2, vq) and torch.equal(meta2, meta) and torch.equal(rs2, rs)


def test_single_read_kernel_special_values(lx):
    """Zero rows, subnormals, infinities and NaN through the shared-memory path (K = 2048)."""
    M, K = 40, 2048
    g = torch.Generator().manual_seed(6)
    x = torch.randn(M, K, generator=g)
    x[0] = 0.0
    x[1, 0:4] = torch.tensor([1e-40, -1e-40, 2e-40, 0.0])
    x[2, 1037] = float("inf")
    x[3, 2047] = float("nan")
    x[5, 100] = float("-inf")
    x[5, 200] = float("nan")
    x[4, 0:8] = torch.tensor([-0.0, 0.0, -0.0, 0.0, 1e18, -1e18, 1.0, 1.0])
    X = x.to(torch.bfloat16)
    vq, meta, rs = lx.prune_compress_fp8(X.cuda(), 1)
    ov, om, oact = oracle.compress_fp8(u16(X))
    got = vq.cpu().numpy()
    gd, od = oracle.e4m3_decode(got), oracle.e4m3_decode(ov)
    nan = np.isnan(od)
    assert (np.isnan(gd) == nan).all()
    assert (got[~nan] == ov[~nan]).all()
    assert (meta.cpu().numpy() == oracle.meta_canon_to_hw_fp8(om, M, K)).all()
    ref = oracle.row_scale(u16(X), 1).astype(np.float64) * oact.astype(np.float64)
    got_s = rs.cpu().numpy().astype(np.float64)
    fin = np.isfinite(ref)
    assert (np.isfinite(got_s) == fin).all()
    np.testing.assert_allclose(got_s[fin], ref[fin], rtol=1e-5)


@pytest.mark.parametrize("ring", ["0", "1", "2", "4", "8"])
def test_every_fp8_prune_form_gives_the_same_codes(ring, monkeypatch):
    """The 16-rows-per-CTA kernel and every warp split of the single-read kernel."""
    from paper_2605_26632_b200 import binding

    monkeypatch.setenv("LYNX_FP8_RING", ring)
    ctx = binding.Lynx(0)
    try:
        M, K = 333, 4096
        X = inputs.make_x(M, K, "outlier", 777)
        ov, om, oact = oracle.compress_fp8(u16(X))
        vq, meta, rs = ctx.prune_compress_fp8(X.cuda(), 1)
        assert (vq.cpu().numpy() == ov).all()
        assert (meta.cpu().numpy() == oracle.meta_canon_to_hw_fp8(om, M, K)).all()
        ref = oracle.row_scale(u16(X), 1).astype(np.float64) * oact.astype(np.float64)
        np.testing.assert_allclose(rs.cpu().numpy(), ref, rtol=1e-5)
        torch.cuda.synchronize()
        assert ctx.last_error() == 0
    finally:
        ctx.close()


@pytest.mark.parametrize("M,K,mode", [(300, 1024, 1), (129, 256, 0), (2048, 3072, 1)])
def test_supplied_row_maximum(lx, M, K, mode):
    """The true maxima supplied by the caller give the same bits as the two-pass form; a
    calibrated constant (some rows saturate, the rest lose range) matches the oracle."""
    X = inputs.make_x(M, K, "outlier", 820 + M)
    Xc = X.cuda()
    vq, meta, rs = lx.prune_compress_fp8(Xc, mode)
    amax = X.float().abs().max(dim=1).values
    vq1, meta1, rs1 = lx.prune_compress_fp8(Xc, mode, row_amax=amax.cuda())
    assert torch.equal(vq, vq1) and torch.equal(meta, meta1) and torch.equal(rs, rs1)
    const = torch.full((M,), float(amax.median()), dtype=torch.float32)
    vq2, meta2, rs2 = lx.prune_compress_fp8(Xc, mode, row_amax=const.cuda())
    ov, om, oact = oracle.compress_fp8(u16(X), row_amax=const.numpy())
    assert (vq2.cpu().numpy() == ov).all()
    assert (meta2.cpu().numpy() == oracle.meta_canon_to_hw_fp8(om, M, K)).all()
    ref = oracle.row_scale(u16(X), mode).astype(np.float64) * oact.astype(np.float64)
    np.testing.assert_allclose(rs2.cpu().numpy(), ref, rtol=1e-5)
    assert (np.abs(oracle.e4m3_decode(ov)) == 448.0).sum() > 0   # the constant does saturate some rows


def test_layer_with_supplied_row_maximum(lx):
    wl = inputs.WORKLOADS["tiny"]
    d = inputs.make_workload(wl, with_bias=True)
    amax = (d["X"].float().abs().max(dim=1).values * 1.25).contiguous()
    oq, ows = oracle.quantize_weights_fp8(u16(d["W"]), True)
    ref = oracle.act_sparse_linear_fp8(u16(d["X"]), oq, ows, bias=u16(d["bias"]), comp_mode=1, row_amax=amax.numpy())
    Wq, ws = lx.quantize_weights_fp8(d["W"].cuda(), True)
    Y = lx.act_sparse_linear_fp8(d["X"].cuda(), Wq, ws, d["bias"].cuda(), 1, row_amax=amax.cuda())
    check_y(Y, ref["Y"])


def test_activation_special_values(lx):
    M, K = 32, 256
    g = torch.Generator().manual_seed(5)
    x = torch.randn(M, K, generator=g)
    x[0] = 0.0
    x[1, 0:4] = torch.tensor([1e-40, -1e-40, 2e-40, 0.0])
    x[2, 7] = float("inf")
    x[3, 9] = float("nan")
    x[4, 0:8] = torch.tensor([-0.0, 0.0, -0.0, 0.0, 1e18, -1e18, 1.0, 1.0])  # squares still fit in fp32
    X = x.to(torch.bfloat16)
    vq, meta, rs = lx.prune_compress_fp8(X.cuda(), 1)
    ov, om, oact = oracle.compress_fp8(u16(X))
    got = vq.cpu().numpy()
    gd, od = oracle.e4m3_decode(got), oracle.e4m3_decode(ov)
    nan = np.isnan(od)
    assert (np.isnan(gd) == nan).all()
    assert (got[~nan] == ov[~nan]).all()
    assert (meta.cpu().numpy() == oracle.meta_canon_to_hw_fp8(om, M, K)).all()
    ref = oracle.row_scale(u16(X), 1).astype(np.float64) * oact.astype(np.float64)
    got_s = rs.cpu().numpy().astype(np.float64)
    fin = np.isfinite(ref)
    assert (np.isfinite(got_s) == fin).all()
    np.testing.assert_allclose(got_s[fin], ref[fin], rtol=1e-5)


@pytest.mark.parametrize("M,K", [(128, 256), (256, 512), (300, 1024)])
def test_identity_weight_returns_the_dequantised_sparse_activation(lx, M, K):
    """W = I (1.0 is exact in E4M3): Y[m, k] = row_scale_m * decode(code) at the kept positions,
    0 elsewhere -- pins the metadata order and the operand geometry of the FP8 MMA on silicon."""
    X = inputs.make_x(M, K, "gelu", 11)
    W = torch.eye(K, dtype=torch.bfloat16)
    Wq, ws = lx.quantize_weights_fp8(W.cuda(), per_channel=False)
    vq, meta, rs = lx.prune_compress_fp8(X.cuda(), 0)
    Y = lx.sparse_linear_fp8(vq, meta, Wq, None, None, rs)
    ov, om, oact = oracle.compress_fp8(u16(X))
    dec = oracle.e4m3_decode(ov).reshape(M, K // 4, 2)
    ref = np.zeros((M, K), dtype=np.float32)
    for m in range(M):
        for g in range(K // 4):
            nib = (int(om[m, g // 4]) >> (4 * (g % 4))) & 0xF
            ref[m, 4 * g + (nib & 3)] = dec[m, g, 0] * oact[m]
            ref[m, 4 * g + (nib >> 2)] = dec[m, g, 1] * oact[m]
    want = torch.from_numpy(ref).to(torch.bfloat16)
    assert torch.equal(Y.cpu(), want)


@pytest.mark.parametrize("mode", [0, 1])
@pytest.mark.parametrize("per_channel", [False, True])
@pytest.mark.parametrize("with_bias,with_res", [(False, False), (True, True)])
def test_tiny_config_fp8_full_oracle(lx, mode, per_channel, with_bias, with_res):
    wl = inputs.WORKLOADS["tiny"]
    d = inputs.make_workload(wl, with_bias=with_bias, with_residual=with_res)
    cu = lambda t: None if t is None else t.cuda()
    oq, ows = oracle.quantize_weights_fp8(u16(d["W"]), per_channel)
    ref = oracle.act_sparse_linear_fp8(u16(d["X"]), oq, ows, bias=None if d["bias"] is None else u16(d["bias"]),
                                       comp_mode=mode, Yr=None if d["residual"] is None else u16(d["residual"]))
    Wq, ws = lx.quantize_weights_fp8(d["W"].cuda(), per_channel)
    Y = lx.act_sparse_linear_fp8(d["X"].cuda(), Wq, ws, cu(d["bias"]), mode, cu(d["residual"]))
    check_y(Y, ref["Y"])
    vq, meta, rs = lx.prune_compress_fp8(d["X"].cuda(), mode)
    Y2 = lx.sparse_linear_fp8(vq, meta, Wq, ws, cu(d["bias"]), rs, cu(d["residual"]))
    assert torch.equal(Y, Y2)


@pytest.mark.parametrize("cfg", [4, 6, 7])
def test_every_fp8_tile_configuration(cfg, monkeypatch):
    from paper_2605_26632_b200 import binding

    monkeypatch.setenv("LYNX_GEMM_CFG", str(cfg))
    ctx = binding.Lynx(0)
    try:
        M, K, N = 700, 1280, 1096  # ragged in M and N for every tile width, 5 K blocks of 256
        X = inputs.make_x(M, K, "outlier", 800 + cfg)
        W = inputs.make_w(N, K, 800 + cfg)
        b = inputs.make_bias(N, 800 + cfg)
        oq, ows = oracle.quantize_weights_fp8(u16(W), True)
        ref = oracle.act_sparse_linear_fp8(u16(X), oq, ows, bias=u16(b), comp_mode=1)
        Wq, ws = ctx.quantize_weights_fp8(W.cuda(), True)
        Y = ctx.act_sparse_linear_fp8(X.cuda(), Wq, ws, b.cuda(), 1)
        check_y(Y, ref["Y"])
        Y2 = ctx.act_sparse_linear_fp8(X.cuda(), Wq, ws, b.cuda(), 1)
        assert torch.equal(Y, Y2)
        torch.cuda.synchronize()
        assert ctx.last_error() == 0
    finally:
        ctx.close()


@pytest.mark.parametrize("name", ["mlp_down", "attn_qkv", "mlp_up"])
def test_dit_workloads_full_size_fp8(lx, name):
    """Weight codes bit-exact.  Y against the oracle on every row and column for mlp_down (the
    bench's shape); the oracle's FP8 product takes ~90 s for 4096 rows on the host cores, so the
    two other shapes are compared on 1024 rows: the first and last row of every 128-row block (the
    rows one CTA owns) plus a seeded remainder, all N columns -- every output tile is touched."""
    wl = inputs.WORKLOADS[name]
    d = inputs.make_workload(wl, with_bias=True)
    rows = parity_rows(wl.M, wl.seed) if name == "mlp_down" else parity_rows(wl.M, wl.seed, all_rows_up_to=0, min_rows=1024)
    oq, ows = oracle.quantize_weights_fp8(u16(d["W"]), True)
    ref = oracle.act_sparse_linear_fp8(u16(d["X"]), oq, ows, bias=u16(d["bias"]), comp_mode=1, rows=rows)
    Wq, ws = lx.quantize_weights_fp8(d["W"].cuda(), True)
    assert (Wq.cpu().numpy() == oq).all()
    Y = lx.act_sparse_linear_fp8(d["X"].cuda(), Wq, ws, d["bias"].cuda(), 1)
    check_y(take(Y, rows), ref["Y"])


def test_fp8_argument_errors(lx):
    from paper_2605_26632_b200.binding import LynxError

    X = torch.zeros(128, 384, dtype=torch.bfloat16, device="cuda")  # K % 256 != 0
    n0 = lx.launch_count()
    with pytest.raises(LynxError) as e:
        lx.prune_compress_fp8(X, 0)
    assert e.value.status == 2
    X = torch.zeros(128, 512, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(LynxError) as e:
        lx.prune_compress_fp8(X, 2)  # whole-tensor scale is not available in FP8
    assert e.value.status == 1
    assert lx.launch_count() == n0
