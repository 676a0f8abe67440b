"""Pins of the CPU oracle against things other than itself (no GPU needed).

Each test fixes the oracle to what the paper's definitions and plain mathematics determine:
hand cases, brute force over a small alphabet, invariants, closed forms, and special cases that
reduce to a library routine (numpy / torch matmul in fp64).
"""
import itertools
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2605_26632_b200 import inputs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def bf16_bits(vals):
    """Exact conversion of floats that are representable in bf16 to their bit patterns."""
    t = torch.tensor(vals, dtype=torch.float32)
    b = t.to(torch.bfloat16)
    assert torch.equal(b.to(torch.float32), t) or torch.isnan(t).any()
    return inputs.as_u16(b)


def tile_group(group_bits, reps=4):
    """A [1, 16] row made of one group repeated (K must be a multiple of 16)."""
    return np.tile(np.asarray(group_bits, dtype=np.uint16), reps)[None, :]


# ---------------------------------------------------------------- selection ------------------

def test_hand_cases_from_golden_file():
    n = 0
    with open(os.path.join(GOLDEN, "topk24_hand_cases.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            lhs, rhs = line.split("->")
            x = [float(v) for v in lhs.split()]
            i0, i1 = (int(v) for v in rhs.split())
            X = tile_group(bf16_bits(x))
            mask = oracle.topk24_mask(X)[0, :4]
            want = np.zeros(4, dtype=np.uint8)
            want[[i0, i1]] = 1
            assert (mask == want).all(), (x, mask, want)
            values, meta = oracle.compress(X)
            assert (meta[0, 0] & 0xF) == (i0 | (i1 << 2))
            assert values[0, 0] == X[0, i0] and values[0, 1] == X[0, i1]
            n += 1
    assert n >= 10


def _brute_force_pair(mags):
    """Independent definition: among the 6 index pairs, the valid ones keep magnitudes that are
    all >= every dropped magnitude; the answer is the lexicographically smallest valid pair."""
    best = None
    for pair in itertools.combinations(range(4), 2):
        dropped = [i for i in range(4) if i not in pair]
        if min(mags[i] for i in pair) >= max(mags[i] for i in dropped):
            if best is None or pair < best:
                best = pair
    return best


def test_brute_force_small_alphabet_exhaustive():
    # +0, -0, +-1, +-2, +-Inf, NaN, smallest subnormal, and a value with low mantissa bits
    alphabet = np.array([0x0000, 0x8000, 0x3F80, 0xBF80, 0x4000, 0xC000, 0x7F80, 0xFF80, 0x7FC0,
                         0x0001, 0x8001, 0x3F81], dtype=np.uint16)
    groups = np.array(list(itertools.product(alphabet, repeat=4)), dtype=np.uint16)  # 20736 x 4
    pad = (-len(groups)) % 4
    groups = np.concatenate([groups, np.zeros((pad, 4), dtype=np.uint16)])
    X = groups.reshape(-1, 16)  # 4 groups per row
    mask = oracle.topk24_mask(X).reshape(-1, 4)
    values, meta = oracle.compress(X)
    nibbles = np.stack([(meta[:, 0] >> (4 * j)) & 0xF for j in range(4)], axis=1).reshape(-1)
    for gi, grp in enumerate(groups):
        mags = [int(b) & 0x7FFF for b in grp]
        i0, i1 = _brute_force_pair(mags)
        assert mask[gi].sum() == 2
        assert mask[gi][i0] == 1 and mask[gi][i1] == 1, (grp, mask[gi], (i0, i1))
        assert nibbles[gi] == (i0 | (i1 << 2))


def test_selection_invariants_random():
    rng = np.random.default_rng(7)
    X = rng.integers(0, 1 << 16, size=(64, 256), dtype=np.uint16)  # every bit pattern class
    mask = oracle.topk24_mask(X)
    g = mask.reshape(64, -1, 4)
    assert (g.sum(-1) == 2).all()
    mag = (X & 0x7FFF).astype(np.int64).reshape(64, -1, 4)
    kept_min = np.where(g == 1, mag, 1 << 20).min(-1)
    drop_max = np.where(g == 0, mag, -1).max(-1)
    assert (kept_min >= drop_max).all()


def test_tie_goes_to_lower_index_everywhere():
    X = np.full((1, 64), 0x3F80, dtype=np.uint16)
    mask = oracle.topk24_mask(X)
    assert (mask.reshape(-1, 4) == np.array([1, 1, 0, 0])).all()
    # sign does not matter for ties
    X[0, 1::2] = 0xBF80
    assert (oracle.topk24_mask(X).reshape(-1, 4) == np.array([1, 1, 0, 0])).all()


# ---------------------------------------------------------------- compression ----------------

LEGAL_NIBBLES = {0x4, 0x8, 0x9, 0xC, 0xD, 0xE}


@pytest.mark.parametrize("dist", ["gelu", "outlier", "gelu_chan"])
def test_compress_decompress_roundtrip(dist):
    X = inputs.as_u16(inputs.make_x(96, 256, dist, 11))
    mask = oracle.topk24_mask(X)
    values, meta = oracle.compress(X)
    back = oracle.decompress(values, meta)
    assert (back == X * mask).all()  # bit-for-bit, incl. sign of kept zeros
    nibs = np.stack([(meta >> (4 * j)) & 0xF for j in range(4)], axis=-1).reshape(-1)
    assert set(np.unique(nibs).tolist()) <= LEGAL_NIBBLES
    # values are exactly the kept entries, in ascending position
    kept = X[mask.astype(bool)].reshape(96, 128)
    assert (kept == values).all()


def test_exactly_two_kept_positions_even_when_values_are_zero():
    X = np.zeros((4, 64), dtype=np.uint16)
    X[0, 5] = 0x4000
    mask = oracle.topk24_mask(X)
    assert (mask.reshape(4, -1, 4).sum(-1) == 2).all()
    values, meta = oracle.compress(X)
    assert (oracle.decompress(values, meta) == X).all()


def _hw_offset_independent(m, k, K):
    """Bit address of logical element (m, k) restated from the tensor-memory picture:
    lane-major 16-byte rows; returns (byte offset, bit in byte)."""
    rb, r = divmod(m, 128)
    kb, kk = divmod(k, 128)
    col, k32 = divmod(kk, 32)           # tensor-memory column = K step
    lane = (r % 8) + 8 * (k32 // 16) + 16 * (r // 16)
    bit = (k32 % 16) + 16 * ((r // 8) % 2)
    byte = (rb * (K // 128) + kb) * 2048 + lane * 16 + col * 4 + bit // 8
    return byte, bit % 8


def test_metadata_hw_permutation_is_bijection_and_matches_layout():
    M, K = 200, 384  # ragged row block
    rng = np.random.default_rng(3)
    X = rng.integers(0, 1 << 16, size=(M, K), dtype=np.uint16)
    _, meta = oracle.compress(X)
    hw = oracle.meta_canon_to_hw(meta, M, K)
    assert hw.size == 2 * 3 * 2048 == oracle.meta_hw_bytes(M, K)
    assert (oracle.meta_hw_to_canon(hw, M, K) == meta).all()
    # every logical element's metadata bit sits where the layout statement says
    for m in [0, 1, 7, 8, 15, 16, 127, 128, 199]:
        for k in [0, 3, 4, 15, 16, 31, 32, 127, 128, 383]:
            canon_bit = (int(meta[m, k // 16]) >> (k % 16)) & 1
            byte, bit = _hw_offset_independent(m, k, K)
            assert ((int(hw[byte]) >> bit) & 1) == canon_bit
    # pad rows hold the legal pattern (positions 0 and 1)
    byte, _ = _hw_offset_independent(255, 0, K)
    assert hw[byte] == 0x44
    # a permutation: each hw byte written exactly once
    marks = oracle.meta_canon_to_hw(np.full((256, K // 16), 0xFFFF, dtype=np.uint16), 256, K)
    assert (marks == 0xFF).all()


# ---------------------------------------------------------------- scale ----------------------

def test_scale_closed_forms():
    # every group [a,a,a,a]: dense norm^2 = 4a^2 G, kept norm^2 = 2a^2 G  ->  s = sqrt(2)
    X = tile_group(bf16_bits([3.0, 3.0, 3.0, 3.0]), reps=16)
    s = oracle.row_scale(X, oracle.COMP_ROW)
    assert abs(s[0] - np.sqrt(2.0)) < 1e-6
    # groups [1,2,2,1]: 10 / 8
    X = tile_group(bf16_bits([1.0, 2.0, 2.0, 1.0]), reps=8)
    assert abs(oracle.row_scale(X, oracle.COMP_ROW)[0] - np.sqrt(1.25)) < 1e-6
    # already 2:4 sparse rows: s = 1 up to eps
    X = tile_group(bf16_bits([0.0, -5.0, 0.0, 0.25]), reps=8)
    assert abs(oracle.row_scale(X, oracle.COMP_ROW)[0] - 1.0) < 1e-7
    # all-zero row: s = 0 (no NaN)
    X = np.zeros((1, 32), dtype=np.uint16)
    assert oracle.row_scale(X, oracle.COMP_ROW)[0] == 0.0
    # mode none
    assert (oracle.row_scale(X, oracle.COMP_NONE) == 1.0).all()


def test_scale_invariant_and_modes():
    Xt = inputs.make_x(32, 512, "gelu", 5)
    X = inputs.as_u16(Xt)
    mask = oracle.topk24_mask(X).astype(np.float64)
    xf = Xt.to(torch.float64).numpy()
    num = (xf ** 2).sum(1)
    den = ((xf * mask) ** 2).sum(1)
    s = oracle.row_scale(X, oracle.COMP_ROW).astype(np.float64)
    # s^2 (den + eps) = num
    np.testing.assert_allclose(s ** 2 * (den + 1e-8), num, rtol=3e-7)
    # rescaled sparse row has the dense row's norm (the stated purpose of the compensation)
    np.testing.assert_allclose(np.sqrt(((s[:, None] * xf * mask) ** 2).sum(1)), np.sqrt(num),
                               rtol=1e-6)
    assert (s >= 1.0).all()
    st = oracle.row_scale(X, oracle.COMP_TENSOR).astype(np.float64)
    assert (st == st[0]).all()
    np.testing.assert_allclose(st[0] ** 2 * (den.sum() + 1e-8), num.sum(), rtol=3e-7)


# ---------------------------------------------------------------- product + epilogue ---------

def test_sparse_path_equals_masked_dense_path_bitwise():
    wl = inputs.Workload("t", 24, 256, 40, "outlier", 21)
    d = inputs.make_workload(wl)
    X, W = inputs.as_u16(d["X"]), inputs.as_u16(d["W"])
    values, meta = oracle.compress(X)
    xm = oracle.decompress(values, meta)
    a = oracle.gemm_masked_f32(xm, W)
    b = oracle.gemm_sparse_f32(values, meta, W)
    assert (a.view(np.uint32) == b.view(np.uint32)).all()
    rows = np.array([3, 0, 23], dtype=np.int64)
    assert (oracle.gemm_sparse_f32(values, meta, W, rows) == b[rows]).all()


def test_gemm_matches_fp64_library_matmul():
    wl = inputs.Workload("t", 16, 512, 48, "gelu", 22)  # N != K catches a transposed W
    d = inputs.make_workload(wl)
    X, W = inputs.as_u16(d["X"]), inputs.as_u16(d["W"])
    mask = torch.from_numpy(oracle.topk24_mask(X).astype(np.float64))
    ref = (d["X"].to(torch.float64) * mask) @ d["W"].to(torch.float64).T
    values, meta = oracle.compress(X)
    xm = oracle.decompress(values, meta)
    got32 = oracle.gemm_masked_f32(xm, W)
    got64 = oracle.gemm_masked_f64(xm, W)
    np.testing.assert_allclose(got64, ref.numpy(), rtol=1e-12, atol=1e-14)
    err = np.linalg.norm(got32 - ref.numpy()) / np.linalg.norm(ref.numpy())
    assert err < 1e-5  # far below the 5e-3 gate applied to the GPU result


def test_already_sparse_input_reduces_to_dense_linear():
    """If X is already 2:4 sparse the whole path is an ordinary linear layer."""
    g = torch.Generator().manual_seed(5)
    M, K, N = 20, 128, 24
    x = torch.randn(M, K, generator=g)
    keep = torch.zeros(M, K // 4, 4)
    for pair_id, pair in enumerate(itertools.combinations(range(4), 2)):
        sel = (torch.arange(M * (K // 4)).reshape(M, K // 4) % 6) == pair_id
        for p in pair:
            keep[..., p] += sel
    keep = keep.reshape(M, K) > 0
    x = torch.where(keep, x + 0.5 * torch.sign(x), torch.zeros(())).to(torch.bfloat16)
    w = inputs.make_w(N, K, 9)
    b = inputs.make_bias(N, 9)
    out = oracle.act_sparse_linear(inputs.as_u16(x), inputs.as_u16(w), bias=inputs.as_u16(b),
                                   comp_mode=oracle.COMP_ROW)
    ref = torch.nn.functional.linear(x.double(), w.double(), b.double()).numpy()
    np.testing.assert_allclose(out["Y"], ref, rtol=2e-5, atol=2e-6)
    np.testing.assert_allclose(out["scale"], 1.0, atol=1e-6)
    assert (oracle.decompress(out["values"], out["meta_canon"]) == inputs.as_u16(x)).all()


def test_integer_valued_case_is_exact():
    rng = np.random.default_rng(0)
    M, K, N = 12, 64, 20
    xi = rng.integers(-8, 9, size=(M, K))
    wi = rng.integers(-4, 5, size=(N, K))
    X = bf16_bits(xi.astype(np.float32).tolist())
    W = bf16_bits(wi.astype(np.float32).tolist())
    mask = oracle.topk24_mask(X).astype(np.int64)
    want = (xi * mask) @ wi.T
    values, meta = oracle.compress(X)
    got = oracle.gemm_sparse_f32(values, meta, W)
    assert (got == want.astype(np.float32)).all()


def test_epilogue_closed_form_and_order():
    acc = np.array([[1.0, -2.0]], dtype=np.float32)
    s = np.array([2.0], dtype=np.float32)
    bias = bf16_bits([0.5, 0.25])
    yr = bf16_bits([[0.25, -1.0]])
    y = oracle.epilogue(acc, 1, s=s, bias=bias, Yr=yr)
    assert y.tolist() == [[2.75, -4.75]]  # s*acc + bias + Yr; bias and Yr are NOT scaled
    assert oracle.epilogue(acc, 1).tolist() == [[1.0, -2.0]]
    assert oracle.epilogue(acc, 1, bias=bias).tolist() == [[1.5, -1.75]]


def test_whole_path_composition_and_row_subset():
    wl = inputs.WORKLOADS["tiny"]
    d = inputs.make_workload(wl, with_bias=True, with_residual=True, M=32)
    X, W = inputs.as_u16(d["X"]), inputs.as_u16(d["W"])
    bias, yr = inputs.as_u16(d["bias"]), inputs.as_u16(d["residual"])
    full = oracle.act_sparse_linear(X, W, bias=bias, comp_mode=oracle.COMP_ROW, Yr=yr)
    mask = oracle.topk24_mask(X).astype(np.float64)
    xf = d["X"].double().numpy()
    s = np.sqrt((xf ** 2).sum(1) / (((xf * mask) ** 2).sum(1) + 1e-8))
    ref = s[:, None] * ((xf * mask) @ d["W"].double().numpy().T) + d["bias"].double().numpy() \
        + d["residual"].double().numpy()
    np.testing.assert_allclose(full["Y"], ref, rtol=3e-5, atol=3e-6)
    rows = np.array([31, 2, 17], dtype=np.int64)
    part = oracle.act_sparse_linear(X, W, bias=bias, comp_mode=oracle.COMP_ROW, Yr=yr, rows=rows)
    assert (part["Y"] == full["Y"][rows]).all()


def test_pruning_error_is_smaller_on_gelu_shaped_rows_than_on_gaussian_rows():
    """Qualitative claim of the motivation section: near-zero-concentrated activations lose
    little under 2:4 pruning.  Sanity only."""
    def rfe(dist):
        x = inputs.make_x(64, 512, dist, 1)
        w = inputs.make_w(64, 512, 1)
        X = inputs.as_u16(x)
        mask = torch.from_numpy(oracle.topk24_mask(X).astype(np.float64))
        full = x.double() @ w.double().T
        sp = (x.double() * mask) @ w.double().T
        return float((full - sp).norm() / full.norm())
    assert rfe("gelu") < 0.6 * rfe("normal")


def test_lora_residual_matches_library_matmul():
    g = torch.Generator().manual_seed(2)
    M, K, R, N = 8, 64, 16, 12
    x = torch.randn(M, K, generator=g).to(torch.bfloat16)
    lb = (torch.randn(R, K, generator=g) * 0.1).to(torch.bfloat16)
    la = (torch.randn(N, R, generator=g) * 0.1).to(torch.bfloat16)
    got = oracle.lora_residual(inputs.as_u16(x), inputs.as_u16(lb), inputs.as_u16(la))
    ref = (x.double() @ lb.double().T) @ la.double().T
    np.testing.assert_allclose(got, ref.numpy(), rtol=1e-5, atol=1e-6)


# ---------------------------------------------------------------- per-group norm compensation ---

def _bf(vals):
    return inputs.as_u16(torch.tensor(vals, dtype=torch.float32).to(torch.bfloat16).reshape(1, -1))


def test_group_scale_closed_forms():
    """[a,a,a,a] keeps two of four equal squares: s = sqrt(2); a group that already has two zeros
    keeps everything: s = 1 and the values are bit copies; a zero group stays zero."""
    x = _bf([1, 1, 1, 1, 3, 4, 0, 0, 0, 0, 0, 0, -2, 0.5, 0.25, 2])
    x = np.tile(x, (1, 8))  # K = 128
    v, meta = oracle.compress_group_scaled(x)
    v0, meta0 = oracle.compress(x)
    assert (meta == meta0).all()
    got = inputs.from_u16(v).float().numpy()[0, :8]
    sqrt2 = float(torch.tensor(2.0 ** 0.5).to(torch.bfloat16))
    assert got[0] == sqrt2 and got[1] == sqrt2
    assert got[2] == 3.0 and got[3] == 4.0
    assert got[4] == 0.0 and got[5] == 0.0
    # [-2, .5, .25, 2]: kept -2 and 2, s = sqrt(8.3125 / 8)
    s = (8.3125 / 8.0) ** 0.5
    ref = torch.tensor([-2 * s, 2 * s]).to(torch.bfloat16).float().numpy()
    assert got[6] == ref[0] and got[7] == ref[1]


def test_group_scale_restores_each_groups_norm_and_matches_fp64():
    g = torch.Generator().manual_seed(21)
    M, K = 64, 512
    x = (torch.randn(M, K, generator=g) * torch.exp(torch.randn(M, K, generator=g))).to(torch.bfloat16)
    X = inputs.as_u16(x)
    v, meta = oracle.compress_group_scaled(X)
    v0, _ = oracle.compress(X)
    vs = inputs.from_u16(v).double().numpy().reshape(M, K // 4, 2)
    kept = inputs.from_u16(v0).double().numpy().reshape(M, K // 4, 2)
    xs = x.double().numpy().reshape(M, K // 4, 4)
    # the scaled pair carries the group's whole norm (up to the bf16 rounding of two values)
    np.testing.assert_allclose((vs ** 2).sum(-1), (xs ** 2).sum(-1), rtol=2.0 ** -7, atol=1e-7)
    # the fp32 reading agrees with the fp64 factors to within one bf16 step, and almost always exactly
    s64 = oracle.group_scale_f64(X)
    ref = torch.from_numpy(kept * s64[..., None]).to(torch.bfloat16).double().numpy()
    assert (np.abs(vs - ref) <= np.abs(ref) * 2.0 ** -7).all()
    assert (vs == ref).mean() > 0.995
    # a scale >= 1 never shrinks a kept value, and it is at most sqrt(2) for Top-2-of-4... of equal
    # magnitudes; in general at most 2 (two kept carry at least half of four squares only when
    # they are the largest two, which they are): |X|^2 <= 2 |X~|^2
    assert (s64 <= 2.0 ** 0.5 + 1e-6).all() and (s64[(xs ** 2).sum(-1) > 1e-6] >= 1.0 - 1e-6).all()


def test_group_mode_equals_row_mode_when_a_row_is_one_group():
    """K = 128 is the smallest K; make 31 of the 32 groups of every row zero: then the row scale
    and the only non-zero group's scale are the same number."""
    g = torch.Generator().manual_seed(22)
    M, K = 48, 128
    x = torch.zeros(M, K)
    x[:, 8:12] = torch.randn(M, 4, generator=g)
    x = x.to(torch.bfloat16)
    X = inputs.as_u16(x)
    v, _ = oracle.compress_group_scaled(X)
    v0, _ = oracle.compress(X)
    s_row = oracle.row_scale(X, oracle.COMP_ROW).astype(np.float64)
    ref = torch.from_numpy(inputs.from_u16(v0).double().numpy() * s_row[:, None]).to(torch.bfloat16).double().numpy()
    got = inputs.from_u16(v).double().numpy()
    assert (np.abs(got - ref) <= np.abs(ref) * 2.0 ** -7).all()
    assert (got == ref).mean() > 0.99


def test_group_mode_whole_path_is_the_product_of_the_scaled_sparse_activation():
    g = torch.Generator().manual_seed(23)
    M, K, N = 16, 256, 40
    x = torch.randn(M, K, generator=g).to(torch.bfloat16)
    w = (torch.randn(N, K, generator=g) * K ** -0.5).to(torch.bfloat16)
    b = (torch.randn(N, generator=g) * 0.1).to(torch.bfloat16)
    out = oracle.act_sparse_linear(inputs.as_u16(x), inputs.as_u16(w), bias=inputs.as_u16(b), comp_mode=oracle.COMP_GROUP)
    v, meta = oracle.compress_group_scaled(inputs.as_u16(x))
    assert (out["values"] == v).all() and (out["meta_canon"] == meta).all()
    xs = inputs.from_u16(oracle.decompress(v, meta)).double()
    ref = xs @ w.double().T + b.double()
    np.testing.assert_allclose(out["Y"], ref.numpy(), rtol=1e-4, atol=1e-5)
    assert (out["scale"] == 1.0).all()


# --------------------------------------------------------------------------- FP8 composition ---

def test_e4m3_codec_matches_the_library_conversion_and_saturates():
    # decode: all 256 codes against torch's float8_e4m3fn
    codes = torch.arange(256, dtype=torch.uint8)
    ref = codes.view(torch.float8_e4m3fn).float().numpy()
    got = oracle.e4m3_decode(codes.numpy())
    assert (np.isnan(got) == np.isnan(ref)).all() and (got[~np.isnan(ref)] == ref[~np.isnan(ref)]).all()
    # encode: random values, every grid point, every midpoint (ties to even), inside the finite range
    g = torch.Generator().manual_seed(31)
    finite = np.sort(ref[~np.isnan(ref) & (ref >= 0)])
    mids = (finite[1:] + finite[:-1]) / 2
    x = np.concatenate([finite, mids, np.nextafter(mids, 0).astype(np.float32), np.nextafter(mids, 1e9).astype(np.float32),
                        (torch.randn(20000, generator=g) * torch.exp(2 * torch.randn(20000, generator=g))).numpy()])
    x = np.concatenate([x, -x]).astype(np.float32)
    x = x[np.abs(x) <= 464.0]
    want = torch.from_numpy(x).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    assert (oracle.e4m3_encode(x) == want).all()
    # satfinite: beyond the range, and Inf, give +-448; NaN stays NaN
    big = oracle.e4m3_encode(np.array([464.0, 465.0, 1e6, np.inf, -500.0, -np.inf], dtype=np.float32))
    assert (big == np.array([0x7E, 0x7E, 0x7E, 0x7E, 0xFE, 0xFE], dtype=np.uint8)).all()
    assert np.isnan(oracle.e4m3_decode(oracle.e4m3_encode(np.array([np.nan], dtype=np.float32)))).all()


def test_fp8_activation_codes_closed_forms():
    """Row amax maps to +-448 exactly; a row of zeros gives zero codes and a zero scale; the mask
    is the bf16 one; the decoded codes times the scale reproduce the kept values to E4M3 accuracy."""
    g = torch.Generator().manual_seed(32)
    M, K = 24, 256
    x = torch.randn(M, K, generator=g)
    x[3] = 0.0
    x[5, 17] = 100.0
    x = x.to(torch.bfloat16)
    X = inputs.as_u16(x)
    vq, meta, sc = oracle.compress_fp8(X)
    v0, meta0 = oracle.compress(X)
    assert (meta == meta0).all()
    dec = oracle.e4m3_decode(vq)
    amax = x.float().abs().max(dim=1).values.numpy()
    assert (np.abs(dec).max(axis=1)[amax > 0] == 448.0).all()
    assert sc[3] == 0.0 and (vq[3] == 0).all()
    np.testing.assert_allclose(sc, amax / 448.0, rtol=1e-6)
    kept = inputs.from_u16(v0).float().numpy()
    err = np.abs(dec * sc[:, None] - kept)
    # E4M3: 3 mantissa bits -> half a step is 2^-4 relative for normals; below 2^-6 of the row's
    # maximum / 448 * ... the grid is absolute (subnormals): 2^-10 * scale
    assert (err <= np.maximum(np.abs(kept) * 2.0 ** -4, sc[:, None] * 2.0 ** -10) * 1.0001).all()


def test_fp8_given_row_maximum():
    """A supplied maximum equal to the true one changes nothing; a larger one scales the codes
    down (same mask); a smaller one saturates at +-448."""
    g = torch.Generator().manual_seed(36)
    M, K = 8, 256
    x = torch.randn(M, K, generator=g).to(torch.bfloat16)
    X = inputs.as_u16(x)
    vq, meta, sc = oracle.compress_fp8(X)
    amax = x.float().abs().max(dim=1).values.numpy()
    vq1, meta1, sc1 = oracle.compress_fp8(X, row_amax=amax)
    assert (vq1 == vq).all() and (meta1 == meta).all() and (sc1 == sc).all()
    vq2, meta2, sc2 = oracle.compress_fp8(X, row_amax=2 * amax)
    assert (meta2 == meta).all() and (sc2 == 2 * sc).all()
    assert np.abs(oracle.e4m3_decode(vq2)).max() == 224.0
    vq3, _, sc3 = oracle.compress_fp8(X, row_amax=0.25 * amax)
    assert np.abs(oracle.e4m3_decode(vq3)).max() == 448.0 and (np.abs(oracle.e4m3_decode(vq3)) == 448.0).sum() > M


def test_fp8_metadata_order_is_the_rows_bytes_block_by_block():
    """Independent restatement: per (128-row, 128-K) block, row r's 16 bytes are the row's 8
    canonical little-endian words of that K block; rows past M are 0x44."""
    g = torch.Generator().manual_seed(35)
    M, K = 200, 384
    X = inputs.as_u16(torch.randn(M, K, generator=g).to(torch.bfloat16))
    _, meta = oracle.compress(X)
    hw = oracle.meta_canon_to_hw_fp8(meta, M, K).reshape(2, 3, 128, 16)
    rows = meta.view(np.uint8).reshape(M, K // 128, 16)          # little-endian host
    for rb in range(2):
        n = min(128, M - rb * 128)
        assert (hw[rb, :, :n, :] == rows[rb * 128: rb * 128 + n].transpose(1, 0, 2)).all()
        assert (hw[rb, :, n:, :] == 0x44).all()


def test_fp8_weight_quantisation_modes():
    g = torch.Generator().manual_seed(33)
    N, K = 12, 64
    w = (torch.randn(N, K, generator=g) * 0.05).to(torch.bfloat16)
    Wq, ws = oracle.quantize_weights_fp8(inputs.as_u16(w), per_channel=False)
    assert (ws == 1.0).all()
    assert (Wq == w.float().to(torch.float8_e4m3fn).view(torch.uint8).numpy()).all()   # a direct cast
    Wq, ws = oracle.quantize_weights_fp8(inputs.as_u16(w), per_channel=True)
    amax = w.float().abs().max(dim=1).values.numpy()
    np.testing.assert_allclose(ws, amax / 448.0, rtol=1e-6)
    assert (np.abs(oracle.e4m3_decode(Wq)).max(axis=1) == 448.0).all()


def test_fp8_whole_path_is_the_product_of_the_dequantised_operands():
    g = torch.Generator().manual_seed(34)
    M, K, N = 16, 256, 24
    x = torch.randn(M, K, generator=g).to(torch.bfloat16)
    w = (torch.randn(N, K, generator=g) * K ** -0.5).to(torch.bfloat16)
    b = (torch.randn(N, generator=g) * 0.1).to(torch.bfloat16)
    X = inputs.as_u16(x)
    for per_channel in (False, True):
        Wq, ws = oracle.quantize_weights_fp8(inputs.as_u16(w), per_channel)
        for mode in (oracle.COMP_NONE, oracle.COMP_ROW):
            out = oracle.act_sparse_linear_fp8(X, Wq, ws, bias=inputs.as_u16(b), comp_mode=mode)
            vq, meta, sc = oracle.compress_fp8(X)
            assert (out["values_q"] == vq).all() and (out["meta_canon"] == meta).all()
            # restated: scatter the decoded codes by the metadata, multiply in fp64
            xs = np.zeros((M, K))
            dec = oracle.e4m3_decode(vq).astype(np.float64).reshape(M, K // 4, 2)
            for m in range(M):
                for gi in range(K // 4):
                    nib = (int(meta[m, gi // 4]) >> (4 * (gi % 4))) & 0xF
                    xs[m, 4 * gi + (nib & 3)] = dec[m, gi, 0]
                    xs[m, 4 * gi + (nib >> 2)] = dec[m, gi, 1]
            s = oracle.row_scale(X, mode).astype(np.float64) * sc.astype(np.float64)
            ref = (xs @ oracle.e4m3_decode(Wq).astype(np.float64).T) * s[:, None] * ws.astype(np.float64)[None, :] \
                + b.double().numpy()[None, :]
            np.testing.assert_allclose(out["Y"], ref, rtol=1e-4, atol=1e-5)
            np.testing.assert_allclose(out["row_scale"], s, rtol=1e-6)
            # and the FP8 layer stays close to the bf16 sparse layer it approximates
            # (per-channel weight scales only: a direct cast of weights this small sits in E4M3's subnormals)
            if per_channel:
                y16 = oracle.act_sparse_linear(X, inputs.as_u16(w), bias=inputs.as_u16(b), comp_mode=mode)["Y"]
                assert np.linalg.norm(out["Y"] - y16) / np.linalg.norm(y16) < 0.06


def test_lora_rows_subset_equals_full_rows():
    g = torch.Generator().manual_seed(12)
    M, K, R, N = 20, 128, 8, 24
    x = torch.randn(M, K, generator=g).to(torch.bfloat16)
    lb = (torch.randn(R, K, generator=g) * 0.1).to(torch.bfloat16)
    la = (torch.randn(N, R, generator=g) * 0.1).to(torch.bfloat16)
    full = oracle.lora_residual(inputs.as_u16(x), inputs.as_u16(lb), inputs.as_u16(la))
    rows = np.array([19, 0, 7], dtype=np.int64)
    sub = oracle.lora_residual(inputs.as_u16(x), inputs.as_u16(lb), inputs.as_u16(la), rows=rows)
    assert (sub == full[rows]).all()


def test_lora_path_uses_the_dense_x_not_the_pruned_one():
    """W = 0 leaves only the LoRA branch: Y must be the DENSE product X (L_A L_B)^T (Algorithm 1
    line 5 applies the low-rank term to X, not to S(X)); a branch fed with the pruned X fails."""
    g = torch.Generator().manual_seed(13)
    M, K, R, N = 16, 128, 8, 40
    x = torch.randn(M, K, generator=g).to(torch.bfloat16)
    w = torch.zeros(N, K, dtype=torch.bfloat16)
    lb = (torch.randn(R, K, generator=g) * 0.2).to(torch.bfloat16)
    la = (torch.randn(N, R, generator=g) * 0.2).to(torch.bfloat16)
    out = oracle.act_sparse_linear_lora(inputs.as_u16(x), inputs.as_u16(w), inputs.as_u16(la), inputs.as_u16(lb),
                                        comp_mode=oracle.COMP_ROW)
    dense = (x.double() @ lb.double().T) @ la.double().T
    np.testing.assert_allclose(out["Y"], dense.numpy(), rtol=2e-5, atol=2e-6)
    mask = torch.from_numpy(oracle.topk24_mask(inputs.as_u16(x)).astype(np.float64))
    pruned = ((x.double() * mask) @ lb.double().T) @ la.double().T
    assert np.abs(out["Y"] - pruned.numpy()).max() > 1e-2


def test_lora_path_on_sparse_input_is_a_dense_linear_with_merged_weights():
    """On an input that already is 2:4 sparse the layer is exact (s = 1, mask = support), so
    Y = X (W + L_A L_B)^T + b: the LoRA term is neither scaled by s nor dropped, and it is
    added once."""
    g = torch.Generator().manual_seed(14)
    M, K, R, N = 12, 256, 16, 24
    x = torch.randn(M, K, generator=g)
    keep = torch.zeros(M, K // 4, 4)
    keep[..., 0] = 1
    keep[..., 2] = 1
    x = torch.where(keep.reshape(M, K) > 0, x, torch.zeros(())).to(torch.bfloat16)
    w = (torch.randn(N, K, generator=g) * K ** -0.5).to(torch.bfloat16)
    b = (torch.randn(N, generator=g) * 0.1).to(torch.bfloat16)
    lb = (torch.randn(R, K, generator=g) * 0.1).to(torch.bfloat16)
    la = (torch.randn(N, R, generator=g) * 0.1).to(torch.bfloat16)
    for mode in (oracle.COMP_NONE, oracle.COMP_ROW, oracle.COMP_TENSOR):
        out = oracle.act_sparse_linear_lora(inputs.as_u16(x), inputs.as_u16(w), inputs.as_u16(la), inputs.as_u16(lb),
                                            bias=inputs.as_u16(b), comp_mode=mode)
        merged = w.double() + la.double() @ lb.double()
        ref = x.double() @ merged.T + b.double()
        np.testing.assert_allclose(out["Y"], ref.numpy(), rtol=1e-4, atol=1e-5)


def test_bf16_rounding_routine_matches_torch():
    g = torch.Generator().manual_seed(3)
    v = torch.randn(4096, generator=g) * 10
    v[:4] = torch.tensor([0.0, -0.0, float("inf"), 1.00390625])  # last one is a tie case
    got = oracle.f32_to_bf16(v.numpy())
    assert (got == inputs.as_u16(v.to(torch.bfloat16))).all()
