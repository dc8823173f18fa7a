"""Pins for the CPU oracle: each test checks it against something other than itself.

The paper prints no worked numeric example, so the pins are: a library fp64 convolution
(sparsity 0), the paper's three stages written out with a library matrix product
(Section 3.2: lowering, dense GEMM on kept rows, zero re-insertion), closed forms,
unit impulses, integer brute force on tiny inputs, and the invariants of the kept list.
"""
import itertools

import numpy as np
import pytest
import torch

import oracle
import workloads as wl


def _rand_case(rng, Nb, H, W, C_in, C_out, kh, kw):
    x = rng.standard_normal((Nb, H, W, C_in)).astype(np.float32)
    w = rng.standard_normal((C_out, kh, kw, C_in)).astype(np.float32)
    b = rng.standard_normal((C_out,)).astype(np.float32)
    return x, w, b


def _torch_bf16(a):
    """bf16 rounding by the library's own conversion, widened to fp64."""
    return torch.from_numpy(np.ascontiguousarray(a)).to(torch.bfloat16).to(torch.float64)


# ----------------------------------------------------------------------------- rounding
def test_bf16_rounding_matches_library_conversion():
    rng = np.random.default_rng(1)
    a = rng.standard_normal(1_000_000).astype(np.float32)
    a[:1000] *= 1e-39                       # denormals
    a[1000:2000] *= 1e30
    # exact ties: bf16 value + half an ulp, both parities
    base = rng.integers(0, 0x7f7f, size=5000).astype(np.uint32) << 16   # finite, positive
    ties = (base | 0x8000).view(np.float32)
    a[2000:7000] = ties
    a[7000:7004] = [np.inf, -np.inf, 0.0, -0.0]
    got = oracle.bf16_round(a)
    ref = torch.from_numpy(a).to(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(got.view(np.uint32), ref.view(np.uint32))
    assert np.isnan(oracle.bf16_round(np.array([np.nan], dtype=np.float32)))[0]


# ----------------------------------------------------------------------------- O1
GEOMS = [  # kh, kw, stride, pad, H, W, C_in, C_out, Nb
    (3, 3, 1, 1, 9, 11, 5, 4, 2),
    (3, 3, 2, 1, 10, 13, 3, 6, 2),
    (1, 1, 1, 0, 6, 7, 8, 3, 1),
    (1, 1, 2, 0, 7, 9, 4, 5, 2),
    (7, 7, 2, 3, 17, 16, 3, 4, 1),
    (5, 5, 1, 2, 8, 8, 2, 2, 1),
    (3, 3, 1, 0, 6, 6, 4, 4, 1),
    (1, 3, 1, 1, 5, 9, 3, 2, 1),
    (3, 2, 2, 2, 9, 8, 2, 3, 2),
]


@pytest.mark.parametrize("g", GEOMS)
@pytest.mark.parametrize("relu", [False, True])
def test_sparsity0_equals_library_conv(g, relu):
    """All-ones mask: the result is the ordinary convolution (the GEMM is unaltered,
    Appendix A), checked against torch.nn.functional.conv2d in fp64."""
    kh, kw, s, p, H, W, C_in, C_out, Nb = g
    rng = np.random.default_rng(hash(g) & 0xffff)
    x, w, b = _rand_case(rng, Nb, H, W, C_in, C_out, kh, kw)
    Ho, Wo = (H + 2 * p - kh) // s + 1, (W + 2 * p - kw) // s + 1
    y = oracle.masked_conv(x, w, b, np.ones(Ho * Wo, np.uint8), s, p, relu)
    xt = _torch_bf16(x).permute(0, 3, 1, 2)
    wt = _torch_bf16(w).permute(0, 3, 1, 2)
    ref = torch.nn.functional.conv2d(xt, wt, torch.from_numpy(b).double(), stride=s, padding=p)
    if relu:
        ref = ref.clamp_min(0)
    ref = ref.permute(0, 2, 3, 1).numpy()
    assert y.shape == ref.shape == (Nb, Ho, Wo, C_out)
    assert np.max(np.abs(y - ref)) <= 1e-12 * max(1.0, np.max(np.abs(ref)))


# ----------------------------------------------------------------------------- O2
def _lowered_matrix(xh, kh, kw, s, p):
    """Explicit lowered activation matrix, one row per sliding window (Section 3),
    K ordered (ky, kx, ci)."""
    Nb, H, W, C = xh.shape
    Ho, Wo = (H + 2 * p - kh) // s + 1, (W + 2 * p - kw) // s + 1
    xp = np.zeros((Nb, H + 2 * p, W + 2 * p, C), dtype=np.float64)
    xp[:, p:p + H, p:p + W, :] = xh
    A = np.empty((Nb, Ho, Wo, kh, kw, C), dtype=np.float64)
    for ky in range(kh):
        for kx in range(kw):
            A[:, :, :, ky, kx, :] = xp[:, ky:ky + s * Ho:s, kx:kx + s * Wo:s, :]
    return A.reshape(Nb * Ho * Wo, kh * kw * C), Ho, Wo


@pytest.mark.parametrize("g", GEOMS)
@pytest.mark.parametrize("per_row", [False, True])
def test_masked_equals_three_stage_pipeline(g, per_row):
    """Section 3.2: (i) lowering with masked rows skipped, (ii) a dense product on the kept
    rows, (iii) zeros inserted at the dropped positions."""
    kh, kw, s, p, H, W, C_in, C_out, Nb = g
    rng = np.random.default_rng(7 + (hash(g) & 0xfff))
    x, w, b = _rand_case(rng, Nb, H, W, C_in, C_out, kh, kw)
    xh, wh = _torch_bf16(x).numpy(), _torch_bf16(w).numpy()
    A, Ho, Wo = _lowered_matrix(xh, kh, kw, s, p)
    rows = Nb * Ho * Wo if per_row else Ho * Wo
    mask = (rng.random(rows) < 0.6).astype(np.uint8)
    full_mask = mask if per_row else np.tile(mask, Nb)
    kept = np.nonzero(full_mask)[0]
    C = np.matmul(A[kept], wh.reshape(C_out, -1).T) + b.astype(np.float64)
    C = np.maximum(C, 0.0)
    ref = np.zeros((Nb * Ho * Wo, C_out))
    ref[kept] = C
    y = oracle.masked_conv(x, w, b, mask, s, p, True).reshape(-1, C_out)
    assert np.max(np.abs(y - ref)) <= 1e-12 * max(1.0, np.max(np.abs(ref)))
    dropped = np.nonzero(full_mask == 0)[0]
    assert np.all(y[dropped] == 0.0)


# ----------------------------------------------------------------------------- O3
def test_closed_form_all_ones_3x3():
    """x = 1, w = 1, 3x3 pad 1 stride 1: each output counts the taps inside the image:
    4 at corners, 6 on edges, 9 inside, times C_in, plus the bias."""
    H, W, C_in, C_out = 6, 8, 5, 3
    x = np.ones((1, H, W, C_in), np.float32)
    w = np.ones((C_out, 3, 3, C_in), np.float32)
    b = np.array([0.5, -1.0, 2.0], np.float32)
    y = oracle.masked_conv(x, w, b, np.ones(H * W, np.uint8), 1, 1, False)[0]
    cnt_y = np.array([2] + [3] * (H - 2) + [2])
    cnt_x = np.array([2] + [3] * (W - 2) + [2])
    ref = (np.outer(cnt_y, cnt_x) * C_in)[:, :, None] + b[None, None, :].astype(np.float64)
    assert np.array_equal(y, ref)


def test_closed_form_1x1_is_per_pixel_matvec():
    rng = np.random.default_rng(3)
    x = rng.integers(-4, 5, (2, 4, 5, 6)).astype(np.float32)
    w = rng.integers(-3, 4, (7, 1, 1, 6)).astype(np.float32)
    y = oracle.masked_conv(x, w, None, np.ones(20, np.uint8), 1, 0, False)
    ref = np.einsum("nhwc,oc->nhwo", x.astype(np.float64), w[:, 0, 0, :].astype(np.float64))
    assert np.array_equal(y, ref)


def test_stride2_shape_and_sampled_positions():
    """1x1 stride 2 with w = identity picks input pixels (2*oy, 2*ox)."""
    C = 3
    x = np.arange(2 * 7 * 9 * C, dtype=np.float32).reshape(2, 7, 9, C) % 251
    w = np.eye(C, dtype=np.float32).reshape(C, 1, 1, C)
    y = oracle.masked_conv(x, w, None, np.ones(4 * 5, np.uint8), 2, 0, False)
    assert y.shape == (2, 4, 5, C)
    assert np.array_equal(y, x[:, ::2, ::2, :].astype(np.float64))


# ----------------------------------------------------------------------------- O4
@pytest.mark.parametrize("s,p", [(1, 1), (2, 1), (1, 0), (2, 3)])
def test_unit_impulse_reads_out_the_filter_unflipped(s, p):
    """A unit impulse at (iy0, ix0, ci0) gives y[oy,ox,co] = w[co][iy0-oy*s+p][ix0-ox*s+p][ci0]
    where that tap exists, else 0: cross-correlation, K ordered (ky, kx, ci)."""
    kh, kw = (3, 3) if p < 3 else (7, 7)
    H, W, C_in, C_out = 9, 10, 3, 2
    rng = np.random.default_rng(11)
    w = rng.integers(-8, 9, (C_out, kh, kw, C_in)).astype(np.float32)
    Ho, Wo = (H + 2 * p - kh) // s + 1, (W + 2 * p - kw) // s + 1
    for iy0, ix0, ci0 in [(0, 0, 0), (4, 5, 1), (H - 1, W - 1, 2), (3, 0, 2)]:
        x = np.zeros((1, H, W, C_in), np.float32)
        x[0, iy0, ix0, ci0] = 1.0
        y = oracle.masked_conv(x, w, None, np.ones(Ho * Wo, np.uint8), s, p, False)[0]
        ref = np.zeros((Ho, Wo, C_out))
        for oy, ox in itertools.product(range(Ho), range(Wo)):
            ky, kx = iy0 - oy * s + p, ix0 - ox * s + p
            if 0 <= ky < kh and 0 <= kx < kw:
                ref[oy, ox, :] = w[:, ky, kx, ci0]
        assert np.array_equal(y, ref)


# ----------------------------------------------------------------------------- O5
def _brute_force_int(x, w, b, mask, s, p, relu):
    """Integer arithmetic with Python ints: exact."""
    Nb, H, W, C_in = x.shape
    C_out, kh, kw, _ = w.shape
    Ho, Wo = (H + 2 * p - kh) // s + 1, (W + 2 * p - kw) // s + 1
    xi, wi, bi = x.astype(int).tolist(), w.astype(int).tolist(), b.astype(int).tolist()
    out = np.zeros((Nb, Ho, Wo, C_out), dtype=np.int64)
    for n, oy, ox in itertools.product(range(Nb), range(Ho), range(Wo)):
        if not mask[oy * Wo + ox]:
            continue
        for co in range(C_out):
            acc = bi[co]
            for ky, kx, ci in itertools.product(range(kh), range(kw), range(C_in)):
                iy, ix = oy * s - p + ky, ox * s - p + kx
                if 0 <= iy < H and 0 <= ix < W:
                    acc += xi[n][iy][ix][ci] * wi[co][ky][kx][ci]
            out[n, oy, ox, co] = max(acc, 0) if relu else acc
    return out


@pytest.mark.parametrize("k,p", [(1, 0), (3, 1), (3, 0)])
@pytest.mark.parametrize("C_in", [1, 2, 3, 4])
@pytest.mark.parametrize("C_out", [1, 2, 3, 4])
def test_tiny_integer_cases_brute_force(k, p, C_in, C_out):
    rng = np.random.default_rng(100 * k + 10 * C_in + C_out)
    H, W = 5, 4
    x = rng.integers(-3, 4, (2, H, W, C_in)).astype(np.float32)
    w = rng.integers(-2, 3, (C_out, k, k, C_in)).astype(np.float32)
    b = rng.integers(-4, 5, (C_out,)).astype(np.float32)
    Ho, Wo = H + 2 * p - k + 1, W + 2 * p - k + 1
    mask = (rng.random(Ho * Wo) < 0.5).astype(np.uint8)
    for relu in (False, True):
        y = oracle.masked_conv(x, w, b, mask, 1, p, relu)
        assert np.array_equal(y, _brute_force_int(x, w, b, mask, 1, p, relu).astype(np.float64))


def test_hand_computed_2x2_input_3x3_filter():
    """Worked by hand: x = [[1,2],[3,4]] (one channel), w = [[1..9]] row-major, pad 1.
    y[0,0] = 5*1+6*2+8*3+9*4 = 77, y[0,1] = 4*1+5*2+7*3+8*4 = 67,
    y[1,0] = 2*1+3*2+5*3+6*4 = 47, y[1,1] = 1*1+2*2+4*3+5*4 = 37; bias 10; mask drops (0,1)."""
    x = np.array([[1, 2], [3, 4]], np.float32).reshape(1, 2, 2, 1)
    w = np.arange(1, 10, dtype=np.float32).reshape(1, 3, 3, 1)
    y = oracle.masked_conv(x, w, np.array([10], np.float32), np.array([1, 0, 1, 1], np.uint8),
                           1, 1, False)
    assert y.reshape(-1).tolist() == [87.0, 0.0, 57.0, 47.0]


# ----------------------------------------------------------------------------- O6
def test_masked_is_mask_times_dense_bit_for_bit():
    rng = np.random.default_rng(21)
    x, w, b = _rand_case(rng, 2, 9, 8, 6, 5, 3, 3)
    mask = (rng.random(72) < 0.5).astype(np.uint8)
    dense = oracle.masked_conv(x, w, b, np.ones(72, np.uint8), 1, 1, True)
    y = oracle.masked_conv(x, w, b, mask, 1, 1, True)
    m = mask.reshape(1, 9, 8, 1).astype(bool)
    assert np.array_equal(y, np.where(m, dense, 0.0))


def test_shared_mask_equals_tiled_per_row_mask():
    rng = np.random.default_rng(22)
    x, w, b = _rand_case(rng, 3, 6, 7, 4, 3, 3, 3)
    mask = (rng.random(42) < 0.5).astype(np.uint8)
    a = oracle.masked_conv(x, w, b, mask, 1, 1, False)
    c = oracle.masked_conv(x, w, b, np.tile(mask, 3), 1, 1, False)
    assert np.array_equal(a, c)
    # a per-row mask that differs between images is honoured image by image
    pm = (rng.random(3 * 42) < 0.5).astype(np.uint8)
    d = oracle.masked_conv(x, w, b, pm, 1, 1, False)
    dense = oracle.masked_conv(x, w, b, np.ones(42, np.uint8), 1, 1, False)
    assert np.array_equal(d, np.where(pm.reshape(3, 6, 7, 1).astype(bool), dense, 0.0))


def test_overlapping_windows_one_masked():
    """Figure 2's situation: two overlapping windows, one masked.  The pixels they share
    still contribute to the window that is kept; the masked one is zero in all channels."""
    x = np.arange(1, 9, dtype=np.float32).reshape(1, 2, 4, 1)      # rows [1 2 3 4], [5 6 7 8]
    w = np.ones((2, 2, 2, 1), np.float32)
    w[1] *= 2
    # 2x2 filter, stride 1, no padding: three windows; the first shares {2, 6} with the second
    y = oracle.masked_conv(x, w, None, np.array([0, 1, 1], np.uint8), 1, 0, False)[0, 0]
    assert y.tolist() == [[0.0, 0.0], [2 + 3 + 6 + 7, 2 * (2 + 3 + 6 + 7)], [3 + 4 + 7 + 8, 2 * (3 + 4 + 7 + 8)]]


def test_dropped_rows_are_skipped_not_multiplied():
    x = np.full((1, 4, 4, 2), np.nan, np.float32)
    w = np.ones((3, 3, 3, 2), np.float32)
    y = oracle.masked_conv(x, w, np.ones(3, np.float32), np.zeros(16, np.uint8), 1, 1, True)
    assert np.all(y == 0.0) and not np.any(np.signbit(y))


def test_kept_list_invariants():
    rng = np.random.default_rng(5)
    for rows in (0, 1, 31, 32, 33, 1000, 4097):
        for q in (0.0, 0.3, 1.0):
            mask = (rng.random(rows) < q).astype(np.uint8)
            kept = oracle.kept_list(mask)
            assert kept.dtype == np.int32
            assert np.array_equal(kept, np.nonzero(mask)[0])
            assert len(kept) == rows - int((mask == 0).sum())
            assert np.all(np.diff(kept) > 0)


def test_rows_variant_equals_full():
    spec = next(iter(wl.iter_small_cases()))
    x, w, b, mask = wl.make_x(spec), wl.make_w(spec), wl.make_b(spec), wl.make_layer_mask(spec)
    full = oracle.masked_conv(x, w, b, mask, spec.stride, spec.pad, True).reshape(-1, spec.N)
    sel = np.random.default_rng(0).integers(0, spec.M, 200)
    got = oracle.masked_conv_rows(x, w, b, mask, spec.stride, spec.pad, True, sel)
    assert np.array_equal(got, full[sel])


# ----------------------------------------------------------------------------- generators
def test_generated_masks_have_the_stated_structure():
    for spec in wl.config(3)[:3] + wl.config(4)[:2] + wl.config(1):
        m = wl.make_layer_mask(spec)
        assert m.size == spec.P and set(np.unique(m)) <= {0, 1}
        nblocks = -(-spec.P // spec.block)
        nd = spec.exact_drop if spec.exact_drop is not None else wl.n_drop_blocks(nblocks, spec.sparsity_pct)
        blocks = m[: (spec.P // spec.block) * spec.block].reshape(-1, spec.block)
        assert np.all(blocks.min(1) == blocks.max(1))
        assert int((np.add.reduceat(m, np.arange(0, spec.P, spec.block)) == 0).sum()) == nd
    assert int((wl.make_layer_mask(wl.config(1)[0]) == 0).sum()) == 1568
    assert len(wl.config(2)) == 20 and len(wl.config(4)) == 31 and len(wl.config(5)) == 18
    dense = sum(2 * s.M * s.K * s.N for s in wl.config(3))
    assert abs(dense / 1e9 - 232.1) < 0.2


# ----------------------------------------------------------------------------- the paper's three stages
@pytest.mark.parametrize("name", ["t_3x3_c64", "t_3x3_s2", "t_1x1_s2", "t_7x7_c3", "t_5x5_c24", "t_3x3_c5_n7"])
def test_definition_equals_the_papers_three_stages_in_fp32(name):
    """Appendix A, Algorithm 2 written out as a separate program (pointer indirection buffer over the
    kept positions, dense product on the reduced range, reverse in-place expansion with the running
    id) reaches the oracle's plain definition up to fp32 rounding; dropped positions are exact zeros."""
    spec = [s for s in wl.iter_small_cases() if s.name == name][0]
    x, w, b, m = wl.make_x(spec), wl.make_w(spec), wl.make_b(spec), wl.make_layer_mask(spec)
    xb, wb = oracle.bf16_round(x), oracle.bf16_round(w)
    for relu in (True, False):
        ref = oracle.masked_conv(x, w, b, m, spec.stride, spec.pad, relu)
        got = oracle.alg2_fp32(xb, wb, b, m, spec.stride, spec.pad, relu).astype(np.float64)
        assert np.linalg.norm(got - ref) <= 2e-6 * np.linalg.norm(ref)
        dropped = np.tile(m, spec.Nb).reshape(spec.Nb, spec.Ho, spec.Wo) == 0
        assert not got[dropped].any() and not ref[dropped].any()


def test_three_stage_expansion_handles_all_kept_and_all_dropped():
    rng = np.random.default_rng(21)
    x = rng.standard_normal((2, 6, 5, 4)).astype(np.float32)
    w = rng.standard_normal((3, 3, 3, 4)).astype(np.float32)
    for mask in (np.ones(30, np.uint8), np.zeros(30, np.uint8)):
        ref = oracle.masked_conv(x, w, None, mask, 1, 1, False)
        got = oracle.alg2_fp32(oracle.bf16_round(x), oracle.bf16_round(w), None, mask, 1, 1, False)
        assert np.allclose(got, ref, rtol=1e-5, atol=1e-5)


# ---- SiLU (the activation of YOLOv5, one of the networks of Section 4)

def _one_by_one(values, bias, act, mask=None):
    """A 1x1 convolution with weight 1 over one row of pixels: the pre-activation is value + bias."""
    x = np.asarray(values, dtype=np.float32).reshape(1, 1, -1, 1)
    w = np.ones((1, 1, 1, 1), dtype=np.float32)
    b = np.asarray([bias], dtype=np.float32)
    m = np.ones(x.shape[2], dtype=np.uint8) if mask is None else np.asarray(mask, dtype=np.uint8)
    return oracle.masked_conv(x, w, b, m, 1, 0, act).ravel()


def test_silu_closed_forms():
    # values exactly representable in bf16, so the pre-activation is known exactly
    z = np.array([0.0, 0.5, 1.0, -2.0, 3.5, -8.0, 16.0, -0.25])
    y = _one_by_one(z, 0.0, "silu")
    import math
    # z sigma(z) written with tanh instead of exp: sigma(z) = (1 + tanh(z / 2)) / 2
    ref = np.array([0.5 * v * (1.0 + math.tanh(0.5 * v)) for v in z])
    np.testing.assert_allclose(y, ref, rtol=1e-14, atol=1e-16)
    assert y[0] == 0.0
    # printed values of z sigma(z): 1 -> 0.7310585786..., -2 -> -0.2384058440...
    assert abs(y[2] - 0.7310585786300049) < 1e-15
    assert abs(y[3] + 0.2384058440442351) < 1e-15
    # odd part: silu(z) - silu(-z) = z
    y2 = _one_by_one(-z, 0.0, "silu")
    np.testing.assert_allclose(y - y2, z, rtol=0, atol=1e-15)
    # bounded below by its minimum -0.27846..., close to z for large z, close to 0 for very negative z
    dense = _one_by_one(np.arange(-64, 64) / 8.0, 0.0, "silu")
    assert dense.min() > -0.2785 and dense.min() < -0.278
    assert abs(y[6] - 16.0) < 2e-6 and -3e-3 < y[5] < 0.0


def test_silu_applies_after_bias_and_only_on_kept_positions():
    z = np.array([1.0, -1.0, 2.0, 0.5])
    y = _one_by_one(z, 0.5, "silu", mask=[1, 0, 1, 0])
    import math
    assert y[1] == 0.0 and y[3] == 0.0                       # not silu(bias)
    for i in (0, 2):
        v = z[i] + 0.5
        assert abs(y[i] - v / (1.0 + math.exp(-v))) < 1e-15
    # the three activation codes differ where they should
    none = _one_by_one(z, 0.5, "none", mask=[1, 1, 1, 1])
    relu = _one_by_one(z, 0.5, "relu", mask=[1, 1, 1, 1])
    np.testing.assert_array_equal(none, z + 0.5)
    np.testing.assert_array_equal(relu, np.maximum(z + 0.5, 0.0))


# ---- fp32 storage (the paper's, Appendix A): inputs taken as given

def test_fp32_storage_equals_library_fp64_conv_on_unrounded_inputs():
    rng = np.random.default_rng(77)
    x = rng.standard_normal((2, 6, 7, 5)).astype(np.float32)
    w = rng.standard_normal((4, 3, 3, 5)).astype(np.float32)
    b = rng.standard_normal(4).astype(np.float32)
    m = (rng.random(42) < 0.6).astype(np.uint8)
    y = oracle.masked_conv(x, w, b, m, 1, 1, False, storage="fp32")
    ref = torch.nn.functional.conv2d(torch.from_numpy(x).double().permute(0, 3, 1, 2),
                                     torch.from_numpy(w).double().permute(0, 3, 1, 2),
                                     torch.from_numpy(b).double(), padding=1).permute(0, 2, 3, 1).numpy()
    ref = ref * np.tile(m, 2).reshape(2, 6, 7, 1)
    np.testing.assert_allclose(y, ref, rtol=0, atol=1e-13)
    # the inputs are not bf16 values, so the bf16-storage result must differ (the option does something)
    assert np.abs(oracle.masked_conv(x, w, b, m, 1, 1, False) - y).max() > 1e-3
    # on bf16-representable inputs both storages agree exactly
    xr, wr = oracle.bf16_round(x), oracle.bf16_round(w)
    np.testing.assert_array_equal(oracle.masked_conv(xr, wr, b, m, 1, 1, True, storage="fp32"),
                                  oracle.masked_conv(x, w, b, m, 1, 1, True))
    sel = np.array([0, 5, 41, 42, 80])
    np.testing.assert_array_equal(oracle.masked_conv_rows(x, w, b, m, 1, 1, "silu", sel, storage="fp32"),
                                  oracle.masked_conv(x, w, b, m, 1, 1, "silu", storage="fp32").reshape(84, 4)[sel])


def test_tf32_operand_keeps_ten_mantissa_bits_and_never_grows():
    """TF32 has 10 explicit mantissa bits: values with at most 11 significant bits are unchanged,
    everything else loses less than 2^-10 of its magnitude, towards zero; the result is idempotent."""
    rng = np.random.default_rng(32)
    a = np.concatenate([rng.standard_normal(100000).astype(np.float32) * np.float32(10.0) ** rng.integers(-20, 20, 100000).astype(np.float32),
                        np.array([0.0, -0.0, 1.0, -1.0, 1.0 + 2.0 ** -10, 1.0 + 2.0 ** -11, 3.0 - 2.0 ** -22, np.inf, -np.inf], np.float32)])
    t = oracle.tf32_operand(a)
    assert np.array_equal(oracle.tf32_operand(t), t)
    fin = np.isfinite(a)
    assert np.all(np.abs(t[fin]) <= np.abs(a[fin])) and np.array_equal(np.signbit(t), np.signbit(a))
    big = fin & (np.abs(a) > 1e-30)
    assert np.all(np.abs(a[big].astype(np.float64) - t[big]) < np.abs(a[big].astype(np.float64)) * 2.0 ** -10)
    assert np.array_equal(t[~fin], a[~fin])
    # 11 significant bits survive, the twelfth is dropped
    assert oracle.tf32_operand(np.float32(1.0 + 2.0 ** -10)) == np.float32(1.0 + 2.0 ** -10)
    assert oracle.tf32_operand(np.float32(1.0 + 2.0 ** -11)) == np.float32(1.0)
    assert oracle.tf32_operand(np.float32(3.0 - 2.0 ** -22)) == np.float32(3.0 - 2.0 ** -9)
    ints = np.arange(-2048, 2049, dtype=np.float32)
    assert np.array_equal(oracle.tf32_operand(ints), ints)
