"""The window-patch form of the fused kernel (a tile's window range loaded once into shared memory, the
filter taps cut out of it into tensor memory) against the CPU oracle, and against the row-gather form.

The library takes this form by itself for stride-1 layers with several filter taps and C_in % 64 == 0
whose mask came from host memory and whose tiles' windows fit the patch buffers; every case below
asserts which form ran, so that a silent change of the choice cannot turn these into tests of the
other form."""
import numpy as np
import pytest
import torch

import oracle
import paper_2309_06626_b200 as asx
import workloads as wl
from gpu_util import check_against_oracle, make_problem, max_abs_tol, to_dev_bf16, REL_FROB_TOL

pytestmark = pytest.mark.gpu


def run_form(spec, x, w, b, mask, flags):
    """Runs the layer and returns (y float64 [M][N], bits, form)."""
    layer = asx.MaskedConvLayer(spec.C_in, spec.C_out, spec.kh, spec.kw, spec.stride, spec.pad)
    layer.set_mask(mask)
    xd, wd = to_dev_bf16(x), to_dev_bf16(w)
    bd = None if b is None else torch.from_numpy(b).cuda()
    out = torch.empty((spec.Nb, spec.Ho, spec.Wo, spec.C_out), dtype=torch.bfloat16, device="cuda")
    out.view(torch.int16).fill_(0x7fc1)
    layer.run(xd, wd, bd, out=out, flags=flags)
    torch.cuda.synchronize()
    assert layer.device_status() == 0
    form = layer.last_run_form()
    layer.close()
    bits = out.view(torch.int16).cpu().numpy().view(np.uint16).reshape(spec.M, spec.C_out)
    return out.float().cpu().numpy().astype(np.float64).reshape(spec.M, spec.C_out), bits, form


def spec_of(name, cin, cout, kh, kw, pad, H, W, Nb, pct, blk, seed):
    return wl.LayerSpec(name, cin, cout, kh, kw, 1, pad, H, W, Nb, pct, blk, "relu", wl.BASE_SEED + 7000 + seed)


CASES = [
    # name, C_in, C_out, kh, kw, pad, H, W, Nb, pct, block
    ("p_3x3_c64_n64", 64, 64, 3, 3, 1, 20, 23, 2, 30, 1),
    ("p_3x3_c64_n64_dense", 64, 64, 3, 3, 1, 20, 23, 2, 0, 1),
    ("p_3x3_c64_56", 64, 64, 3, 3, 1, 56, 56, 3, 50, 4),          # the ResNet layer1 shape
    ("p_3x3_c128_28", 128, 128, 3, 3, 1, 28, 28, 4, 50, 4),       # layer2: two slices
    ("p_3x3_c256_14", 256, 256, 3, 3, 1, 14, 14, 6, 50, 4),       # layer3: tiles cross image borders, two column tiles
    ("p_3x3_c64_n24", 64, 24, 3, 3, 1, 17, 19, 2, 25, 1),         # narrow tile (BN = 32), odd width
    ("p_3x3_c64_n200", 64, 200, 3, 3, 1, 12, 13, 2, 40, 2),       # two column tiles of 112, the second ragged
    ("p_5x5_c64", 64, 40, 5, 5, 2, 15, 13, 2, 50, 1),
    ("p_2x2_c64_p0", 64, 32, 2, 2, 0, 16, 16, 3, 50, 1),
    ("p_1x3_c64", 64, 32, 1, 3, 1, 9, 30, 2, 30, 1),              # pad applies to both axes: Ho = H + 2
    ("p_3x1_c64_p0", 64, 32, 3, 1, 0, 12, 10, 2, 30, 1),
    ("p_3x3_c320", 320, 72, 3, 3, 1, 12, 12, 1, 10, 1),           # five slices
    ("p_3x3_c64_p2", 64, 64, 3, 3, 2, 10, 11, 2, 20, 1),          # padding wider than the filter needs
    ("p_7x7_c64", 64, 16, 7, 7, 3, 12, 12, 2, 50, 2),
]


@pytest.mark.parametrize("case", CASES, ids=[c[0] for c in CASES])
@pytest.mark.parametrize("act", [asx.ACT_RELU, 0, asx.ACT_SILU], ids=["relu", "none", "silu"])
def test_window_patch_against_oracle(case, act):
    spec = spec_of(*case, seed=CASES.index(case))
    x, w, b, mask = make_problem(spec)
    layer = asx.MaskedConvLayer(spec.C_in, spec.C_out, spec.kh, spec.kw, 1, spec.pad)
    layer.set_mask(mask)
    layer.run(to_dev_bf16(x), to_dev_bf16(w), torch.from_numpy(b).cuda(), flags=act | asx.IMPL_WINDOW_PATCH)
    torch.cuda.synchronize()
    assert layer.last_run_form() == asx.FORM_WINDOW_PATCH, "this case is meant to take the window-patch form"
    layer.close()
    check_against_oracle(spec, x, w, b, mask, act | asx.IMPL_WINDOW_PATCH)
    check_against_oracle(spec, x, w, b, mask, act | asx.RECOMPACT | asx.IMPL_WINDOW_PATCH)
    check_against_oracle(spec, x, w, b, mask, act)                        # whichever form the library picks


@pytest.mark.parametrize("kept_rows", [0, 1, 127, 128, 129, 255, 256, 257, "all"])
def test_tile_boundaries(kept_rows):
    spec = wl.LayerSpec("edge64", 64, 32, 3, 3, 1, 1, 20, 20, 1, 0, 1, "relu", 4243)
    x, w, b, _ = make_problem(spec)
    mask = np.zeros(spec.P, np.uint8)
    if kept_rows == "all":
        mask[:] = 1
    else:
        mask[np.random.default_rng(kept_rows).permutation(spec.P)[:kept_rows]] = 1
    check_against_oracle(spec, x, w, b, mask, asx.ACT_RELU | asx.IMPL_WINDOW_PATCH)
    y, bits, form = run_form(spec, x, w, b, mask, asx.ACT_RELU | asx.IMPL_WINDOW_PATCH)
    assert form == asx.FORM_WINDOW_PATCH or kept_rows == 0      # with nothing kept there are no tiles to cut


def test_per_row_mask():
    spec = spec_of("p_rowmask", 64, 64, 3, 3, 1, 18, 21, 3, 40, 2, seed=50)
    x, w, b, mask = make_problem(spec, per_row=True)
    check_against_oracle(spec, x, w, None, mask, asx.IMPL_WINDOW_PATCH)
    assert run_form(spec, x, w, None, mask, asx.IMPL_WINDOW_PATCH)[2] == asx.FORM_WINDOW_PATCH


def test_tiny_integer_case_is_bit_exact_and_equals_row_gather():
    """Small integers: every product and sum is exact, so both forms must reproduce the oracle exactly."""
    spec = wl.LayerSpec("pint", 64, 16, 3, 3, 1, 1, 9, 8, 2, 50, 1, "smallint", 777)
    x, w, b, mask = make_problem(spec)
    ref = oracle.masked_conv(x, w, b, mask, 1, 1, True).reshape(spec.M, spec.C_out)
    ya, _, fa = run_form(spec, x, w, b, mask, asx.ACT_RELU | asx.IMPL_WINDOW_PATCH)
    yb, _, fb = run_form(spec, x, w, b, mask, asx.ACT_RELU | asx.IMPL_ROW_GATHER)
    assert fa == asx.FORM_WINDOW_PATCH and fb == asx.FORM_ROW_GATHER_TMA
    assert np.array_equal(ya, ref) and np.array_equal(yb, ref)


def test_more_tiles_than_the_row_coordinate_ring():
    """Enough kept rows that a block works through more tiles than the ring of decoded tiles holds
    (8 per block): the row-coordinate warp, the ring's reuse and the patch buffers' turn-taking all run.
    Checked on sampled rows (the oracle computes them one by one)."""
    spec = spec_of("p_many", 64, 64, 3, 3, 1, 56, 56, 64, 10, 4, seed=60)      # 180 000 kept rows: more than 9 tiles per block
    x, w, b, mask = make_problem(spec)
    rng = np.random.default_rng(5)
    sel = np.sort(rng.choice(spec.M, 1536, replace=False)).astype(np.int64)
    check_against_oracle(spec, x, w, b, mask, asx.ACT_RELU | asx.IMPL_WINDOW_PATCH, rows_sel=sel)
    y, bits, form = run_form(spec, x, w, b, mask, asx.ACT_RELU | asx.IMPL_WINDOW_PATCH)
    assert form == asx.FORM_WINDOW_PATCH
    # and the whole tensor equals the row-gather form to within two bf16 roundings of the same sums
    y2, bits2, form2 = run_form(spec, x, w, b, mask, asx.ACT_RELU | asx.IMPL_ROW_GATHER)
    assert form2 == asx.FORM_ROW_GATHER_TMA
    assert np.array_equal(bits == 0, bits2 == 0) or np.abs(y - y2).max() < 0.1
    assert np.abs(y - y2).max() <= 2 * max_abs_tol(spec.K, oracle.bf16_round(x), oracle.bf16_round(w))
    assert np.linalg.norm(y - y2) / np.linalg.norm(y2) <= REL_FROB_TOL


def test_residual_add():
    spec = spec_of("p_res", 64, 64, 3, 3, 1, 14, 14, 3, 50, 4, seed=70)
    x, w, b, mask = make_problem(spec)
    rng = np.random.default_rng(9)
    res = rng.standard_normal((spec.M, spec.C_out)).astype(np.float32)
    resd = to_dev_bf16(res.reshape(spec.Nb, spec.Ho, spec.Wo, spec.C_out))
    layer = asx.MaskedConvLayer(64, 64, 3, 3, 1, 1)
    layer.set_mask(mask)
    layer.set_residual(resd)
    out = layer.run(to_dev_bf16(x), to_dev_bf16(w), torch.from_numpy(b).cuda(), flags=asx.ACT_RELU | asx.IMPL_WINDOW_PATCH)
    torch.cuda.synchronize()
    assert layer.device_status() == 0 and layer.last_run_form() == asx.FORM_WINDOW_PATCH
    layer.close()
    pre = oracle.masked_conv(x, w, b, mask, 1, 1, False).reshape(spec.M, spec.C_out)
    fm = np.tile(mask, spec.Nb).astype(bool)
    ref = np.where(fm[:, None], np.maximum(pre + oracle.bf16_round(res).astype(np.float64), 0.0), 0.0)
    got = out.float().cpu().numpy().astype(np.float64).reshape(spec.M, spec.C_out)
    assert np.linalg.norm(got - ref) / np.linalg.norm(ref) <= REL_FROB_TOL
    assert np.abs(got - ref).max() <= max_abs_tol(spec.K, oracle.bf16_round(x), oracle.bf16_round(w)) + 2.0 ** -7 * np.abs(ref).max()


@pytest.mark.parametrize("pct", [75, 90, 97])
def test_sparse_masks_cut_into_short_tiles(pct):
    """At high sparsity the windows of 128 kept rows span more input rows than a patch buffer holds, so
    the host cuts shorter tiles (or the planner prefers the row gather): the result must not depend on it."""
    spec = spec_of("p_sparse", 64, 64, 3, 3, 1, 56, 56, 2, pct, 1, seed=80 + pct)
    x, w, b, mask = make_problem(spec)
    check_against_oracle(spec, x, w, b, mask, asx.ACT_RELU)
    check_against_oracle(spec, x, w, b, mask, asx.ACT_RELU | asx.IMPL_ROW_GATHER)
    check_against_oracle(spec, x, w, b, mask, asx.ACT_RELU | asx.IMPL_WINDOW_PATCH)
    assert run_form(spec, x, w, b, mask, asx.ACT_RELU | asx.IMPL_WINDOW_PATCH)[2] == asx.FORM_WINDOW_PATCH


def test_wide_rows_cut_into_short_tiles():
    """112 x 112 x 64: one padded input row is 15 KB, a patch buffer holds five of them, so most tiles are
    cut before they reach 128 rows."""
    spec = spec_of("p_wide", 64, 32, 3, 3, 1, 112, 112, 1, 30, 2, seed=95)
    x, w, b, mask = make_problem(spec)
    check_against_oracle(spec, x, w, b, mask, asx.ACT_RELU | asx.RECOMPACT | asx.IMPL_WINDOW_PATCH)


def test_device_masks_take_the_row_gather():
    """A mask given as a device pointer is not known to the host: no window-patch plan."""
    spec = spec_of("p_devmask", 64, 64, 3, 3, 1, 20, 20, 2, 30, 1, seed=90)
    x, w, b, mask = make_problem(spec)
    layer = asx.MaskedConvLayer(64, 64, 3, 3, 1, 1)
    layer.set_mask(torch.from_numpy(mask).cuda())
    out = layer.run(to_dev_bf16(x), to_dev_bf16(w), torch.from_numpy(b).cuda(), flags=asx.ACT_RELU | asx.RECOMPACT)
    torch.cuda.synchronize()
    assert layer.last_run_form() == asx.FORM_ROW_GATHER_TMA
    layer.close()
    ref = oracle.masked_conv(x, w, b, mask, 1, 1, True).reshape(spec.M, spec.C_out)
    got = out.float().cpu().numpy().astype(np.float64).reshape(spec.M, spec.C_out)
    assert np.linalg.norm(got - ref) / np.linalg.norm(ref) <= REL_FROB_TOL


def test_compact_output():
    """With ASX_OUT_COMPACT the kept rows go to y[n*P' + j] in kept order and nothing else is written."""
    spec = spec_of("p_compact", 64, 48, 3, 3, 1, 20, 23, 3, 40, 2, seed=96)
    x, w, b, mask = make_problem(spec)
    kept = int(mask.sum())
    layer = asx.MaskedConvLayer(64, 48, 3, 3, 1, 1)
    layer.set_mask(mask)
    y = torch.full((spec.Nb * kept + 4, spec.C_out), float("nan"), dtype=torch.bfloat16, device="cuda")
    st = int(torch.cuda.current_stream().cuda_stream)
    xd, wd, bd = to_dev_bf16(x), to_dev_bf16(w), torch.from_numpy(b).cuda()
    rc = layer.run_raw(xd.data_ptr(), spec.Nb, spec.H, spec.W, wd.data_ptr(), bd.data_ptr(), y.data_ptr(),
                       asx.ACT_RELU | asx.OUT_COMPACT | asx.IMPL_WINDOW_PATCH, st)
    assert rc == 0
    torch.cuda.synchronize()
    assert layer.device_status() == 0 and layer.last_run_form() == asx.FORM_WINDOW_PATCH
    layer.close()
    got = y.float().cpu().numpy().astype(np.float64)
    assert np.isnan(got[spec.Nb * kept:]).all(), "rows behind the compact output were written"
    rows = (np.arange(spec.Nb)[:, None] * spec.P + np.flatnonzero(mask)[None, :]).reshape(-1)
    ref = oracle.masked_conv(x, w, b, mask, 1, 1, True).reshape(spec.M, spec.C_out)[rows]
    got = got[:spec.Nb * kept]
    assert not np.isnan(got).any()
    assert np.linalg.norm(got - ref) / np.linalg.norm(ref) <= REL_FROB_TOL
    assert np.abs(got - ref).max() <= max_abs_tol(spec.K, oracle.bf16_round(x), oracle.bf16_round(w))


STEM_CASES = [
    # name, C_in, C_out, k, pad, H, W, Nb, pct, block: stride-2 first layers, which reach the window-patch form
    # through the 2x2-block staging (pixels are overlapping runs of four 32-byte blocks)
    ("stem_7x7_c3_64", 3, 64, 7, 3, 64, 64, 2, 50, 4),
    ("stem_7x7_c3_224", 3, 64, 7, 3, 224, 224, 1, 50, 4),         # the ResNet stem: four patch buffers, eight epilogue warps
    ("stem_7x7_c3_n32", 3, 32, 7, 3, 32, 48, 3, 30, 1),
    ("stem_7x7_c3_dense", 3, 64, 7, 3, 96, 160, 2, 0, 1),
    ("stem_7x7_c1_n16", 1, 16, 7, 3, 40, 40, 2, 75, 4),
    ("stem_7x7_c3_n128", 3, 128, 7, 3, 64, 64, 2, 50, 4),
    ("stem_7x7_c3_pad2", 3, 64, 7, 2, 64, 64, 2, 50, 4),
    ("stem_7x7_c4_w_odd_blocks", 4, 64, 7, 3, 36, 52, 2, 40, 2),  # staged rows padded up to whole 128-byte units
]


@pytest.mark.parametrize("case", STEM_CASES, ids=[c[0] for c in STEM_CASES])
@pytest.mark.parametrize("recompact", [False, True], ids=["stored_list", "recompact"])
def test_first_layer_in_the_window_patch_form(case, recompact):
    name, cin, cout, k, pad, H, W, Nb, pct, blk = case
    spec = wl.LayerSpec(name, cin, cout, k, k, 2, pad, H, W, Nb, pct, blk, "relu", wl.BASE_SEED + 7700 + len(name))
    x, w, b, mask = make_problem(spec, per_row=False)
    flags = asx.ACT_RELU | asx.IMPL_WINDOW_PATCH | (asx.RECOMPACT if recompact else 0)
    check_against_oracle(spec, x, w, b, mask, flags)
    _, bits_p, form_p = run_form(spec, x, w, b, mask, flags)
    assert form_p == asx.FORM_WINDOW_PATCH
    # and the row-gather form of the same staged problem gives the same bits (same products, same order of k-blocks)
    _, bits_g, form_g = run_form(spec, x, w, b, mask, (flags & ~asx.IMPL_WINDOW_PATCH) | asx.IMPL_ROW_GATHER)
    assert form_g != asx.FORM_WINDOW_PATCH
    fm = (mask if mask.size == spec.M else np.tile(mask, spec.Nb)).astype(bool)
    assert not np.any(bits_p[~fm]) and not np.any(bits_g[~fm])
    yp = torch.from_numpy(bits_p.view(np.int16)).view(torch.bfloat16).float().numpy()
    yg = torch.from_numpy(bits_g.view(np.int16)).view(torch.bfloat16).float().numpy()
    assert np.max(np.abs(yp - yg)) <= 2.0 ** -6 * max(1.0, float(np.max(np.abs(yg))))
