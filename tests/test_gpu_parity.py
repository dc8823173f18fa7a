"""Parity of the CUDA path against the CPU oracle, through the C ABI.

Kept-row list and dropped-row zeros bit-exact; kept values within a relative Frobenius
error of 5e-3 and a max abs error of 1e-2*sqrt(K)*max|x|*max|w| (bf16-rounded inputs)."""
import itertools

import numpy as np
import pytest
import torch

import oracle
import paper_2309_06626_b200 as asx
import workloads as wl
from gpu_util import check_against_oracle, make_problem, run_library, to_dev_bf16
from philox_ref import random_block_mask

pytestmark = pytest.mark.gpu

SMALL = list(wl.iter_small_cases())
IMPLS = [("naive", asx.IMPL_NAIVE), ("tcgen05", 0), ("row_gather", asx.IMPL_ROW_GATHER)]


@pytest.mark.parametrize("impl", IMPLS, ids=[i[0] for i in IMPLS])
@pytest.mark.parametrize("spec", SMALL, ids=[s.name for s in SMALL])
def test_small_cases_full_compare(spec, impl):
    x, w, b, mask = make_problem(spec)
    check_against_oracle(spec, x, w, b, mask, asx.ACT_RELU | impl[1])


@pytest.mark.parametrize("impl", IMPLS, ids=[i[0] for i in IMPLS])
def test_per_row_mask_and_no_relu_no_bias(impl):
    for spec in SMALL[:4]:
        x, w, b, mask = make_problem(spec, per_row=True)
        check_against_oracle(spec, x, w, None, mask, impl[1])


@pytest.mark.parametrize("impl", IMPLS, ids=[i[0] for i in IMPLS])
@pytest.mark.parametrize("kept_rows", [0, 1, 127, 128, 129, 255, 256, 257, "all"])
def test_tile_boundaries(kept_rows, impl):
    """Kept-row counts around the 128-row tile size, all kept and all dropped."""
    spec = wl.LayerSpec("edge", 16, 32, 3, 3, 1, 1, 20, 20, 1, 0, 1, "relu", 4242)
    x, w, b, _ = make_problem(spec)
    mask = np.zeros(spec.P, np.uint8)
    if kept_rows == "all":
        mask[:] = 1
    else:
        mask[np.random.default_rng(kept_rows).permutation(spec.P)[:kept_rows]] = 1
    check_against_oracle(spec, x, w, b, mask, asx.ACT_RELU | impl[1])


@pytest.mark.parametrize("impl", IMPLS, ids=[i[0] for i in IMPLS])
@pytest.mark.parametrize("k,p", [(1, 0), (3, 1)])
def test_tiny_integer_cases_bit_exact(k, p, impl):
    """1x1 and 3x3, C_in, C_out in 1..4, small integers: every product and sum is exact in
    bf16/fp32, so the GPU must reproduce the oracle exactly."""
    for C_in, C_out in itertools.product(range(1, 5), range(1, 5)):
        spec = wl.LayerSpec("tiny", C_in, C_out, k, k, 1, p, 5, 4, 2, 50, 1, "smallint",
                            1000 * k + 10 * C_in + C_out)
        x, w, b, mask = make_problem(spec)
        for relu in (0, asx.ACT_RELU):
            y, bits, kept = run_library(spec, x, w, b, mask, relu | impl[1], prefill=0x7fc1)
            ref = oracle.masked_conv(x, w, b, mask, 1, p, bool(relu)).reshape(spec.M, C_out)
            assert np.array_equal(y, ref), (C_in, C_out, relu)
            assert np.array_equal(kept, oracle.kept_list(mask))


@pytest.mark.parametrize("impl", IMPLS, ids=[i[0] for i in IMPLS])
@pytest.mark.parametrize("spec", SMALL, ids=[s.name for s in SMALL])
def test_small_cases_silu(spec, impl):
    """The SiLU epilogue (own kernel instances) on every small case, split-K layers included."""
    x, w, b, mask = make_problem(spec)
    check_against_oracle(spec, x, w, b, mask, asx.ACT_SILU | impl[1])


def test_silu_values_on_exact_preactivations():
    """1x1, weight 1, inputs exact in bf16: the pre-activation is x + bias exactly, so the output
    is bf16(silu(x + bias)) up to the error of the fast exponential (well inside half a bf16 ulp
    except at rounding ties, hence one ulp allowed)."""
    vals = np.array([0.0, 0.5, 1.0, -2.0, 3.5, -8.0, 16.0, -0.25, -40.0, 40.0, -100.0, 6.0], dtype=np.float32)
    spec = wl.LayerSpec("silu1x1", 8, 8, 1, 1, 1, 0, 3, 4, 1, 0, 1, "relu", 1)
    x = np.zeros((1, 3, 4, 8), np.float32)
    x[0, :, :, 0] = vals.reshape(3, 4)
    w = np.zeros((8, 1, 1, 8), np.float32)
    w[:, 0, 0, 0] = 1.0
    b = np.full(8, 0.5, np.float32)
    mask = np.ones(12, np.uint8)
    mask[5] = 0
    y, bits, kept = run_library(spec, x, w, b, mask, asx.ACT_SILU, prefill=0x7fc1)
    ref = oracle.masked_conv(x, w, b, mask, 1, 0, "silu").reshape(12, 8)
    assert not np.any(bits[5])
    ulp = np.maximum(np.abs(ref), 2.0 ** -126) * 2.0 ** -7
    assert np.all(np.abs(y - ref) <= ulp), np.abs(y - ref).max()
    assert np.all(np.isfinite(y))


def test_relu_and_silu_together_are_rejected():
    layer = asx.MaskedConvLayer(8, 8, 1, 1, 1, 0)
    layer.set_mask(np.ones(4, np.uint8))
    x = torch.zeros((1, 2, 2, 8), dtype=torch.bfloat16, device="cuda")
    w = torch.zeros((8, 1, 1, 8), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(asx.AsxError):
        layer.run(x, w, None, flags=asx.ACT_RELU | asx.ACT_SILU)
    layer.close()


def test_all_dropped_ignores_nan_input():
    spec = wl.LayerSpec("nan", 8, 16, 3, 3, 1, 1, 9, 9, 2, 100, 1, "relu", 7)
    x, w, b, _ = make_problem(spec)
    x[:] = np.nan
    y, bits, kept = run_library(spec, x, w, b, np.zeros(spec.P, np.uint8), asx.ACT_RELU, prefill=0x7fc1)
    assert kept.size == 0 and not np.any(bits)


def test_generated_mask_matches_documented_rule():
    layer = asx.MaskedConvLayer(8, 8, 3, 3, 1, 1)
    for rows, s, blk, seed in [(3136, 0.5, 1, 1), (784, 0.3, 4, 2**40 + 5), (1000, 0.9, 16, 3), (49, 0.0, 2, 4)]:
        layer.set_mask_random(rows, s, blk, seed)
        got = layer.mask(rows)
        assert np.array_equal(got, random_block_mask(rows, s, blk, seed))
        assert np.array_equal(layer.kept(), oracle.kept_list(got))
    layer.close()


def test_recompact_flag_and_mask_change():
    spec = SMALL[0]
    x, w, b, mask = make_problem(spec)
    layer = asx.MaskedConvLayer(spec.C_in, spec.C_out, 3, 3, spec.stride, spec.pad)
    from gpu_util import to_dev_bf16
    xd, wd, bd = to_dev_bf16(x), to_dev_bf16(w), torch.from_numpy(b).cuda()
    layer.set_mask(mask)
    y1 = layer.run(xd, wd, bd, flags=asx.ACT_RELU | asx.RECOMPACT)
    y2 = layer.run(xd, wd, bd, flags=asx.ACT_RELU)
    assert torch.equal(y1.view(torch.int16), y2.view(torch.int16))
    mask2 = 1 - mask
    layer.set_mask(torch.from_numpy(mask2).cuda())           # device-side mask
    y3 = layer.run(xd, wd, bd, flags=asx.ACT_RELU)
    torch.cuda.synchronize()
    ref = oracle.masked_conv(x, w, b, mask2, spec.stride, spec.pad, True)
    assert np.array_equal(layer.kept(), oracle.kept_list(mask2))
    got = y3.float().cpu().numpy().astype(np.float64)
    assert np.linalg.norm(got - ref) / np.linalg.norm(ref) < 5e-3
    layer.close()


def test_run_argument_errors_on_device():
    layer = asx.MaskedConvLayer(64, 64, 3, 3, 1, 1)
    layer.set_mask(np.ones(100, np.uint8))
    x = torch.zeros((1, 12, 12, 64), dtype=torch.bfloat16, device="cuda")
    w = torch.zeros((64, 3, 3, 64), dtype=torch.bfloat16, device="cuda")
    y = torch.zeros((1, 12, 12, 64), dtype=torch.bfloat16, device="cuda")
    st = int(torch.cuda.current_stream().cuda_stream)
    assert layer.run_raw(x.data_ptr(), 1, 12, 12, w.data_ptr(), 0, y.data_ptr(), 0, st) == 4      # 144 != 100
    assert layer.run_raw(x.data_ptr() + 2, 1, 10, 10, w.data_ptr(), 0, y.data_ptr(), 0, st) == 5   # alignment
    assert layer.run_raw(x.data_ptr(), 1, 10, 10, w.data_ptr(), 0, x.data_ptr(), 0, st) == 1       # y aliases x
    assert layer.run_raw(x.data_ptr(), 1, 10, 10, w.data_ptr(), 0, y.data_ptr(), 0, st) == 0
    torch.cuda.synchronize()
    assert layer.device_status() == 0
    layer.close()


def test_config1_full():
    spec = wl.config(1)[0]
    x, w, b, mask = make_problem(spec)
    assert int(mask.sum()) == 1568
    check_against_oracle(spec, x, w, b, mask, asx.ACT_RELU)


def test_shared_k_blocks_give_the_same_bits_every_run():
    """Few kept rows and a long reduction: the k-blocks of a tile are shared between thread blocks
    that exchange fp32 partial tiles.  The partials are added in a fixed order, so repeated runs
    (and a run on the same layer handle after the workspace was used) agree bit for bit."""
    spec = [s for s in SMALL if s.name == "t_3x3_c512"][0]
    x, w, b, mask = make_problem(spec)
    layer = asx.MaskedConvLayer(spec.C_in, spec.C_out, spec.kh, spec.kw, spec.stride, spec.pad)
    layer.set_mask(mask)
    xd, wd, bd = to_dev_bf16(x), to_dev_bf16(w), torch.from_numpy(b).cuda()
    runs = []
    for flags in (asx.ACT_RELU, asx.ACT_RELU | asx.RECOMPACT, asx.ACT_RELU):
        y = layer.run(xd, wd, bd, flags=flags)
        torch.cuda.synchronize()
        runs.append(y.view(torch.int16).cpu().numpy().copy())
    assert layer.device_status() == 0
    layer.close()
    assert np.array_equal(runs[0], runs[1]) and np.array_equal(runs[0], runs[2])
    ref = oracle.masked_conv(x, w, b, mask, spec.stride, spec.pad, True)
    got = torch.from_numpy(runs[0]).view(torch.bfloat16).float().numpy().astype(np.float64).reshape(ref.shape)
    assert np.linalg.norm(got - ref) / np.linalg.norm(ref) < 5e-3


def test_masks_from_one_score_across_resolutions():
    """Algorithm 1's getMask through the layer API: three layers at different resolutions take their
    masks from one input-resolution score; the stored masks equal the oracle's bit for bit and the
    convolutions under them match the oracle."""
    rng = np.random.default_rng(2309)
    score = rng.random((32, 48)).astype(np.float32)
    for (cin, cout, k, s, p, H, W, sparsity) in [(3, 16, 3, 2, 1, 32, 48, 0.3), (16, 32, 3, 1, 1, 16, 24, 0.5),
                                                 (64, 64, 1, 2, 0, 16, 24, 0.25)]:
        spec = wl.LayerSpec("scores", cin, cout, k, k, s, p, H, W, 2, int(sparsity * 100), 1, "relu", wl.BASE_SEED + 77)
        x, w, b = wl.make_x(spec), wl.make_w(spec), wl.make_b(spec)
        want = oracle.get_mask(score, spec.Ho, spec.Wo, sparsity)
        layer = asx.MaskedConvLayer(cin, cout, k, k, s, p)
        layer.set_mask_from_scores(score, spec.Ho, spec.Wo, sparsity)
        assert np.array_equal(layer.mask(spec.P), want)
        y = layer.run(to_dev_bf16(x), to_dev_bf16(w), torch.from_numpy(b).cuda(), flags=asx.ACT_RELU | asx.RECOMPACT)
        torch.cuda.synchronize()
        assert layer.device_status() == 0
        assert np.array_equal(layer.kept(), oracle.kept_list(want))
        layer.close()
        ref = oracle.masked_conv(x, w, b, want, s, p, True)
        got = y.float().cpu().numpy().astype(np.float64).reshape(ref.shape)
        assert np.linalg.norm(got - ref) / np.linalg.norm(ref) < 5e-3
        dropped = np.tile(want, spec.Nb) == 0
        assert not got.reshape(spec.M, cout)[dropped].any()
