"""fp32 storage (ASX_F32; Appendix A, Algorithm 2 stores fp32) through the C ABI against the CPU oracle.

The tensor cores read fp32 operands as TF32 (the lower 13 mantissa bits are ignored), so the oracle
is the plain definition on `oracle.tf32_operand(x)`, `oracle.tf32_operand(w)` with fp32 storage;
products of two TF32 values are exact in fp32, which leaves the order and rounding of the fp32
accumulation as the only difference.  Tolerances: relative Frobenius error 2e-4 and max abs error
1e-3 * sqrt(K) * max|x| * max|w| (an fp32 sum of K <= 4608 terms: K * 2^-24 = 2.7e-4 of the sum of
magnitudes at worst, about sqrt(K) * 2^-24 typically); kept list and dropped-row zero bits exact."""
import itertools
import math

import numpy as np
import pytest
import torch

import oracle
import paper_2309_06626_b200 as asx
import workloads as wl
from gpu_util import full_row_mask, make_problem

pytestmark = pytest.mark.gpu

SMALL = list(wl.iter_small_cases())
IMPLS = [("naive", asx.IMPL_NAIVE), ("tcgen05", 0)]
REL_TOL_F32 = 2e-4


def run_f32(spec, x, w, b, mask, flags, prefill=0x7fc00001):
    """(y fp64 [M][N], raw uint32 bits, kept list) of one ASX_F32 call."""
    layer = asx.MaskedConvLayer(spec.C_in, spec.C_out, spec.kh, spec.kw, spec.stride, spec.pad)
    layer.set_mask(mask)
    xd = torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).cuda()
    wd = torch.from_numpy(np.ascontiguousarray(w, dtype=np.float32)).cuda()
    bd = None if b is None else torch.from_numpy(b).cuda()
    out = torch.empty((spec.Nb, spec.Ho, spec.Wo, spec.C_out), dtype=torch.float32, device="cuda")
    out.view(torch.int32).fill_(prefill)          # NaN canary
    layer.run(xd, wd, bd, out=out, flags=flags | asx.F32)
    torch.cuda.synchronize()
    status = layer.device_status()
    kept = layer.kept()
    layer.close()
    assert status == 0, f"device status {status}"
    bits = out.view(torch.int32).cpu().numpy().view(np.uint32).reshape(spec.M, spec.C_out)
    return out.cpu().numpy().astype(np.float64).reshape(spec.M, spec.C_out), bits, kept


def check_f32(spec, x, w, b, mask, flags, rows_sel=None):
    """x and w must already be TF32 values (see the module docstring)."""
    act = "silu" if flags & asx.ACT_SILU else bool(flags & asx.ACT_RELU)
    y, bits, kept = run_f32(spec, x, w, b, mask, flags)
    assert np.array_equal(kept, oracle.kept_list(mask)), "kept-row list differs"
    fm = full_row_mask(spec, mask).astype(bool)
    assert not np.any(bits[~fm]), "dropped rows are not all-zero bits"
    assert not np.any(np.isnan(y)), "an output element was never written"
    if rows_sel is None:
        ref = oracle.masked_conv(x, w, b, mask, spec.stride, spec.pad, act, storage="fp32").reshape(spec.M, spec.C_out)
        got = y
    else:
        ref = oracle.masked_conv_rows(x, w, b, mask, spec.stride, spec.pad, act, rows_sel, storage="fp32")
        got = y[rows_sel]
    diff = got - ref
    rel = float(np.linalg.norm(diff)) / max(float(np.linalg.norm(ref)), 1e-30)
    mx = float(np.max(np.abs(diff))) if diff.size else 0.0
    tol = 1e-3 * math.sqrt(spec.K) * float(np.max(np.abs(x))) * float(np.max(np.abs(w)))
    assert rel <= REL_TOL_F32, f"{spec.name}: relative Frobenius error {rel:.3e}"
    assert mx <= tol, f"{spec.name}: max abs error {mx:.3e} > {tol:.3e}"
    return rel, mx


def tf32_problem(spec, per_row=False):
    x, w, b, mask = make_problem(spec, per_row)
    return oracle.tf32_operand(x), oracle.tf32_operand(w), b, mask


@pytest.mark.parametrize("impl", IMPLS, ids=[i[0] for i in IMPLS])
@pytest.mark.parametrize("spec", SMALL, ids=[s.name for s in SMALL])
def test_small_cases_full_compare(spec, impl):
    x, w, b, mask = tf32_problem(spec)
    check_f32(spec, x, w, b, mask, asx.ACT_RELU | impl[1])


@pytest.mark.parametrize("spec", SMALL[:6], ids=[s.name for s in SMALL[:6]])
def test_silu_per_row_mask_and_recompact(spec):
    x, w, b, mask = tf32_problem(spec, per_row=True)
    check_f32(spec, x, w, None, mask, asx.ACT_SILU)
    x, w, b, mask = tf32_problem(spec)
    check_f32(spec, x, w, b, mask, asx.RECOMPACT)


@pytest.mark.parametrize("impl", IMPLS, ids=[i[0] for i in IMPLS])
@pytest.mark.parametrize("kept_rows", [0, 1, 127, 128, 129, 257, "all"])
def test_tile_boundaries(kept_rows, impl):
    spec = wl.LayerSpec("edge32", 16, 36, 3, 3, 1, 1, 20, 20, 1, 0, 1, "relu", 4343)
    x, w, b, _ = tf32_problem(spec)
    mask = np.zeros(spec.P, np.uint8)
    if kept_rows == "all":
        mask[:] = 1
    else:
        mask[np.random.default_rng(kept_rows).permutation(spec.P)[:kept_rows]] = 1
    check_f32(spec, x, w, b, mask, asx.ACT_RELU | impl[1])


@pytest.mark.parametrize("impl", IMPLS, ids=[i[0] for i in IMPLS])
@pytest.mark.parametrize("k,p", [(1, 0), (3, 1)])
def test_tiny_integer_cases_bit_exact(k, p, impl):
    """Small integers: every product and sum is exact, so the fp32 output equals the oracle exactly."""
    for C_in, C_out in itertools.product(range(1, 5), range(1, 5)):
        spec = wl.LayerSpec("tiny", C_in, C_out, k, k, 1, p, 5, 4, 2, 50, 1, "smallint", 2000 * k + 10 * C_in + C_out)
        x, w, b, mask = make_problem(spec)
        for relu in (0, asx.ACT_RELU):
            y, bits, kept = run_f32(spec, x, w, b, mask, relu | impl[1])
            ref = oracle.masked_conv(x, w, b, mask, 1, p, bool(relu), storage="fp32").reshape(spec.M, C_out)
            assert np.array_equal(y, ref), (C_in, C_out, relu)


def test_lower_mantissa_bits_of_the_operands_are_ignored():
    """The contraction reads only the TF32 part of an fp32 operand: full-precision inputs give the
    same bits as the inputs with their lower 13 mantissa bits cleared.  Note what this does and does
    not show: it compares the GPU with ITSELF (two runs of the same kernel), which is how the reading
    "the lower 13 bits are dropped towards zero" of the tensor core's TF32 conversion was confirmed;
    it is not a comparison with the oracle.  Parity with the oracle proper (the other tests of this
    file) runs on inputs that are already TF32 values, where no reading of the conversion enters."""
    for spec in (SMALL[0], SMALL[2], SMALL[6]):
        x, w, b, mask = make_problem(spec)
        y_full, bits_full, _ = run_f32(spec, x, w, b, mask, asx.ACT_RELU)
        y_t, bits_t, _ = run_f32(spec, oracle.tf32_operand(x), oracle.tf32_operand(w), b, mask, asx.ACT_RELU)
        assert np.array_equal(bits_full, bits_t), spec.name


def test_unrounded_inputs_stay_within_the_tf32_error_of_the_fp32_definition():
    """Against the definition on the unrounded fp32 inputs the error is that of dropping 13 mantissa
    bits per operand: each product loses less than 2 * 2^-10 of its magnitude."""
    spec = SMALL[0]
    x, w, b, mask = make_problem(spec)
    y, _, _ = run_f32(spec, x, w, b, mask, 0)
    ref = oracle.masked_conv(x, w, b, mask, spec.stride, spec.pad, False, storage="fp32").reshape(spec.M, spec.C_out)
    bound = oracle.masked_conv(np.abs(x), np.abs(w), None, mask, spec.stride, spec.pad, False,
                               storage="fp32").reshape(spec.M, spec.C_out) * 2.0 ** -9
    assert np.all(np.abs(y - ref) <= bound + 1e-6)


def test_large_layer_sampled_rows_and_both_gpu_implementations():
    """A ResNet-18 layer1 shape at batch 8 (M = 25088, 98 kept tiles at 50 %): sampled rows against the
    oracle, every element against the one-thread-per-output kernel."""
    spec = wl.LayerSpec("layer1_f32", 64, 64, 3, 3, 1, 1, 56, 56, 8, 50, 4, "relu", 777)
    x, w, b, mask = tf32_problem(spec)
    rng = np.random.default_rng(5)
    sel = np.sort(rng.choice(spec.M, 600, replace=False))
    check_f32(spec, x, w, b, mask, asx.ACT_RELU, rows_sel=sel)
    y_fast, _, _ = run_f32(spec, x, w, b, mask, asx.ACT_RELU)
    y_naive, _, _ = run_f32(spec, x, w, b, mask, asx.ACT_RELU | asx.IMPL_NAIVE)
    assert np.linalg.norm(y_fast - y_naive) <= REL_TOL_F32 * np.linalg.norm(y_naive)


def test_unsupported_combinations_are_refused():
    spec = SMALL[0]
    x, w, b, mask = tf32_problem(spec)
    layer = asx.MaskedConvLayer(spec.C_in, spec.C_out, spec.kh, spec.kw, spec.stride, spec.pad)
    layer.set_mask(mask)
    xd, wd = torch.from_numpy(x).cuda(), torch.from_numpy(w).cuda()
    out = torch.empty((spec.Nb, spec.Ho, spec.Wo, spec.C_out), dtype=torch.float32, device="cuda")
    for extra in (asx.OUT_COMPACT, asx.IN_COMPACT):
        rc = layer.run_raw(xd.data_ptr(), spec.Nb, spec.H, spec.W, wd.data_ptr(), 0, out.data_ptr(), asx.F32 | extra, 0)
        assert rc == 2      # ASX_ERR_UNSUPPORTED
    layer.close()


def test_resnet18_batch64_stack_full_size_sampled_rows():
    """Configuration 3 in fp32 storage, launched as `bench.py --dtype f32` launches it (ASX_RECOMPACT,
    ReLU): kept list and zero rows in full, 768 sampled rows per layer against the oracle."""
    rng = np.random.default_rng(33)
    for spec in wl.config(3):
        x, w, b, mask = tf32_problem(spec)
        xd, wd, bd = torch.from_numpy(x).cuda(), torch.from_numpy(w).cuda(), torch.from_numpy(b).cuda()
        y = torch.empty((spec.Nb, spec.Ho, spec.Wo, spec.C_out), dtype=torch.float32, device="cuda")
        y.view(torch.int32).fill_(0x7fc00001)
        layer = asx.MaskedConvLayer(spec.C_in, spec.C_out, spec.kh, spec.kw, spec.stride, spec.pad)
        layer.set_mask(mask)
        layer.run(xd, wd, bd, out=y, flags=asx.ACT_RELU | asx.RECOMPACT | asx.F32)
        torch.cuda.synchronize()
        assert layer.device_status() == 0
        kept = layer.kept()
        layer.close()
        assert np.array_equal(kept, oracle.kept_list(mask)), spec.name
        y2 = y.view(spec.Nb, spec.P, spec.C_out)
        md = torch.from_numpy(mask.astype(bool)).cuda()
        assert not bool(y2[:, ~md, :].view(torch.int32).any()), f"{spec.name}: dropped rows are not all-zero bits"
        assert not bool(torch.isnan(y2[:, md, :]).any()), f"{spec.name}: a kept element was never written"
        kept_rows = np.nonzero(np.tile(mask, spec.Nb))[0]
        sel = rng.choice(kept_rows, size=min(768, kept_rows.size), replace=False)
        sel = np.unique(np.concatenate([sel, kept_rows[:2], kept_rows[-2:], rng.integers(0, spec.M, 16)])).astype(np.int64)
        ref = oracle.masked_conv_rows(x, w, b, mask, spec.stride, spec.pad, True, sel, storage="fp32")
        got = y.view(spec.M, spec.C_out)[torch.from_numpy(sel).cuda()].cpu().numpy().astype(np.float64)
        diff = got - ref
        rel = float(np.linalg.norm(diff)) / max(float(np.linalg.norm(ref)), 1e-30)
        tol = 1e-3 * math.sqrt(spec.K) * float(np.abs(x).max()) * float(np.abs(w).max())
        assert rel <= REL_TOL_F32, f"{spec.name}: relative Frobenius error {rel:.3e}"
        assert float(np.abs(diff).max()) <= tol, f"{spec.name}: max abs error {np.abs(diff).max():.3e} > {tol:.3e}"
        del xd, wd, y, y2
