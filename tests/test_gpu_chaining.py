"""Layer chaining without re-densifying (compact outputs and inputs) against the oracle.

The oracle has no notion of compact tensors: a compact output must equal the kept rows of the
oracle's dense output, and a convolution fed with a compact input must equal the oracle's
convolution of the dense tensor that has zeros at the dropped positions."""
import numpy as np
import pytest
import torch

import oracle
import paper_2309_06626_b200 as asx
import workloads as wl
from gpu_util import to_dev_bf16

pytestmark = pytest.mark.gpu


def _run_raw(layer, x_dev, Nb, H, W, w_dev, b_dev, y_dev, flags):
    st = int(torch.cuda.current_stream().cuda_stream)
    rc = layer.run_raw(x_dev.data_ptr(), Nb, H, W, w_dev.data_ptr(), b_dev.data_ptr() if b_dev is not None else 0,
                       y_dev.data_ptr(), flags, st)
    assert rc == 0, f"asx_run returned {rc}"
    torch.cuda.synchronize()
    assert layer.device_status() == 0


def _rel(a, b):
    return np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-30)


def _close(got, ref, K, x_in, w, extra_abs=0.0):
    """The bar of the plain layers: relative Frobenius error <= 5e-3 and, element by element,
    |got - ref| <= 1e-2 * sqrt(K) * max|x| * max|w| on the bf16-rounded operands of THIS layer
    (plus extra_abs where something else is rounded on the way, e.g. an added residual)."""
    assert got.shape == ref.shape
    assert _rel(got, ref) <= 5e-3, f"relative Frobenius error {_rel(got, ref):.3e}"
    tol = 1e-2 * np.sqrt(K) * float(np.abs(oracle.bf16_round(np.asarray(x_in, np.float32))).max()) * \
        float(np.abs(oracle.bf16_round(np.asarray(w, np.float32))).max()) + extra_abs
    worst = float(np.abs(got - ref).max()) if got.size else 0.0
    assert worst <= tol, f"max abs error {worst:.3e} > {tol:.3e}"


CASES = [
    # C_in, C_mid, C_out, k1, s1, p1, k2, s2, p2, H, W, Nb, sparsity1 %, sparsity2 %, block
    (64, 64, 48, 3, 1, 1, 3, 1, 1, 20, 23, 2, 40, 30, 1),        # TMA gather on both layers
    (16, 32, 24, 3, 2, 1, 3, 1, 1, 29, 31, 2, 50, 50, 4),        # cp.async gather on the second layer
    (64, 128, 256, 1, 1, 0, 3, 2, 1, 14, 14, 3, 25, 60, 2),      # 1x1 then a strided 3x3
    (128, 512, 64, 3, 1, 1, 3, 1, 1, 7, 7, 4, 50, 50, 1),        # few rows, long reduction: shared k-blocks on layer 2
]


@pytest.mark.parametrize("case", CASES, ids=[f"c{i}" for i in range(len(CASES))])
def test_two_layers_chained_compact(case):
    cin, cmid, cout, k1, s1, p1, k2, s2, p2, H, W, Nb, sp1, sp2, blk = case
    l1 = wl.LayerSpec("chain1", cin, cmid, k1, k1, s1, p1, H, W, Nb, sp1, blk, "relu", wl.BASE_SEED + 301)
    l2 = wl.LayerSpec("chain2", cmid, cout, k2, k2, s2, p2, l1.Ho, l1.Wo, Nb, sp2, blk, "relu", wl.BASE_SEED + 302)
    x, w1, b1, m1 = wl.make_x(l1), wl.make_w(l1), wl.make_b(l1), wl.make_layer_mask(l1)
    w2, b2, m2 = wl.make_w(l2), wl.make_b(l2), wl.make_layer_mask(l2)
    # oracle: two dense layers; the intermediate is stored as bf16 by the GPU path
    y1_ref = oracle.masked_conv(x, w1, b1, m1, s1, p1, True)
    y1_bf = oracle.bf16_round(y1_ref.astype(np.float32)).astype(np.float64)
    y2_ref = oracle.masked_conv(y1_bf.astype(np.float32), w2, b2, m2, s2, p2, True)

    kept1, kept2 = int(m1.sum()), int(m2.sum())
    A = asx.MaskedConvLayer(cin, cmid, k1, k1, s1, p1)
    B = asx.MaskedConvLayer(cmid, cout, k2, k2, s2, p2)
    A.set_mask(m1)
    B.set_mask(m2)
    B.set_input_mask(m1)
    xd, w1d, w2d = to_dev_bf16(x), to_dev_bf16(w1), to_dev_bf16(w2)
    b1d, b2d = torch.from_numpy(b1).cuda(), torch.from_numpy(b2).cuda()
    y1c = torch.full((Nb * kept1, cmid), float("nan"), dtype=torch.bfloat16, device="cuda")
    y2c = torch.full((Nb * kept2, cout), float("nan"), dtype=torch.bfloat16, device="cuda")
    _run_raw(A, xd, Nb, H, W, w1d, b1d, y1c, asx.ACT_RELU | asx.RECOMPACT | asx.OUT_COMPACT)
    _run_raw(B, y1c, Nb, l1.Ho, l1.Wo, w2d, b2d, y2c, asx.ACT_RELU | asx.RECOMPACT | asx.IN_COMPACT | asx.OUT_COMPACT)
    A.close(); B.close()

    rows1 = (np.arange(Nb)[:, None] * l1.P + np.flatnonzero(m1)[None, :]).reshape(-1)
    rows2 = (np.arange(Nb)[:, None] * l2.P + np.flatnonzero(m2)[None, :]).reshape(-1)
    got1 = y1c.float().cpu().numpy().astype(np.float64)
    got2 = y2c.float().cpu().numpy().astype(np.float64)
    assert not np.isnan(got1).any() and not np.isnan(got2).any(), "a compact row was never written"
    _close(got1, y1_ref.reshape(l1.M, cmid)[rows1], l1.K, x, w1)
    _close(got2, y2_ref.reshape(l2.M, cout)[rows2], l2.K, y1_bf, w2)


def test_compact_input_into_dense_output_and_errors():
    spec = wl.LayerSpec("cin_only", 64, 64, 3, 3, 1, 1, 17, 19, 2, 30, 1, "relu", wl.BASE_SEED + 303)
    x, w, b, m = wl.make_x(spec), wl.make_w(spec), wl.make_b(spec), wl.make_layer_mask(spec)
    rng = np.random.default_rng(4)
    m_in = (rng.random(spec.H * spec.W) < 0.6).astype(np.uint8)
    x_masked = x * np.tile(m_in, spec.Nb).reshape(spec.Nb, spec.H, spec.W, 1)
    ref = oracle.masked_conv(x_masked, w, b, m, spec.stride, spec.pad, True)
    rows_in = (np.arange(spec.Nb)[:, None] * spec.H * spec.W + np.flatnonzero(m_in)[None, :]).reshape(-1)
    xc = to_dev_bf16(x.reshape(-1, spec.C_in)[rows_in])
    layer = asx.MaskedConvLayer(spec.C_in, spec.C_out, 3, 3, 1, 1)
    layer.set_mask(m)
    wd, bd = to_dev_bf16(w), torch.from_numpy(b).cuda()
    y = torch.full((spec.Nb, spec.Ho, spec.Wo, spec.C_out), float("nan"), dtype=torch.bfloat16, device="cuda")
    st = int(torch.cuda.current_stream().cuda_stream)
    args = (xc.data_ptr(), spec.Nb, spec.H, spec.W, wd.data_ptr(), bd.data_ptr(), y.data_ptr())
    assert layer.run_raw(*args, asx.ACT_RELU | asx.IN_COMPACT, st) == 3                       # no input mask yet
    layer.set_input_mask(torch.from_numpy(m_in).cuda())                                       # from device memory
    assert layer.run_raw(*args, asx.ACT_RELU | asx.IN_COMPACT | asx.IMPL_NAIVE, st) == 1      # not with the reference kernel
    assert layer.run_raw(xc.data_ptr(), spec.Nb, spec.H + 1, spec.W, wd.data_ptr(), bd.data_ptr(), y.data_ptr(),
                         asx.ACT_RELU | asx.IN_COMPACT, st) in (4,)                            # mask length != H*W
    assert layer.run_raw(*args, asx.ACT_RELU | asx.IN_COMPACT, st) == 0
    torch.cuda.synchronize()
    assert layer.device_status() == 0
    layer.close()
    got = y.float().cpu().numpy().astype(np.float64).reshape(ref.shape)
    assert not np.isnan(got).any()
    _close(got, ref, spec.K, x, w)
    assert not got.reshape(spec.M, -1)[np.tile(m, spec.Nb) == 0].any()


def test_compact_output_next_to_its_input_in_memory():
    """A compact output is smaller than the dense one: an input that starts right behind it does not
    overlap it (the overlap check once used the dense extent and refused such calls)."""
    spec = wl.LayerSpec("adjacent", 8, 16, 3, 3, 1, 1, 12, 10, 1, 90, 1, "relu", wl.BASE_SEED + 304)
    x, w, b, m = wl.make_x(spec), wl.make_w(spec), wl.make_b(spec), wl.make_layer_mask(spec)
    kept = int(m.sum())
    y_elems = ((kept * spec.C_out + 63) // 64) * 64                       # keeps x 16-byte aligned
    arena = torch.zeros(y_elems + x.size, dtype=torch.bfloat16, device="cuda")
    yc = arena[:kept * spec.C_out].view(kept, spec.C_out)
    xd = arena[y_elems:].view(x.shape)
    xd.copy_(to_dev_bf16(x))
    layer = asx.MaskedConvLayer(spec.C_in, spec.C_out, 3, 3, 1, 1)
    layer.set_mask(m)
    _run_raw(layer, xd, 1, spec.H, spec.W, to_dev_bf16(w), torch.from_numpy(b).cuda(), yc, asx.ACT_RELU | asx.OUT_COMPACT)
    layer.close()
    ref = oracle.masked_conv(x, w, b, m, 1, 1, True).reshape(spec.M, spec.C_out)[np.flatnonzero(m)]
    _close(yc.float().cpu().numpy().astype(np.float64), ref, spec.K, x, w)


RES_CASES = [
    # C_in, C_out, k, s, p, H, W, Nb, sparsity %, block, compact output
    (64, 64, 3, 1, 1, 20, 23, 2, 40, 1, False),      # TMA gather, dense output
    (16, 40, 3, 2, 1, 29, 31, 2, 50, 4, False),      # cp.async gather, 48-wide tile with a 16-column tail
    (64, 64, 3, 1, 1, 14, 14, 3, 30, 2, True),       # compact output: the residual is compact too
    (512, 64, 3, 1, 1, 7, 7, 4, 50, 1, False),       # few rows, long reduction: the add happens after the k shares are summed
    (5, 7, 3, 1, 1, 12, 11, 2, 30, 1, False),        # odd channel counts: element-wise loads and stores
]


@pytest.mark.parametrize("act", ["relu", "silu"])
@pytest.mark.parametrize("case", RES_CASES, ids=[f"r{i}" for i in range(len(RES_CASES))])
def test_residual_add_before_the_activation(case, act):
    """y = mask ? act(conv + bias + residual) : 0, the shortcut of a residual block fused into the
    epilogue.  The oracle gives conv + bias without activation; the rest is written out here."""
    cin, cout, k, s, p, H, W, Nb, sp, blk, compact = case
    act_flag = asx.ACT_RELU if act == "relu" else asx.ACT_SILU
    f = (lambda z: np.maximum(z, 0.0)) if act == "relu" else (lambda z: z / (1.0 + np.exp(-z)))
    spec = wl.LayerSpec("res", cin, cout, k, k, s, p, H, W, Nb, sp, blk, "relu", wl.BASE_SEED + 310)
    x, w, b, m = wl.make_x(spec), wl.make_w(spec), wl.make_b(spec), wl.make_layer_mask(spec)
    rng = np.random.default_rng(12)
    res = oracle.bf16_round(rng.standard_normal((spec.M, cout)).astype(np.float32)).astype(np.float64)
    fm = np.tile(m, Nb).astype(bool)
    lin = oracle.masked_conv(x, w, b, m, s, p, False).reshape(spec.M, cout)
    ref = np.where(fm[:, None], f(lin + res), 0.0)
    rows = np.flatnonzero(fm)
    layer = asx.MaskedConvLayer(cin, cout, k, k, s, p)
    layer.set_mask(m)
    xd, wd, bd = to_dev_bf16(x), to_dev_bf16(w), torch.from_numpy(b).cuda()
    if compact:
        rd = to_dev_bf16(res[rows].astype(np.float32))
        y = torch.full((rows.size, cout), float("nan"), dtype=torch.bfloat16, device="cuda")
        flags = act_flag | asx.RECOMPACT | asx.OUT_COMPACT
    else:
        rd = to_dev_bf16(res.astype(np.float32))
        y = torch.full((spec.M, cout), float("nan"), dtype=torch.bfloat16, device="cuda")
        flags = act_flag | asx.RECOMPACT
    layer.set_residual(rd)
    st = int(torch.cuda.current_stream().cuda_stream)
    assert layer.run_raw(xd.data_ptr(), Nb, H, W, wd.data_ptr(), bd.data_ptr(), y.data_ptr(), flags | asx.IMPL_NAIVE, st) == 1
    _run_raw(layer, xd, Nb, H, W, wd, bd, y, flags)
    got = y.float().cpu().numpy().astype(np.float64)
    assert not np.isnan(got).any()
    want = ref[rows] if compact else ref
    # the sum with the residual is rounded to bf16 once more: half an ulp of the largest result
    _close(got, want, spec.K, x, w, extra_abs=2.0 ** -8 * float(np.abs(want).max()))
    if not compact:
        assert not got[~fm].any()
    # switching the residual off gives the plain layer again
    layer.set_residual(None)
    _run_raw(layer, xd, Nb, H, W, wd, bd, y, flags)
    layer.close()
    plain = np.where(fm[:, None], f(lin), 0.0)
    _close(y.float().cpu().numpy().astype(np.float64), plain[rows] if compact else plain, spec.K, x, w)
