"""Parity at the benchmark's full sizes (configurations 2-5), in the launch configuration bench.py
times: mask compaction + fused kernel through the C ABI.  The kept-row list and the zero rows are
checked in full and bit-exact; kept values are checked on sampled rows that the CPU oracle
evaluates one by one (relative Frobenius error <= 5e-3, max abs error <= 1e-2*sqrt(K)*max|x|*max|w|).
"""
import math

import numpy as np
import pytest
import torch

import oracle
import paper_2309_06626_b200 as asx
import workloads as wl

pytestmark = pytest.mark.gpu

N_SAMPLED_ROWS = 1536


def _check_layer(spec, rng):
    x, w, b, mask = wl.make_x(spec), wl.make_w(spec), wl.make_b(spec), wl.make_layer_mask(spec)
    xd = torch.from_numpy(x).to(torch.bfloat16).cuda()
    wd = torch.from_numpy(w).to(torch.bfloat16).cuda()
    bd = torch.from_numpy(b).cuda()
    y = torch.empty((spec.Nb, spec.Ho, spec.Wo, spec.C_out), dtype=torch.bfloat16, device="cuda")
    y.view(torch.int16).fill_(0x7fc1)                                   # NaN canary: every element must be written
    layer = asx.MaskedConvLayer(spec.C_in, spec.C_out, spec.kh, spec.kw, spec.stride, spec.pad)
    layer.set_mask(mask)
    layer.run(xd, wd, bd, out=y, flags=asx.ACT_RELU | asx.RECOMPACT)
    torch.cuda.synchronize()
    assert layer.device_status() == 0
    kept = layer.kept()
    layer.close()
    assert np.array_equal(kept, oracle.kept_list(mask)), f"{spec.name}: kept-row list differs"
    y2 = y.view(spec.Nb, spec.P, spec.C_out)
    md = torch.from_numpy(mask.astype(bool)).cuda()
    assert not bool(y2[:, ~md, :].view(torch.int16).any()), f"{spec.name}: dropped rows are not all-zero bits"
    assert not bool(torch.isnan(y2[:, md, :]).any()), f"{spec.name}: a kept element was never written"
    # sampled rows: mostly kept ones, from every image region, plus the first and last rows
    full = np.tile(mask, spec.Nb)
    kept_rows = np.nonzero(full)[0]
    sel = rng.choice(kept_rows, size=min(N_SAMPLED_ROWS, kept_rows.size), replace=False) if kept_rows.size else np.array([], np.int64)
    sel = np.unique(np.concatenate([sel, kept_rows[:2], kept_rows[-2:], rng.integers(0, spec.M, 32)])).astype(np.int64)
    ref = oracle.masked_conv_rows(x, w, b, mask, spec.stride, spec.pad, True, sel)
    got = y.view(spec.M, spec.C_out)[torch.from_numpy(sel).cuda()].float().cpu().numpy().astype(np.float64)
    diff = got - ref
    nref = float(np.linalg.norm(ref))
    rel = float(np.linalg.norm(diff)) / nref if nref > 0 else float(np.linalg.norm(diff))
    tol = 1e-2 * math.sqrt(spec.K) * float(np.abs(oracle.bf16_round(x)).max()) * float(np.abs(oracle.bf16_round(w)).max())
    assert rel <= 5e-3, f"{spec.name}: relative Frobenius error {rel:.3e}"
    assert float(np.abs(diff).max()) <= tol, f"{spec.name}: max abs error {np.abs(diff).max():.3e} > {tol:.3e}"


@pytest.mark.parametrize("cfg", [2, 3])
def test_resnet18_stack_full_size(cfg):
    rng = np.random.default_rng(cfg)
    for spec in wl.config(cfg):
        _check_layer(spec, rng)


def test_detection_stack_full_size():
    rng = np.random.default_rng(4)
    for spec in wl.config(4):
        _check_layer(spec, rng)


def test_sparsity_sweep_full_size():
    rng = np.random.default_rng(5)
    for spec in wl.config(5):          # all 18 (sparsity, block) combinations
        _check_layer(spec, rng)
