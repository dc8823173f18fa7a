"""Helpers for the GPU parity tests: run one layer problem through the C-ABI library and
compare with the CPU oracle under the stated tolerances."""
import math

import numpy as np
import torch

import oracle
import paper_2309_06626_b200 as asx
import workloads as wl

REL_FROB_TOL = 5e-3           # relative Frobenius error of the kept values


def max_abs_tol(K, xh, wh):
    """1e-2 * sqrt(K) * max|x| * max|w| on the bf16-rounded inputs."""
    return 1e-2 * math.sqrt(K) * float(np.max(np.abs(xh))) * float(np.max(np.abs(wh)))


def to_dev_bf16(a):
    return torch.from_numpy(np.ascontiguousarray(a)).to(torch.bfloat16).cuda().contiguous()


def run_library(spec, x, w, b, mask, flags, prefill=None):
    """Returns (y as float64 numpy [M][N], raw uint16 bits [M][N], kept list)."""
    layer = asx.MaskedConvLayer(spec.C_in, spec.C_out, spec.kh, spec.kw, spec.stride, spec.pad)
    layer.set_mask(mask)
    xd, wd = to_dev_bf16(x), to_dev_bf16(w)
    bd = None if b is None else torch.from_numpy(b).cuda()
    out = torch.empty((spec.Nb, spec.Ho, spec.Wo, spec.C_out), dtype=torch.bfloat16, device="cuda")
    if prefill is not None:
        out.view(torch.int16).fill_(prefill)
    layer.run(xd, wd, bd, out=out, flags=flags)
    torch.cuda.synchronize()
    status = layer.device_status()
    kept = layer.kept()
    layer.close()
    assert status == 0, f"device status {status}"
    bits = out.view(torch.int16).cpu().numpy().view(np.uint16).reshape(spec.M, spec.C_out)
    y = out.float().cpu().numpy().astype(np.float64).reshape(spec.M, spec.C_out)
    return y, bits, kept


def full_row_mask(spec, mask):
    return mask if mask.size == spec.M else np.tile(mask, spec.Nb)


def check_against_oracle(spec, x, w, b, mask, flags, rows_sel=None):
    """Full comparison (rows_sel None) or comparison on selected lowered rows."""
    relu = "silu" if flags & asx.ACT_SILU else bool(flags & asx.ACT_RELU)      # the oracle's activation argument
    y, bits, kept = run_library(spec, x, w, b, mask, flags, prefill=0x7fc1)   # NaN canary
    # kept list: bit-exact
    assert np.array_equal(kept, oracle.kept_list(mask)), "kept-row list differs"
    fm = full_row_mask(spec, mask).astype(bool)
    # dropped rows: the bit pattern 0x0000 in every channel
    assert not np.any(bits[~fm]), "dropped rows are not all-zero bits"
    assert not np.any(np.isnan(y)), "an output element was never written"
    xh, wh = oracle.bf16_round(x), oracle.bf16_round(w)
    if rows_sel is None:
        ref = oracle.masked_conv(x, w, b, mask, spec.stride, spec.pad, relu).reshape(spec.M, spec.C_out)
        got = y
    else:
        ref = oracle.masked_conv_rows(x, w, b, mask, spec.stride, spec.pad, relu, rows_sel)
        got = y[rows_sel]
    diff = got - ref
    nref = float(np.linalg.norm(ref))
    rel = float(np.linalg.norm(diff)) / nref if nref > 0 else float(np.linalg.norm(diff))
    mx = float(np.max(np.abs(diff))) if diff.size else 0.0
    tol = max_abs_tol(spec.K, xh, wh)
    assert rel <= REL_FROB_TOL, f"{spec.name}: relative Frobenius error {rel:.3e}"
    assert mx <= tol, f"{spec.name}: max abs error {mx:.3e} > {tol:.3e}"
    return rel, mx


def make_problem(spec, per_row=False):
    return (wl.make_x(spec), wl.make_w(spec), wl.make_b(spec), wl.make_layer_mask(spec, per_row))
