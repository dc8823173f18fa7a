"""The bounded waits of the fused kernel, exercised from the host in the safe form.

A layer with few kept rows and a long reduction shares each tile's k-blocks between thread blocks;
the blocks of a tile meet at an arrival counter.  The test overwrites one tile's counter with a value
the arrivals can never lift to the number of shares and shortens the wait limit to about a
millisecond: the waiting blocks must give up, every role of the kernel must leave, the kernel must
return, the status word must say so, and the next run on the same handle must be correct again.
Nothing here faults, traps or hangs the GPU: the wait simply runs out."""
import numpy as np
import pytest
import torch

import oracle
import paper_2309_06626_b200 as asx
import workloads as wl
from gpu_util import make_problem, max_abs_tol, to_dev_bf16, REL_FROB_TOL

pytestmark = pytest.mark.gpu

ASX_ERR_TIMEOUT = 8


def test_a_wait_that_runs_out_is_reported_and_the_layer_recovers():
    spec = [s for s in wl.iter_small_cases() if s.name == "t_3x3_c256_n40_longk"][0]
    x, w, b, mask = make_problem(spec)
    ref = oracle.masked_conv(x, w, b, mask, spec.stride, spec.pad, True).reshape(spec.M, spec.C_out)
    tol = max_abs_tol(spec.K, oracle.bf16_round(x), oracle.bf16_round(w))
    layer = asx.MaskedConvLayer(spec.C_in, spec.C_out, spec.kh, spec.kw, spec.stride, spec.pad)
    layer.set_mask(mask)
    xd, wd, bd = to_dev_bf16(x), to_dev_bf16(w), torch.from_numpy(b).cuda()
    flags = asx.ACT_RELU | asx.IMPL_ROW_GATHER             # the form that shares k-blocks between blocks
    st = int(torch.cuda.current_stream().cuda_stream)

    def run_and_compare():
        y = layer.run(xd, wd, bd, flags=flags)
        torch.cuda.synchronize()
        assert layer.device_status() == 0
        got = y.float().cpu().numpy().astype(np.float64).reshape(spec.M, spec.C_out)
        assert np.linalg.norm(got - ref) / np.linalg.norm(ref) <= REL_FROB_TOL
        assert np.abs(got - ref).max() <= tol

    run_and_compare()
    # the plan of this layer shares k-blocks: the counters exist (else this case tests nothing)
    rc = asx.lib().asx_debug_set_split_counter(layer._h, 0, -100000, st)
    assert rc == 0, f"the layer was expected to share k-blocks between blocks (status {rc})"
    assert asx.lib().asx_debug_set_split_counter(layer._h, 1 << 40, 0, st) == 1       # outside the workspace
    layer.set_wait_limit(2_000_000)                        # about a millisecond of GPU clock cycles
    t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    layer.run(xd, wd, bd, flags=flags)
    t1.record()
    torch.cuda.synchronize()
    assert t0.elapsed_time(t1) < 500.0, "the kernel did not leave its wait within the limit"
    assert layer.device_status() == ASX_ERR_TIMEOUT
    assert layer.device_status() == 0                       # the word is cleared by the query
    layer.set_wait_limit(0)                                 # back to the default
    run_and_compare()
    run_and_compare()
    layer.close()


def test_hook_refuses_layers_without_shared_k_blocks():
    spec = wl.LayerSpec("nosplit", 64, 64, 3, 3, 1, 1, 20, 20, 2, 30, 1, "relu", 99)
    x, w, b, mask = make_problem(spec)
    layer = asx.MaskedConvLayer(64, 64, 3, 3, 1, 1)
    layer.set_mask(mask)
    layer.run(to_dev_bf16(x), to_dev_bf16(w), torch.from_numpy(b).cuda(), flags=asx.ACT_RELU)
    torch.cuda.synchronize()
    st = int(torch.cuda.current_stream().cuda_stream)
    assert asx.lib().asx_debug_set_split_counter(layer._h, 0, 5, st) == 2       # ASX_ERR_UNSUPPORTED
    layer.close()
