"""Data-dependent masks: the CUDA kernel against the oracle rule (bit-exact), and a masked
convolution driven by such a mask (one entry per lowered row, set from device memory)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2309_06626_b200 as asx
import workloads as wl
from gpu_util import to_dev_bf16

pytestmark = pytest.mark.gpu


def _activation(rng, rows, C, zero_frac=0.5):
    x = rng.standard_normal((rows, C)).astype(np.float32)
    x = np.maximum(x, 0.0)                                   # what a ReLU leaves
    dead = rng.random(rows) < zero_frac
    x[dead] = -np.abs(rng.standard_normal((int(dead.sum()), C)).astype(np.float32)) * (rng.random((int(dead.sum()), 1)) < 0.5)
    return x


@pytest.mark.parametrize("rows,C", [(1, 8), (5, 3), (1000, 5), (4097, 8), (3001, 16), (777, 32), (50_000, 64),
                                    (1234, 128), (517, 256), (300, 512), (129, 24), (0, 64)])
def test_kernel_equals_oracle(rows, C):
    rng = np.random.default_rng(rows * 31 + C)
    x = _activation(rng, rows, C)
    xd = to_dev_bf16(x).reshape(rows, C)
    got = asx.mask_from_activation(xd).cpu().numpy()
    want = oracle.mask_from_activation(xd.float().cpu().numpy()) if rows else np.zeros(0, np.uint8)
    assert np.array_equal(got, want)
    if rows > 100:
        assert 0 < int(want.sum()) < rows


def test_special_values_and_unaligned_input():
    vals = torch.tensor([0.0, -0.0, float("nan"), float("inf"), -float("inf"), 1e-40, -1e-40, 1.0, -1.0],
                        dtype=torch.float32).to(torch.bfloat16)
    x = torch.zeros((len(vals), 64), dtype=torch.bfloat16)
    x[torch.arange(len(vals)), torch.arange(len(vals)) * 7 % 64] = vals
    xd = x.cuda()
    want = oracle.mask_from_activation(x.float().numpy())
    assert want.tolist() == [0, 0, 0, 1, 0, 1, 0, 1, 0]
    assert asx.mask_from_activation(xd).cpu().numpy().tolist() == want.tolist()
    # a view that starts 2 bytes into an allocation: the generic kernel
    flat = torch.zeros(len(vals) * 64 + 1, dtype=torch.bfloat16, device="cuda")
    flat[1:] = xd.reshape(-1)
    out = torch.empty(len(vals), dtype=torch.uint8, device="cuda")
    rc = asx.lib().asx_mask_from_activation(flat.data_ptr() + 2, len(vals), 64, out.data_ptr(),
                                            int(torch.cuda.current_stream().cuda_stream))
    torch.cuda.synchronize()
    assert rc == 0 and out.cpu().numpy().tolist() == want.tolist()


def test_masked_convolution_driven_by_an_activation_mask():
    """The previous layer's output decides which positions the next convolution computes."""
    spec = wl.LayerSpec("from_act", 32, 48, 3, 3, 1, 1, 18, 22, 3, 0, 1, "relu", wl.BASE_SEED + 99)
    rng = np.random.default_rng(5)
    x, w, b = wl.make_x(spec), wl.make_w(spec), wl.make_b(spec)
    act = _activation(rng, spec.M, 16, zero_frac=0.4)        # [M][16]: one row per output position of the layer
    act_d = to_dev_bf16(act).reshape(spec.M, 16)
    mask_d = asx.mask_from_activation(act_d)
    want = oracle.mask_from_activation(act_d.float().cpu().numpy())
    layer = asx.MaskedConvLayer(spec.C_in, spec.C_out, spec.kh, spec.kw, spec.stride, spec.pad)
    layer.set_mask(mask_d)                                   # device pointer, one entry per lowered row
    y = layer.run(to_dev_bf16(x), to_dev_bf16(w), torch.from_numpy(b).cuda(), flags=asx.ACT_RELU | asx.RECOMPACT)
    torch.cuda.synchronize()
    assert layer.device_status() == 0
    assert np.array_equal(layer.kept(), oracle.kept_list(want))
    layer.close()
    ref = oracle.masked_conv(x, w, b, want, spec.stride, spec.pad, True)
    got = y.float().cpu().numpy().astype(np.float64).reshape(ref.shape)
    assert np.linalg.norm(got - ref) / np.linalg.norm(ref) < 5e-3
    assert not got.reshape(spec.M, spec.C_out)[want == 0].any()
