"""Seeded random layer geometries against the oracle: channel counts around every staging path
(1..6, multiples of 8 and 64, odd counts), filter sizes 1..8, strides 1..3, paddings up to the
filter size, ragged images, shared and per-row masks, with and without bias and ReLU."""
import numpy as np
import pytest

import paper_2309_06626_b200 as asx
import workloads as wl
from gpu_util import check_against_oracle, make_problem

pytestmark = pytest.mark.gpu


def _random_spec(i):
    rng = np.random.default_rng(90_000 + i)
    cin = int(rng.choice([1, 2, 3, 4, 5, 6, 8, 16, 24, 32, 40, 64, 64, 96, 128, 192, 256]))
    cout = int(rng.choice([1, 7, 8, 16, 24, 40, 64, 64, 72, 128, 136, 256, 264]))
    k = int(rng.choice([1, 2, 3, 3, 3, 4, 5, 7, 8]))
    stride = int(rng.choice([1, 1, 2, 2, 3]))
    pad = int(rng.integers(0, k))                      # 0 .. k-1
    # keep K = k*k*cin moderate so that the oracle stays fast
    while k * k * cin > 6000:
        cin //= 2
    H = int(rng.integers(max(k - 2 * pad, 1) + 2, 34))
    W = int(rng.integers(max(k - 2 * pad, 1) + 2, 34))
    if rng.random() < 0.5:                             # even sizes reach the pixel-pair and 2x2-block forms
        H += H % 2
        W += W % 2
    Nb = int(rng.integers(1, 4))
    pct = int(rng.choice([0, 10, 30, 50, 50, 75, 95, 100]))
    block = int(rng.choice([1, 1, 2, 4, 16]))
    return wl.LayerSpec(f"rnd{i}", cin, cout, k, k, stride, pad, H, W, Nb, pct, block, "relu", wl.BASE_SEED + 40_000 + i)


@pytest.mark.parametrize("i", range(60))
def test_random_geometry(i):
    spec = _random_spec(i)
    rng = np.random.default_rng(7 * i + 1)
    per_row = bool(rng.random() < 0.3)
    x, w, b, mask = make_problem(spec, per_row=per_row)
    flags = (asx.ACT_RELU if rng.random() < 0.7 else 0) | (asx.RECOMPACT if rng.random() < 0.5 else 0)
    check_against_oracle(spec, x, w, b if rng.random() < 0.8 else None, mask, flags)


def _random_patch_spec(i):
    """Geometries the window-patch form takes: stride 1, several taps, C_in a multiple of 64."""
    rng = np.random.default_rng(555_000 + i)
    cin = int(rng.choice([64, 64, 128, 192, 256]))
    cout = int(rng.choice([8, 16, 24, 40, 64, 64, 72, 128, 136, 200, 256, 264]))
    kh = int(rng.choice([1, 2, 3, 3, 3, 4, 5]))
    kw = int(rng.choice([1, 2, 3, 3, 3, 4, 5]))
    if kh * kw < 2:
        kw = 3
    pad = int(rng.integers(0, 3))
    H = int(rng.integers(max(kh - 2 * pad, 1) + 1, 30))
    W = int(rng.integers(max(kw - 2 * pad, 1) + 1, 30))
    Nb = int(rng.integers(1, 7))
    pct = int(rng.choice([0, 10, 30, 50, 50, 75, 90, 97]))
    blk = int(rng.choice([1, 1, 2, 4, 8]))
    while kh * kw * cin * cout > 3_000_000:
        cout = max(8, cout // 2)
    return wl.LayerSpec(f"rp{i}", cin, cout, kh, kw, 1, pad, H, W, Nb, pct, blk, "relu", wl.BASE_SEED + 60_000 + i)


@pytest.mark.parametrize("i", range(40))
def test_random_geometry_window_patch(i):
    """The same kind of sweep with the window-patch form forced (300 such cases, each run three times with
    bit-identical results, were run once; this is their first 40)."""
    spec = _random_patch_spec(i)
    per_row = bool(np.random.default_rng(11 * i + 3).random() < 0.3)
    x, w, b, mask = make_problem(spec, per_row=per_row)
    flags = asx.ACT_RELU | asx.IMPL_WINDOW_PATCH | (asx.RECOMPACT if i % 2 else 0)
    check_against_oracle(spec, x, w, b, mask, flags)
