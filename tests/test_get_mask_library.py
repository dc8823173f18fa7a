"""The library's host-side mask generator (Algorithm 1, getMask) against the oracle, bit for bit,
through the C ABI.  No GPU is needed: asx_mask_from_scores makes no CUDA call."""
import numpy as np
import pytest

import oracle
import paper_2309_06626_b200 as asx

CASES = [
    # H0, W0, Ho, Wo, sparsity
    (224, 224, 112, 112, 0.5), (224, 224, 56, 56, 0.3), (224, 224, 28, 28, 0.1), (224, 224, 14, 14, 0.75),
    (224, 224, 7, 7, 0.9), (64, 96, 16, 12, 0.4), (10, 11, 3, 5, 0.4), (56, 56, 56, 56, 0.25),
    (33, 47, 33, 47, 0.0), (33, 47, 11, 15, 1.0), (5, 5, 1, 1, 0.5),
]


@pytest.mark.parametrize("H0,W0,Ho,Wo,s", CASES)
def test_mask_from_scores_equals_oracle(H0, W0, Ho, Wo, s):
    rng = np.random.default_rng(H0 * 1000 + Ho)
    score = rng.random((H0, W0)).astype(np.float32)
    assert np.array_equal(asx.mask_from_scores(score, Ho, Wo, s), oracle.get_mask(score, Ho, Wo, s))


def test_ties_and_quantised_scores_equal_oracle():
    rng = np.random.default_rng(3)
    score = rng.integers(0, 4, size=(48, 48)).astype(np.float32)      # many equal pooled scores
    for Ho, s in ((48, 0.3), (24, 0.5), (12, 0.2), (6, 0.6)):
        assert np.array_equal(asx.mask_from_scores(score, Ho, Ho, s), oracle.get_mask(score, Ho, Ho, s))


def test_argument_errors():
    score = np.zeros((8, 8), np.float32)
    out = np.zeros(64, np.uint8)
    L = asx.lib()
    assert L.asx_mask_from_scores(score.ctypes.data, 8, 8, 9, 8, 0.5, out.ctypes.data) == 1      # layer larger than score
    assert L.asx_mask_from_scores(score.ctypes.data, 8, 8, 4, 4, 1.5, out.ctypes.data) == 1      # sparsity out of range
    assert L.asx_mask_from_scores(None, 8, 8, 4, 4, 0.5, out.ctypes.data) == 1
    assert L.asx_mask_from_scores(score.ctypes.data, 8, 8, 4, 4, 0.5, None) == 1
