"""Pins for the oracle of Algorithm 1's getMask (random score -> average pooling -> ranking).

The paper prints no numbers for it, so the pins are: the library's own average pooling and
sorting routines on cases where the readings do not matter (distinct scores, dividing
resolutions), a hand-worked 4x4 example, the count rule, tie order, and the property that makes
the masks "propagate consistently": a layer's dropped set is a function of the pooled score only.
"""
import numpy as np
import pytest
import torch

import oracle


def test_hand_worked_4x4_to_2x2():
    # windows:  [[1,2],[5,6]] -> 3.5   [[3,4],[7,8]] -> 5.5   [[9,10],[13,14]] -> 11.5   [[11,12],[15,16]] -> 13.5
    score = np.arange(1, 17, dtype=np.float32).reshape(4, 4)
    assert np.array_equal(oracle.pooled_score(score, 2, 2), np.array([[3.5, 5.5], [11.5, 13.5]]))
    assert oracle.get_mask(score, 2, 2, 0.5).tolist() == [0, 0, 1, 1]
    assert oracle.get_mask(score, 2, 2, 0.25).tolist() == [0, 1, 1, 1]
    assert oracle.get_mask(-score, 2, 2, 0.25).tolist() == [1, 1, 1, 0]
    # sparsity 1/8 of 4 positions: floor(0.5 + 0.5) = 1 dropped; 0.1 of 4: floor(0.9) = 0 dropped
    assert int(oracle.get_mask(score, 2, 2, 0.125).sum()) == 3
    assert int(oracle.get_mask(score, 2, 2, 0.1).sum()) == 4


@pytest.mark.parametrize("H0,W0,Ho,Wo", [(224, 224, 112, 112), (224, 224, 7, 7), (64, 96, 16, 12), (56, 56, 56, 56)])
def test_pooling_matches_library_avg_pool(H0, W0, Ho, Wo):
    rng = np.random.default_rng(7)
    score = rng.random((H0, W0)).astype(np.float32)
    ref = torch.nn.functional.avg_pool2d(torch.from_numpy(score).double()[None, None], (H0 // Ho, W0 // Wo))[0, 0].numpy()
    got = oracle.pooled_score(score, Ho, Wo)
    assert got.shape == (Ho, Wo)
    np.testing.assert_allclose(got, ref, rtol=1e-14, atol=0)


def test_non_dividing_resolution_uses_floor_ratio_and_ignores_the_rest():
    rng = np.random.default_rng(8)
    score = rng.random((10, 11)).astype(np.float32)
    got = oracle.pooled_score(score, 3, 5)          # ratio 3 x 2: rows 0..8, columns 0..9 are used
    ref = score[:9, :10].astype(np.float64).reshape(3, 3, 5, 2).mean(axis=(1, 3))
    np.testing.assert_allclose(got, ref, rtol=1e-14)
    changed = score.copy()
    changed[9, :] = 100.0
    changed[:, 10] = -100.0
    assert np.array_equal(oracle.get_mask(score, 3, 5, 0.4), oracle.get_mask(changed, 3, 5, 0.4))


@pytest.mark.parametrize("s", [0.0, 0.1, 0.3, 0.5, 0.9, 1.0])
def test_dropped_set_is_the_k_smallest_pooled_scores(s):
    rng = np.random.default_rng(9)
    score = rng.random((48, 40)).astype(np.float32)
    Ho, Wo = 12, 10
    P = Ho * Wo
    mask = oracle.get_mask(score, Ho, Wo, s)
    k = int(np.floor(s * P + 0.5))
    assert mask.dtype == np.uint8 and mask.shape == (P,) and int(mask.sum()) == P - k
    pooled = torch.nn.functional.avg_pool2d(torch.from_numpy(score).double()[None, None], 4).reshape(-1).numpy()
    dropped = np.flatnonzero(mask == 0)
    # library sort: the k smallest values (distinct with probability one)
    assert set(dropped.tolist()) == set(np.argsort(pooled, kind="stable")[:k].tolist())
    if 0 < k < P:
        assert pooled[dropped].max() < pooled[mask == 1].min()


def test_ties_are_dropped_in_raster_order():
    score = np.zeros((8, 8), dtype=np.float32)
    mask = oracle.get_mask(score, 4, 4, 0.25)
    assert mask.tolist() == [0] * 4 + [1] * 12
    score[0:2, 0:2] = 1.0                                  # position 0 now has the largest score
    assert oracle.get_mask(score, 4, 4, 0.25).tolist() == [1, 0, 0, 0, 0] + [1] * 11


def test_masks_of_two_layers_come_from_the_same_score():
    """Consistency across resolutions (Section 3.1): the coarse layer's pooled score is the mean of the
    fine layer's over each 2x2 group, so a coarse position whose four fine positions are all among the
    fine layer's dropped set, with every other fine position scoring higher, is dropped first."""
    rng = np.random.default_rng(10)
    score = (rng.random((32, 32)).astype(np.float32) + 1.0)
    score[8:16, 16:24] = 0.0                              # one 8x8 patch with the lowest scores
    fine = oracle.get_mask(score, 8, 8, 4 / 64).reshape(8, 8)       # ratio 4: the patch is 2x2 fine cells
    coarse = oracle.get_mask(score, 4, 4, 1 / 16).reshape(4, 4)     # ratio 8: exactly one coarse cell
    assert np.argwhere(fine == 0).tolist() == [[2, 4], [2, 5], [3, 4], [3, 5]]
    assert np.argwhere(coarse == 0).tolist() == [[1, 2]]
    np.testing.assert_allclose(oracle.pooled_score(score, 4, 4),
                               oracle.pooled_score(score, 8, 8).reshape(4, 2, 4, 2).mean(axis=(1, 3)), rtol=1e-14)


def test_mask_from_activation_special_values_and_library_reduction():
    x = np.zeros((9, 4), dtype=np.float32)
    x[1, 2] = 1.0                                   # one positive channel
    x[2, :] = -1.0                                  # only negatives
    x[3, 0] = -0.0
    x[4, 1] = np.nan                                # NaN is not positive
    x[5, 3] = np.float32(1e-40)                     # a denormal is positive
    x[6, :] = [np.nan, -1.0, 0.0, 2.0]              # NaN beside a positive
    x[7, 0] = np.inf
    x[8, 0] = -np.inf
    assert oracle.mask_from_activation(x).tolist() == [0, 1, 0, 0, 0, 1, 1, 1, 0]
    rng = np.random.default_rng(11)
    y = rng.standard_normal((3, 5, 7, 6)).astype(np.float32)
    y[rng.random(y.shape[:-1]) < 0.4] = -np.abs(y[rng.random(y.shape[:-1]) < 0.4][0])   # many all-negative positions
    ref = (torch.from_numpy(y) > 0).any(dim=-1).reshape(-1).numpy().astype(np.uint8)
    assert np.array_equal(oracle.mask_from_activation(y), ref)
