"""Oracle for the mask generator of the paper's training pipeline (Algorithm 1, function getMask):
test infrastructure, not part of the product.

getMask draws one random 2-D score at the input image's resolution, brings it to each layer's
resolution with an average pooling whose window and stride are ratio = input_res // layer_res,
ranks the layer's positions by their pooled score and sets the mask to 0 at the ranked fraction s.

The paper does not say which end of the ranking is masked, how ties are ordered, how s * P is
rounded, or what happens when the resolutions do not divide.  The readings taken here (the same
ones the library documents): the k = floor(s * P + 1/2) positions with the SMALLEST pooled score are
dropped; equal scores are ordered by position index (raster order); the pooling window of output
cell (i, j) is rows i*rh .. i*rh + rh - 1 and columns j*rw .. j*rw + rw - 1 of the score with
rh = H0 // Ho, rw = W0 // Wo (so rows and columns of the score beyond Ho*rh, Wo*rw are unused);
scores are fp32 values, window sums are accumulated in fp64 in raster order of the window and
divided by rh*rw in fp64, and the ranking compares those fp64 values.

Plain numpy with explicit loops over the output cells; no blocking, no vectorised tricks."""
from __future__ import annotations

import numpy as np


def pooled_score(score: np.ndarray, Ho: int, Wo: int) -> np.ndarray:
    """avg_pool2d(score, ratio) of Algorithm 1 at a layer of Ho x Wo positions; fp64 [Ho][Wo]."""
    score = np.asarray(score, dtype=np.float32)
    H0, W0 = score.shape
    rh, rw = H0 // Ho, W0 // Wo
    if rh < 1 or rw < 1:
        raise ValueError("the layer's resolution exceeds the score's")
    out = np.zeros((Ho, Wo), dtype=np.float64)
    for i in range(Ho):
        for j in range(Wo):
            acc = 0.0
            for a in range(rh):
                for b in range(rw):
                    acc += float(score[i * rh + a, j * rw + b])
            out[i, j] = acc / float(rh * rw)
    return out


def get_mask(score: np.ndarray, Ho: int, Wo: int, sparsity: float) -> np.ndarray:
    """The layer's binary mask (uint8 [Ho*Wo], 1 keep / 0 drop) of Algorithm 1's getMask."""
    P = Ho * Wo
    pooled = pooled_score(score, Ho, Wo).reshape(P)
    k = int(np.floor(sparsity * P + 0.5))
    k = max(0, min(P, k))
    # rankPixels: ascending by (pooled score, position); a stable sort keeps equal scores in raster order
    order = sorted(range(P), key=lambda p: (pooled[p], p))
    mask = np.ones(P, dtype=np.uint8)
    for p in order[:k]:
        mask[p] = 0
    return mask


def mask_from_activation(x: np.ndarray) -> np.ndarray:
    """Data-dependent mask of the family the paper contrasts itself with (Section 2: sparsity that
    comes from the activations themselves, e.g. ReLU zeros): a lowered row / spatial position is kept
    iff at least one of its channels is strictly positive.  x: [..., C] real values (already rounded
    to the storage precision by the caller); NaN and zeros of either sign count as not positive.
    Returns uint8 [prod(leading dims)]."""
    x = np.asarray(x, dtype=np.float64)
    C = x.shape[-1]
    rows = x.reshape(-1, C)
    out = np.zeros(rows.shape[0], dtype=np.uint8)
    for r in range(rows.shape[0]):
        keep = 0
        for c in range(C):
            if rows[r, c] > 0.0:
                keep = 1
        out[r] = keep
    return out
