"""Philox4x32-10 written from its published definition (Salmon et al., SC'11), test side.

Used to re-derive, independently of the library, the mask that asx_set_mask_random
generates.  Pinned in test_abi.py against the known-answer vectors of the reference
implementation's test suite.
"""
import numpy as np

M0, M1 = 0xD2511F53, 0xCD9E8D57
W0, W1 = 0x9E3779B9, 0xBB67AE85
MASK32 = 0xFFFFFFFF


def philox4x32_10(ctr, key):
    c0, c1, c2, c3 = ctr
    k0, k1 = key
    for _ in range(10):
        p0, p1 = M0 * c0, M1 * c2
        c0, c1, c2, c3 = ((p1 >> 32) ^ c1 ^ k0) & MASK32, p1 & MASK32, ((p0 >> 32) ^ c3 ^ k1) & MASK32, p0 & MASK32
        k0, k1 = (k0 + W0) & MASK32, (k1 + W1) & MASK32
    return c0, c1, c2, c3


def random_block_mask(rows: int, sparsity: float, block: int, seed: int) -> np.ndarray:
    """The documented rule of asx_set_mask_random: score each block with Philox, drop the
    floor(sparsity*nblocks + 1/2) blocks with the smallest (score, index)."""
    nblocks = -(-rows // block)
    n_drop = min(nblocks, int(sparsity * nblocks + 0.5))
    key = (seed & MASK32, (seed >> 32) & MASK32)
    scores = []
    for b in range(nblocks):
        o = philox4x32_10((b & MASK32, (b >> 32) & MASK32, 0, 0), key)
        scores.append(((o[1] << 32) | o[0], b))
    scores.sort()
    mask = np.ones(rows, dtype=np.uint8)
    for _, b in scores[:n_drop]:
        mask[b * block:(b + 1) * block] = 0
    return mask
