"""Seeded synthetic inputs for the masked conv-GEMM path.

This module only *describes* layer problems and draws random tensors and masks
for them.  It holds none of the method's arithmetic (no convolution, no
compaction, no rounding of results) and is the one module that both the CPU
oracle's tests and the CUDA path's tests/bench may import.

The paper evaluates trained ResNet / YOLO networks on image datasets; neither
the datasets nor trained weights or masks are available, so each configuration
below is a stack of independent convolution problems that has the tensor
shapes of those networks (224x224 classification, 640x640 detection), with
random post-activation inputs, Kaiming-normal weights and a uniformly drawn
row mask.  Layers are independent: there is no residual add, pooling or
normalisation between them (normalisation is assumed folded into w and b).

Notation (paper, Section 3: the lowered activation matrix has one entry per
sliding window; here a "row" is one output spatial position):
  x[Nb][H][W][C_in], w[C_out][kh][kw][C_in], b[C_out], mask[rows],
  Ho = (H + 2*pad - kh)//stride + 1, P = Ho*Wo, M = Nb*P, K = kh*kw*C_in.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Iterator, List, Optional

import numpy as np

BASE_SEED = 230906626


@dataclass(frozen=True)
class LayerSpec:
    name: str
    C_in: int
    C_out: int
    kh: int
    kw: int
    stride: int
    pad: int
    H: int
    W: int
    Nb: int
    sparsity_pct: int          # percentage of mask blocks dropped
    block: int                 # consecutive rows kept/dropped together
    x_dist: str                # "relu" | "normal" | "silu" | "smallint"
    seed: int
    relu: bool = True
    exact_drop: Optional[int] = None   # drop exactly this many blocks instead of pct

    @property
    def Ho(self) -> int:
        return (self.H + 2 * self.pad - self.kh) // self.stride + 1

    @property
    def Wo(self) -> int:
        return (self.W + 2 * self.pad - self.kw) // self.stride + 1

    @property
    def P(self) -> int:
        return self.Ho * self.Wo

    @property
    def M(self) -> int:
        return self.Nb * self.P

    @property
    def K(self) -> int:
        return self.kh * self.kw * self.C_in

    @property
    def N(self) -> int:
        return self.C_out


def n_drop_blocks(nblocks: int, pct: int) -> int:
    """Blocks dropped for a percentage: round-half-up of pct% of nblocks, in integers."""
    return (pct * nblocks + 50) // 100


def _streams(seed: int):
    ss = np.random.SeedSequence(seed)
    return [np.random.Generator(np.random.PCG64(s)) for s in ss.spawn(4)]


def make_mask(rows: int, pct: int, block: int, seed: int,
              exact_drop: Optional[int] = None) -> np.ndarray:
    """Row mask (uint8, 1 = keep, 0 = drop).  Blocks of `block` consecutive flat
    row indices (raster order; the last block may be short) are dropped together.
    The dropped blocks are the first n_drop entries of a seeded permutation."""
    rng = _streams(seed)[3]
    nblocks = (rows + block - 1) // block
    nd = n_drop_blocks(nblocks, pct) if exact_drop is None else exact_drop
    perm = rng.permutation(nblocks)
    keep_block = np.ones(nblocks, dtype=np.uint8)
    keep_block[perm[:nd]] = 0
    return np.repeat(keep_block, block)[:rows].copy()


def make_x(spec: LayerSpec) -> np.ndarray:
    rng = _streams(spec.seed)[0]
    shape = (spec.Nb, spec.H, spec.W, spec.C_in)
    if spec.x_dist == "smallint":
        return rng.integers(-3, 4, size=shape).astype(np.float32)
    z = rng.standard_normal(shape, dtype=np.float32)
    if spec.x_dist == "relu":
        np.maximum(z, 0.0, out=z)
    elif spec.x_dist == "silu":
        z = (z / (1.0 + np.exp(-z))).astype(np.float32)
    elif spec.x_dist != "normal":
        raise ValueError(spec.x_dist)
    return z


def make_w(spec: LayerSpec) -> np.ndarray:
    rng = _streams(spec.seed)[1]
    shape = (spec.C_out, spec.kh, spec.kw, spec.C_in)
    if spec.x_dist == "smallint":
        return rng.integers(-2, 3, size=shape).astype(np.float32)
    std = np.float32(np.sqrt(2.0 / spec.K))
    return rng.standard_normal(shape, dtype=np.float32) * std


def make_b(spec: LayerSpec) -> np.ndarray:
    rng = _streams(spec.seed)[2]
    if spec.x_dist == "smallint":
        return rng.integers(-4, 5, size=(spec.C_out,)).astype(np.float32)
    return rng.standard_normal((spec.C_out,), dtype=np.float32) * np.float32(0.01)


def make_layer_mask(spec: LayerSpec, per_row: bool = False) -> np.ndarray:
    """Mask of P entries shared by every image of the batch (the paper's case: one
    constant mask per layer), or of M entries (one bit per lowered row)."""
    rows = spec.M if per_row else spec.P
    return make_mask(rows, spec.sparsity_pct, spec.block, spec.seed, spec.exact_drop)


def _resnet18(Nb: int, pct: int, block: int, cfg: int) -> List[LayerSpec]:
    L: List[LayerSpec] = []

    def add(name, cin, cout, k, s, p, H, dist="relu"):
        L.append(LayerSpec(name, cin, cout, k, k, s, p, H, H, Nb, pct, block, dist,
                           BASE_SEED + 1000 * cfg + len(L)))

    add("conv1", 3, 64, 7, 2, 3, 224, "normal")
    for i in range(2):
        add(f"layer1.{i}.conv1", 64, 64, 3, 1, 1, 56)
        add(f"layer1.{i}.conv2", 64, 64, 3, 1, 1, 56)
    c, H = 64, 56
    for stage in (2, 3, 4):
        c2, H2 = 2 * c, H // 2
        add(f"layer{stage}.0.conv1", c, c2, 3, 2, 1, H)
        add(f"layer{stage}.0.conv2", c2, c2, 3, 1, 1, H2)
        add(f"layer{stage}.0.proj", c, c2, 1, 2, 0, H)
        add(f"layer{stage}.1.conv1", c2, c2, 3, 1, 1, H2)
        add(f"layer{stage}.1.conv2", c2, c2, 3, 1, 1, H2)
        c, H = c2, H2
    return L


def _csp_darknet_like(Nb: int, pct: int, block: int, cfg: int) -> List[LayerSpec]:
    """A synthetic detection-backbone-shaped stack: a 3x3/2 stem, then four stages of a
    3x3/2 down-convolution followed by a cross-stage-partial block of 1x1 and 3x3 convs."""
    L: List[LayerSpec] = []

    def add(name, cin, cout, k, s, p, H, dist="silu"):
        L.append(LayerSpec(name, cin, cout, k, k, s, p, H, H, Nb, pct, block, dist,
                           BASE_SEED + 1000 * cfg + len(L)))

    add("stem", 3, 32, 3, 2, 1, 640, "normal")
    for i, (c, n, H) in enumerate([(64, 1, 160), (128, 2, 80), (256, 3, 40), (512, 1, 20)], 1):
        add(f"s{i}.down", c // 2, c, 3, 2, 1, 2 * H)
        add(f"s{i}.csp.a", c, c // 2, 1, 1, 0, H)
        add(f"s{i}.csp.b", c, c // 2, 1, 1, 0, H)
        for j in range(n):
            add(f"s{i}.m{j}.pw", c // 2, c // 2, 1, 1, 0, H)
            add(f"s{i}.m{j}.conv", c // 2, c // 2, 3, 1, 1, H)
        add(f"s{i}.csp.out", c, c, 1, 1, 0, H)
    return L


SWEEP_SPARSITY = (0, 10, 25, 50, 75, 90)
SWEEP_BLOCK = (1, 4, 16)


def config(cfg: int) -> List[LayerSpec]:
    """The five benchmark configurations (1-based)."""
    if cfg == 1:
        return [LayerSpec("conv3x3_56x56x64", 64, 64, 3, 3, 1, 1, 56, 56, 1, 50, 1, "relu",
                          BASE_SEED + 1000, exact_drop=1568)]
    if cfg == 2:
        return _resnet18(1, 30, 1, 2)
    if cfg == 3:
        return _resnet18(64, 50, 4, 3)
    if cfg == 4:
        return _csp_darknet_like(16, 40, 2, 4)
    if cfg == 5:
        out = []
        for s in SWEEP_SPARSITY:
            for blk in SWEEP_BLOCK:
                out.append(LayerSpec(f"sweep_s{s}_b{blk}", 256, 256, 3, 3, 1, 1, 28, 28, 128,
                                     s, blk, "relu", BASE_SEED + 5000 + len(out)))
        return out
    raise ValueError(f"unknown config {cfg}")


def with_batch(spec: LayerSpec, Nb: int) -> LayerSpec:
    return replace(spec, Nb=Nb)


def with_sparsity(spec: LayerSpec, pct: int) -> LayerSpec:
    return replace(spec, sparsity_pct=pct, exact_drop=None)


def touched_input_pixels(spec: LayerSpec, mask: np.ndarray) -> int:
    """U: number of distinct input pixels (per whole batch) covered by at least one kept
    window.  Pure index bookkeeping used for the algorithmic byte count."""
    per_row = mask.size == spec.M and spec.Nb > 1
    total = 0
    masks = mask.reshape(spec.Nb, spec.Ho, spec.Wo) if per_row else mask.reshape(1, spec.Ho, spec.Wo)
    for m in masks:
        cover = np.zeros((spec.H + 2 * spec.pad + spec.kh, spec.W + 2 * spec.pad + spec.kw), dtype=bool)
        oy, ox = np.nonzero(m)
        for ky in range(spec.kh):
            for kx in range(spec.kw):
                cover[oy * spec.stride + ky, ox * spec.stride + kx] = True
        total += int(cover[spec.pad:spec.pad + spec.H, spec.pad:spec.pad + spec.W].sum())
    return total if per_row else total * spec.Nb


def algorithmic_flops(spec: LayerSpec, kept_rows: int) -> int:
    return 2 * kept_rows * spec.K * spec.N


def make_score(cfg: int, H0: int, W0: int) -> np.ndarray:
    """The random 2-D score of Algorithm 1's getMask at the network's input resolution: uniform
    fp32 in [0, 1), one per configuration (every layer of the stack derives its mask from it)."""
    rng = np.random.Generator(np.random.PCG64(BASE_SEED + 500_000 + cfg))
    return rng.random((H0, W0), dtype=np.float32)


def algorithmic_bytes(spec: LayerSpec, mask: np.ndarray, elem_bytes: int = 2) -> int:
    """Bytes the method must move for one layer call: touched input pixels, weights,
    bias, the full output (zero rows included), the mask and the kept-row list.
    elem_bytes: storage size of x, w and y (2 for bf16, 4 for fp32)."""
    Pk = int(mask.sum())
    U = touched_input_pixels(spec, mask)
    e = elem_bytes
    return e * spec.C_in * U + e * spec.K * spec.N + 4 * spec.N + e * spec.M * spec.N + mask.size + 4 * Pk


def iter_small_cases() -> Iterator[LayerSpec]:
    """Small random-shaped problems that span several 128-row tiles and ragged tails."""
    cases = [
        # name, C_in, C_out, k, s, p, H, W, Nb, pct, block
        ("t_3x3_c64", 64, 64, 3, 1, 1, 20, 23, 2, 30, 1),
        ("t_3x3_s2", 32, 48, 3, 2, 1, 29, 31, 2, 50, 4),
        ("t_1x1_c128", 128, 256, 1, 1, 0, 14, 14, 3, 40, 2),
        ("t_1x1_s2", 64, 128, 1, 2, 0, 28, 28, 2, 50, 4),
        ("t_7x7_c3", 3, 64, 7, 2, 3, 64, 64, 2, 50, 4),
        ("t_3x3_c3", 3, 32, 3, 2, 1, 48, 40, 2, 40, 2),
        ("t_3x3_c8", 8, 24, 3, 1, 1, 17, 19, 1, 25, 1),
        ("t_3x3_c16_n512", 16, 512, 3, 1, 0, 18, 18, 1, 10, 1),
        ("t_5x5_c24", 24, 40, 5, 1, 2, 15, 13, 2, 75, 16),
        ("t_3x3_c256", 256, 256, 3, 1, 1, 14, 14, 2, 50, 4),
        ("t_3x3_c5_n7", 5, 7, 3, 1, 1, 12, 11, 2, 30, 1),
        ("t_3x3_c512", 512, 512, 3, 1, 1, 7, 7, 4, 50, 4),
        # tiny channel counts under stride 2: even width (pixel pairs, odd and even padding),
        # odd width (plain channel padding), and stride 1
        ("t_3x3_c3_s2_oddw", 3, 16, 3, 2, 1, 33, 41, 2, 40, 2),
        ("t_5x5_c4_s2_p2", 4, 24, 5, 2, 2, 30, 32, 2, 30, 1),
        ("t_2x2_c1_s2_p0", 1, 8, 2, 2, 0, 16, 16, 3, 50, 1),
        ("t_4x4_c2_s2_p1", 2, 40, 4, 2, 1, 18, 22, 2, 25, 4),
        ("t_3x3_c4_s1", 4, 16, 3, 1, 1, 14, 15, 2, 50, 1),
        # stems that take the 2x2-block form: 7-wide with even padding, 8-wide
        ("t_7x7_c4_s2_p2", 4, 16, 7, 2, 2, 22, 26, 1, 40, 2),
        ("t_8x8_c2_s2_p2", 2, 24, 8, 2, 2, 20, 24, 2, 30, 1),
        # few rows and a long reduction: the k-blocks of a tile are shared between blocks
        ("t_3x3_c256_n40_longk", 256, 40, 3, 1, 1, 9, 10, 2, 20, 1),
        ("t_3x3_c320_n264_longk", 320, 264, 3, 1, 1, 12, 12, 1, 0, 1),
    ]
    for i, (name, cin, cout, k, s, p, H, W, Nb, pct, blk) in enumerate(cases):
        yield LayerSpec(name, cin, cout, k, k, s, p, H, W, Nb, pct, blk, "relu",
                        BASE_SEED + 9000 + i)
