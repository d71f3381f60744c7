"""Seeded synthetic inputs for pivoted (PBP) fully-connected layers.

This module only *draws* inputs: permutations, kept-tile sets, tile values,
biases and activation vectors.  It contains none of the method's arithmetic
(no products, no permutation application, no packing), so both the CPU oracle's
tests and the CUDA path's tests can use it without sharing any computation.

A layer is described in the paper's PBP form (Eq. 1): a sparse matrix equals
row-permutation x block matrix x column-permutation.  Here a layer is the
tuple (M, N, B, row_perm, col_perm, tile_list, tile_values, bias):

* ``row_perm[i]`` / ``col_perm[j]``: original index of pivoted row i / column j
  (index-array convention of Section 4.1.4: gathering "abc" with [2,0,1]
  gives "cab").  Both are bijections on the padded ranges [0, Mb*B) / [0, Nb*B).
* ``tile_list[t] = (block_row, block_col)`` of kept tile t in pivoted space.
* ``tile_values[t]`` is the dense B x B tile, row-major, in the weight dtype
  (fp16 tiles are rounded once here, so every consumer sees the same bits).

Draw order per layer is fixed: row_perm, col_perm, tile set, tile values,
bias; the activation vector x is drawn last from the first layer's generator.
Seed = 20171201 + 100*config + layer.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional

import numpy as np

BASE_SEED = 20171201

ACT_IDENTITY = 0
ACT_RELU = 1


@dataclass
class Layer:
    M: int
    N: int
    B: int
    row_perm: np.ndarray          # int32 [Mb*B]
    col_perm: np.ndarray          # int32 [Nb*B]
    tile_list: np.ndarray         # int32 [T, 2]
    tile_values: np.ndarray       # float32 or float16 [T, B, B]
    bias: Optional[np.ndarray]    # float32 [M] or None
    act: int = ACT_IDENTITY
    seed: int = 0

    @property
    def Mb(self) -> int:
        return -(-self.M // self.B)

    @property
    def Nb(self) -> int:
        return -(-self.N // self.B)

    @property
    def T(self) -> int:
        return int(self.tile_list.shape[0])

    @property
    def wdtype(self) -> str:
        return "f16" if self.tile_values.dtype == np.float16 else "f32"


@dataclass
class Workload:
    name: str
    layers: List[Layer]
    x: np.ndarray                 # [batch, N0] (or [steps, I] for the recurrent config)
    note: str = ""
    extra: dict = field(default_factory=dict)


def _seed(config: int, layer: int) -> int:
    return BASE_SEED + 100 * config + layer


def balanced_tiles(rng: np.random.Generator, Mb: int, Nb: int, k: int) -> np.ndarray:
    """Exactly k kept tiles in every block-row, columns drawn without replacement, sorted."""
    rows = []
    for br in range(Mb):
        cols = np.sort(rng.choice(Nb, size=k, replace=False))
        rows.append(np.stack([np.full(k, br, dtype=np.int64), cols], axis=1))
    if not rows:
        return np.zeros((0, 2), dtype=np.int32)
    return np.concatenate(rows, axis=0).astype(np.int32)


def uniform_tiles(rng: np.random.Generator, Mb: int, Nb: int, T: int) -> np.ndarray:
    """T kept tiles drawn without replacement from the whole Mb x Nb grid (unbalanced rows)."""
    flat = np.sort(rng.choice(Mb * Nb, size=T, replace=False))
    return np.stack([flat // Nb, flat % Nb], axis=1).astype(np.int32)


def make_layer(seed: int, M: int, N: int, B: int, *, wdtype: str,
               tiles: str, k: int = 0, density: float = 0.0,
               bias_std: Optional[float] = None, act: int = ACT_IDENTITY,
               identity_perms: bool = False, w_std: Optional[float] = None,
               integer_values: bool = False) -> tuple[Layer, np.random.Generator]:
    """Draw one layer.  ``tiles`` is "balanced" (k per block-row) or "uniform"
    (round(density*Mb*Nb) tiles over the whole grid).  Weights ~ N(0, 1/N)
    (variance 1/N) unless ``w_std`` is given; ``integer_values`` draws small
    integers in [-4, 4] instead (every partial sum is then exact in fp16/fp32)."""
    rng = np.random.default_rng(seed)
    Mb, Nb = -(-M // B), -(-N // B)
    if identity_perms:
        row_perm = np.arange(Mb * B, dtype=np.int32)
        col_perm = np.arange(Nb * B, dtype=np.int32)
    else:
        row_perm = rng.permutation(Mb * B).astype(np.int32)
        col_perm = rng.permutation(Nb * B).astype(np.int32)
    if tiles == "balanced":
        tile_list = balanced_tiles(rng, Mb, Nb, k)
    elif tiles == "uniform":
        tile_list = uniform_tiles(rng, Mb, Nb, int(round(density * Mb * Nb)))
    else:
        raise ValueError(tiles)
    T = tile_list.shape[0]
    if integer_values:
        vals = rng.integers(-4, 5, size=(T, B, B)).astype(np.float32)
    else:
        std = w_std if w_std is not None else 1.0 / np.sqrt(N)
        vals = (rng.standard_normal((T, B, B)) * std).astype(np.float32)
    if wdtype == "f16":
        vals = vals.astype(np.float16)          # round-to-nearest-even, once
    elif wdtype != "f32":
        raise ValueError(wdtype)
    bias = None
    if bias_std is not None:
        if integer_values:
            bias = rng.integers(-8, 9, size=M).astype(np.float32)
        else:
            bias = (rng.standard_normal(M) * bias_std).astype(np.float32)
    return Layer(M, N, B, row_perm, col_perm, tile_list, vals, bias, act, seed), rng


def draw_x(rng: np.random.Generator, batch: int, N: int, lo: float, hi: float,
           dtype: str, integer_values: bool = False) -> np.ndarray:
    if integer_values:
        x = rng.integers(-2, 3, size=(batch, N)).astype(np.float32)
    else:
        x = rng.uniform(lo, hi, size=(batch, N)).astype(np.float32)
    return x.astype(np.float16) if dtype == "f16" else x


# --------------------------------------------------------------------------- #
# The five workloads.  ``scale`` < 1 shrinks the matrix edge (kept a multiple of
# B) for tests that need the oracle to finish quickly; scale=1 is the full size.
# --------------------------------------------------------------------------- #

def config1(batch: int = 1, scale: float = 1.0, **kw) -> Workload:
    """1024 x 1024 fp32, B=32, 8 of 32 tiles per block-row, bias, ReLU."""
    B = 32
    n = max(B * 8, int(1024 * scale) // B * B)
    lay, rng = make_layer(_seed(1, 0), n, n, B, wdtype="f32", tiles="balanced", k=8,
                          bias_std=0.1, act=ACT_RELU, **kw)
    x = draw_x(rng, batch, n, -1.0, 1.0, "f32", kw.get("integer_values", False))
    return Workload("cfg1_fc1024_f32_b32_d25", [lay], x)


def config2(batch: int = 1, scale: float = 1.0, **kw) -> Workload:
    """4096 x 4096 fp32, B=64, 8 of 64 tiles per block-row, no bias, identity."""
    B = 64
    n = max(B * 8, int(4096 * scale) // B * B)
    lay, rng = make_layer(_seed(2, 0), n, n, B, wdtype="f32", tiles="balanced", k=8,
                          act=ACT_IDENTITY, **kw)
    x = draw_x(rng, batch, n, -1.0, 1.0, "f32", kw.get("integer_values", False))
    return Workload("cfg2_fc4096_f32_b64_d12.5", [lay], x)


def config3(batch: int = 1, scale: float = 1.0, **kw) -> Workload:
    """9216 -> 4096 -> 4096 -> 1000, fp16 weights/activations, B=32, densities
    10/10/25 % drawn over the whole tile grid, bias, ReLU between layers."""
    B = 32
    d0 = max(B * 4, int(9216 * scale) // B * B)
    d1 = max(B * 4, int(4096 * scale) // B * B)
    d3 = 1000 if scale == 1.0 else max(B * 2 - 7, int(1000 * scale))
    dims = [d0, d1, d1, d3]
    dens = [0.10, 0.10, 0.25]
    acts = [ACT_RELU, ACT_RELU, ACT_IDENTITY]
    layers, rng0 = [], None
    for l in range(3):
        lay, rng = make_layer(_seed(3, l), dims[l + 1], dims[l], B, wdtype="f16",
                              tiles="uniform", density=dens[l], bias_std=0.1,
                              act=acts[l], **kw)
        layers.append(lay)
        if l == 0:
            rng0 = rng
    x = draw_x(rng0, batch, dims[0], 0.0, 1.0, "f16", kw.get("integer_values", False))
    return Workload("cfg3_chain_9216_4096_4096_1000_f16_b32", layers, x)


def config4(steps: int = 256, scale: float = 1.0, **kw) -> Workload:
    """LSTM gate matrix 4H x (I+H), H = I = 2048, fp16, B=16, 51 of 256 tiles
    per block-row (round(0.2*256)); x holds ``steps`` input vectors."""
    B = 16
    H = max(B * 2, int(2048 * scale) // B * B)
    I = H
    Nb = (I + H) // B
    k = int(round(0.2 * Nb))
    lay, rng = make_layer(_seed(4, 0), 4 * H, I + H, B, wdtype="f16", tiles="balanced",
                          k=k, act=ACT_IDENTITY, **kw)
    x = draw_x(rng, steps, I, -1.0, 1.0, "f16")
    return Workload("cfg4_lstm_h2048_f16_b16_d20", [lay], x, extra={"H": H, "I": I})


def config5(k: int = 128, batch: int = 1, scale: float = 1.0, **kw) -> Workload:
    """8192 x 8192 fp16, B=64, k of 128 tiles per block-row (k=128 is density 1),
    no bias, identity."""
    B = 64
    n = max(B * 4, int(8192 * scale) // B * B)
    Nb = n // B
    kk = max(1, int(round(k * Nb / 128)))
    lay, rng = make_layer(_seed(5, 0) + k, n, n, B, wdtype="f16", tiles="balanced", k=kk,
                          act=ACT_IDENTITY, **kw)
    x = draw_x(rng, batch, n, -1.0, 1.0, "f16", kw.get("integer_values", False))
    return Workload(f"cfg5_fc8192_f16_b64_k{k}", [lay], x)


# --------------------------------------------------------------------------- #
# Irregular block structure (Section 4.1.5): W_piv holds rectangles of any size.
# --------------------------------------------------------------------------- #

@dataclass
class BlockLayer:
    M: int
    N: int
    B: int                        # grid the library lays the blocks over; fixes the padded sizes
    row_perm: np.ndarray          # int32 [ceil(M/B)*B]
    col_perm: np.ndarray          # int32 [ceil(N/B)*B]
    blocks: np.ndarray            # int32 [nb, 4] = first pivoted row, first pivoted column, height, width
    block_values: np.ndarray      # float32 or float16, the blocks one after the other, each row-major
    bias: Optional[np.ndarray]
    act: int = ACT_IDENTITY
    seed: int = 0

    @property
    def wdtype(self) -> str:
        return "f16" if self.block_values.dtype == np.float16 else "f32"

    @property
    def block_bytes(self) -> int:
        return int(self.block_values.size * self.block_values.dtype.itemsize)


def _block_values(rng, blocks, N, wdtype, integer_values):
    n = int(np.sum(blocks[:, 2].astype(np.int64) * blocks[:, 3])) if len(blocks) else 0
    if integer_values:
        v = rng.integers(-4, 5, size=n).astype(np.float32)
    else:
        v = (rng.standard_normal(n) / np.sqrt(N)).astype(np.float32)
    return v.astype(np.float16) if wdtype == "f16" else v


def paper_square(size: int, blocks_per_side: int, B: int, *, wdtype: str = "f32", batch: int = 1,
                 integer_values: bool = False, seed: Optional[int] = None) -> Workload:
    """The geometry the paper measures (Section 5): a size x size matrix with
    ``blocks_per_side`` identical square blocks of edge size/blocks_per_side on the
    diagonal of the pivoted matrix (fill-in = 1/blocks_per_side), random index arrays,
    x ~ U(-1, 1), no bias."""
    edge = size // blocks_per_side
    if edge * blocks_per_side != size:
        raise ValueError("size must be a multiple of blocks_per_side")
    seed = _seed(6, 0) + size + blocks_per_side if seed is None else seed
    rng = np.random.default_rng(seed)
    pad = -(-size // B) * B
    row_perm = rng.permutation(pad).astype(np.int32)
    col_perm = rng.permutation(pad).astype(np.int32)
    blocks = np.array([[k * edge, k * edge, edge, edge] for k in range(blocks_per_side)], dtype=np.int32)
    vals = _block_values(rng, blocks, size, wdtype, integer_values)
    lay = BlockLayer(size, size, B, row_perm, col_perm, blocks, vals, None, ACT_IDENTITY, seed)
    x = draw_x(rng, batch, size, -1.0, 1.0, wdtype, integer_values)
    return Workload(f"paper_square_{size}_fill{100.0 / blocks_per_side:g}_{wdtype}_grid{B}", [lay], x)


def irregular_blocks(seed: int, M: int, N: int, B: int, *, wdtype: str, n_row_cuts: int, n_col_cuts: int,
                     keep: float, batch: int = 1, bias_std: Optional[float] = None, act: int = ACT_IDENTITY,
                     integer_values: bool = False, aligned: bool = False) -> Workload:
    """Rectangles of mixed sizes: random cut lines split the padded pivoted matrix into a grid of
    unequal cells and a random fraction ``keep`` of the cells become blocks (so blocks differ in height
    and width, several share their rows, none overlap).  ``aligned`` puts the cuts on multiples of B."""
    rng = np.random.default_rng(seed)
    Mp, Np = -(-M // B) * B, -(-N // B) * B
    row_perm = rng.permutation(Mp).astype(np.int32)
    col_perm = rng.permutation(Np).astype(np.int32)

    def cuts(n, length):
        if aligned:
            inner = rng.choice(np.arange(1, length // B), size=min(n, length // B - 1), replace=False) * B
        else:
            inner = rng.choice(np.arange(1, length), size=min(n, length - 1), replace=False)
        return np.concatenate([[0], np.sort(inner), [length]]).astype(np.int64)

    rc, cc = cuts(n_row_cuts, Mp), cuts(n_col_cuts, Np)
    cells = [(i, j) for i in range(len(rc) - 1) for j in range(len(cc) - 1)]
    chosen = rng.permutation(len(cells))[:max(1, int(round(keep * len(cells))))]
    blocks = np.array([[rc[cells[c][0]], cc[cells[c][1]], rc[cells[c][0] + 1] - rc[cells[c][0]],
                        cc[cells[c][1] + 1] - cc[cells[c][1]]] for c in chosen], dtype=np.int32)
    vals = _block_values(rng, blocks, N, wdtype, integer_values)
    bias = None
    if bias_std is not None:
        bias = rng.integers(-8, 9, size=M).astype(np.float32) if integer_values else \
            (rng.standard_normal(M) * bias_std).astype(np.float32)
    lay = BlockLayer(M, N, B, row_perm, col_perm, blocks, vals, bias, act, seed)
    x = draw_x(rng, batch, N, -1.0, 1.0, wdtype, integer_values)
    return Workload(f"irregular_{M}x{N}_{wdtype}_grid{B}", [lay], x)


# The 4 x 4 example worked by hand (values are part of the test fixtures, not drawn).
def hand_example() -> Layer:
    return Layer(
        M=4, N=4, B=2,
        row_perm=np.array([2, 0, 3, 1], dtype=np.int32),
        col_perm=np.array([1, 3, 0, 2], dtype=np.int32),
        tile_list=np.array([[0, 1], [1, 0]], dtype=np.int32),
        tile_values=np.array([[[1, 2], [3, 4]], [[5, 6], [7, 8]]], dtype=np.float32),
        bias=np.array([0.5, -0.5, 1.0, -20.0], dtype=np.float32),
        act=ACT_RELU,
    )
