"""Seeded synthetic inputs for the SDVG hot path (Sec. 4.1 workload shapes).

This module only draws random numbers and packs them; it contains none of the
method's arithmetic (no RoPE, no softmax, no routing rule, no ring indexing).
Both the CUDA tests/bench and the CPU oracle tests read inputs from here so
that they see the same bits.

bf16 tensors are carried as ``numpy.uint16`` bit patterns.  Streams are
``numpy.random.Generator(PCG64(SeedSequence([...])))`` keyed by
``(config_seed, block, source, tensor)`` so that any tensor can be regenerated
alone.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

# tensor ids
Q, K, V = 0, 1, 2
# source ids: who produced the tensor in the speculative schedule
SRC_DRAFT_STEP = 0      # drafter denoise step s (source = SRC_DRAFT_STEP + s)
SRC_DRAFT_CLEAN = 8     # drafter's final K/V of the block
SRC_TARGET_STEP = 16    # target denoise step s (rejected block)
SRC_TARGET_CLEAN = 24   # target's final K/V after regeneration
SRC_ACCEPT_CLEAN = 32   # target-shaped K/V of an accepted draft block


@dataclass(frozen=True)
class Shape:
    """One model shape of the workload (Sec. 4.1: 3 latent frames per block)."""
    name: str
    heads: int
    head_dim: int
    frames: int          # latent frames per block
    grid_h: int
    grid_w: int
    slots: int           # ring slots = visible prior blocks + self

    @property
    def block_tokens(self) -> int:
        return self.frames * self.grid_h * self.grid_w

    @property
    def scale(self) -> float:
        return 1.0 / float(np.sqrt(np.float64(self.head_dim)))


TINY = Shape("tiny", heads=2, head_dim=64, frames=2, grid_h=4, grid_w=8, slots=3)
WAN_1_3B = Shape("wan1.3b-drafter", heads=12, head_dim=128, frames=3, grid_h=30, grid_w=52, slots=3)
WAN_14B = Shape("wan14b-target", heads=40, head_dim=128, frames=3, grid_h=30, grid_w=52, slots=7)


def _rng(*key: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(np.random.SeedSequence([int(k) for k in key])))


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Pack float32 values to bf16 bit patterns, round-to-nearest-even (finite inputs)."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + bias) >> np.uint32(16)).astype(np.uint16)


def normal_bf16(shape, *key: int, mean: float = 0.0, std: float = 1.0) -> np.ndarray:
    """bf16 bit patterns of N(mean, std) samples, stream keyed by ``key``."""
    x = _rng(*key).standard_normal(size=shape, dtype=np.float32)
    if std != 1.0:
        x *= np.float32(std)
    if mean != 0.0:
        x += np.float32(mean)
    return f32_to_bf16_bits(x)


def block_tensor(shape: Shape, seed: int, block: int, source: int, tensor: int,
                 std: float = 1.0) -> np.ndarray:
    """One [block_tokens, heads, head_dim] bf16 tensor ~ N(0, std)."""
    return normal_bf16((shape.block_tokens, shape.heads, shape.head_dim),
                       seed, block, source, tensor, std=std)


class TensorPool:
    """Cheap per-(block, source, tensor) tensors for the long sweeps.

    A pool of ``n`` base tensors is drawn once; tensor (block, source, tensor)
    is base ``i`` rolled by ``r`` elements along the flattened axis, with
    (i, r) drawn from the key's own stream.  Every tensor keeps the N(0,1)
    value distribution and distinct keys give distinct bits, at the cost of a
    memcpy instead of a fresh 24M-sample draw.
    """

    def __init__(self, shape: Shape, seed: int, n: int = 4):
        self.shape = shape
        self.seed = seed
        self.base = [block_tensor(shape, seed, 1_000_000 + i, 0, 0).reshape(-1) for i in range(n)]

    def get(self, block: int, source: int, tensor: int) -> np.ndarray:
        g = _rng(self.seed, block, source, tensor, 77)
        i = int(g.integers(0, len(self.base)))
        # roll by a multiple of head_dim so rows stay rows
        nrows = self.base[i].size // self.shape.head_dim
        r = int(g.integers(1, nrows)) * self.shape.head_dim
        out = np.roll(self.base[i], r)
        return out.reshape(self.shape.block_tokens, self.shape.heads, self.shape.head_dim)


def uniform_scores(num_blocks: int, frames: int, lo: float, hi: float, *key: int) -> np.ndarray:
    """fp32 per-frame scores ~ U(lo, hi), shape [num_blocks, frames]."""
    return _rng(*key).uniform(lo, hi, size=(num_blocks, frames)).astype(np.float32)


def normal_scores(num_blocks: int, frames: int, mean: float, std: float, *key: int) -> np.ndarray:
    """fp32 per-frame scores ~ N(mean, std), shape [num_blocks, frames]."""
    return (_rng(*key).standard_normal(size=(num_blocks, frames)) * std + mean).astype(np.float32)


# Accept rates reported in Table 1 (P(block minimum >= tau), block 0 excluded).
TABLE1_TAU = np.array([-2.5, -2.0, -1.5, -1.0, -0.9, -0.8, -0.7])
TABLE1_ACCEPT = np.array([0.889, 0.875, 0.834, 0.780, 0.764, 0.749, 0.731])


def calibrated_scores(num_blocks: int, frames: int, *key: int) -> np.ndarray:
    """Scores whose per-block minimum follows the accept-rate curve of Table 1.

    The block minimum is drawn by inverting a piecewise-linear survival
    function through the seven (tau, accept-rate) points of Table 1, extended
    linearly to 1 at tau=-4 and to 0 at tau=+0.5; the other frames sit a
    non-negative jitter above it, and the position of the worst frame is
    random.  Only the distribution of inputs is shaped here; the routing rule
    itself lives elsewhere.
    """
    g = _rng(*key)
    taus = np.concatenate([[-4.0], TABLE1_TAU, [0.5]])
    surv = np.concatenate([[1.0], TABLE1_ACCEPT, [0.0]])
    u = g.uniform(0.0, 1.0, size=num_blocks)
    # survival is decreasing in tau: invert on the reversed arrays
    qmin = np.interp(u, surv[::-1], taus[::-1])
    jitter = g.exponential(0.4, size=(num_blocks, frames))
    pos = g.integers(0, frames, size=num_blocks)
    jitter[np.arange(num_blocks), pos] = 0.0
    return (qmin[:, None] + jitter).astype(np.float32)


def ragged_scores(frame_counts, mean: float, std: float, *key: int):
    """Ragged per-block scores: returns (flat fp32 scores, int32 offsets[B+1])."""
    counts = np.asarray(frame_counts, dtype=np.int64)
    offsets = np.zeros(counts.size + 1, dtype=np.int32)
    offsets[1:] = np.cumsum(counts)
    flat = (_rng(*key).standard_normal(size=int(offsets[-1])) * std + mean).astype(np.float32)
    return flat, offsets
