"""Seeded synthetic inputs for the memory-slice hot path.

This module only draws random inputs and describes workloads: sequence lengths, which logical
blocks of a sequence live in the lent arena, free-list permutations, N(0,1) bf16 values. It holds
none of the method's arithmetic (no gather, attention or migration), so both the CUDA path and
the CPU oracle can be fed from it without sharing code.

The workloads mirror the shapes of the paper's serving experiments (Section 6.1: variable-length
requests, continuous batching); the paper's own traces are not available, so lengths are drawn from
the stated uniform / lognormal ranges instead.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional

import numpy as np

BLOCK_TOKENS = 16
HEAD_DIM = 128

AUTO, LOCAL, LENT = 0, 1, 2


@dataclass
class Workload:
    """A named decode workload: shapes, batch and placement rule."""
    name: str
    num_layers: int
    num_q_heads: int
    num_kv_heads: int
    batch: int
    len_lo: int
    len_hi: int
    lent_fraction: float
    ring_slots: int = 2
    head_dim: int = HEAD_DIM
    block_tokens: int = BLOCK_TOKENS

    @property
    def block_bytes(self) -> int:
        return 2 * self.block_tokens * self.num_kv_heads * self.head_dim * 2

    @property
    def kv_bytes_per_token(self) -> int:
        return 2 * self.num_kv_heads * self.head_dim * 2


# The decode workloads of the benchmark definition.
WORKLOADS: Dict[str, Workload] = {
    # 1: single-layer correctness case, plain multi-head attention.
    "single_layer_mha": Workload("single_layer_mha", 1, 8, 8, 4, 100, 500, 0.25),
    # 2: Llama-3-8B-shaped decode.
    "llama3_8b_decode": Workload("llama3_8b_decode", 32, 32, 8, 64, 512, 4096, 0.40),
    # 4: Llama-3-70B-shaped per-GPU decode.
    "llama3_70b_decode": Workload("llama3_70b_decode", 80, 64, 8, 32, 4096, 8192, 0.50),
}


def draw_lengths(rng: np.random.Generator, batch: int, lo: int, hi: int) -> np.ndarray:
    """Sequence lengths, uniform over the integers lo..hi inclusive."""
    return rng.integers(lo, hi + 1, size=batch).astype(np.int64)


def blocks_for(length: int, block_tokens: int = BLOCK_TOKENS) -> int:
    return (int(length) + block_tokens - 1) // block_tokens


def choose_lent(rng: np.random.Generator, num_blocks: int, fraction: float) -> np.ndarray:
    """Boolean mask over a sequence's logical blocks: exactly round(fraction * nb) are lent."""
    n_lent = int(round(fraction * num_blocks))
    mask = np.zeros(num_blocks, dtype=bool)
    if n_lent > 0:
        mask[rng.choice(num_blocks, size=n_lent, replace=False)] = True
    return mask


def free_order(rng: np.random.Generator, n: int) -> np.ndarray:
    """A seeded permutation of 0..n-1: the order in which a free list hands out block ids."""
    return rng.permutation(n).astype(np.uint32)


@dataclass
class Placement:
    """Lengths and per-block tier hints of one batch, plus capacities that fit it."""
    lengths: np.ndarray                      # [batch] tokens
    hints: List[np.ndarray]                  # per sequence: LOCAL / LENT per logical block
    local_blocks: int
    lent_blocks: int
    staging_blocks: int                      # lent blocks in use by the whole batch
    local_free_order: Optional[np.ndarray] = None
    lent_free_order: Optional[np.ndarray] = None
    seq_ids: List[int] = field(default_factory=list)

    @property
    def total_blocks(self) -> int:
        return int(sum(len(h) for h in self.hints))

    @property
    def total_tokens(self) -> int:
        return int(self.lengths.sum())


def make_placement(wl: Workload, seed: int, slack_blocks: int = 16, permute: bool = True,
                   lengths: Optional[np.ndarray] = None) -> Placement:
    """Draw lengths, choose the lent blocks of every sequence and size both arenas."""
    rng = np.random.default_rng(seed)
    if lengths is None:
        lengths = draw_lengths(rng, wl.batch, wl.len_lo, wl.len_hi)
    hints = []
    n_local = n_lent = 0
    for n in lengths:
        nb = blocks_for(n, wl.block_tokens)
        mask = choose_lent(rng, nb, wl.lent_fraction)
        hints.append(np.where(mask, LENT, LOCAL).astype(np.int32))
        n_lent += int(mask.sum())
        n_local += nb - int(mask.sum())
    local_blocks = n_local + slack_blocks
    lent_blocks = n_lent + slack_blocks
    lo = free_order(rng, local_blocks) if permute else None
    ro = free_order(rng, lent_blocks) if permute else None
    return Placement(np.asarray(lengths, np.int64), hints, local_blocks, lent_blocks, n_lent, lo, ro,
                     list(range(len(lengths))))


def normal_bf16_bits(rng: np.random.Generator, shape) -> np.ndarray:
    """N(0,1) samples rounded to bf16 (nearest even), returned as uint16 bit patterns."""
    x = rng.standard_normal(size=shape, dtype=np.float32)
    u = x.view(np.uint32)
    lsb = (u >> 16) & 1
    return ((u + 0x7FFF + lsb) >> 16).astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns to float32 (a format change, not arithmetic)."""
    return (bits.astype(np.uint32) << 16).view(np.float32)


BF16_NAN = np.uint16(0x7FC0)


# ---------------------------------------------------------------------------------------------
# Bursty growth workload (Poisson arrivals, lognormal output lengths)
# ---------------------------------------------------------------------------------------------
@dataclass
class Arrival:
    step: int
    prompt_len: int
    output_len: int


def bursty_arrivals(seed: int, steps: int, rate: float = 8.0, prompt_lo: int = 256,
                    prompt_hi: int = 2048, out_median: float = 512.0, out_sigma: float = 1.0,
                    out_clip: int = 8192) -> List[Arrival]:
    """Requests arriving per decode step ~ Poisson(rate); prompts uniform; outputs lognormal."""
    rng = np.random.default_rng(seed)
    out: List[Arrival] = []
    for t in range(steps):
        for _ in range(int(rng.poisson(rate))):
            p = int(rng.integers(prompt_lo, prompt_hi + 1))
            o = int(np.clip(round(float(rng.lognormal(np.log(out_median), out_sigma))), 1, out_clip))
            out.append(Arrival(t, p, o))
    return out
