"""Seeded synthetic inputs shaped like the paper's MT decoding workloads.

This module serves both the CUDA path and the CPU oracle, so it holds none of
the method's arithmetic: only lengths, Gaussian activations, the rounding of
those activations to the storage dtype, and the named workload shapes.

The paper decodes with 6-layer decoders, 8 heads, beam 4 and sentences of at
most 80 words (Section 4.1).  Its test sets are not available here; Gaussian
activations with the same tensor shapes and a uniform source-length mix stand
in for them.

Every tensor is drawn from its own counter-based stream keyed by
``(seed, tag, step, layer)``, so any step of a long decode can be produced
without drawing its predecessors, and the draw never depends on which consumer
asks first.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict, List, Tuple

import numpy as np

F32 = "f32"
BF16 = "bf16"

# stream tags (arbitrary distinct integers)
TAG_LEN, TAG_Q_SELF, TAG_K_SELF, TAG_V_SELF = 1, 2, 3, 4
TAG_Q_ENC, TAG_K_MEM, TAG_V_MEM, TAG_X_AAN, TAG_PREFIX, TAG_PARENT = 5, 6, 7, 8, 9, 10
TAG_S_FULL = 11


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bfloat16 (ties to even); result is float32."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32).astype(np.uint64)
    bias = ((u >> 16) & 1) + 0x7FFF
    r = ((u + bias) >> 16) << 16
    return r.astype(np.uint32).view(np.float32).reshape(x.shape)


def bf16_bits(x: np.ndarray) -> np.ndarray:
    """Upper 16 bits of float32 values that are already exactly representable in bfloat16."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    return (x.view(np.uint32) >> 16).astype(np.uint16).reshape(x.shape)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    b = np.ascontiguousarray(b, dtype=np.uint16)
    return (b.astype(np.uint32) << 16).view(np.float32).reshape(b.shape)


def normal(seed: int, tag: int, step: int, layer: int, shape, dtype: str) -> np.ndarray:
    """Standard-normal float32 tensor, rounded to ``dtype`` (returned as float32)."""
    rng = np.random.default_rng([int(seed), int(tag), int(step), int(layer)])
    x = rng.standard_normal(size=shape, dtype=np.float32)
    if dtype == BF16:
        x = round_to_bf16(x)
    return x


def integers(seed: int, tag: int, lo: int, hi: int, n: int) -> np.ndarray:
    """``n`` integers uniform in ``[lo, hi]`` (both ends included), int32."""
    rng = np.random.default_rng([int(seed), int(tag)])
    return rng.integers(lo, hi + 1, size=n, dtype=np.int64).astype(np.int32)


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    dtype: str
    n_layers: int
    n_heads: int
    d_head: int
    n_sent: int
    beam: int
    self_blocks: Tuple[int, ...]      # block sizes, bottom-up; ignored when self_is_aan
    encdec_blocks: Tuple[int, ...]
    src_lo: int
    src_hi: int
    tgt_rule: str                     # "ratio1.1" | "fixed"
    tgt_fixed: int
    ragged_prefix: bool
    self_is_aan: bool
    seed: int

    @property
    def n_seqs(self) -> int:
        return self.n_sent * self.beam

    @property
    def d_model(self) -> int:
        return self.n_heads * self.d_head

    @property
    def elem_bytes(self) -> int:
        return 4 if self.dtype == F32 else 2

    def src_lens(self) -> np.ndarray:
        """Source length of every sentence."""
        return integers(self.seed, TAG_LEN, self.src_lo, self.src_hi, self.n_sent)

    def tgt_lens(self) -> np.ndarray:
        """Number of decode steps of every sentence (all its beams run that long)."""
        if self.tgt_rule == "fixed":
            return np.full(self.n_sent, self.tgt_fixed, dtype=np.int32)
        # ceil(1.1 * Ls) in exact integer arithmetic
        ls = self.src_lens().astype(np.int64)
        return ((11 * ls + 9) // 10).astype(np.int32)

    def max_src_len(self) -> int:
        return int(self.src_hi)

    def max_tgt_len(self) -> int:
        if self.tgt_rule == "fixed":
            return int(self.tgt_fixed)
        return int((11 * self.src_hi + 9) // 10)

    def prefix_lens(self) -> np.ndarray:
        """Positions already cached per *sequence* before the first timed/checked step."""
        t = np.repeat(self.tgt_lens(), self.beam)
        if not self.ragged_prefix:
            return np.zeros_like(t)
        rng = np.random.default_rng([int(self.seed), TAG_PREFIX])
        u = rng.integers(0, 1 << 30, size=t.shape[0], dtype=np.int64)
        return (u % t.astype(np.int64)).astype(np.int32)      # uniform in [0, T_s)


WORKLOADS: Dict[str, Workload] = {
    # the five configurations, in order
    "tiny": Workload("tiny", F32, 6, 8, 64, 1, 4, (2, 2, 2), (3, 3), 16, 16, "fixed", 16, False, False, 0),
    "base": Workload("base", BF16, 6, 8, 64, 64, 4, (2, 2, 2), (6,), 10, 60, "ratio1.1", 0, False, False, 1),
    "big": Workload("big", BF16, 6, 16, 64, 128, 4, (3, 3), (6,), 20, 100, "ratio1.1", 0, True, False, 2),
    "long": Workload("long", BF16, 12, 8, 64, 32, 4, (4, 4, 4), (12,), 512, 512, "fixed", 512, False, False, 3),
    "aan": Workload("aan", BF16, 6, 8, 64, 64, 4, (1, 1, 1, 1, 1, 1), (2, 2, 2), 10, 60, "fixed", 80, False, True, 4),
}


def unshared(w: Workload) -> Workload:
    """Same workload with sharing switched off (every block has one layer)."""
    ones = tuple([1] * w.n_layers)
    return dataclasses.replace(w, name=w.name + "-unshared", self_blocks=ones, encdec_blocks=ones)


def scaled(w: Workload, n_sent: int, name: str | None = None) -> Workload:
    """Same workload with fewer (or more) sentences; lengths keep the same distribution."""
    return dataclasses.replace(w, n_sent=int(n_sent), name=name or f"{w.name}-{n_sent}")


def self_qkv(w: Workload, step: int, layer: int):
    """q, k, v of one decode step for one layer: each ``[n_seqs, H, d_h]`` float32."""
    shp = (w.n_seqs, w.n_heads, w.d_head)
    return (normal(w.seed, TAG_Q_SELF, step, layer, shp, w.dtype),
            normal(w.seed, TAG_K_SELF, step, layer, shp, w.dtype),
            normal(w.seed, TAG_V_SELF, step, layer, shp, w.dtype))


def encdec_q(w: Workload, step: int, layer: int) -> np.ndarray:
    return normal(w.seed, TAG_Q_ENC, step, layer, (w.n_seqs, w.n_heads, w.d_head), w.dtype)


def encoder_memory(w: Workload, layer: int):
    """Encoder-memory keys and values of one layer, padded: ``[n_sent, max_src, H, d_h]``.

    Rows at or beyond a sentence's source length are drawn too (so the stream
    does not depend on the lengths) but no consumer may read them.
    """
    shp = (w.n_sent, w.max_src_len(), w.n_heads, w.d_head)
    return (normal(w.seed, TAG_K_MEM, 0, layer, shp, w.dtype),
            normal(w.seed, TAG_V_MEM, 0, layer, shp, w.dtype))


def aan_x(w: Workload, step: int, layer: int) -> np.ndarray:
    return normal(w.seed, TAG_X_AAN, step, layer, (w.n_seqs, w.d_model), w.dtype)


def beam_parents(w: Workload, step: int, keep_prob: float = 0.0) -> np.ndarray:
    """A parent beam (0..beam-1) for every sequence, as beam search would pick: with probability
    ``keep_prob`` a hypothesis continues itself, otherwise its parent is drawn uniformly."""
    rng = np.random.default_rng([int(w.seed), TAG_PARENT, int(step)])
    parent = rng.integers(0, w.beam, size=w.n_seqs, dtype=np.int64).astype(np.int32)
    if keep_prob > 0.0:
        keep = rng.random(w.n_seqs) < keep_prob
        parent = np.where(keep, np.arange(w.n_seqs) % w.beam, parent).astype(np.int32)
    return parent


def self_prefill(w: Workload, layer: int):
    """Keys and values already cached before the first checked step: ``[n_seqs, max_tgt, H, d_h]``.

    Rows at or beyond a sequence's prefix length are drawn but never used.
    """
    shp = (w.n_seqs, w.max_tgt_len(), w.n_heads, w.d_head)
    return (normal(w.seed, TAG_PREFIX, 1, layer, shp, w.dtype),
            normal(w.seed, TAG_PREFIX, 2, layer, shp, w.dtype))
