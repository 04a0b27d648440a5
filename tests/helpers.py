"""Shared test helpers: driving the oracle over a synthetic workload (no CUDA here)."""
from __future__ import annotations

import itertools

import numpy as np

from oracle import san_oracle as so
from paper_1906_11024_b200 import synth


def compositions(M):
    """Every way to cut M layers into runs of adjacent layers (2^(M-1) policies)."""
    out = []
    for cuts in itertools.product([0, 1], repeat=M - 1):
        sizes, run = [], 1
        for c in cuts:
            if c:
                sizes.append(run)
                run = 1
            else:
                run += 1
        sizes.append(run)
        out.append(tuple(sizes))
    return out


def make_oracle(w: synth.Workload, shared_context=False) -> so.Oracle:
    return so.Oracle(w.n_layers, w.n_heads, w.d_head, w.n_sent, w.beam, w.max_tgt_len(), w.max_src_len(),
                     w.self_blocks, w.encdec_blocks, shared_context)


def load_memory(o: so.Oracle, w: synth.Workload):
    """Fill the oracle's encoder memory from the workload (K only for block-first layers)."""
    src = w.src_lens()
    first = set(np.cumsum((0,) + tuple(w.encdec_blocks))[:-1].tolist())
    for l in range(w.n_layers):
        K, V = synth.encoder_memory(w, l)
        for g in range(w.n_sent):
            o.mem_set(l, g, K[g, :src[g]] if l in first else None, V[g, :src[g]])
    return src
