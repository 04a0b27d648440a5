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


# --------------------------------------------------------------------------- error measures
def normwise_err(x: np.ndarray, y: np.ndarray) -> float:
    """max over vectors (last axis) of ||x - y||_inf / ||y||_inf, y being the reference."""
    num = np.abs(x.astype(np.float64) - y).max(-1)
    den = np.abs(y).max(-1)
    den = np.where(den > 0, den, 1.0)
    return float((num / den).max()) if num.size else 0.0


def weights_err(S: np.ndarray, ref: np.ndarray, floor: float = 1e-7) -> float:
    """max element-wise |S - ref| / max(ref, floor)."""
    if S.size == 0:
        return 0.0
    return float((np.abs(S.astype(np.float64) - ref) / np.maximum(ref, floor)).max())


TOL = {"f32": 1e-5, "bf16": 1e-2}     # output tolerance per input dtype
TOL_S = 1e-5                          # S is float32 computed from exactly representable inputs


class OracleRun:
    """Drives the oracle through the same decode schedule as the CUDA driver."""

    def __init__(self, w: synth.Workload, shared_context=False):
        self.w = w
        self.o = make_oracle(w, shared_context)
        self.shared_context = shared_context
        self.self_first = list(np.cumsum((0,) + tuple(w.self_blocks))[:-1])
        self.enc_first = list(np.cumsum((0,) + tuple(w.encdec_blocks))[:-1])
        self.src = load_memory_for(self.o, w, shared_context)

    def prefill(self, seq_ids, n_rows):
        """Rows [0, n_rows[i]) of every listed sequence from the workload's prefill draw."""
        w = self.w
        for l in range(w.n_layers):
            K, V = synth.self_prefill(w, l)
            seq_ids = np.asarray(seq_ids)
            n_rows = np.asarray(n_rows)
            for p in range(int(n_rows.max()) if len(n_rows) else 0):
                ids = seq_ids[n_rows > p]
                self.o.self_append(l, ids, np.full(len(ids), p), K[ids, p] if l in self.self_first else None, V[ids, p])

    def step(self, host, seq_ids, pos, want_S=True):
        """One decode step with the host inputs returned by ``Decoder.fill_step_inputs``.
        Returns dict with S_self [N_s][n][H][ld], O_self [M][n][H][dh], S_enc, O_enc (float64)."""
        w, o = self.w, self.o
        seq_ids = np.asarray(seq_ids, np.int32)
        pos = np.asarray(pos, np.int32)
        out = {}
        if w.self_is_aan:
            out["O_self"] = np.stack([o.aan_step(l, seq_ids, pos + 1, host["x"][l]).reshape(len(seq_ids), w.n_heads, w.d_head)
                                      for l in range(w.n_layers)])
        else:
            S_list, O_list = [], []
            for l in range(w.n_layers):
                first = l in self.self_first
                b = self.self_first.index(l) if first else None
                o.self_append(l, seq_ids, pos, host["k"][b] if first else None, host["v"][l])
            for l in range(w.n_layers):
                first = l in self.self_first
                b = self.self_first.index(l) if first else None
                S, O = o.self_attend(l, seq_ids, pos + 1, host["q"][b] if first else None, want_S=first and want_S)
                if first and want_S:
                    S_list.append(S)
                O_list.append(O)
            out["S_self"] = np.stack(S_list) if S_list else None
            out["O_self"] = np.stack(O_list)
        beams = host["beams"]
        S_list, O_list = [], []
        for l in range(w.n_layers):
            first = l in self.enc_first
            c = self.enc_first.index(l) if first else None
            S, O = o.encdec_attend(l, beams, host["q_enc"][c] if first else None, want_S=first and want_S)
            if first and want_S:
                S_list.append(S)
            if first or not self.shared_context:
                O_list.append(O)
        out["S_enc"] = np.stack(S_list) if S_list else None
        out["O_enc"] = np.stack(O_list)
        return out


def load_memory_for(o, w, shared_context):
    """Encoder memory into the oracle.  With shared context (Eq. 5) only block-first layers own
    memory; the oracle's upper layers return the block's stored output and never read any."""
    src = w.src_lens()
    first = set(np.cumsum((0,) + tuple(w.encdec_blocks))[:-1].tolist())
    for l in range(w.n_layers):
        if shared_context and l not in first:
            continue
        K, V = synth.encoder_memory(w, l)
        for g in range(w.n_sent):
            o.mem_set(l, g, K[g, :src[g]] if l in first else None, V[g, :src[g]])
    return src


def cached_row_order(rows_bits: np.ndarray, pos, dtype: str) -> np.ndarray:
    """How the library stores cache rows: bf16 rows have their eight 16-byte chunks permuted,
    logical chunk c of the row at position ``pos`` sitting at chunk ``c ^ (pos & 7)``; float32
    rows are stored as they are.  ``rows_bits``: [..., 64] bit patterns; ``pos``: broadcastable
    to the leading axes."""
    if dtype != synth.BF16:
        return rows_bits
    x = rows_bits.reshape(rows_bits.shape[:-1] + (8, 8))
    pos = np.broadcast_to(np.asarray(pos), rows_bits.shape[:-1])
    phys = np.arange(8)
    src = phys[None, :] ^ (pos.reshape(-1, 1) & 7)            # physical chunk pc holds logical pc ^ (pos & 7)
    flat = x.reshape(-1, 8, 8)
    out = np.take_along_axis(flat, src[:, :, None], axis=1)
    return out.reshape(rows_bits.shape)
