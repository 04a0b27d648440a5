"""Decode-step driver over the C ABI: device buffers, uploads and the call sequence.

This is plumbing for tests, the smoke check and the benchmark: torch supplies device
memory and streams, every attention step runs in the library's kernels.  A decode step
for a synthetic workload (every layer's q/k/v known up front) is

    san_cache_append(SELF, all layers)                      one launch
    per self block:    san_attn_weights, san_attn_apply      (all layers of the block)
    per enc-dec block: san_attn_weights, san_attn_apply
  or, with average attention in place of self-attention,
    san_aan_step(all layers) followed by the enc-dec calls.
"""
from __future__ import annotations

import dataclasses
from typing import List, Optional

import numpy as np
import torch

from . import binding as B
from . import synth


def to_device(x_f32: np.ndarray, dtype: str, device) -> torch.Tensor:
    """float32 host values (already rounded to ``dtype``) -> device tensor of that dtype."""
    if dtype == synth.BF16:
        bits = synth.bf16_bits(x_f32)
        return torch.from_numpy(bits.view(np.int16)).to(device).view(torch.bfloat16)
    return torch.from_numpy(np.ascontiguousarray(x_f32, dtype=np.float32)).to(device)


def to_host_f32(t: torch.Tensor) -> np.ndarray:
    return t.detach().to("cpu").to(torch.float32).numpy()


@dataclasses.dataclass
class StepBuffers:
    """Device inputs and outputs of one decode step (one replica)."""
    ids: torch.Tensor            # [n] int32 sequence ids
    pos: torch.Tensor            # [n] int32 row written by this step
    lens: torch.Tensor           # [n] int32 cache length after the append (= pos + 1)
    sent_ids: torch.Tensor       # [n_sent] int32
    src_lens: torch.Tensor       # [n_sent] int32
    q_self: Optional[torch.Tensor]   # [N_s][n][H][64]
    k_new: Optional[torch.Tensor]    # [N_s][n][H][64]
    v_new: Optional[torch.Tensor]    # [M][n][H][64]
    x_aan: Optional[torch.Tensor]    # [M][n][d]
    t_aan: Optional[torch.Tensor]    # [n] int32, 1-based
    q_enc: torch.Tensor          # [N_e][n_sent][beam][H][64]
    S_self: Optional[torch.Tensor]   # [N_s][n][H][ld_t] float32
    O_self: torch.Tensor         # [M][n][H][64]
    S_enc: torch.Tensor          # [N_e][n_sent*beam][H][ld_s] float32
    O_enc: torch.Tensor          # [M or N_e][n_sent*beam][H][64]
    max_len: int                 # host bound on lens
    max_src: int                 # host bound on src_lens


class Decoder:
    """One library context over torch-allocated device buffers for a workload shape."""

    def __init__(self, w: synth.Workload, device="cuda:0", encdec_shared_context: bool = False):
        self.w = w
        self.device = torch.device(device)
        self.shared_ctx = bool(encdec_shared_context)
        self._host_step_args = {}
        self.tdtype = torch.bfloat16 if w.dtype == synth.BF16 else torch.float32
        self.cfg = B.san_config(
            n_layers=w.n_layers, n_heads=w.n_heads, d_head=w.d_head, max_sent=w.n_sent, beam=w.beam,
            max_tgt_len=w.max_tgt_len(), max_src_len=w.max_src_len(),
            dtype=B.SAN_BF16 if w.dtype == synth.BF16 else B.SAN_F32,
            self_is_aan=int(w.self_is_aan), encdec_shared_context=int(self.shared_ctx))
        self.self_sizes = list(w.self_blocks)
        self.enc_sizes = list(w.encdec_blocks)
        rc, cb, wb = B.san_query_bytes(self.cfg, len(self.self_sizes), len(self.enc_sizes))
        B.check(rc, "san_query_bytes")
        self.cache_bytes, self.ws_bytes = cb, wb
        with torch.cuda.device(self.device):
            self.cache = torch.empty(cb, dtype=torch.uint8, device=self.device)
            self.ws = torch.empty(wb, dtype=torch.uint8, device=self.device)
            rc, self.ctx = B.san_create(self.cfg, self.self_sizes, self.enc_sizes, self.cache, cb, self.ws, wb)
        B.check(rc, "san_create")
        # the lowest layer of every block, as the library's own policy tables have it
        rc, _, self.self_first = B.san_policy_get_map(self.ctx, B.SAN_SELF)
        B.check(rc, "san_policy_get_map")
        rc, _, self.enc_first = B.san_policy_get_map(self.ctx, B.SAN_ENCDEC)
        B.check(rc, "san_policy_get_map")
        self.ld_t = (w.max_tgt_len() + 3) // 4 * 4
        self.ld_s = (w.max_src_len() + 3) // 4 * 4

    def close(self):
        if getattr(self, "ctx", None):
            B.san_destroy(self.ctx)
            self.ctx = None
        self._host_step_args = {}

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ------------------------------------------------------------------ buffers
    def new_step_buffers(self, n: Optional[int] = None, n_sent: Optional[int] = None) -> StepBuffers:
        w, dev = self.w, self.device
        n = w.n_seqs if n is None else n
        n_sent = w.n_sent if n_sent is None else n_sent
        M, H, dh = w.n_layers, w.n_heads, w.d_head
        Ns, Ne = len(self.self_sizes), len(self.enc_sizes)
        i32 = dict(dtype=torch.int32, device=dev)
        e = dict(dtype=self.tdtype, device=dev)
        f = dict(dtype=torch.float32, device=dev)
        aan = w.self_is_aan
        n_enc_out = Ne if self.shared_ctx else M
        return StepBuffers(
            ids=torch.zeros(n, **i32), pos=torch.zeros(n, **i32), lens=torch.ones(n, **i32),
            sent_ids=torch.zeros(n_sent, **i32), src_lens=torch.ones(n_sent, **i32),
            q_self=None if aan else torch.zeros(Ns, n, H, dh, **e),
            k_new=None if aan else torch.zeros(Ns, n, H, dh, **e),
            v_new=None if aan else torch.zeros(M, n, H, dh, **e),
            x_aan=torch.zeros(M, n, H * dh, **e) if aan else None,
            t_aan=torch.ones(n, **i32) if aan else None,
            q_enc=torch.zeros(Ne, n_sent, w.beam, H, dh, **e),
            S_self=None if aan else torch.zeros(Ns, n, H, self.ld_t, **f),
            O_self=torch.zeros(M, n, H, dh, **e),
            S_enc=torch.zeros(Ne, n_sent * w.beam, H, self.ld_s, **f),
            O_enc=torch.zeros(n_enc_out, n_sent * w.beam, H, dh, **e),
            max_len=w.max_tgt_len(), max_src=w.max_src_len())

    # ------------------------------------------------------------------- calls
    def load_encoder_memory(self, stream=None):
        """Upload the workload's encoder memory and write it into the caches (one call)."""
        w, dev = self.w, self.device
        M = w.n_layers
        src = w.src_lens()
        sent_ids = torch.arange(w.n_sent, dtype=torch.int32, device=dev)
        nrows = torch.from_numpy(src).to(dev)
        layers = self.enc_first if self.shared_ctx else list(range(M))
        Ks, Vs = [], []
        for l in range(M):
            if l in self.enc_first or l in layers:
                K, V = synth.encoder_memory(w, l)
                if l in self.enc_first:
                    Ks.append(K)
                if l in layers:
                    Vs.append(V)
        k_dev = to_device(np.stack(Ks), w.dtype, dev)
        if self.shared_ctx:
            # Eq. 5: only block-first layers own encoder memory; one call per such layer
            for i, l in enumerate(self.enc_first):
                v_dev = to_device(Vs[i], w.dtype, dev)
                B.check(B.san_cache_append(self.ctx, B.SAN_ENCDEC, l, l + 1, k_dev[i], v_dev, sent_ids, None, nrows,
                                           w.n_sent, w.max_src_len(), stream), "san_cache_append(ENCDEC)")
        else:
            v_dev = to_device(np.stack(Vs), w.dtype, dev)
            B.check(B.san_cache_append(self.ctx, B.SAN_ENCDEC, 0, M, k_dev, v_dev, sent_ids, None, nrows,
                                       w.n_sent, w.max_src_len(), stream), "san_cache_append(ENCDEC)")
        torch.cuda.synchronize(dev)     # uploads above are temporaries
        return src

    def step(self, sb: StepBuffers, stream=None) -> int:
        """Issue every attention call of one decode step; returns the number of launches."""
        w, ctx = self.w, self.ctx
        M = w.n_layers
        n, n_sent = sb.ids.shape[0], sb.sent_ids.shape[0]
        launches = 0
        if w.self_is_aan:
            B.check(B.san_aan_step(ctx, 0, M, sb.x_aan, sb.ids, sb.t_aan, n, sb.O_self, stream), "san_aan_step")
            launches += 1
        else:
            B.check(B.san_cache_append(ctx, B.SAN_SELF, 0, M, sb.k_new, sb.v_new, sb.ids, sb.pos, None, n, 1, stream),
                    "san_cache_append")
            launches += 1
            for b, (first, size) in enumerate(zip(self.self_first, self.self_sizes)):
                B.check(B.san_attn_weights(ctx, B.SAN_SELF, b, sb.q_self[b], sb.ids, sb.lens, n, sb.max_len,
                                           sb.S_self[b], self.ld_t, stream), "san_attn_weights")
                B.check(B.san_attn_apply(ctx, B.SAN_SELF, b, first, first + size, sb.S_self[b], self.ld_t, sb.ids,
                                         None, sb.lens, n, sb.max_len, sb.O_self[first], 0, stream), "san_attn_apply")
                launches += 2
        for c, (first, size) in enumerate(zip(self.enc_first, self.enc_sizes)):
            B.check(B.san_attn_weights(ctx, B.SAN_ENCDEC, c, sb.q_enc[c], sb.sent_ids, sb.src_lens, n_sent, sb.max_src,
                                       sb.S_enc[c], self.ld_s, stream), "san_attn_weights(ENCDEC)")
            if self.shared_ctx:
                B.check(B.san_attn_apply(ctx, B.SAN_ENCDEC, c, first, first + 1, sb.S_enc[c], self.ld_s, sb.sent_ids,
                                         None, sb.src_lens, n_sent, sb.max_src, sb.O_enc[c], 0, stream),
                        "san_attn_apply(ENCDEC)")
            else:
                B.check(B.san_attn_apply(ctx, B.SAN_ENCDEC, c, first, first + size, sb.S_enc[c], self.ld_s, sb.sent_ids,
                                         None, sb.src_lens, n_sent, sb.max_src, sb.O_enc[first], 0, stream),
                        "san_attn_apply(ENCDEC)")
            launches += 2
        return launches

    def step_fused(self, sb: StepBuffers, stream=None) -> int:
        """The same decode step as ``step`` in one launch (san_decode_step)."""
        w = self.w
        n, n_sent = sb.ids.shape[0], sb.sent_ids.shape[0]
        kw = dict(d_seq_ids=sb.ids, n_seqs=n, max_len=sb.max_len, d_O_self=sb.O_self,
                  d_q_enc=sb.q_enc, d_sent_ids=sb.sent_ids, d_src_lens=sb.src_lens, n_sent=n_sent, max_src=sb.max_src,
                  d_S_enc=sb.S_enc, ld_s=self.ld_s, d_O_enc=sb.O_enc, stream=stream)
        if w.self_is_aan:
            kw.update(d_x_aan=sb.x_aan, d_t=sb.t_aan)
        else:
            kw.update(d_q_self=sb.q_self, d_k_new=sb.k_new, d_v_new=sb.v_new, d_pos=sb.pos, d_S_self=sb.S_self,
                      ld_t=self.ld_t)
        B.check(B.san_decode_step(self.ctx, **kw), "san_decode_step")
        return 1

    def _dev_step_args(self, sb: StepBuffers) -> dict:
        w = self.w
        n, n_sent = sb.ids.shape[0], sb.sent_ids.shape[0]
        kw = dict(d_seq_ids=sb.ids, n_seqs=n, max_len=sb.max_len, d_O_self=sb.O_self,
                  d_q_enc=sb.q_enc, d_sent_ids=sb.sent_ids, d_src_lens=sb.src_lens, n_sent=n_sent, max_src=sb.max_src,
                  d_S_enc=sb.S_enc, ld_s=self.ld_s, d_O_enc=sb.O_enc)
        if w.self_is_aan:
            kw.update(d_x_aan=sb.x_aan, d_t=sb.t_aan)
        else:
            kw.update(d_q_self=sb.q_self, d_k_new=sb.k_new, d_v_new=sb.v_new, d_pos=sb.pos, d_S_self=sb.S_self,
                      ld_t=self.ld_t)
        return kw

    def host_buffers(self, sb: StepBuffers, want_S: bool = False) -> dict:
        """Pinned host copies of the step's inputs and pinned room for its outputs, keyed by
        the san_step_args field they stand for."""
        names_in = {"d_seq_ids": sb.ids, "d_sent_ids": sb.sent_ids, "d_src_lens": sb.src_lens, "d_q_enc": sb.q_enc}
        if self.w.self_is_aan:
            names_in.update(d_x_aan=sb.x_aan, d_t=sb.t_aan)
        else:
            names_in.update(d_pos=sb.pos, d_q_self=sb.q_self, d_k_new=sb.k_new, d_v_new=sb.v_new)
        names_out = {"d_O_self": sb.O_self, "d_O_enc": sb.O_enc}
        if want_S:
            names_out["d_S_enc"] = sb.S_enc
            if sb.S_self is not None:
                names_out["d_S_self"] = sb.S_self
        hb = {k: t.cpu().pin_memory() for k, t in names_in.items()}
        hb.update({k: torch.empty_like(t, device="cpu").pin_memory() for k, t in names_out.items()})
        hb["_in"], hb["_out"] = list(names_in), list(names_out)
        return hb

    def step_fused_host(self, sb: StepBuffers, hb: dict, stream=None) -> int:
        """The decode step through san_decode_step_host: inputs come from and outputs go to the
        pinned host tensors of ``hb``; the library issues the copies around its one launch."""
        # the two argument structs hold raw pointers and bounds: built once per pair of buffer sets and
        # rebuilt when the step's bounds change (a serving loop calls this every step)
        key = (id(sb), id(hb))
        cached = self._host_step_args.get(key)
        if cached is None or cached[2] != (sb.max_len, sb.max_src):
            host = B.step_args(**{k: hb[k] for k in hb["_in"] + hb["_out"]})
            dev = B.step_args(**self._dev_step_args(sb))
            cached = (host, dev, (sb.max_len, sb.max_src), sb, hb)      # keeps the buffers alive with their pointers
            self._host_step_args[key] = cached
        B.check(B.san_decode_step_host(self.ctx, cached[0], cached[1], stream), "san_decode_step_host")
        return 1

    def device_status(self, stream=None):
        rc, first_error, detail = B.san_device_status(self.ctx, stream)
        B.check(rc, "san_device_status")
        return first_error, detail

    # ------------------------------------------------- filling step inputs from the workload
    def fill_step_inputs(self, sb: StepBuffers, step: int, seq_ids: np.ndarray, pos: np.ndarray,
                         sent_ids: Optional[np.ndarray] = None):
        """Upload the workload's synthetic inputs of decode step ``step`` for the listed sequences.

        Enc-dec queries are uploaded for whole sentences (all beams of ``sent_ids``).
        Returns the host copies (float32) for the caller's bookkeeping.
        """
        w, dev = self.w, self.device
        seq_ids = np.asarray(seq_ids, np.int32)
        pos = np.asarray(pos, np.int32)
        if sent_ids is None:
            sent_ids = np.unique(seq_ids // w.beam).astype(np.int32)
        src = w.src_lens()
        host = {}
        sb.ids.copy_(torch.from_numpy(seq_ids))
        sb.pos.copy_(torch.from_numpy(pos))
        sb.lens.copy_(torch.from_numpy(pos + 1))
        sb.sent_ids.copy_(torch.from_numpy(sent_ids))
        sb.src_lens.copy_(torch.from_numpy(src[sent_ids]))
        # the host knows where every hypothesis stands: the bounds of this step, not of the whole run
        sb.max_len = int(pos.max()) + 1 if len(pos) else 1
        sb.max_src = int(src[sent_ids].max()) if len(sent_ids) else 1
        if w.self_is_aan:
            xs = np.stack([synth.aan_x(w, step, l)[seq_ids] for l in range(w.n_layers)])
            sb.x_aan.copy_(to_device(xs, w.dtype, dev))
            sb.t_aan.copy_(torch.from_numpy(pos + 1))
            host["x"] = xs
        else:
            qs, ks, vs = [], [], []
            for l in range(w.n_layers):
                q, k, v = synth.self_qkv(w, step, l)
                vs.append(v[seq_ids])
                if l in self.self_first:
                    qs.append(q[seq_ids])
                    ks.append(k[seq_ids])
            host["q"], host["k"], host["v"] = np.stack(qs), np.stack(ks), np.stack(vs)
            sb.q_self.copy_(to_device(host["q"], w.dtype, dev))
            sb.k_new.copy_(to_device(host["k"], w.dtype, dev))
            sb.v_new.copy_(to_device(host["v"], w.dtype, dev))
        beams = (sent_ids[:, None] * w.beam + np.arange(w.beam)[None, :]).reshape(-1)
        qe = np.stack([synth.encdec_q(w, step, l)[beams] for l in self.enc_first])
        host["q_enc"] = qe          # [N_e][n_sent*beam][H][64]
        sb.q_enc.copy_(to_device(qe, w.dtype, dev).view(sb.q_enc.shape))
        host["beams"] = beams
        return host
