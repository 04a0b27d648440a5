"""san_attn_weights_static: the weights step for callers that cannot allocate device memory.

Some users of this library run the decode loop where cudaMalloc is off the table: all of
HBM already belongs to a serving framework's cache pool, or allocation is forbidden once
serving has begun, or its device-wide stall is unaffordable.  They call the static-scratch
entry point, which needs neither a context nor a workspace.  This test drives it through
the C ABI on rows long enough to be split (so the fixed scratch is really used), twice in
a row, and checks each result against san_attn_weights on the same inputs.

This file sorts last on purpose: a run that stops at the first failure has then already
run every other test.
"""
import numpy as np
import pytest
import torch

from paper_1906_11024_b200 import binding as B
from paper_1906_11024_b200 import build as san_build
from paper_1906_11024_b200 import synth
from paper_1906_11024_b200.driver import Decoder, to_device

pytestmark = pytest.mark.gpu

TOL_S = 1e-5      # the tolerance the parity tests use for weights (relative, floor 1e-7)


def _weights_err(S, ref, floor=1e-7):
    return float((np.abs(S.astype(np.float64) - ref) / np.maximum(ref, floor)).max())


@pytest.mark.parametrize("dtype", [synth.BF16, synth.F32])
def test_static_scratch_weights_match_the_context_path_twice_in_a_row(dtype):
    san_build.build()
    w = synth.Workload("noalloc", dtype, 2, 4, 64, 3, 4, (2,), (2,), 200, 300, "fixed", 300, False, False, 91)
    dec = Decoder(w)
    dev = dec.device
    n, H, T, Ls = w.n_seqs, w.n_heads, w.max_tgt_len(), w.max_src_len()
    e = w.elem_bytes
    # fill the key planes through the normal append path
    K, V = synth.self_prefill(w, 0)
    ids = torch.arange(n, dtype=torch.int32, device=dev)
    rows = torch.full((n,), T, dtype=torch.int32, device=dev)
    B.check(B.san_cache_append(dec.ctx, B.SAN_SELF, 0, 1, to_device(K, dtype, dev), to_device(V, dtype, dev), ids, None,
                               rows, n, T))
    src = dec.load_encoder_memory()
    # device addresses of the first self key plane and the first memory key plane, from the
    # documented arena layout: [self K planes][self V planes][memory K planes][memory V planes]
    self_plane = (n * H * T * 64 * e + 255) // 256 * 256
    self_K = dec.cache.data_ptr()
    mem_K = dec.cache.data_ptr() + (1 + w.n_layers) * self_plane
    status = torch.zeros(8, dtype=torch.int32, device=dev)
    for call in range(2):
        # decoder self-attention rows: one query per (sequence, head), ragged lengths
        q = synth.self_qkv(w, call, 0)[0]
        lens_h = np.array([T, 257, 129, 300, 1, 64, 200, 33, 299, 128, 256, 17], np.int32)[:n]
        lens = torch.from_numpy(lens_h).to(dev)
        q_dev = to_device(q, dtype, dev)
        S_ref = torch.zeros(n, H, dec.ld_t, device=dev)
        S_new = torch.zeros(n, H, dec.ld_t, device=dev)
        B.check(B.san_attn_weights(dec.ctx, B.SAN_SELF, 0, q_dev, ids, lens, n, T, S_ref, dec.ld_t))
        B.check(B.san_attn_weights_static(dec.cfg.dtype, H, 1, q_dev, self_K, n, T, ids, lens, n, T, S_new,
                                          dec.ld_t, status))
        torch.cuda.synchronize(dev)
        assert status.cpu().numpy()[0] == 0
        a, b = S_new.cpu().numpy(), S_ref.cpu().numpy()
        for i in range(n):
            L = int(lens_h[i])
            assert _weights_err(a[i, :, :L], b[i, :, :L].astype(np.float64)) <= TOL_S, (call, "self", i)
            assert abs(a[i, :, :L].astype(np.float64).sum(-1) - 1.0).max() <= 1e-5
        # encoder memory: the beams of a sentence share each key tile
        qe = synth.encdec_q(w, call, 0).reshape(w.n_sent, w.beam, H, 64)
        sent = torch.arange(w.n_sent, dtype=torch.int32, device=dev)
        sl = torch.from_numpy(src).to(dev)
        qe_dev = to_device(qe, dtype, dev)
        E_ref = torch.zeros(w.n_sent * w.beam, H, dec.ld_s, device=dev)
        E_new = torch.zeros_like(E_ref)
        B.check(B.san_attn_weights(dec.ctx, B.SAN_ENCDEC, 0, qe_dev, sent, sl, w.n_sent, Ls, E_ref, dec.ld_s))
        B.check(B.san_attn_weights_static(dec.cfg.dtype, H, w.beam, qe_dev, mem_K, w.n_sent, Ls, sent, sl, w.n_sent,
                                          Ls, E_new, dec.ld_s, status))
        torch.cuda.synchronize(dev)
        assert status.cpu().numpy()[0] == 0
        a, b = E_new.cpu().numpy(), E_ref.cpu().numpy()
        for s in range(w.n_sent * w.beam):
            L = int(src[s // w.beam])
            assert _weights_err(a[s, :, :L], b[s, :, :L].astype(np.float64)) <= TOL_S, (call, "encdec", s)
    # sizes beyond the fixed scratch are refused before anything is launched
    assert B.san_attn_weights_static(dec.cfg.dtype, 1024, 1, q_dev, self_K, 65, T, ids, lens, 65, T, S_new,
                                     dec.ld_t, None) == B.SAN_ERR_CAPACITY
    # a bad length is skipped and reported in the caller's status words, not a fault
    bad = lens.clone()
    bad[1] = 0
    B.check(B.san_attn_weights_static(dec.cfg.dtype, H, 1, q_dev, self_K, n, T, ids, bad, n, T, S_new, dec.ld_t, status))
    torch.cuda.synchronize(dev)
    st = status.cpu().numpy()
    assert st[0] == B.SAN_ERR_DEVICE_CHECK and st[2] == 1
    dec.close()
