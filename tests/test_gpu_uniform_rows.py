"""Parity of the one-launch decode step on rows of one length: every sequence sits at the same
cache length (or every sentence has the same source length), for lengths on both sides of the
tile boundaries (24 key rows beside the queries in an item's first tile, 32 rows per tile) and
for blocks of 1, 2, 3 and 6 layers.  One launch per test over rows of one shape, which also
makes these the cases to count a kernel's instructions per row on."""
import numpy as np
import pytest
import torch

from paper_1906_11024_b200 import binding as B
from paper_1906_11024_b200 import build as san_build
from paper_1906_11024_b200 import synth
from paper_1906_11024_b200.driver import Decoder, to_device, to_host_f32
from tests.helpers import TOL, TOL_S, OracleRun, normwise_err, weights_err

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    san_build.build()
    B.lib()


# which kernel runs the step and how it cuts the rows (san_step_kernel_select): the automatic choice, the team
# pipeline with its own cut (up to four heads to a warp), and the team pipeline with one head
# to a warp in tiles of 16 positions
CUTS = {"auto": None, "team": (2,), "team-1head-tile16": (2, 0, 1, 16, 0, 1)}


def _select(dec, cut):
    if CUTS[cut] is not None:
        B.check(B.san_step_kernel_select(dec.ctx, *CUTS[cut]), "san_step_kernel_select")


def _wl(pi_self, pi_enc, src, T, n_sent=16):
    return synth.Workload(name=f"uniform-{pi_self}-{pi_enc}-{src}-{T}", dtype=synth.BF16, n_layers=6, n_heads=8, d_head=64,
                          n_sent=n_sent, beam=4, self_blocks=(pi_self,) * (6 // pi_self),
                          encdec_blocks=(pi_enc,) * (6 // pi_enc), src_lo=src, src_hi=src, tgt_rule="fixed",
                          tgt_fixed=T, ragged_prefix=False, self_is_aan=False, seed=5)


@pytest.mark.parametrize("cut", sorted(CUTS))
@pytest.mark.parametrize("L", [8, 21, 24, 25, 40, 56, 88])
@pytest.mark.parametrize("pi", [1, 2, 3])
def test_self_attention_rows_of_one_length(L, pi, cut):
    """Self-attention only (no sentence in the step): prefill L-1 rows, decode the L-th."""
    w = _wl(pi, 1, 8, L)
    dec, orc = Decoder(w), OracleRun(w)
    _select(dec, cut)
    n = w.n_seqs
    ids = np.arange(n, dtype=np.int32)
    if L > 1:
        rows = np.full(n, L - 1, np.int32)
        orc.prefill(ids, rows)
        for l in range(w.n_layers):
            K, V = synth.self_prefill(w, l)
            B.check(B.san_cache_append(dec.ctx, B.SAN_SELF, l, l + 1, to_device(K, w.dtype, dec.device) if l in dec.self_first else None,
                                       to_device(V, w.dtype, dec.device), torch.from_numpy(ids).cuda(), None,
                                       torch.from_numpy(rows).cuda(), n, w.max_tgt_len()), "prefill")
    pos = np.full(n, L - 1, np.int32)
    full = dec.new_step_buffers()
    host = dec.fill_step_inputs(full, 0, ids, pos)
    sb = dec.new_step_buffers(n, 0)                          # the same step without its enc-dec part
    for name in ("ids", "pos", "lens", "q_self", "k_new", "v_new"):
        getattr(sb, name).copy_(getattr(full, name))
    sb.max_len = L
    dec.step_fused(sb)
    assert dec.device_status()[0] == 0
    for l in range(w.n_layers):
        first = l in orc.self_first
        b = orc.self_first.index(l) if first else None
        orc.o.self_append(l, ids, pos, host["k"][b] if first else None, host["v"][l])
    S_ref, O_ref = [], []
    for l in range(w.n_layers):
        first = l in orc.self_first
        S, O = orc.o.self_attend(l, ids, pos + 1, host["q"][orc.self_first.index(l)] if first else None, want_S=first)
        O_ref.append(O)
        if first:
            S_ref.append(S)
    assert normwise_err(to_host_f32(sb.O_self), np.stack(O_ref)) <= TOL[w.dtype]
    assert weights_err(to_host_f32(sb.S_self)[..., :L], np.stack(S_ref)[..., :L]) <= TOL_S
    dec.close()


@pytest.mark.parametrize("cut", sorted(CUTS))
@pytest.mark.parametrize("Ls", [16, 24, 38, 60])
@pytest.mark.parametrize("pi", [1, 3, 6])
def test_encoder_memory_rows_of_one_length(Ls, pi, cut):
    """Encoder-decoder attention only (no sequence in the step's self-attention part)."""
    w = _wl(1, pi, Ls, 8)
    dec, orc = Decoder(w), OracleRun(w)
    _select(dec, cut)
    dec.load_encoder_memory()
    ids = np.arange(w.n_seqs, dtype=np.int32)
    full = dec.new_step_buffers()
    host = dec.fill_step_inputs(full, 0, ids, np.zeros(w.n_seqs, np.int32))
    sb = dec.new_step_buffers(0, w.n_sent)
    for name in ("sent_ids", "src_lens", "q_enc"):
        getattr(sb, name).copy_(getattr(full, name))
    sb.max_src = Ls
    dec.step_fused(sb)
    assert dec.device_status()[0] == 0
    S_ref, O_ref = [], []
    for l in range(w.n_layers):
        first = l in orc.enc_first
        S, O = orc.o.encdec_attend(l, host["beams"], host["q_enc"][orc.enc_first.index(l)] if first else None, want_S=first)
        O_ref.append(O)
        if first:
            S_ref.append(S)
    assert normwise_err(to_host_f32(sb.O_enc), np.stack(O_ref)) <= TOL[w.dtype]
    assert weights_err(to_host_f32(sb.S_enc)[..., :Ls], np.stack(S_ref)[..., :Ls]) <= TOL_S
    dec.close()
