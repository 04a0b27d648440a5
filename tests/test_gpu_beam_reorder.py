"""Beam-search cache reorder (san_beam_reorder) against the oracle and against a host-side
gather: integer work, so the cache contents are compared bit for bit; attention after the
reorder is compared with the oracle within the usual tolerances."""
import numpy as np
import pytest
import torch

from paper_1906_11024_b200 import binding as B
from paper_1906_11024_b200 import build as san_build
from paper_1906_11024_b200 import synth
from paper_1906_11024_b200.driver import Decoder, to_device, to_host_f32
from tests.helpers import TOL, TOL_S, OracleRun, cached_row_order, normwise_err, weights_err

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    san_build.build()
    B.lib()


def _wl(dtype=synth.BF16, **kw):
    base = dict(name="reorder", dtype=dtype, n_layers=4, n_heads=2, d_head=64, n_sent=5, beam=4,
                self_blocks=(1, 3), encdec_blocks=(4,), src_lo=5, src_hi=9, tgt_rule="fixed", tgt_fixed=40,
                ragged_prefix=False, self_is_aan=False, seed=91)
    base.update(kw)
    return synth.Workload(**base)


def _i32(x, dev):
    return torch.tensor(np.asarray(x, np.int32), dtype=torch.int32, device=dev)


# parents per sentence: identity, a permutation, everyone from one parent, duplicates, a swap
PARENTS4 = [[0, 1, 2, 3], [3, 2, 1, 0], [2, 2, 2, 2], [0, 0, 3, 3], [1, 0, 2, 3]]


@pytest.mark.parametrize("dtype,T", [(synth.BF16, 40), (synth.F32, 40), (synth.BF16, 300)])
def test_cache_after_reorder_equals_host_gather_bit_for_bit(dtype, T):
    """Rows are appended from known host values, so the expected arena is built on the host
    (never read from the device): a gather of whole rows by parent, first lens rows only, rows
    beyond the taken length and untouched beams unchanged.  T = 300 spans several tiles."""
    w = _wl(dtype, tgt_fixed=T)
    dec = Decoder(w)
    dev = dec.device
    M, H, dh, n = w.n_layers, w.n_heads, w.d_head, w.n_seqs
    Ns, e = len(w.self_blocks), w.elem_bytes
    udt = np.uint16 if dtype == synth.BF16 else np.uint32
    bits = (lambda a: synth.bf16_bits(a)) if dtype == synth.BF16 else (lambda a: a.view(np.uint32))
    dec.cache.zero_()
    rng = np.random.default_rng(5)
    fill = rng.integers(T // 2, T + 1, size=n).astype(np.int32)            # rows each sequence holds
    expK = np.zeros((Ns, n, H, T, dh), udt)
    expV = np.zeros((M, n, H, T, dh), udt)
    ids = np.arange(n, dtype=np.int32)
    for l in range(M):
        K, V = synth.self_prefill(w, l)                                     # [n][T][H][64]
        first = l in dec.self_first
        B.check(B.san_cache_append(dec.ctx, B.SAN_SELF, l, l + 1, to_device(K, dtype, dev) if first else None,
                                   to_device(V, dtype, dev), _i32(ids, dev), None, _i32(fill, dev), n, T), "append")
        rowpos = np.arange(T)[:, None]
        for s in range(n):
            f = fill[s]
            expV[l, s, :, :f] = cached_row_order(bits(V[s, :f]), rowpos[:f], dtype).transpose(1, 0, 2)
            if first:
                expK[dec.self_first.index(l), s, :, :f] = cached_row_order(bits(K[s, :f]), rowpos[:f], dtype).transpose(1, 0, 2)
    torch.cuda.synchronize()

    def check_arena():
        raw = dec.cache.cpu().numpy()
        plane = n * H * T * dh * e
        assert np.array_equal(raw[:Ns * plane].view(udt).reshape(Ns, n, H, T, dh), expK)
        assert np.array_equal(raw[Ns * plane:(Ns + M) * plane].view(udt).reshape(M, n, H, T, dh), expV)

    check_arena()
    sent_order = np.array([4, 0, 2, 1, 3], np.int32)                        # items need not be in sentence order
    for rnd in range(3):                                                    # reorders compose
        parent = np.array([PARENTS4[(g + rnd) % len(PARENTS4)] for g in sent_order], np.int32)
        lens = np.zeros((len(sent_order), w.beam), np.int32)
        for i, g in enumerate(sent_order):
            for s in range(w.beam):
                full = fill[g * w.beam + parent[i, s]]
                lens[i, s] = full if (rnd + s) % 3 else rng.integers(0, full + 1)     # some take only a prefix
        B.check(B.san_beam_reorder(dec.ctx, _i32(sent_order, dev), _i32(parent, dev), _i32(lens, dev),
                                   len(sent_order), int(lens.max())), "san_beam_reorder")
        oldK, oldV = expK.copy(), expV.copy()
        for i, g in enumerate(sent_order):
            for s in range(w.beam):
                src, dst, L = g * w.beam + parent[i, s], g * w.beam + s, lens[i, s]
                expK[:, dst, :, :L] = oldK[:, src, :, :L]
                expV[:, dst, :, :L] = oldV[:, src, :, :L]
        assert dec.device_status()[0] == 0
        check_arena()
    dec.close()


def _decode_reorder_decode(w, fused):
    """Decode, reorder by parent beams on both sides, decode on: outputs must keep matching."""
    dec = Decoder(w)
    orc = OracleRun(w)
    dec.load_encoder_memory()
    n = w.n_seqs
    ids = np.arange(n, dtype=np.int32)
    sent = np.arange(w.n_sent, dtype=np.int32)
    src_seq = np.repeat(w.src_lens(), w.beam)
    tol = TOL[w.dtype]
    rng = np.random.default_rng(17)
    worst = 0.0
    for step in range(9):
        pos = np.full(n, step, np.int32)
        sb = dec.new_step_buffers()
        host = dec.fill_step_inputs(sb, step, ids, pos, sent)
        (dec.step_fused if fused else dec.step)(sb)
        ref = orc.step(host, ids, pos)
        assert dec.device_status()[0] == 0
        for got, want in ((sb.O_self, ref["O_self"]), (sb.O_enc, ref["O_enc"])):
            err = normwise_err(to_host_f32(got), want)
            worst = max(worst, err)
            assert err <= tol, (step, err)
        if not w.self_is_aan:
            S = to_host_f32(sb.S_self)[..., :step + 1]
            assert weights_err(S, ref["S_self"][..., :step + 1]) <= TOL_S
        if step in (2, 3, 6):                                               # the beam search picks survivors
            parent = rng.integers(0, w.beam, size=(w.n_sent, w.beam)).astype(np.int32)
            if step == 3:
                parent[0] = np.arange(w.beam)                               # one sentence keeps its beams
            lens = np.full((w.n_sent, w.beam), step + 1, np.int32)
            B.check(B.san_beam_reorder(dec.ctx, _i32(sent, dec.device), _i32(parent, dec.device),
                                       _i32(lens, dec.device), w.n_sent, step + 1), "san_beam_reorder")
            orc.o.beam_reorder((sent[:, None] * w.beam + parent).reshape(-1), lens.reshape(-1))
    dec.close()
    return worst


@pytest.mark.parametrize("fused", [True, False])
@pytest.mark.parametrize("dtype", [synth.BF16, synth.F32])
def test_attention_after_reorder_matches_oracle(dtype, fused):
    _decode_reorder_decode(_wl(dtype, tgt_fixed=12), fused)


def test_running_average_after_reorder_matches_oracle():
    """With AAN in place of self-attention the reorder hands on the parent's running sum."""
    _decode_reorder_decode(_wl(synth.BF16, tgt_fixed=12, self_is_aan=True, encdec_blocks=(2, 2)), True)


def test_bad_parent_or_length_is_skipped_and_reported():
    w = _wl(synth.BF16, tgt_fixed=16)
    dec = Decoder(w)
    dev = dec.device
    dec.cache.zero_()
    before = dec.cache.clone()
    sent = np.arange(w.n_sent, dtype=np.int32)
    parent = np.tile(np.array([1, 0, 3, 2], np.int32), (w.n_sent, 1))
    lens = np.full((w.n_sent, w.beam), 8, np.int32)
    bad = parent.copy(); bad[2, 1] = w.beam                                # parent outside the sentence's beams
    B.check(B.san_beam_reorder(dec.ctx, _i32(sent, dev), _i32(bad, dev), _i32(lens, dev), w.n_sent, 8), "reorder")
    err, detail = dec.device_status()
    assert err == B.SAN_ERR_DEVICE_CHECK and detail[1] == 2 * w.beam + 1 and detail[2] == w.beam
    badl = lens.copy(); badl[1, 0] = 9                                     # beyond the host bound
    B.check(B.san_beam_reorder(dec.ctx, _i32(sent, dev), _i32(parent, dev), _i32(badl, dev), w.n_sent, 8), "reorder")
    err, detail = dec.device_status()
    assert err == B.SAN_ERR_DEVICE_CHECK and detail[2] == 9 and detail[3] == 8
    assert torch.equal(before, dec.cache)                                  # an all-zero arena stays all zero
    # host-visible mistakes never launch
    assert B.san_beam_reorder(dec.ctx, None, _i32(parent, dev), _i32(lens, dev), w.n_sent, 8) == B.SAN_ERR_NULL
    assert B.san_beam_reorder(dec.ctx, _i32(sent, dev), _i32(parent, dev), _i32(lens, dev), w.n_sent + 1, 8) == B.SAN_ERR_SHAPE
    assert B.san_beam_reorder(dec.ctx, _i32(sent, dev), _i32(parent, dev), _i32(lens, dev), w.n_sent, 17) == B.SAN_ERR_SHAPE
    assert B.san_beam_reorder(dec.ctx, _i32(sent, dev), _i32(parent, dev), _i32(lens, dev), 0, 8) == B.SAN_OK
    dec.close()
