"""san_seq_reset: the running sums of the listed sequences start again from zero in the middle
of a count.  The oracle has no reset; "the sum is zero" is the same as "every earlier input of
that sequence was zero", so the expected values come from a second oracle run that is fed zero
rows for the positions before the reset."""
import numpy as np
import pytest
import torch

from oracle import san_oracle as so
from paper_1906_11024_b200 import binding as B
from paper_1906_11024_b200 import build as san_build
from paper_1906_11024_b200 import synth
from paper_1906_11024_b200.driver import Decoder, to_device, to_host_f32
from tests.helpers import TOL, normwise_err

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    san_build.build()
    B.lib()


def _i32(x, dev):
    return torch.tensor(np.asarray(x, np.int32), dtype=torch.int32, device=dev)


@pytest.mark.parametrize("dtype", [synth.BF16, synth.F32])
def test_reset_in_the_middle_of_a_count_then_continue(dtype):
    w = synth.Workload(name="reset", dtype=dtype, n_layers=3, n_heads=2, d_head=64, n_sent=3, beam=2,
                       self_blocks=(3,), encdec_blocks=(3,), src_lo=4, src_hi=6, tgt_rule="fixed", tgt_fixed=12,
                       ragged_prefix=False, self_is_aan=True, seed=93)
    dec = Decoder(w)
    dev = dec.device
    M, n, d = w.n_layers, w.n_seqs, w.n_heads * w.d_head
    ids = np.arange(n, dtype=np.int32)
    kept = so.Oracle(M, w.n_heads, w.d_head, w.n_sent, w.beam, 12, 6, [3], [3])      # sequences that are not reset
    fresh = so.Oracle(M, w.n_heads, w.d_head, w.n_sent, w.beam, 12, 6, [3], [3])     # history replaced by zeros
    reset_ids = np.array([4, 1], np.int32)
    out = torch.zeros(M, n, d, dtype=dec.tdtype, device=dev)
    zeros = np.zeros((n, d), np.float32)

    def step(t, check_reset):
        xs = np.stack([synth.aan_x(w, t, l) for l in range(M)])                      # [M][n][d], rounded to dtype
        B.check(B.san_aan_step(dec.ctx, 0, M, to_device(xs, dtype, dev), _i32(ids, dev), _i32(np.full(n, t + 1), dev),
                               n, out), "san_aan_step")
        got = to_host_f32(out)
        for l in range(M):
            ref_kept = kept.aan_step(l, ids, np.full(n, t + 1), xs[l])
            ref_fresh = fresh.aan_step(l, ids, np.full(n, t + 1), xs[l] if check_reset else zeros)
            for s in range(n):
                ref = ref_fresh[s] if (check_reset and s in reset_ids) else ref_kept[s]
                assert normwise_err(got[l, s][None], ref[None]) <= TOL[dtype], (t, l, s)

    for t in range(4):
        step(t, False)
    B.check(B.san_seq_reset(dec.ctx, _i32(reset_ids, dev), len(reset_ids)), "san_seq_reset")
    for t in range(4, 7):                     # the count goes on: t = 5, 6, 7 over sums that restarted at zero
        step(t, True)
    err, detail = dec.device_status()
    assert err == 0, (err, detail)
    # the sums of the other sequences were not touched: bit-identical to a run without the reset
    dec2 = Decoder(w)
    out2 = torch.zeros_like(out)
    for t in range(7):
        xs = np.stack([synth.aan_x(w, t, l) for l in range(M)])
        B.check(B.san_aan_step(dec2.ctx, 0, M, to_device(xs, dtype, dev), _i32(ids, dev), _i32(np.full(n, t + 1), dev),
                               n, out2), "san_aan_step")
    others = np.setdiff1d(ids, reset_ids)
    assert torch.equal(out[:, others], out2[:, others])
    dec.close(); dec2.close()


def test_reset_argument_checks():
    w = synth.Workload(name="reset", dtype=synth.BF16, n_layers=2, n_heads=2, d_head=64, n_sent=2, beam=2,
                       self_blocks=(2,), encdec_blocks=(2,), src_lo=4, src_hi=6, tgt_rule="fixed", tgt_fixed=8,
                       ragged_prefix=False, self_is_aan=True, seed=94)
    dec = Decoder(w)
    dev = dec.device
    assert B.san_seq_reset(dec.ctx, None, 1) == B.SAN_ERR_NULL
    assert B.san_seq_reset(dec.ctx, _i32([0], dev), w.n_seqs + 1) == B.SAN_ERR_SHAPE
    assert B.san_seq_reset(dec.ctx, None, 0) == B.SAN_OK
    B.check(B.san_seq_reset(dec.ctx, _i32([1, w.n_seqs], dev), 2), "san_seq_reset")   # an id out of range is skipped
    err, detail = dec.device_status()
    assert err == B.SAN_ERR_DEVICE_CHECK and detail[1] == 1 and detail[2] == w.n_seqs
    dec.close()
    w2 = synth.Workload(name="reset", dtype=synth.BF16, n_layers=2, n_heads=2, d_head=64, n_sent=2, beam=2,
                        self_blocks=(2,), encdec_blocks=(2,), src_lo=4, src_hi=6, tgt_rule="fixed", tgt_fixed=8,
                        ragged_prefix=False, self_is_aan=False, seed=94)
    dec = Decoder(w2)
    assert B.san_seq_reset(dec.ctx, _i32([0], dev), 1) == B.SAN_ERR_UNSUPPORTED
    dec.close()
