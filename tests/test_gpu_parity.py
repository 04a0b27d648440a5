"""Parity of the CUDA path (through the C ABI) against the CPU oracle, element by element.

Tolerances: outputs O within 1e-5 (float32) / 1e-2 (bf16 inputs, float32 accumulation),
measured per output vector as ||x - ref||_inf / ||ref||_inf; weights S within 1e-5
element-wise (relative, floor 1e-7) with rows summing to one; cache contents bit-exact.
"""
import dataclasses

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


def _compare(w, dec, sb, ref, n, lens, src_lens_per_seq, tag):
    tol = TOL[w.dtype]
    first_error, detail = dec.device_status()
    assert first_error == 0, (tag, first_error, detail)
    if not w.self_is_aan:
        S = to_host_f32(sb.S_self)
        for b in range(S.shape[0]):
            for i in range(n):
                L = int(lens[i])
                err = weights_err(S[b, i, :, :L], ref["S_self"][b, i, :, :L])
                assert err <= TOL_S, (tag, "S_self", b, i, err)
                assert np.abs(S[b, i, :, :L].astype(np.float64).sum(-1) - 1.0).max() <= 1e-5
    O = to_host_f32(sb.O_self)
    err = normwise_err(O, ref["O_self"])
    assert err <= tol, (tag, "O_self", err)
    S = to_host_f32(sb.S_enc)
    for c in range(S.shape[0]):
        for i in range(S.shape[1]):
            L = int(src_lens_per_seq[i])
            e2 = weights_err(S[c, i, :, :L], ref["S_enc"][c, i, :, :L])
            assert e2 <= TOL_S, (tag, "S_enc", c, i, e2)
    O = to_host_f32(sb.O_enc)
    err = normwise_err(O, ref["O_enc"])
    assert err <= tol, (tag, "O_enc", err)


STEP_KERNEL = [0]        # which kernel san_decode_step is told to launch (see san_step_kernel_select); tests set it


def _run(w, check_steps=None, max_steps=None, shared_context=False, jumps=None, fused=False):
    """Decode the workload on both sides.  Sequences start at their prefix length, advance in
    lock-step and drop out when their sentence is done.  ``jumps`` = list of (start_pos, n_steps)
    segments for long runs: the caches are re-prefilled to start_pos before each segment."""
    dec = Decoder(w, encdec_shared_context=shared_context)
    if STEP_KERNEL[0]:
        sel = STEP_KERNEL[0] if isinstance(STEP_KERNEL[0], tuple) else (STEP_KERNEL[0],)
        B.check(B.san_step_kernel_select(dec.ctx, *sel), "san_step_kernel_select")
    orc = OracleRun(w, shared_context)
    dec.load_encoder_memory()
    T = np.repeat(w.tgt_lens(), w.beam)
    src_seq = np.repeat(w.src_lens(), w.beam)
    all_ids = np.arange(w.n_seqs, dtype=np.int32)
    segments = jumps if jumps else [(None, max_steps if max_steps else int(T.max()))]
    checked = 0
    for start, n_steps in segments:
        pos = w.prefix_lens().astype(np.int32) if start is None else np.full(w.n_seqs, start, np.int32)
        if not w.self_is_aan and pos.max() > 0:
            _prefill(dec, orc, w, all_ids, pos)
        for g in range(n_steps):
            active = all_ids[pos < T]
            if len(active) == 0:
                break
            # whole sentences stay active together (all beams of a sentence share T)
            sent = np.unique(active // w.beam).astype(np.int32)
            sb = dec.new_step_buffers(len(active), len(sent))
            step_id = g if start is None else 100000 + start + g
            host = dec.fill_step_inputs(sb, step_id, active, pos[active], sent)
            (dec.step_fused if fused else dec.step)(sb)
            if fused and STEP_KERNEL[0]:
                want = STEP_KERNEL[0][0] if isinstance(STEP_KERNEL[0], tuple) else STEP_KERNEL[0]
                assert B.san_step_kernel_used(dec.ctx)[1] == want                # the forced kernel is the one that ran
            do_check = check_steps is None or g in check_steps
            ref = orc.step(host, active, pos[active], want_S=do_check)
            if do_check:
                _compare(w, dec, sb, ref, len(active), pos[active] + 1, src_seq[host["beams"]], (w.name, start, g))
                checked += 1
            pos[active] += 1
    assert checked > 0
    dec.close()


def _prefill(dec, orc, w, ids, n_rows):
    orc.prefill(ids, n_rows)
    dev = dec.device
    t_ids = torch.from_numpy(ids).to(dev)
    t_rows = torch.from_numpy(n_rows.astype(np.int32)).to(dev)
    for l in range(w.n_layers):
        K, V = synth.self_prefill(w, l)
        k_dev = to_device(K, w.dtype, dev) if l in dec.self_first else None
        v_dev = to_device(V, w.dtype, dev)
        B.check(B.san_cache_append(dec.ctx, B.SAN_SELF, l, l + 1, k_dev, v_dev, t_ids, None, t_rows,
                                   len(ids), w.max_tgt_len()), "prefill")
    torch.cuda.synchronize(dev)


def test_tiny_fp32_every_step():
    """First configuration in full: float32, blocks {2,2,2} / {3,3}, 16 steps, tolerance 1e-5."""
    _run(synth.WORKLOADS["tiny"])


def test_tiny_fp32_unshared_equals_standard_attention():
    _run(synth.unshared(synth.WORKLOADS["tiny"]))


def test_base_bf16_scaled_every_step():
    _run(synth.scaled(synth.WORKLOADS["base"], 8))


def test_base_bf16_full_size_sampled_steps():
    w = synth.WORKLOADS["base"]
    last = int(w.tgt_lens().max()) - 1
    _run(w, check_steps={0, 1, 17, 33, last})


def test_big_bf16_ragged_scaled_every_step():
    _run(synth.scaled(synth.WORKLOADS["big"], 6))


def test_big_bf16_full_size_sampled_steps():
    _run(synth.WORKLOADS["big"], check_steps={0, 5, 40}, max_steps=41)


def test_long_bf16_split_rows_scaled():
    """Few rows and long caches: rows are split over several warps (ticket combine)."""
    w = synth.scaled(synth.WORKLOADS["long"], 2)
    _run(w, jumps=[(0, 3), (30, 4), (62, 4), (126, 4), (254, 4), (508, 4)])


def test_long_bf16_full_size_sampled_steps():
    _run(synth.WORKLOADS["long"], jumps=[(0, 2), (63, 3), (255, 3), (510, 2)])


def test_aan_bf16_scaled_every_step():
    _run(synth.scaled(synth.WORKLOADS["aan"], 8), max_steps=80)


def test_aan_bf16_full_size_sampled_steps():
    _run(synth.WORKLOADS["aan"], check_steps={0, 1, 40, 79})


def test_learned_policy_blocks_separate_calls():
    """Uneven blocks, as the policy learner of Section 3.3 produces on the paper's Figure 2."""
    _run(dataclasses.replace(synth.scaled(synth.WORKLOADS["base"], 6), self_blocks=(1, 5), encdec_blocks=(4, 2),
                             name="learned"), max_steps=12)


def test_encdec_shared_context_eq5():
    """Eq. 5: one output per enc-dec block; upper layers of the block reuse it."""
    _run(synth.scaled(synth.WORKLOADS["base"], 4), max_steps=6, shared_context=True)
    _run(dataclasses.replace(synth.scaled(synth.WORKLOADS["tiny"], 2), encdec_blocks=(3, 3)), max_steps=4,
         shared_context=True)


@pytest.mark.parametrize("beam", [1, 2, 3, 5, 8, 12, 20])
def test_other_beam_sizes(beam):
    """The paper sweeps beam sizes 4..20 (Figure 5); a key tile is scored for up to eight beams at a
    time, wider beams go through in groups of eight."""
    w = dataclasses.replace(synth.scaled(synth.WORKLOADS["base"], 3), beam=beam, name=f"beam{beam}")
    _run(w, max_steps=5)


def test_fp32_long_rows_and_splits():
    w = dataclasses.replace(synth.WORKLOADS["tiny"], name="tiny-long", src_lo=300, src_hi=300,
                            tgt_rule="fixed", tgt_fixed=300)
    _run(w, jumps=[(0, 2), (127, 3), (255, 3), (297, 3)])


# ------------------------------------------------------------------ the one-launch decode step
FUSED_CASES = {
    "tiny": lambda: _run(synth.WORKLOADS["tiny"], fused=True),
    "tiny-unshared": lambda: _run(synth.unshared(synth.WORKLOADS["tiny"]), fused=True),
    "base-scaled": lambda: _run(synth.scaled(synth.WORKLOADS["base"], 8), fused=True),
    "base-full": lambda: _run(synth.WORKLOADS["base"], check_steps={0, 1, 17, 33, 65}, fused=True),
    "big-scaled-ragged": lambda: _run(synth.scaled(synth.WORKLOADS["big"], 6), fused=True),
    "big-full": lambda: _run(synth.WORKLOADS["big"], check_steps={0, 5, 40}, max_steps=41, fused=True),
    "long-scaled-split": lambda: _run(synth.scaled(synth.WORKLOADS["long"], 2),
                                      jumps=[(0, 3), (30, 4), (62, 4), (126, 4), (254, 4), (508, 4)], fused=True),
    "long-full": lambda: _run(synth.WORKLOADS["long"], jumps=[(0, 2), (63, 3), (255, 3), (510, 2)], fused=True),
    "aan-scaled": lambda: _run(synth.scaled(synth.WORKLOADS["aan"], 8), max_steps=80, fused=True),
    "aan-full": lambda: _run(synth.WORKLOADS["aan"], check_steps={0, 1, 40, 79}, fused=True),
    # the policies the paper's Figure 2 leads to: layer 1 alone then layers 2-6 (self), {4,2} (enc-dec)
    "learned-policy-blocks": lambda: _run(dataclasses.replace(synth.scaled(synth.WORKLOADS["base"], 6), self_blocks=(1, 5),
                                                              encdec_blocks=(4, 2), name="learned"), max_steps=12, fused=True),
    # sharing off on the big shape: about 500 list slots per CTA, so every CTA decodes and drains in rounds
    "big-unshared-many-rounds": lambda: _run(synth.unshared(synth.WORKLOADS["big"]), check_steps={0, 3}, max_steps=4, fused=True),
    "eq5-shared-context": lambda: _run(synth.scaled(synth.WORKLOADS["base"], 4), max_steps=6, shared_context=True,
                                       fused=True),
    "fp32-long-rows": lambda: _run(dataclasses.replace(synth.WORKLOADS["tiny"], name="tiny-long", src_lo=300, src_hi=300,
                                                       tgt_rule="fixed", tgt_fixed=300),
                                   jumps=[(0, 2), (127, 3), (255, 3), (297, 3)], fused=True),
}


@pytest.mark.parametrize("case", sorted(FUSED_CASES))
def test_one_launch_step_matches_oracle(case):
    FUSED_CASES[case]()


TEAM_CASES = [c for c in sorted(FUSED_CASES) if not c.startswith(("tiny", "fp32"))]      # the team pipeline is bf16 only


@pytest.mark.parametrize("case", TEAM_CASES)
def test_one_launch_step_team_pipeline_matches_oracle(case):
    """The same cases with the team-pipeline kernel forced (automatically it only takes steps with split rows)."""
    STEP_KERNEL[0] = 2
    try:
        FUSED_CASES[case]()
    finally:
        STEP_KERNEL[0] = 0


ROWS_CASES = [c for c in TEAM_CASES if c.startswith(("base", "aan", "learned", "eq5"))]   # rows of at most 96 positions


@pytest.mark.parametrize("case", ROWS_CASES)
def test_one_launch_step_short_rows_kernel_matches_oracle(case):
    """The same cases with the short-rows kernel forced (whole planes per copy, scores in registers)."""
    STEP_KERNEL[0] = 3
    try:
        FUSED_CASES[case]()
    finally:
        STEP_KERNEL[0] = 0


def test_short_rows_kernel_every_length_up_to_its_limit():
    """One sentence per source length 1..96, decoded for 96 steps: every block count and every ragged tail."""
    w = dataclasses.replace(synth.WORKLOADS["base"], name="rows-all-lengths", n_sent=12, src_lo=1, src_hi=96,
                            tgt_rule="fixed", tgt_fixed=96, self_blocks=(1, 2, 3), encdec_blocks=(5, 1))
    STEP_KERNEL[0] = 3
    try:
        _run(w, fused=True)
    finally:
        STEP_KERNEL[0] = 0


def _rows_kernel_args(heads):
    """san_step_kernel_select arguments: short-rows kernel, heads per item for (self, encoder-decoder) attention."""
    return (3, -1, heads[0] + ((heads[1] + 1) << 8), 64, 0, 1)


@pytest.mark.parametrize("heads", [(1, 1), (2, 1), (2, 2), (4, 1), (4, 2)])
def test_short_rows_kernel_heads_per_item(heads):
    """Items of 1, 2 or 4 heads for self-attention and 1 or 2 for encoder-decoder attention, on rows short
    enough for four heads of a plane to fit a warp's ring (the kernel takes fewer where they would not)."""
    w = dataclasses.replace(synth.WORKLOADS["base"], name=f"rows-heads-{heads[0]}-{heads[1]}", n_sent=6, src_lo=5, src_hi=30,
                            tgt_rule="fixed", tgt_fixed=34, self_blocks=(3, 1, 2), encdec_blocks=(2, 4))
    STEP_KERNEL[0] = _rows_kernel_args(heads)
    try:
        _run(w, fused=True)
    finally:
        STEP_KERNEL[0] = 0
    dec = Decoder(w)
    B.check(B.san_step_kernel_select(dec.ctx, *_rows_kernel_args(heads)), "san_step_kernel_select")
    dec.load_encoder_memory()
    sb = dec.new_step_buffers()
    dec.fill_step_inputs(sb, 0, np.arange(w.n_seqs, dtype=np.int32), np.zeros(w.n_seqs, np.int32))
    dec.step_fused(sb)
    rc, which, rpu = B.san_step_kernel_used(dec.ctx)
    assert rc == 0 and which == 3 and rpu == [heads[0], heads[1]], (which, rpu)      # the first step's rows are one position long
    dec.close()


@pytest.mark.parametrize("kernel", [0, 2, 3])
@pytest.mark.parametrize("beam", [1, 2, 3, 5, 8, 12, 20])
def test_one_launch_step_other_beam_sizes(beam, kernel):
    w = dataclasses.replace(synth.scaled(synth.WORKLOADS["base"], 3), beam=beam, name=f"beam{beam}")
    STEP_KERNEL[0] = kernel
    try:
        _run(w, max_steps=5, fused=True)
    finally:
        STEP_KERNEL[0] = 0


def test_automatic_kernel_choice():
    """Rows long enough to be split over a team go to the team pipeline, sentence-sized rows to the per-warp kernel,
    launches without self-attention to the short-rows kernel."""
    for name, want in (("base", 1), ("long", 2)):
        w = synth.scaled(synth.WORKLOADS[name], 2)
        dec = Decoder(w)
        dec.load_encoder_memory()
        sb = dec.new_step_buffers()
        dec.fill_step_inputs(sb, 0, np.arange(w.n_seqs, dtype=np.int32), np.zeros(w.n_seqs, np.int32))
        dec.step_fused(sb)
        rc, which, rpu = B.san_step_kernel_used(dec.ctx)
        assert rc == 0 and which == want, (name, which, rpu)
        assert dec.device_status()[0] == 0
        dec.close()
    # a beam wider than one query group: the launches after the first hold encoder-decoder attention alone
    # and go to the short-rows kernel (the last launch is the one reported)
    w = dataclasses.replace(synth.scaled(synth.WORKLOADS["base"], 2), beam=12, name="beam12")
    dec = Decoder(w)
    dec.load_encoder_memory()
    sb = dec.new_step_buffers()
    dec.fill_step_inputs(sb, 0, np.arange(w.n_seqs, dtype=np.int32), np.zeros(w.n_seqs, np.int32))
    dec.step_fused(sb)
    rc, which, rpu = B.san_step_kernel_used(dec.ctx)
    assert rc == 0 and which == 3 and rpu[1] == 1, (which, rpu)
    assert dec.device_status()[0] == 0
    dec.close()


def test_one_launch_step_writes_the_cache_like_append():
    """After a fused step the caches hold this step's rows bit for bit (same as san_cache_append)."""
    w = synth.scaled(synth.WORKLOADS["base"], 3)
    a, b = Decoder(w), Decoder(w)
    for d in (a, b):
        d.cache.zero_()
        d.load_encoder_memory()
    ids = np.arange(w.n_seqs, dtype=np.int32)
    for step in range(4):
        pos = np.full(w.n_seqs, step, np.int32)
        sa, sb_ = a.new_step_buffers(), b.new_step_buffers()
        a.fill_step_inputs(sa, step, ids, pos)
        b.fill_step_inputs(sb_, step, ids, pos)
        a.step(sa)
        b.step_fused(sb_)
    torch.cuda.synchronize()
    assert a.device_status()[0] == 0 and b.device_status()[0] == 0
    assert torch.equal(a.cache, b.cache)
    a.close(); b.close()


@pytest.mark.parametrize("name", ["tiny", "aan"])
def test_host_buffer_step_equals_oracle(name):
    """san_decode_step_host: inputs in pinned host memory, outputs read back by the library."""
    w = synth.WORKLOADS[name] if name == "tiny" else synth.scaled(synth.WORKLOADS[name], 3)
    dec = Decoder(w)
    orc = OracleRun(w)
    dec.load_encoder_memory()
    ids = np.arange(w.n_seqs, dtype=np.int32)
    tol = TOL[w.dtype]
    for step in range(5):
        pos = np.full(w.n_seqs, step, np.int32)
        sb = dec.new_step_buffers()
        host = dec.fill_step_inputs(sb, step, ids, pos)
        hb = dec.host_buffers(sb, want_S=True)
        for k in hb["_in"]:                       # the device copies of the inputs must come from the host side
            if hb[k].dtype != torch.int32:
                getattr(sb, {"d_q_enc": "q_enc", "d_q_self": "q_self", "d_k_new": "k_new", "d_v_new": "v_new",
                             "d_x_aan": "x_aan"}[k]).zero_()
        dec.step_fused_host(sb, hb)
        torch.cuda.synchronize()
        assert dec.device_status()[0] == 0
        ref = orc.step(host, ids, pos)
        for key, want in (("d_O_self", ref["O_self"]), ("d_O_enc", ref["O_enc"])):
            assert normwise_err(hb[key].to(torch.float32).numpy(), want) <= tol, (name, step, key)
        L = step + 1
        if not w.self_is_aan:
            assert weights_err(hb["d_S_self"].numpy()[..., :L], ref["S_self"][..., :L]) <= TOL_S
        src_seq = np.repeat(w.src_lens(), w.beam)
        S = hb["d_S_enc"].numpy()
        for i in range(S.shape[1]):
            assert weights_err(S[:, i, :, :src_seq[i]], ref["S_enc"][:, i, :, :src_seq[i]]) <= TOL_S
    dec.close()
