"""Full-sequence shared attention (san_full_block) against the oracle: S within 1e-5
element-wise (relative, floor 1e-7), outputs within 1e-2 per vector (bf16 inputs and outputs,
float32 accumulation)."""
import numpy as np
import pytest
import torch

from oracle import san_oracle as so
from paper_1906_11024_b200 import binding as B
from paper_1906_11024_b200 import build as san_build
from paper_1906_11024_b200 import synth
from paper_1906_11024_b200.driver import to_device, to_host_f32
from tests.helpers import TOL, TOL_S, normwise_err, weights_err

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    san_build.build()
    B.lib()


def _inputs(seed, n_seq, cap, H, n_layers):
    rng = np.random.default_rng([seed, n_seq, cap, H])
    r = lambda *shape: synth.round_to_bf16(rng.standard_normal(shape, dtype=np.float32))
    return r(n_seq, cap, H, 64), r(n_seq, cap, H, 64), r(n_layers, n_seq, cap, H, 64)


def _run(lens, cap, H, n_layers, causal, max_len=0, want_S=True, seed=3):
    n_seq = len(lens)
    Q, K, V = _inputs(seed, n_seq, cap, H, n_layers)
    dev = "cuda"
    dq, dk, dv = (to_device(x, synth.BF16, dev) for x in (Q, K, V))
    dl = torch.tensor(lens, dtype=torch.int32, device=dev)
    ld = cap + 3
    dS = torch.full((n_seq, H, cap, ld), -7.0, dtype=torch.float32, device=dev) if want_S else None
    dO = torch.full((n_layers, n_seq, cap, H, 64), -7.0, dtype=torch.bfloat16, device=dev)
    rc = B.san_full_block(B.SAN_BF16, H, n_layers, causal, dq, dk, dv, dl, n_seq, cap, max_len, dS, ld, dO)
    assert rc == B.SAN_OK
    torch.cuda.synchronize()
    O = to_host_f32(dO)
    S = dS.cpu().numpy() if want_S else None
    for i, l in enumerate(lens):
        if l == 0:
            assert (O[:, i] == -7.0).all()
            continue
        S_ref, O_ref = so.full_block(Q[i, :l], K[i, :l], V[:, i, :l], causal)
        assert normwise_err(O[:, i, :l], O_ref) <= TOL[synth.BF16], (i, l)
        assert (O[:, i, l:] == -7.0).all()                       # rows beyond the sequence are not written
        if want_S:
            assert weights_err(S[i, :, :l, :l], S_ref) <= TOL_S, (i, l)
            assert np.abs(S[i, :, :l, :l].astype(np.float64).sum(-1) - 1.0).max() <= 1e-5
            assert (S[i, :, :l, l:] == -7.0).all() and (S[i, :, l:] == -7.0).all()


@pytest.mark.parametrize("causal", [False, True])
def test_ragged_batch_short_sentences(causal):
    """Encoder-sized sentences: lengths around the 16-row warp tile and the 64-row CTA tile."""
    _run([1, 2, 15, 16, 17, 63, 64, 65, 80, 33, 0], cap=80, H=3, n_layers=3, causal=causal)


@pytest.mark.parametrize("causal", [False, True])
def test_long_sequences_several_key_chunks(causal):
    _run([300, 257, 129, 512], cap=512, H=2, n_layers=2, causal=causal)


def test_block_of_one_layer_and_of_six_without_S():
    _run([40, 70], cap=72, H=8, n_layers=1, causal=False)
    _run([40, 70], cap=72, H=8, n_layers=6, causal=False, want_S=False)


def test_host_bound_cuts_longer_sequences():
    """max_len below a length: the sequence is treated as max_len long (documented)."""
    n_seq, cap, H = 2, 96, 2
    Q, K, V = _inputs(9, n_seq, cap, H, 2)
    dq, dk, dv = (to_device(x, synth.BF16, "cuda") for x in (Q, K, V))
    dl = torch.tensor([96, 50], dtype=torch.int32, device="cuda")
    dO = torch.zeros((2, n_seq, cap, H, 64), dtype=torch.bfloat16, device="cuda")
    assert B.san_full_block(B.SAN_BF16, H, 2, 0, dq, dk, dv, dl, n_seq, cap, 64, None, 0, dO) == B.SAN_OK
    O = to_host_f32(dO)
    for i, l in enumerate([64, 50]):
        _, O_ref = so.full_block(Q[i, :l], K[i, :l], V[:, i, :l], False)
        assert normwise_err(O[:, i, :l], O_ref) <= TOL[synth.BF16]


def test_argument_checks():
    t = torch.zeros(64, dtype=torch.bfloat16, device="cuda")
    l = torch.ones(1, dtype=torch.int32, device="cuda")
    f = B.san_full_block
    assert f(B.SAN_BF16, 1, 1, 0, None, t, t, l, 1, 1, 0, None, 0, t) == B.SAN_ERR_NULL
    assert f(B.SAN_F32, 1, 1, 0, t, t, t, l, 1, 1, 0, None, 0, t) == B.SAN_ERR_UNSUPPORTED
    assert f(B.SAN_BF16, 1, 7, 0, t, t, t, l, 1, 1024, 0, None, 0, t) == B.SAN_ERR_UNSUPPORTED   # 7 layers: mma.sync kernel, 512 at most
    assert f(B.SAN_BF16, 1, 1, 0, t, t, t, l, 1, 1, 2, None, 0, t) == B.SAN_ERR_SHAPE
    assert f(B.SAN_BF16, 1, 1, 0, t, t, t, l, 0, 1, 0, None, 0, t) == B.SAN_OK


@pytest.mark.parametrize("causal", [False, True])
def test_tensor_memory_path_ragged_lengths(causal):
    """A length bound of 128 or more selects the tcgen05 kernel (128-query tiles, accumulators in
    tensor memory): lengths on both sides of the 64-key chunk and the 128-query tile, an empty
    and a one-token sequence in the same batch."""
    _run([1, 63, 64, 65, 127, 128, 129, 200, 0], cap=200, H=2, n_layers=3, causal=causal)


def test_tensor_memory_path_beyond_512_positions():
    """The tcgen05 kernel streams the keys in chunks and has no length limit of its own."""
    _run([700, 513], cap=704, H=1, n_layers=2, causal=True)


def test_tensor_memory_path_one_and_six_layers():
    _run([150, 333], cap=336, H=3, n_layers=1, causal=False)
    _run([150, 333], cap=336, H=3, n_layers=6, causal=True, want_S=False)
