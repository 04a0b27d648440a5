"""Device part of the policy learner (san_js_matrix) against the oracle.

Tolerance: the kernel takes the fast logarithm (absolute error about 2^-21 on (0, 2]) of
float32 ratios and sums a row in float32; every term x*ln(x/m) carries an error of a few 1e-7
times x and the x of a row sum to one, so a (row, head) value is within about 1e-6 absolute of
the double result, and so is the mean."""
import math

import numpy as np
import pytest
import torch

from oracle import san_oracle as so
from paper_1906_11024_b200 import binding as B
from paper_1906_11024_b200 import build as san_build
from paper_1906_11024_b200 import synth
from paper_1906_11024_b200.driver import Decoder, to_host_f32
from tests.helpers import OracleRun

pytestmark = pytest.mark.gpu
TOL_JS = 2e-6


@pytest.fixture(scope="module", autouse=True)
def _built():
    san_build.build()
    B.lib()


def _oracle_matrix(S64, lens):
    M = S64.shape[0]
    js = np.zeros((M, M))
    for a in range(M):
        for b in range(a + 1, M):
            js[a, b] = js[b, a] = so.layer_js(S64[a], S64[b], lens)
    return js


@pytest.mark.parametrize("M,n,H,ld", [(6, 37, 8, 70), (2, 1, 1, 1), (12, 5, 3, 520), (3, 300, 2, 33)])
def test_js_matrix_on_seeded_distributions(M, n, H, ld):
    """Seeded float32 distributions (softmax of scaled normals, some exact zeros, ragged
    lengths including 0 and 1): both sides get the same float32 values."""
    rng = np.random.default_rng([7, M, n, ld])
    lens = rng.integers(0, ld + 1, size=n).astype(np.int32)
    lens[0] = ld
    if n > 1:
        lens[1] = 1
    S = np.zeros((M, n, H, ld), np.float32)
    for l in range(M):
        z = rng.standard_normal((n, H, ld)) * (0.5 + l)
        for i in range(n):
            L = lens[i]
            if L == 0:
                continue
            e = np.exp(z[i, :, :L] - z[i, :, :L].max(-1, keepdims=True))
            e[:, rng.random(L) < 0.1] *= (L == 1)          # exact zeros: 0 ln 0 = 0
            if not e.sum(-1).all():
                e[:, 0] = 1.0
            S[l, i, :, :L] = (e / e.sum(-1, keepdims=True)).astype(np.float32)
    want = _oracle_matrix(S.astype(np.float64), lens)
    dS = torch.from_numpy(S).cuda()
    dl = torch.from_numpy(lens).cuda()
    djs = torch.full((M, M), 123.0, dtype=torch.float64, device="cuda")        # cleared by the call
    B.check(B.san_js_matrix(M, dS, n * H * ld, ld, n, H, dl, djs), "san_js_matrix")
    got = djs.cpu().numpy()
    assert np.array_equal(got, got.T) and not got.diagonal().any()
    assert np.abs(got - want).max() <= TOL_JS
    assert got.min() >= 0.0 and got.max() <= math.log(2) + TOL_JS


def test_identical_and_disjoint_layers():
    """Closed forms: equal layers give 0, layers with disjoint supports give ln 2."""
    n, H, ld = 9, 2, 40
    a = np.zeros((n, H, ld), np.float32); a[..., :20] = 1.0 / 20
    b = np.zeros((n, H, ld), np.float32); b[..., 20:] = 1.0 / 20
    S = np.stack([a, a, b])
    djs = torch.zeros(3, 3, dtype=torch.float64, device="cuda")
    lens = torch.full((n,), ld, dtype=torch.int32, device="cuda")
    B.check(B.san_js_matrix(3, torch.from_numpy(S).cuda(), n * H * ld, ld, n, H, lens, djs), "san_js_matrix")
    got = djs.cpu().numpy()
    assert got[0, 1] == 0.0
    assert got[0, 2] == pytest.approx(math.log(2), abs=TOL_JS) and got[1, 2] == pytest.approx(math.log(2), abs=TOL_JS)


def test_policy_learned_from_an_unshared_decode_step():
    """The whole learner: decode with block size 1 so that every layer writes its own S, take
    the JS matrix of those weights on the device, search the policy on the host.  The oracle
    does the same from its own S.  Thresholds are taken midway between the similarity values
    the oracle sees, so that the float32 weights cannot tip a decision."""
    w = synth.unshared(synth.scaled(synth.WORKLOADS["base"], 6))
    dec = Decoder(w)
    orc = OracleRun(w)
    dec.load_encoder_memory()
    ids = np.arange(w.n_seqs, dtype=np.int32)
    for step in range(7):
        pos = np.full(w.n_seqs, step, np.int32)
        sb = dec.new_step_buffers()
        host = dec.fill_step_inputs(sb, step, ids, pos)
        dec.step_fused(sb)
        ref = orc.step(host, ids, pos)
    assert dec.device_status()[0] == 0
    M, H = w.n_layers, w.n_heads
    src_seq = np.repeat(w.src_lens(), w.beam).astype(np.int32)
    for S_dev, S_ref, lens, ld in ((sb.S_self, ref["S_self"], np.full(w.n_seqs, 7, np.int32), dec.ld_t),
                                   (sb.S_enc, ref["S_enc"], src_seq, dec.ld_s)):
        djs = torch.zeros(M, M, dtype=torch.float64, device="cuda")
        B.check(B.san_js_matrix(M, S_dev, S_dev.stride(0), ld, w.n_seqs, H, torch.from_numpy(lens).cuda(), djs), "js")
        got = djs.cpu().numpy()
        want = _oracle_matrix(np.ascontiguousarray(S_ref), lens)
        assert np.abs(got - want).max() <= 1e-5          # S itself differs by up to 1e-5 relative
        sims = sorted({so.block_sim(want, m, n) for m in range(1, M) for n in range(m + 1, M + 1)})
        thetas = [(a + b) / 2 for a, b in zip(sims, sims[1:]) if b - a > 1e-3][:12]
        assert thetas
        for theta in thetas:
            rc, sizes = B.san_policy_search(got, M, theta)
            assert rc == B.SAN_OK and sizes == so.greedy_policy(want, theta)
    dec.close()
