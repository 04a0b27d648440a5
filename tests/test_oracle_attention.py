"""Pins for the CPU oracle's attention: none of these re-type the oracle's own loops.

Each test names what fixes the expected value: a library routine on a special
case, a closed form, an invariant, a hand-worked example or brute force.
"""
import math

import numpy as np
import pytest
import torch

from oracle import san_oracle as so
from paper_1906_11024_b200 import synth
from tests.helpers import compositions


def _fill(o, rng, M, n, H, dh, T, first_layers):
    """Append T random positions to every layer; returns K, V as [M, n, T, H, dh] float32."""
    K = rng.standard_normal((M, n, T, H, dh)).astype(np.float32)
    V = rng.standard_normal((M, n, T, H, dh)).astype(np.float32)
    ids = np.arange(n)
    for l in range(M):
        for t in range(T):
            o.self_append(l, ids, np.full(n, t), K[l, :, t] if l in first_layers else None, V[l, :, t])
    return K, V


def test_block_size_one_is_textbook_multihead_attention():
    """Eq. 1-2 with no sharing: equals torch's scaled_dot_product_attention in float64."""
    rng = np.random.default_rng(10)
    M, n, H, dh, T = 3, 5, 4, 64, 23
    o = so.Oracle(M, H, dh, n, 1, T, 4, [1] * M, [1] * M)
    K, V = _fill(o, rng, M, n, H, dh, T, set(range(M)))
    lens = rng.integers(1, T + 1, size=n)
    for l in range(M):
        q = rng.standard_normal((n, H, dh)).astype(np.float32)
        S, O = o.self_attend(l, np.arange(n), lens, q)
        for s in range(n):
            L = int(lens[s])
            tq = torch.from_numpy(q[s].astype(np.float64))[:, None, :]                 # [H,1,dh]
            tk = torch.from_numpy(K[l, s, :L].astype(np.float64)).permute(1, 0, 2)    # [H,L,dh]
            tv = torch.from_numpy(V[l, s, :L].astype(np.float64)).permute(1, 0, 2)
            ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, scale=1.0 / math.sqrt(dh))
            np.testing.assert_allclose(O[s], ref[:, 0, :].numpy(), rtol=1e-12, atol=1e-13)
            assert np.all(S[s, :, L:] == 0.0)


def test_softmax_without_max_subtraction_extended_precision():
    """S equals exp(z)/sum exp(z) evaluated directly in long double (no max trick)."""
    rng = np.random.default_rng(11)
    n, H, dh, T = 3, 2, 64, 17
    o = so.Oracle(1, H, dh, n, 1, T, 4, [1], [1])
    K, V = _fill(o, rng, 1, n, H, dh, T, {0})
    q = rng.standard_normal((n, H, dh)).astype(np.float32)
    S, _ = o.self_attend(0, np.arange(n), np.full(n, T), q)
    z = np.einsum("nhd,nthd->nht", q.astype(np.longdouble), K[0].astype(np.longdouble)) / np.sqrt(np.longdouble(dh))
    e = np.exp(z)
    ref = e / e.sum(-1, keepdims=True)
    np.testing.assert_allclose(S, ref.astype(np.float64), rtol=1e-13, atol=1e-16)


def test_rows_of_S_are_distributions():
    rng = np.random.default_rng(12)
    n, H, dh, T = 6, 8, 64, 40
    o = so.Oracle(2, H, dh, n, 1, T, 4, [2], [2])
    _fill(o, rng, 2, n, H, dh, T, {0})
    lens = rng.integers(1, T + 1, size=n)
    S, _ = o.self_attend(0, np.arange(n), lens, (5 * rng.standard_normal((n, H, dh))).astype(np.float32))
    assert np.all(S >= 0.0) and np.all(S <= 1.0)
    np.testing.assert_allclose(S.sum(-1), 1.0, rtol=0, atol=1e-12)


def test_shared_layer_applies_first_layers_weights_to_its_own_values():
    """Eq. 4: O of layer m+i = S^m . V^{m+i}, recomputed with a separate numpy matmul."""
    rng = np.random.default_rng(13)
    M, n, H, dh, T = 6, 4, 8, 64, 19
    sizes = [2, 3, 1]
    first = {0, 2, 5}
    o = so.Oracle(M, H, dh, n, 1, T, 4, sizes, [M])
    K, V = _fill(o, rng, M, n, H, dh, T, first)
    lens = rng.integers(1, T + 1, size=n)
    bol, fl = so.policy_from_sizes(sizes, M)
    S_first = {}
    for l in range(M):
        is_first = l in first
        q = rng.standard_normal((n, H, dh)).astype(np.float32) if is_first else None
        S, O = o.self_attend(l, np.arange(n), lens, q)
        if is_first:
            S_first[bol[l]] = S.copy()
        np.testing.assert_array_equal(S, S_first[bol[l]])      # the very same weights
        for s in range(n):
            L = int(lens[s])
            ref = np.einsum("ht,thd->hd", S_first[bol[l]][s, :, :L], V[l, s, :L].astype(np.float64))
            np.testing.assert_allclose(O[s], ref, rtol=0, atol=1e-13)


def test_shared_layer_never_reads_its_own_keys_or_query():
    """A non-first layer gets no q and no K, and still produces S^m . V."""
    rng = np.random.default_rng(14)
    n, H, dh, T = 2, 2, 64, 7
    o = so.Oracle(2, H, dh, n, 1, T, 4, [2], [2])
    K, V = _fill(o, rng, 2, n, H, dh, T, {0})
    q = rng.standard_normal((n, H, dh)).astype(np.float32)
    S0, _ = o.self_attend(0, np.arange(n), np.full(n, T), q)
    S1, O1 = o.self_attend(1, np.arange(n), np.full(n, T), None)
    np.testing.assert_array_equal(S0, S1)
    np.testing.assert_allclose(O1, np.einsum("nht,nthd->nhd", S0, V[1].astype(np.float64)), atol=1e-13)
    with pytest.raises(so.OracleError):
        o.self_attend(0, np.arange(n), np.full(n, T), None)    # a first layer needs its query


def test_hand_worked_example():
    """d_h = 4 so the scale is 1/2; q = (2,0,0,0); keys (0,..), (ln2,..), (ln3,..).
    z = (0, ln2, ln3), so S = (1,2,3)/6.  Values with first column (6,12,18) give 14; a
    second layer of the same block with first column (6,0,0) gives 1."""
    o = so.Oracle(2, 1, 4, 1, 1, 3, 1, [2], [2])
    keys = [0.0, math.log(2.0), math.log(3.0)]
    v0, v1 = [6.0, 12.0, 18.0], [6.0, 0.0, 0.0]
    for t in range(3):
        k = np.array([[[keys[t], 0, 0, 0]]], np.float32)
        o.self_append(0, [0], [t], k, np.array([[[v0[t], 1, 0, -1]]], np.float32))
        o.self_append(1, [0], [t], None, np.array([[[v1[t], 2, 0, 0]]], np.float32))
    S, O = o.self_attend(0, [0], [3], np.array([[[2.0, 0, 0, 0]]], np.float32))
    # float32 storage of ln2, ln3 perturbs z by ~1e-8
    np.testing.assert_allclose(S[0, 0], [1 / 6, 1 / 3, 1 / 2], rtol=0, atol=1e-7)
    np.testing.assert_allclose(O[0, 0], [14.0, 1.0, 0.0, -1.0], rtol=0, atol=2e-6)
    _, O1 = o.self_attend(1, [0], [3], None)
    np.testing.assert_allclose(O1[0, 0], [1.0, 2.0, 0.0, 0.0], rtol=0, atol=2e-6)


def test_closed_forms():
    rng = np.random.default_rng(15)
    n, H, dh, T = 3, 2, 64, 11
    o = so.Oracle(1, H, dh, n, 1, T, 4, [1], [1])
    K, V = _fill(o, rng, 1, n, H, dh, T, {0})
    ids = np.arange(n)
    q = rng.standard_normal((n, H, dh)).astype(np.float32)
    # (i) a cache of one position: S = [1], O = V_0
    S, O = o.self_attend(0, ids, np.ones(n), q)
    np.testing.assert_array_equal(S[:, :, 0], 1.0)
    np.testing.assert_array_equal(O, V[0, :, 0].astype(np.float64))
    # (ii) q = 0: uniform weights and O = prefix mean of V
    lens = np.array([T, 5, 2])
    S, O = o.self_attend(0, ids, lens, np.zeros_like(q))
    for s in range(n):
        np.testing.assert_allclose(S[s, :, :lens[s]], 1.0 / lens[s], rtol=1e-15)
        np.testing.assert_allclose(O[s], V[0, s, :lens[s]].astype(np.float64).mean(0), atol=1e-14)
    # (iii) adding the same vector c to every key leaves S unchanged
    S_ref, O_ref = o.self_attend(0, ids, np.full(n, T), q)
    c = rng.standard_normal((1, H, dh)).astype(np.float32)
    o2 = so.Oracle(1, H, dh, n, 1, T, 4, [1], [1])
    for t in range(T):
        o2.self_append(0, ids, np.full(n, t), K[0, :, t] + c, V[0, :, t])
    S2, _ = o2.self_attend(0, ids, np.full(n, T), q)
    np.testing.assert_allclose(S2, S_ref, rtol=0, atol=2e-6)        # K + c rounds in float32
    # (iv) permuting cache positions permutes S and leaves O unchanged
    perm = rng.permutation(T)
    o3 = so.Oracle(1, H, dh, n, 1, T, 4, [1], [1])
    for t in range(T):
        o3.self_append(0, ids, np.full(n, t), K[0, :, perm[t]], V[0, :, perm[t]])
    S3, O3 = o3.self_attend(0, ids, np.full(n, T), q)
    np.testing.assert_allclose(S3, S_ref[:, :, perm], rtol=1e-13)
    np.testing.assert_allclose(O3, O_ref, atol=1e-13)
    # (v) one key aligned with a huge query: S -> one-hot, O -> that position's value
    o4 = so.Oracle(1, 1, dh, 1, 1, T, 4, [1], [1])
    for t in range(T):
        k = np.zeros((1, 1, dh), np.float32)
        k[0, 0, t] = 1.0
        o4.self_append(0, [0], [t], k, V[0, :1, t, :1])
    qq = np.zeros((1, 1, dh), np.float32)
    qq[0, 0, 6] = 4000.0
    S4, O4 = o4.self_attend(0, [0], [T], qq)
    assert S4[0, 0, 6] == 1.0 and S4[0, 0].sum() == 1.0
    np.testing.assert_array_equal(O4[0, 0], V[0, 0, 6, 0].astype(np.float64))


def test_aan_is_the_prefix_mean_and_matches_uniform_attention():
    rng = np.random.default_rng(16)
    n, H, dh, T = 3, 2, 64, 9
    d = H * dh
    o = so.Oracle(2, H, dh, n, 1, T, 4, [1, 1], [2])
    X = rng.standard_normal((T, n, d)).astype(np.float32)
    ids = np.arange(n)
    outs = np.stack([o.aan_step(1, ids, np.full(n, t + 1), X[t]) for t in range(T)])
    ref = np.cumsum(X.astype(np.float64), 0) / np.arange(1, T + 1)[:, None, None]
    np.testing.assert_allclose(outs, ref, rtol=0, atol=1e-14)
    np.testing.assert_array_equal(outs[0], X[0].astype(np.float64))             # t = 1 returns x_1
    c = np.full((n, d), 0.375, np.float32)
    o2 = so.Oracle(1, H, dh, n, 1, T, 4, [1], [1])
    for t in range(T):
        np.testing.assert_array_equal(o2.aan_step(0, ids, np.full(n, t + 1), c), 0.375)
    # the same rows as cached values under uniform attention (q = 0) give the same mean
    o3 = so.Oracle(1, H, dh, n, 1, T, 4, [1], [1])
    for t in range(T):
        o3.self_append(0, ids, np.full(n, t), np.zeros((n, H, dh), np.float32), X[t].reshape(n, H, dh))
    _, O = o3.self_attend(0, ids, np.full(n, T), np.zeros((n, H, dh), np.float32))
    np.testing.assert_allclose(O.reshape(n, d), outs[-1], atol=1e-14)
    # ragged counts: sequences at different t in one call
    o4 = so.Oracle(1, H, dh, n, 1, T, 4, [1], [1])
    for t in range(3):
        o4.aan_step(0, [0, 1], [t + 1, t + 1], X[t, :2])
    got = o4.aan_step(0, [2, 0], [1, 4], X[3, [2, 0]])
    np.testing.assert_array_equal(got[0], X[3, 2].astype(np.float64))
    np.testing.assert_allclose(got[1], X[:4, 0].astype(np.float64).mean(0), atol=1e-14)


@pytest.mark.parametrize("dh", [4, 64])
def test_brute_force_every_policy_of_tiny_stacks(dh):
    """Every composition of M <= 3 layers: the oracle equals a per-layer restatement that
    recomputes S from the block's lowest layer with plain Python loops."""
    rng = np.random.default_rng(17)
    n, H = 2, 2
    for M in (1, 2, 3):
        for sizes in compositions(M):
            T = int(rng.integers(1, 6))
            bol, first = so.policy_from_sizes(sizes, M)
            o = so.Oracle(M, H, dh, n, 1, T, 4, sizes, [M])
            K, V = _fill(o, rng, M, n, H, dh, T, set(first.tolist()))
            Q = rng.standard_normal((M, n, H, dh)).astype(np.float32)
            lens = rng.integers(1, T + 1, size=n)
            for l in range(M):
                m = int(first[bol[l]])
                _, O = o.self_attend(l, np.arange(n), lens, Q[l] if l == m else None)
                for s in range(n):
                    for h in range(H):
                        L = int(lens[s])
                        z = [sum(float(Q[m, s, h, d]) * float(K[m, s, j, h, d]) for d in range(dh)) / math.sqrt(dh)
                             for j in range(L)]
                        e = [math.exp(x) for x in z]
                        for d in range(dh):
                            ref = sum(e[j] / sum(e) * float(V[l, s, j, h, d]) for j in range(L))
                            assert abs(O[s, h, d] - ref) <= 1e-12 * max(1.0, abs(ref))


def test_encdec_beams_share_memory_and_both_value_modes():
    """Keys and values come from the encoder output (Section 2): all beams of a sentence
    read the same rows.  Own-V mode (Table 4, 'Shared V = no') applies the block's S to
    each layer's own memory values; shared-context mode (Eq. 5) returns the first layer's
    output for every layer of the block."""
    rng = np.random.default_rng(18)
    M, H, dh, n_sent, beam, Ls_max = 4, 2, 64, 3, 2, 9
    src = [9, 1, 5]
    Kmem = rng.standard_normal((M, n_sent, Ls_max, H, dh)).astype(np.float32)
    Vmem = rng.standard_normal((M, n_sent, Ls_max, H, dh)).astype(np.float32)
    sizes = [3, 1]
    first = {0, 3}
    n = n_sent * beam
    q = rng.standard_normal((M, n, H, dh)).astype(np.float32)
    for shared_ctx in (False, True):
        o = so.Oracle(M, H, dh, n_sent, beam, 4, Ls_max, [M], sizes, shared_ctx)
        for l in range(M):
            for g in range(n_sent):
                o.mem_set(l, g, Kmem[l, g, :src[g]] if l in first else None, Vmem[l, g, :src[g]])
        ids = np.arange(n)
        O_first = None
        for l in range(M):
            m = 0 if l < 3 else 3
            S, O = o.encdec_attend(l, ids, q[l] if l in first else None)
            if l in first:
                O_first = O.copy()
            for s in range(n):
                g, L = s // beam, src[s // beam]
                tq = torch.from_numpy(q[m, s].astype(np.float64))[:, None, :]
                tk = torch.from_numpy(Kmem[m, g, :L].astype(np.float64)).permute(1, 0, 2)
                vl = m if shared_ctx else l
                tv = torch.from_numpy(Vmem[vl, g, :L].astype(np.float64)).permute(1, 0, 2)
                ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, scale=1 / math.sqrt(dh))
                np.testing.assert_allclose(O[s], ref[:, 0].numpy(), rtol=1e-12, atol=1e-13)
                np.testing.assert_allclose(S[s, :, :L].sum(-1), 1.0, atol=1e-12)
            if shared_ctx:
                np.testing.assert_array_equal(O, O_first)
    # Eq. 5 premise: when the layers' values are the same tensor, own-V mode gives equal outputs
    o = so.Oracle(2, H, dh, n_sent, beam, 4, Ls_max, [2], [2], False)
    for l in range(2):
        for g in range(n_sent):
            o.mem_set(l, g, Kmem[0, g, :src[g]] if l == 0 else None, Vmem[0, g, :src[g]])
    _, Oa = o.encdec_attend(0, np.arange(n), q[0])
    _, Ob = o.encdec_attend(1, np.arange(n), None)
    np.testing.assert_array_equal(Oa, Ob)


def test_subset_of_sequences_and_order_of_ids():
    """Finished sequences drop out of the id list; results do not depend on list order."""
    rng = np.random.default_rng(19)
    n, H, dh, T = 6, 2, 64, 8
    o = so.Oracle(1, H, dh, n, 1, T, 4, [1], [1])
    _fill(o, rng, 1, n, H, dh, T, {0})
    q = rng.standard_normal((n, H, dh)).astype(np.float32)
    lens = rng.integers(1, T + 1, size=n)
    S_all, O_all = o.self_attend(0, np.arange(n), lens, q)
    pick = np.array([4, 1, 5])
    S_p, O_p = o.self_attend(0, pick, lens[pick], q[pick])
    np.testing.assert_array_equal(S_p, S_all[pick])
    np.testing.assert_array_equal(O_p, O_all[pick])


def test_beam_reorder_is_a_gather_of_cached_rows():
    rng = np.random.default_rng(20)
    M, n_sent, beam, H, dh, T = 2, 2, 3, 2, 64, 6
    n = n_sent * beam
    o = so.Oracle(M, H, dh, n_sent, beam, T, 4, [1, 1], [2])
    K, V = _fill(o, rng, M, n, H, dh, T, {0, 1})
    src = np.array([2, 0, 0, 4, 4, 3])          # parents stay within a sentence's beams
    lens = np.array([6, 4, 6, 5, 5, 1])
    o.beam_reorder(src, lens)
    q = rng.standard_normal((n, H, dh)).astype(np.float32)
    for l in range(M):
        _, O = o.self_attend(l, np.arange(n), lens, q)
        for s in range(n):
            L = int(lens[s])
            tq = torch.from_numpy(q[s].astype(np.float64))[:, None, :]
            tk = torch.from_numpy(K[l, src[s], :L].astype(np.float64)).permute(1, 0, 2)
            tv = torch.from_numpy(V[l, src[s], :L].astype(np.float64)).permute(1, 0, 2)
            ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, scale=1 / math.sqrt(dh))
            np.testing.assert_allclose(O[s], ref[:, 0].numpy(), rtol=1e-12, atol=1e-13)


def test_beam_reorder_carries_the_running_average_of_the_parent():
    """With average attention a hypothesis continues the prefix mean of the hypothesis it
    extends: after a reorder, the next step's output is the mean of the PARENT's inputs at
    positions 1..len plus the new input, written out here with cumsum/arange over the gathered
    parent rows.  Parents differ per beam and one hypothesis keeps a shorter prefix."""
    rng = np.random.default_rng(22)
    M, n_sent, beam, H, dh, T = 2, 2, 3, 2, 64, 7
    n, d = n_sent * beam, H * dh
    o = so.Oracle(M, H, dh, n_sent, beam, T, 4, [1, 1], [2])
    hist = 5
    X = rng.standard_normal((M, hist, n, d)).astype(np.float32)
    ids = np.arange(n)
    for l in range(M):
        for t in range(hist):
            o.aan_step(l, ids, np.full(n, t + 1), X[l, t])
    src = np.array([1, 2, 0, 5, 3, 3])            # every beam changes parent, two share one
    lens = np.array([5, 5, 3, 5, 5, 5])           # sequence 2 keeps only 3 positions of its parent
    o.beam_reorder(src, lens)
    x_new = rng.standard_normal((M, n, d)).astype(np.float32)
    for l in range(M):
        got = o.aan_step(l, ids, lens + 1, x_new[l])
        for s in range(n):
            L = int(lens[s])
            rows = np.concatenate([X[l, :L, src[s]], x_new[l, s][None]], 0).astype(np.float64)
            ref = (np.cumsum(rows, 0) / np.arange(1, L + 2)[:, None])[-1]
            np.testing.assert_allclose(got[s], ref, rtol=0, atol=1e-14)
            assert np.abs(got[s] - (X[l, :L, s].astype(np.float64).sum(0) + x_new[l, s]) / (L + 1)).max() > 1e-3


@pytest.mark.parametrize("causal", [False, True])
def test_full_sequence_block_matches_library_attention(causal):
    """Encoder-side SAN (Table 5): S is l x l, computed once, applied to each layer's V."""
    rng = np.random.default_rng(21)
    l, H, dh, nl = 13, 3, 64, 3
    Q = rng.standard_normal((l, H, dh)).astype(np.float32)
    K = rng.standard_normal((l, H, dh)).astype(np.float32)
    V = rng.standard_normal((nl, l, H, dh)).astype(np.float32)
    S, O = so.full_block(Q, K, V, causal)
    tq = torch.from_numpy(Q.astype(np.float64)).permute(1, 0, 2)
    tk = torch.from_numpy(K.astype(np.float64)).permute(1, 0, 2)
    for a in range(nl):
        tv = torch.from_numpy(V[a].astype(np.float64)).permute(1, 0, 2)
        ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=causal, scale=1 / math.sqrt(dh))
        np.testing.assert_allclose(O[a], ref.permute(1, 0, 2).numpy(), rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(S.sum(-1), 1.0, atol=1e-12)
    if causal:
        assert np.all(np.triu(S, 1) == 0.0)


def test_oracle_rejects_bad_arguments():
    o = so.Oracle(2, 1, 4, 2, 1, 3, 2, [2], [2])
    v = np.zeros((1, 1, 4), np.float32)
    with pytest.raises(so.OracleError):
        o.self_append(0, [0], [3], v, v)            # position beyond capacity
    with pytest.raises(so.OracleError):
        o.self_append(2, [0], [0], v, v)            # no such layer
    with pytest.raises(so.OracleError):
        o.self_attend(0, [0], [0], v)               # empty cache
    with pytest.raises(so.OracleError):
        o.encdec_attend(0, [0], v)                  # memory never set
    with pytest.raises(so.OracleError):
        o.aan_step(0, [0], [0], np.zeros((1, 4), np.float32))
