"""Pins for the oracle's integer policy tables and the policy learner (Eq. 6, Section 3.3)."""
import math
import os

import numpy as np
import pytest
from scipy.spatial.distance import jensenshannon

from oracle import san_oracle as so

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _fig2(name):
    return np.loadtxt(os.path.join(GOLD, name), comments="#")


@pytest.mark.parametrize("sizes,expect_map,expect_first", [
    ((2, 2, 2), [0, 0, 1, 1, 2, 2], [0, 2, 4]),
    ((3, 3), [0, 0, 0, 1, 1, 1], [0, 3]),
    ((6,), [0, 0, 0, 0, 0, 0], [0]),
    ((4, 4, 4), [0, 0, 0, 0, 1, 1, 1, 1, 2, 2, 2, 2], [0, 4, 8]),
    ((12,), [0] * 12, [0]),
    ((1, 5), [0, 1, 1, 1, 1, 1], [0, 1]),
    ((1, 1, 1, 1, 1, 1), [0, 1, 2, 3, 4, 5], [0, 1, 2, 3, 4, 5]),
    ((2, 4), [0, 0, 1, 1, 1, 1], [0, 2]),      # the pi_1 = 2, pi_2 = 4 example of Section 3.2
])
def test_block_tables_listed_explicitly(sizes, expect_map, expect_first):
    bol, first = so.policy_from_sizes(sizes, sum(sizes))
    assert bol.tolist() == expect_map and first.tolist() == expect_first
    s2, f2 = so.policy_from_map(expect_map)
    assert s2.tolist() == list(sizes) and f2.tolist() == expect_first


@pytest.mark.parametrize("sizes,M", [((2, 2), 6), ((3, 4), 6), ((2, 0, 4), 6), ((-1, 7), 6), ((), 6)])
def test_invalid_sizes_rejected(sizes, M):
    with pytest.raises(so.OracleError):
        so.policy_from_sizes(sizes, M)


@pytest.mark.parametrize("bmap", [[1, 1, 2], [0, 2, 2], [0, 1, 0], [0, 0, -1]])
def test_invalid_maps_rejected(bmap):
    with pytest.raises(so.OracleError):
        so.policy_from_map(bmap)


def test_js_divergence_properties_and_library_value():
    rng = np.random.default_rng(30)
    p = rng.random(17); p /= p.sum()
    q = rng.random(17); q /= q.sum()
    assert so.js_divergence(p, p) == 0.0
    assert so.js_divergence(p, q) == pytest.approx(so.js_divergence(q, p), rel=1e-15)
    a = np.array([0.5, 0.5, 0.0, 0.0]); b = np.array([0.0, 0.0, 0.25, 0.75])
    assert so.js_divergence(a, b) == pytest.approx(math.log(2.0), rel=1e-15)    # disjoint supports: the bound
    assert 0.0 < so.js_divergence(p, q) < math.log(2.0)
    assert so.js_divergence(p, q) == pytest.approx(jensenshannon(p, q) ** 2, rel=1e-12)   # scipy returns the root
    # p = (1,0), q = (1/2,1/2): JS = 3/4 ln(4/3) + 1/4 ln 2 - ... worked out by hand:
    # m = (3/4, 1/4); KL(p||m) = ln(4/3); KL(q||m) = 1/2 ln(2/3) + 1/2 ln 2
    hand = 0.5 * math.log(4 / 3) + 0.5 * (0.5 * math.log(2 / 3) + 0.5 * math.log(2.0))
    assert so.js_divergence([1.0, 0.0], [0.5, 0.5]) == pytest.approx(hand, rel=1e-14)


def test_layer_js_averages_over_rows_and_heads():
    rng = np.random.default_rng(31)
    n, H, ld = 4, 3, 9
    lens = np.array([9, 1, 4, 7])
    Sa = np.zeros((n, H, ld)); Sb = np.zeros((n, H, ld))
    tot = 0.0
    for i in range(n):
        for h in range(H):
            a = rng.random(lens[i]); b = rng.random(lens[i])
            Sa[i, h, :lens[i]] = a / a.sum(); Sb[i, h, :lens[i]] = b / b.sum()
            tot += jensenshannon(Sa[i, h, :lens[i]], Sb[i, h, :lens[i]]) ** 2
    assert so.layer_js(Sa, Sb, lens) == pytest.approx(tot / (n * H), rel=1e-12)


def test_block_similarity_special_cases():
    """Eq. 6 on matrices where the answer is known without evaluating the double sum."""
    M = 5
    JS = np.full((M, M), 0.2); np.fill_diagonal(JS, 0.0)
    for m in range(1, M):
        for n in range(m + 1, M + 1):
            assert so.block_sim(JS, m, n) == pytest.approx(math.log(2) - 0.2, rel=1e-14)   # all pairs alike
    JS2 = np.zeros((3, 3)); JS2[0, 1] = JS2[1, 0] = 0.1; JS2[0, 2] = JS2[2, 0] = 0.3; JS2[1, 2] = JS2[2, 1] = 0.5
    assert so.block_sim(JS2, 1, 2) == pytest.approx(math.log(2) - 0.1, rel=1e-14)        # a pair: mu itself
    assert so.block_sim(JS2, 1, 3) == pytest.approx(math.log(2) - 0.3, rel=1e-14)        # mean JS of 3 pairs = 0.3
    assert so.block_sim(JS2, 2, 3) == pytest.approx(math.log(2) - 0.5, rel=1e-14)        # indices are 1-based


def test_figure2_self_attention_policy_is_layer1_alone_then_layers_2_to_6():
    """Section 3.3 says a good choice for Figure 2(a) is to share layers 2-6 and leave
    layer 1; thresholds in the range the paper found for self-attention give that."""
    JS = _fig2("fig2_js_self.txt")
    assert np.array_equal(JS, JS.T)
    for theta in (0.30, 0.35, 0.40, 0.50):
        assert so.greedy_policy(JS, theta) == [1, 5]
    # sim(1,2) is ln2 - 0.5429: layer 1 does not pair with layer 2 at any theta above it
    assert so.block_sim(JS, 1, 2) == pytest.approx(math.log(2) - 0.5429, rel=1e-14)
    assert so.greedy_policy(JS, 0.15) == [6]
    assert so.greedy_policy(JS, 0.68) == [1, 1, 1, 1, 1, 1]


def test_figure2_encdec_policies():
    """Figure 2(b): good similarity only among two or three adjacent layers (Section 3.1)."""
    JS = _fig2("fig2_js_encdec.txt")
    assert np.array_equal(JS, JS.T)
    assert so.block_sim(JS, 1, 2) == pytest.approx(math.log(2) - 0.0175, rel=1e-14)
    # sizes always sum to the layer count, blocks listed bottom-up
    for theta in np.linspace(0.0, 0.7, 29):
        sizes = so.greedy_policy(JS, float(theta))
        assert sum(sizes) == 6 and min(sizes) >= 1
    assert so.greedy_policy(JS, 0.30) == [6]
    assert so.greedy_policy(JS, 0.40) == [4, 2]
    assert so.greedy_policy(JS, 0.50) == [3, 1, 2]
    # more sharing as theta falls: the number of blocks never decreases with theta
    counts = [len(so.greedy_policy(JS, float(t))) for t in np.linspace(0.0, 0.7, 71)]
    assert all(b >= a for a, b in zip(counts, counts[1:]))
