"""Host part of the policy learner through the C ABI (no GPU needed): Eq. 6 and the
bottom-up search of Section 3.3, against the oracle, the Figure 2 matrices and brute force."""
import math
import os

import numpy as np
import pytest

from oracle import san_oracle as so
from paper_1906_11024_b200 import binding as B
from paper_1906_11024_b200 import build as san_build

GOLD = os.path.join(os.path.dirname(__file__), "golden")


@pytest.fixture(scope="module", autouse=True)
def _built():
    san_build.build()
    B.lib()


def _fig2(name):
    return np.loadtxt(os.path.join(GOLD, name), comments="#")


def test_figure2_policies_through_the_abi():
    js = _fig2("fig2_js_self.txt")
    for theta in (0.30, 0.35, 0.40, 0.50):
        assert B.san_policy_search(js, 6, theta) == (B.SAN_OK, [1, 5])
    assert B.san_policy_search(js, 6, 0.15) == (B.SAN_OK, [6])
    assert B.san_policy_search(js, 6, 0.68) == (B.SAN_OK, [1] * 6)
    js = _fig2("fig2_js_encdec.txt")
    assert B.san_policy_search(js, 6, 0.30) == (B.SAN_OK, [6])
    assert B.san_policy_search(js, 6, 0.40) == (B.SAN_OK, [4, 2])
    assert B.san_policy_search(js, 6, 0.50) == (B.SAN_OK, [3, 1, 2])
    rc, sim = B.san_block_similarity(js, 6, 0, 1)
    assert rc == B.SAN_OK and sim == pytest.approx(math.log(2) - 0.0175, rel=1e-14)


def test_similarity_and_search_equal_the_oracle_on_random_matrices():
    """Same double arithmetic on both sides: the integer result (block sizes) must be equal for
    every threshold, the similarities to rounding order."""
    rng = np.random.default_rng(44)
    for M in (1, 2, 3, 6, 12, 17):
        a = rng.random((M, M)) * math.log(2)
        js = (a + a.T) / 2
        np.fill_diagonal(js, 0.0)
        for m in range(M):
            for n in range(m + 1, M):
                rc, sim = B.san_block_similarity(js, M, m, n)
                assert rc == B.SAN_OK and sim == pytest.approx(so.block_sim(js, m + 1, n + 1), rel=1e-13)
        for theta in np.linspace(-0.1, 0.8, 37):
            rc, sizes = B.san_policy_search(js, M, float(theta))
            assert rc == B.SAN_OK and sizes == so.greedy_policy(js, float(theta))
            assert sum(sizes) == M


def test_search_against_brute_force_restatement():
    """The search restated from Section 3.3 with the double sum of Eq. 6 written out in numpy."""
    rng = np.random.default_rng(45)
    M = 7
    a = rng.random((M, M)) * 0.6
    js = (a + a.T) / 2
    np.fill_diagonal(js, 0.0)
    mu = math.log(2) - js

    def sim(m, n):      # 0-based inclusive
        idx = np.arange(m, n + 1)
        sub = mu[np.ix_(idx, idx)]
        return (sub.sum() - np.trace(sub)) / ((n - m + 1) * (n - m))

    for theta in (0.2, 0.3, 0.4, 0.5):
        sizes, m = [], 0
        while m < M:
            n = m
            while n + 1 < M and sim(m, n + 1) >= theta:
                n += 1
            sizes.append(n - m + 1)
            m = n + 1
        assert B.san_policy_search(js, M, theta) == (B.SAN_OK, sizes)


def test_argument_checks():
    js = np.zeros((3, 3))
    assert B.san_block_similarity(js, 3, 1, 1)[0] == B.SAN_ERR_RANGE       # a block of one layer has no pair
    assert B.san_block_similarity(js, 3, 0, 3)[0] == B.SAN_ERR_RANGE
    assert B.san_policy_search(js, 3, float("nan"))[0] == B.SAN_ERR_RANGE
    assert B.lib().san_policy_search(None, 3, 0.5, None, None) == B.SAN_ERR_NULL
    assert B.lib().san_js_matrix(0, None, 0, 0, 0, 0, None, None, None) == B.SAN_ERR_NULL
