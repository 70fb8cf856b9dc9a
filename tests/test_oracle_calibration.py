"""Pins of the calibration oracle (last attention row, Eq. 3, Eq. 4)."""

import math

import numpy as np
from scipy.spatial.distance import jensenshannon

from oracle import calibration as C
from oracle import prefill_attention as P


def test_js_closed_forms():
    a = np.array([0.2, 0.3, 0.5])
    assert C.js_divergence(a, a) == 0.0
    # disjoint supports: m = a/2 on a's support, KL(a || m) = ln 2
    assert abs(C.js_divergence([1.0, 0.0], [0.0, 1.0]) - math.log(2)) < 1e-15
    assert abs(C.js_divergence([0.5, 0.5, 0, 0], [0, 0, 0.25, 0.75]) - math.log(2)) < 1e-15
    # two-point example by hand: a = (1, 0), b = (1/2, 1/2): m = (3/4, 1/4)
    want = 0.5 * (math.log(4 / 3) + 0.5 * math.log(2 / 3) + 0.5 * math.log(2))
    assert abs(C.js_divergence([1.0, 0.0], [0.5, 0.5]) - want) < 1e-15


def test_js_symmetric_bounded_and_equal_to_scipy():
    rng = np.random.default_rng(0)
    for _ in range(20):
        a, b = rng.random(37), rng.random(37)
        a[rng.integers(37)] = 0.0
        a, b = a / a.sum(), b / b.sum()
        j = C.js_divergence(a, b)
        assert abs(j - C.js_divergence(b, a)) < 1e-15
        assert 0.0 <= j <= math.log(2)
        assert abs(j - jensenshannon(a, b) ** 2) < 1e-12       # SciPy returns the square root, natural log


def test_last_row_is_the_last_row_of_the_prefill_attention_matrix():
    rng = np.random.default_rng(1)
    N, T, Hq, Hkv, D = 2, 23, 4, 2, 8
    q, k, v = rng.standard_normal((N, T, Hq, D)), rng.standard_normal((N, T, Hkv, D)), rng.standard_normal((N, T, Hkv, D))
    _, probs = P.prefill_lazy_attention(q, k, v, [0] * T, [0, 0], P.MODE_VLA_QC, return_probs=True)
    for l in range(N):
        want = np.mean([probs[l][h][-1] for h in range(Hq)], axis=0)
        got = C.last_row_attention(q[l, -1], k[l], 1.0 / math.sqrt(D))
        np.testing.assert_allclose(got, want, rtol=0, atol=1e-14)
        assert abs(got.sum() - 1.0) < 1e-13


def test_similarity_is_the_sample_mean():
    rng = np.random.default_rng(2)
    rows = [[(lambda x: x / x.sum())(rng.random(11)) for _ in range(4)] for _ in range(3)]
    S = C.adjacent_similarity(rows)
    assert S.shape == (3,)
    for l in range(3):
        assert abs(S[l] - np.mean([C.js_divergence(r[l], r[l + 1]) for r in rows])) < 1e-15
    same = [[rows[0][0]] * 4]
    assert np.all(C.adjacent_similarity(same) == 0.0)


def test_lazy_blocks_follow_the_threshold():
    S = [0.30, 0.01, 0.02, 0.40, 0.03, 0.03, 0.03, 0.50]
    assert C.lazy_blocks(S, 0.05) == [0, 0, 1, 1, 0, 1, 1, 1, 0]
    assert C.lazy_blocks(S, 0.05, max_block=2) == [0, 0, 1, 0, 0, 1, 0, 1, 0]
    assert C.lazy_blocks(S, 0.005) == [0] * 9                      # nothing is similar enough
    assert C.lazy_blocks(S, 1.0) == [0] + [1] * 8                  # everything is (eps at its upper end)
    assert C.lazy_blocks([], 0.1) == [0]
