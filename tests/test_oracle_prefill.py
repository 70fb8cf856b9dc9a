"""Pins of the prefill oracle (Eq. 1, Eq. 5, Eq. 7) to things other than itself."""

import math

import numpy as np
import pytest
import torch

from oracle import prefill_attention as P
from oracle.lazy_attention import LazyAttentionOracle

MODES = [P.MODE_VLA_QC, P.MODE_VLA_EQ8, P.MODE_GLA]


def _rand(rng, *shape):
    return rng.standard_normal(shape)


def test_ordinary_layer_is_library_causal_attention():
    rng = np.random.default_rng(1)
    N, T, Hq, Hkv, D = 2, 37, 4, 2, 16
    q, k, v = _rand(rng, N, T, Hq, D), _rand(rng, N, T, Hkv, D), _rand(rng, N, T, Hkv, D)
    kind = rng.integers(0, 2, T)
    out = P.prefill_lazy_attention(q, k, v, kind, [0, 0], P.MODE_VLA_QC)
    for l in range(N):
        tq = torch.from_numpy(q[l]).permute(1, 0, 2)                       # [Hq, T, D]
        tk = torch.from_numpy(k[l]).permute(1, 0, 2).repeat_interleave(2, dim=0)
        tv = torch.from_numpy(v[l]).permute(1, 0, 2).repeat_interleave(2, dim=0)
        ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True)
        np.testing.assert_allclose(out[l], ref.permute(1, 0, 2).numpy(), rtol=0, atol=1e-12)


def test_hand_example_three_tokens():
    """D = 1, scale 1, tokens (text, visual, text).  Leader: q = (1, 0, 2), k = (0, 1, 0);
    lazy layer: q = (2, 5, 1), k = (1, 7, 0.5), V = (10, 20, 30)."""
    q = np.array([[1.0, 0.0, 2.0], [2.0, 5.0, 1.0]]).reshape(2, 3, 1, 1)
    k = np.array([[0.0, 1.0, 0.0], [1.0, 7.0, 0.5]]).reshape(2, 3, 1, 1)
    v = np.array([[1.0, 2.0, 3.0], [10.0, 20.0, 30.0]]).reshape(2, 3, 1, 1)
    kind = [0, 1, 0]
    e, r = math.e, math.sqrt(math.e)
    # Eq. 7: queries (own 2, leader 0, own 1), keys (own 1, leader 1, own 0.5)
    for mode in (P.MODE_VLA_QC, P.MODE_VLA_EQ8):
        out = P.prefill_lazy_attention(q, k, v, kind, [0, 1], mode, scale=1.0)
        want = [10.0, 15.0, (10 * e + 20 * e + 30 * r) / (2 * e + r)]
        np.testing.assert_allclose(out[1, :, 0, 0], want, rtol=0, atol=1e-13)
    # Eq. 5: the leader's queries and keys; last row logits (0, 2, 0)
    out = P.prefill_lazy_attention(q, k, v, kind, [0, 1], P.MODE_GLA, scale=1.0)
    want = [10.0, 15.0, (10 + 20 * e * e + 30) / (2 + e * e)]     # row 1: leader q = 0, uniform over two keys
    np.testing.assert_allclose(out[1, :, 0, 0], want, rtol=0, atol=1e-13)
    # the leader itself (Eq. 1): row 2 has q = 2, logits (0, 2, 0), V = (1, 2, 3)
    np.testing.assert_allclose(out[0, 2, 0, 0], (1 + 2 * e * e + 3) / (2 + e * e), rtol=0, atol=1e-13)
    # a wrong selection would give something else: own q for the visual row would weight v0 by e^35
    assert abs(out[1, 1, 0, 0] - 20.0) > 1.0


@pytest.mark.parametrize("mode", MODES)
def test_lazy_equals_ordinary_when_leader_qk_equal_own(mode):
    rng = np.random.default_rng(2)
    N, T, Hq, Hkv, D = 3, 29, 4, 2, 8
    q, k, v = _rand(rng, N, T, Hq, D), _rand(rng, N, T, Hkv, D), _rand(rng, N, T, Hkv, D)
    q[1], k[1] = q[0], k[0]
    q[2], k[2] = q[0], k[0]
    kind = rng.integers(0, 2, T)
    lazy = P.prefill_lazy_attention(q, k, v, kind, [0, 1, 1], mode)
    full = P.prefill_lazy_attention(q, k, v, kind, [0, 0, 0], mode)
    assert np.array_equal(lazy, full)


def test_gla_reuses_the_leaders_attention_matrix_and_rows_sum_to_one():
    rng = np.random.default_rng(3)
    N, T, Hq, Hkv, D = 2, 23, 2, 1, 8
    q, k, v = _rand(rng, N, T, Hq, D), _rand(rng, N, T, Hkv, D), _rand(rng, N, T, Hkv, D)
    kind = rng.integers(0, 2, T)
    out, probs = P.prefill_lazy_attention(q, k, v, kind, [0, 1], P.MODE_GLA, return_probs=True)
    for h in range(Hq):
        assert np.array_equal(probs[1][h], probs[0][h])
        np.testing.assert_allclose(out[1, :, h], probs[0][h] @ v[1, :, 0], rtol=0, atol=1e-13)
        np.testing.assert_allclose(probs[0][h].sum(axis=1), 1.0, rtol=0, atol=1e-13)
        assert np.all(np.triu(probs[0][h], 1) == 0.0)


@pytest.mark.parametrize("mode", MODES)
def test_causality_later_tokens_do_not_change_earlier_rows(mode):
    rng = np.random.default_rng(4)
    N, T, Hq, Hkv, D = 2, 19, 2, 2, 8
    q, k, v = _rand(rng, N, T, Hq, D), _rand(rng, N, T, Hkv, D), _rand(rng, N, T, Hkv, D)
    kind = rng.integers(0, 2, T)
    a = P.prefill_lazy_attention(q, k, v, kind, [0, 1], mode)
    q2, k2, v2 = q.copy(), k.copy(), v.copy()
    q2[:, 11:], k2[:, 11:], v2[:, 11:] = 5.0, -3.0, 7.0
    b = P.prefill_lazy_attention(q2, k2, v2, kind, [0, 1], mode)
    assert np.array_equal(a[:, :11], b[:, :11])
    assert not np.allclose(a[:, 11:], b[:, 11:])


@pytest.mark.parametrize("mode", [P.MODE_VLA_EQ8, P.MODE_GLA])
def test_last_prompt_row_agrees_with_the_decode_oracle(mode):
    """Prefilling T tokens and reading row T-1 must equal caching T-1 tokens and decoding the
    T-th (a text token): Eq. 1 row vs Eq. 2, Eq. 5 row vs Eq. 6, Eq. 7 text row vs Eq. 8."""
    rng = np.random.default_rng(5)
    N, T, Hq, Hkv, D = 4, 41, 4, 2, 16
    q, k, v = _rand(rng, N, T, Hq, D), _rand(rng, N, T, Hkv, D), _rand(rng, N, T, Hkv, D)
    kind = rng.integers(0, 2, T)
    kind[-1] = 0
    layer_kind = [0, 1, 0, 1]
    out = P.prefill_lazy_attention(q, k, v, kind, layer_kind, mode)
    dec = LazyAttentionOracle(N, Hq, Hkv, D, layer_kind, mode, n_seqs=1)
    dec.prefill_append(0, kind[:-1].tolist(), k[:, :-1], v[:, :-1])
    ref, _ = dec.decode_step(0, q[:, -1], k[:, -1], v[:, -1])
    np.testing.assert_allclose(out[:, -1], ref, rtol=0, atol=1e-12)


def test_ordinary_rows_of_vla_qc_agree_with_decode_and_lazy_rows_follow_eq7():
    """With the cached-query decode reading, ordinary layers still agree row for row; the lazy
    layer's prefill row is Eq. 7's (own query on every key), which that decode reading changes."""
    rng = np.random.default_rng(6)
    N, T, Hq, Hkv, D = 2, 17, 2, 1, 8
    q, k, v = _rand(rng, N, T, Hq, D), _rand(rng, N, T, Hkv, D), _rand(rng, N, T, Hkv, D)
    kind = np.array([0] * 3 + [1] * 9 + [0] * 5)
    out = P.prefill_lazy_attention(q, k, v, kind, [0, 1], P.MODE_VLA_QC)
    dec = LazyAttentionOracle(N, Hq, Hkv, D, [0, 1], P.MODE_VLA_QC, n_seqs=1)
    dec.prefill_append(0, kind[:-1].tolist(), k[:, :-1], v[:, :-1])
    ref, _ = dec.decode_step(0, q[:, -1], k[:, -1], v[:, -1])
    np.testing.assert_allclose(out[0, -1], ref[0], rtol=0, atol=1e-12)
    assert not np.allclose(out[1, -1], ref[1])
