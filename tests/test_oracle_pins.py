"""Pins of the fp64 oracle against what the paper and the mathematics fix (CPU only).

Each test is chosen so that a plausible mistake in the oracle (a dropped term, a wrong
query or key source, a swapped stream, a missing new token, a wrong GQA head map, two
softmaxes instead of one) makes at least one of them fail.
"""

import itertools
import math

import numpy as np
import pytest

from oracle import lazy_attention as la
from oracle.lazy_attention import (LAYER_FULL, LAYER_LAZY, MODE_GLA, MODE_VLA_EQ8, MODE_VLA_QC,
                                   LazyAttentionOracle)

MODES = (MODE_VLA_QC, MODE_VLA_EQ8, MODE_GLA)
E = math.e


# ------------------------------------------------------------------------------------------
# hand-worked example: D = 1, scale = 1, one head, layers [ordinary, lazy]
# prompt: text t0, visual v0, v1.  All numbers are exactly representable.
#   layer 0: K = (t0 0, v0 1, v1 0), V = (1, 2, 3); step: q = 1, k = 0, v = 4
#   layer 1: own K(t0) = 1 (its visual K is not kept), V = (10, 20, 30); step: q = 2, k = .5, v = 40
# Eq. 2 for layer 0: logits (t0 0, v0 1, v1 0, new 0) -> weights (1, e, 1, 1).
# Eq. 8 (VLA_EQ8), layer 1: own q on own text K and on the leader's visual K:
#   logits (t0 2, v0 2, v1 0, new 1).
# VLA_QC, layer 1: visual keys scored by the cached leader query 1: (t0 2, v0 1, v1 0, new 1).
# Eq. 6 (GLA), layer 1: leader's weights (1, e, 1, 1) on the own V (10, 20, 30, 40).
# ------------------------------------------------------------------------------------------

def _hand(mode):
    o = LazyAttentionOracle(2, 1, 1, 1, [LAYER_FULL, LAYER_LAZY], mode, n_seqs=1, scale=1.0)
    kind = [0, 1, 1]
    k = np.array([[0.0, 1.0, 0.0], [1.0, 77.0, -55.0]]).reshape(2, 3, 1, 1)   # lazy visual K is never used
    v = np.array([[1.0, 2.0, 3.0], [10.0, 20.0, 30.0]]).reshape(2, 3, 1, 1)
    o.prefill_append(0, kind, k, v)
    q = np.array([1.0, 2.0]).reshape(2, 1, 1)
    kn = np.array([0.0, 0.5]).reshape(2, 1, 1)
    vn = np.array([4.0, 40.0]).reshape(2, 1, 1)
    return o.decode_step(0, q, kn, vn)


def test_hand_example_closed_forms():
    out, lse = _hand(MODE_VLA_QC)
    assert out[0, 0, 0] == pytest.approx((8 + 2 * E) / (3 + E), abs=1e-13)
    assert lse[0, 0] == pytest.approx(math.log(3 + E), abs=1e-13)
    assert out[1, 0, 0] == pytest.approx((10 * E**2 + 60 * E + 30) / (E + 1) ** 2, abs=1e-12)
    assert lse[1, 0] == pytest.approx(math.log((E + 1) ** 2), abs=1e-13)

    out, lse = _hand(MODE_VLA_EQ8)
    assert out[0, 0, 0] == pytest.approx((8 + 2 * E) / (3 + E), abs=1e-13)
    assert out[1, 0, 0] == pytest.approx((30 * E**2 + 40 * E + 30) / (2 * E**2 + E + 1), abs=1e-12)

    out, lse = _hand(MODE_GLA)
    assert out[1, 0, 0] == pytest.approx((80 + 20 * E) / (3 + E), abs=1e-12)
    assert out[1, 0, 0] == pytest.approx(10 * out[0, 0, 0], abs=1e-12)   # leader's weights, V scaled by 10
    assert lse[1, 0] == pytest.approx(lse[0, 0], abs=1e-13)


# ------------------------------------------------------------------------------------------
# independent brute force written from Eq. 2 / 6 / 8 with Python floats only
# ------------------------------------------------------------------------------------------

def _brute(mode, kinds, layer_kind, K, V, q, kn, vn, scale, g):
    """K, V: [N][T][Hkv][D] lists; q: [N][Hq][D]; kn, vn: [N][Hkv][D].  Returns out[N][Hq][D]."""
    N, Hq, D = len(layer_kind), len(q[0]), len(q[0][0])
    out = [[[0.0] * D for _ in range(Hq)] for _ in range(N)]
    leader = 0
    for l in range(N):
        if layer_kind[l] == LAYER_FULL:
            leader = l
        lazy = layer_kind[l] == LAYER_LAZY
        for h in range(Hq):
            kv = h // g
            logits, vals = [], []
            for t, kind in enumerate(kinds):          # cached prompt tokens, original order
                if not lazy:
                    qq, kk = q[l][h], K[l][t][kv]
                elif mode == MODE_GLA:
                    qq, kk = q[leader][h], K[leader][t][kv]
                elif kind == 1:                        # visual token in a VLA lazy layer
                    qq = q[leader][h] if mode == MODE_VLA_QC else q[l][h]
                    kk = K[leader][t][kv]
                else:
                    qq, kk = q[l][h], K[l][t][kv]
                logits.append(scale * sum(a * b for a, b in zip(qq, kk)))
                vals.append(V[l][t][kv])
            if lazy and mode == MODE_GLA:              # the new token
                logits.append(scale * sum(a * b for a, b in zip(q[leader][h], kn[leader][kv])))
            else:
                logits.append(scale * sum(a * b for a, b in zip(q[l][h], kn[l][kv])))
            vals.append(vn[l][kv])
            z = sum(math.exp(s) for s in logits)
            for d in range(D):
                out[l][h][d] = sum(math.exp(s) / z * v[d] for s, v in zip(logits, vals))
    return out


@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("layer_kind,g", [([0, 1], 1), ([0, 1, 1], 2), ([0, 0, 1, 0, 1], 1)])
def test_brute_force_small(mode, layer_kind, g):
    rng = np.random.default_rng(11 + mode + len(layer_kind))
    N, Hkv, D = len(layer_kind), 2, 2
    Hq = Hkv * g
    for kinds in itertools.product([0, 1], repeat=3):      # every text/visual pattern of 3 tokens
        T = len(kinds)
        K = rng.integers(-3, 4, size=(N, T, Hkv, D)) / 2.0
        V = rng.integers(-3, 4, size=(N, T, Hkv, D)) / 2.0
        q = rng.integers(-3, 4, size=(N, Hq, D)) / 2.0
        kn = rng.integers(-3, 4, size=(N, Hkv, D)) / 2.0
        vn = rng.integers(-3, 4, size=(N, Hkv, D)) / 2.0
        o = LazyAttentionOracle(N, Hq, Hkv, D, layer_kind, mode, n_seqs=1)
        o.prefill_append(0, list(kinds), K, V)
        out, _ = o.decode_step(0, q, kn, vn)
        ref = _brute(mode, kinds, layer_kind, K.tolist(), V.tolist(), q.tolist(), kn.tolist(),
                     vn.tolist(), 1.0 / math.sqrt(D), g)
        np.testing.assert_allclose(out, np.array(ref), rtol=0, atol=1e-13)


# ------------------------------------------------------------------------------------------
# closed forms and invariants on random multi-layer states
# ------------------------------------------------------------------------------------------

def _random_state(mode, rng, layer_kind=(0, 1, 0, 1, 1), Hq=4, Hkv=2, D=8, n_text=5, n_vis=9, n_seqs=2,
                  q_scale=1.0):
    N = len(layer_kind)
    o = LazyAttentionOracle(N, Hq, Hkv, D, layer_kind, mode, n_seqs=n_seqs)
    kinds = [0] * 2 + [1] * n_vis + [0] * (n_text - 2)
    data = {}
    for s in range(n_seqs):
        K = rng.standard_normal((N, len(kinds), Hkv, D))
        V = rng.standard_normal((N, len(kinds), Hkv, D))
        o.prefill_append(s, kinds, K, V)
        data[s] = (K, V)
    return o, kinds, data


@pytest.mark.parametrize("mode", MODES)
def test_zero_queries_give_mean_of_own_values(mode):
    rng = np.random.default_rng(5)
    o, kinds, data = _random_state(mode, rng)
    N = o.N
    for step in range(3):
        q = np.zeros((N, o.Hq, o.D))
        kn, vn = rng.standard_normal((N, o.Hkv, o.D)), rng.standard_normal((N, o.Hkv, o.D))
        out, lse = o.decode_step(1, q, kn, vn)
        for l in range(N):
            vals = np.concatenate([o.V_T[l][1].rows(), o.V_V[l][1].rows()])
            for h in range(o.Hq):
                np.testing.assert_allclose(out[l, h], vals[:, h // o.g].mean(axis=0), atol=1e-14)
                assert lse[l, h] == pytest.approx(math.log(vals.shape[0]), abs=1e-13)


@pytest.mark.parametrize("mode", MODES)
def test_probability_rows_sum_to_one(mode):
    rng = np.random.default_rng(6)
    o, _, _ = _random_state(mode, rng)
    N = o.N
    q = 3 * rng.standard_normal((N, o.Hq, o.D))
    out, lse, probs = o.decode_step(0, q, rng.standard_normal((N, o.Hkv, o.D)),
                                    rng.standard_normal((N, o.Hkv, o.D)), return_probs=True)
    for l in range(N):
        for h in range(o.Hq):
            p = probs[l][h]
            assert p.shape[0] == o.V_T[l][0].n + o.V_V[l][0].n
            assert np.all(p >= 0)
            assert abs(p.sum() - 1.0) <= 1e-12


@pytest.mark.parametrize("mode", MODES)
def test_dominant_key_selects_its_value(mode):
    """One key whose logit exceeds all others by > 60 takes all the weight."""
    rng = np.random.default_rng(7)
    N, H, D = 2, 1, 4
    o = LazyAttentionOracle(N, H, H, D, [0, 1], mode, n_seqs=1, scale=1.0)
    kinds = [0, 1, 1, 1, 0]
    K = 0.01 * rng.standard_normal((N, 5, H, D))
    V = rng.standard_normal((N, 5, H, D))
    K[:, 2, 0, :] = [100.0, 0, 0, 0]          # visual token 2 dominates (in both layers' K)
    o.prefill_append(0, kinds, K, V)
    q = np.zeros((N, H, D))
    q[:, 0, 0] = 1.0
    out, _ = o.decode_step(0, q, 0.01 * rng.standard_normal((N, H, D)), rng.standard_normal((N, H, D)))
    for l in range(N):
        np.testing.assert_allclose(out[l, 0], V[l, 2, 0], atol=1e-20, rtol=1e-15)


@pytest.mark.parametrize("mode", MODES)
def test_lazy_equals_full_when_shared_q_and_k_equal_own(mode):
    """If every lazy layer's q and K are copies of its leader's, each mode reproduces plain
    attention (Eq. 2) with the layer's own V -- bit for bit, the summation order being equal."""
    rng = np.random.default_rng(8)
    layer_kind = [0, 1, 1, 0, 1]
    N, Hq, Hkv, D = 5, 4, 2, 8
    leader = la.leaders_of(layer_kind)
    kinds = [0, 1, 1, 0, 1, 0, 0, 1]
    K = rng.standard_normal((N, len(kinds), Hkv, D))
    V = rng.standard_normal((N, len(kinds), Hkv, D))
    for l in range(N):
        K[l] = K[leader[l]]
    lazy = LazyAttentionOracle(N, Hq, Hkv, D, layer_kind, mode, n_seqs=1)
    full = LazyAttentionOracle(N, Hq, Hkv, D, [0] * N, mode, n_seqs=1)
    lazy.prefill_append(0, kinds, K, V)
    full.prefill_append(0, kinds, K, V)
    for step in range(4):
        q = rng.standard_normal((N, Hq, D))
        kn = rng.standard_normal((N, Hkv, D))
        vn = rng.standard_normal((N, Hkv, D))
        for l in range(N):
            q[l], kn[l] = q[leader[l]], kn[leader[l]]
        a, la_ = lazy.decode_step(0, q, kn, vn)
        b, lb_ = full.decode_step(0, q, kn, vn)
        assert np.array_equal(a, b)
        assert np.array_equal(la_, lb_)


def test_modes_differ_exactly_where_the_query_source_differs():
    """Leader query 0, lazy query != 0: VLA_QC's visual logits are all 0, VLA_EQ8's are not;
    GLA ignores the lazy layer's q and k entirely."""
    rng = np.random.default_rng(9)
    N, H, D = 2, 2, 4
    kinds = [0, 1, 1, 1, 0]
    K = rng.standard_normal((N, 5, H, D))
    V = rng.standard_normal((N, 5, H, D))
    q = rng.standard_normal((N, H, D))
    q[0] = 0.0
    kn, vn = rng.standard_normal((N, H, D)), rng.standard_normal((N, H, D))
    outs, probs = {}, {}
    for mode in MODES:
        o = LazyAttentionOracle(N, H, H, D, [0, 1], mode, n_seqs=1)
        o.prefill_append(0, kinds, K, V)
        outs[mode], _, probs[mode] = o.decode_step(0, q, kn, vn, return_probs=True)
    n_text = 3   # two prompt text tokens + the new one; probabilities are (text, visual) ordered
    p_qc = probs[MODE_VLA_QC][1][0]
    assert np.allclose(p_qc[n_text:], p_qc[n_text], atol=1e-15)          # equal visual weights
    p_eq8 = probs[MODE_VLA_EQ8][1][0]
    assert np.ptp(p_eq8[n_text:]) > 1e-3
    p_gla = probs[MODE_GLA][1][0]
    assert np.allclose(p_gla, 1.0 / 6, atol=1e-15)                        # leader's q = 0 -> uniform
    # GLA must not depend on the lazy layer's own q / k
    o = LazyAttentionOracle(N, H, H, D, [0, 1], MODE_GLA, n_seqs=1)
    o.prefill_append(0, kinds, K, V)
    q2, kn2 = q.copy(), kn.copy()
    q2[1] += 5.0
    kn2[1] -= 3.0
    out2, _ = o.decode_step(0, q2, kn2, vn)
    assert np.array_equal(out2, outs[MODE_GLA])
    assert not np.allclose(outs[MODE_VLA_QC][1], outs[MODE_VLA_EQ8][1])


def test_vla_without_visual_tokens_is_plain_attention():
    rng = np.random.default_rng(10)
    N, H, D = 3, 2, 4
    K, V = rng.standard_normal((N, 4, H, D)), rng.standard_normal((N, 4, H, D))
    q, kn, vn = (rng.standard_normal((N, H, D)) for _ in range(3))
    ref = LazyAttentionOracle(N, H, H, D, [0, 0, 0], MODE_VLA_QC, n_seqs=1)
    ref.prefill_append(0, [0] * 4, K, V)
    want, _ = ref.decode_step(0, q, kn, vn)
    for mode in (MODE_VLA_QC, MODE_VLA_EQ8):
        o = LazyAttentionOracle(N, H, H, D, [0, 1, 1], mode, n_seqs=1)
        o.prefill_append(0, [0] * 4, K, V)
        got, _ = o.decode_step(0, q, kn, vn)
        assert np.array_equal(got, want)


def test_full_layer_matches_library_softmax():
    """Eq. 2 reduces to textbook attention: compare with torch's float64 softmax and matmul,
    including the GQA head map h -> h // g."""
    import torch

    rng = np.random.default_rng(12)
    N, Hq, Hkv, D, T = 2, 6, 2, 16, 37
    K, V = rng.standard_normal((N, T, Hkv, D)), rng.standard_normal((N, T, Hkv, D))
    kinds = list(rng.integers(0, 2, size=T))
    q, kn, vn = rng.standard_normal((N, Hq, D)), rng.standard_normal((N, Hkv, D)), rng.standard_normal((N, Hkv, D))
    o = LazyAttentionOracle(N, Hq, Hkv, D, [0, 0], MODE_VLA_QC, n_seqs=1)
    o.prefill_append(0, kinds, K, V)
    out, lse = o.decode_step(0, q, kn, vn)
    for l in range(N):
        Kt = torch.from_numpy(np.concatenate([K[l], kn[l][None]]))      # [T+1, Hkv, D]
        Vt = torch.from_numpy(np.concatenate([V[l], vn[l][None]]))
        for h in range(Hq):
            s = (Kt[:, h // 3] @ torch.from_numpy(q[l, h])) / math.sqrt(D)
            ref = torch.softmax(s, dim=0) @ Vt[:, h // 3]
            np.testing.assert_allclose(out[l, h], ref.numpy(), atol=1e-14)
            assert lse[l, h] == pytest.approx(float(torch.logsumexp(s, 0)), abs=1e-13)


def test_key_order_does_not_matter():
    rng = np.random.default_rng(13)
    q, K, V = rng.standard_normal(8), rng.standard_normal((20, 8)), rng.standard_normal((20, 8))
    o1, l1, _ = la.softmax_attention([(q, K)], V, 0.3)
    perm = rng.permutation(20)
    o2, l2, _ = la.softmax_attention([(q, K[perm])], V[perm], 0.3)
    np.testing.assert_allclose(o1, o2, atol=1e-14)
    assert l1 == pytest.approx(l2, abs=1e-13)


def test_split_merge_equals_single_pass():
    rng = np.random.default_rng(14)
    for trial in range(20):
        L, D = int(rng.integers(1, 70)), 16
        q, K, V = 2 * rng.standard_normal(D), rng.standard_normal((L, D)), rng.standard_normal((L, D))
        o1, l1, _ = la.softmax_attention([(q, K)], V, 0.25)
        cuts = sorted(set(rng.integers(0, L + 1, size=int(rng.integers(0, 6))).tolist()))
        o2, l2 = la.split_attention(q, K, V, 0.25, cuts)
        np.testing.assert_allclose(o1, o2, atol=1e-12)
        assert l1 == pytest.approx(l2, abs=1e-12)


def test_merge_is_shift_invariant_and_handles_far_apart_maxima():
    a = (0.0, 2.0, np.array([2.0, 4.0]))       # two keys of logit 0 with values (1,2),(1,2)
    b = (-800.0, 1.0, np.array([5.0, 5.0]))    # negligible chunk
    o, lse = la.merge_partials([a, b])
    np.testing.assert_allclose(o, [1.0, 2.0], atol=1e-15)
    assert lse == pytest.approx(math.log(2.0), abs=1e-15)
    o2, lse2 = la.merge_partials([(a[0] + 7, a[1], a[2]), (b[0] + 7, b[1], b[2])])
    np.testing.assert_allclose(o, o2, atol=1e-15)
    assert lse2 == pytest.approx(lse + 7, abs=1e-12)


def test_qslot_follows_the_most_recent_ordinary_layer():
    """The Q Cache is refreshed by every ordinary layer and read by the lazy layers after it."""
    rng = np.random.default_rng(15)
    layer_kind = [0, 1, 0, 0, 1, 1]
    N, H, D = 6, 1, 4
    o = LazyAttentionOracle(N, H, H, D, layer_kind, MODE_GLA, n_seqs=1)
    K, V = rng.standard_normal((N, 3, H, D)), rng.standard_normal((N, 3, H, D))
    o.prefill_append(0, [0, 1, 0], K, V)
    q, kn, vn = (rng.standard_normal((N, H, D)) for _ in range(3))
    out, lse = o.decode_step(0, q, kn, vn)
    assert np.array_equal(o.qslot[0], q[3])
    assert o.leader == [0, 0, 2, 3, 3, 3]
    # GLA: a lazy layer's softmax statistics equal its leader's
    assert lse[1, 0] == lse[0, 0] and lse[4, 0] == lse[3, 0] and lse[5, 0] == lse[3, 0]
    assert lse[2, 0] != lse[0, 0]


def test_lazy_layer_zero_is_rejected():
    with pytest.raises(ValueError):
        LazyAttentionOracle(2, 1, 1, 4, [1, 0], MODE_GLA, n_seqs=1)


@pytest.mark.parametrize("mode", MODES)
def test_storage_rule_and_saving_closed_form(mode):
    """Token-exact saving at the end of prefill equals the paper's closed form:
    GLA n/(2N); VLA |V|/(|V|+|T|) * n/(2N)  (section "Efficiency Analysis")."""
    from fractions import Fraction

    rng = np.random.default_rng(16)
    layer_kind = [0, 0, 1, 0, 1, 1, 0, 1]
    N, n = len(layer_kind), sum(layer_kind)
    n_text, n_vis = 7, 29
    o = LazyAttentionOracle(N, 2, 2, 4, layer_kind, mode, n_seqs=1)
    kinds = [0] * 3 + [1] * n_vis + [0] * (n_text - 3)
    o.prefill_append(0, kinds, rng.standard_normal((N, len(kinds), 2, 4)), rng.standard_normal((N, len(kinds), 2, 4)))
    saved = Fraction(o.rows_all_full() - o.rows_stored(), o.rows_all_full())
    if mode == MODE_GLA:
        assert saved == Fraction(n, 2 * N)
    else:
        assert saved == Fraction(n_vis, n_vis + n_text) * Fraction(n, 2 * N)
    for l in range(N):
        lazy = layer_kind[l] == LAYER_LAZY
        assert (o.K_V[l][0] is None) == lazy
        assert (o.K_T[l][0] is None) == (lazy and mode == MODE_GLA)
        assert o.V_T[l][0].n == n_text and o.V_V[l][0].n == n_vis
