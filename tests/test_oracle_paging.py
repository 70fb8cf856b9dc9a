"""Pins of the allocator's integer model and of the KV-saving accounting (CPU only)."""

import math
from fractions import Fraction

import numpy as np
import pytest

from oracle.paging import (K_T, K_V, V_T, V_V, MODE_GLA, MODE_VLA_EQ8, MODE_VLA_QC, OutOfPages,
                           PagedCacheModel)
from paper_2602_01901_b200 import workloads as W


def _golden():
    vals = {}
    import os

    with open(os.path.join(os.path.dirname(__file__), "golden", "paper_values.txt")) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if "=" in line:
                k, v = [x.strip() for x in line.split("=", 1)]
                vals[k] = v
    return vals


def test_hand_enumerated_page_ids():
    """3 layers [ordinary, lazy, ordinary], VLA, page 4: pop order written out by hand."""
    m = PagedCacheModel([0, 1, 0], MODE_VLA_QC, page_size=4, n_pages=64, max_seqs=2)
    m.prefill_append([0], [3], [5])          # 3 text, 5 visual -> 1 text page, 2 visual pages per stream
    # layer 0: K_T [0], K_V [1,2], V_T [3], V_V [4,5]; layer 1 (lazy): K_T [6], V_T [7], V_V [8,9];
    # layer 2: K_T [10], K_V [11,12], V_T [13], V_V [14,15]
    assert m.page_table(0, K_T, 0) == ([0], 3, 0)
    assert m.page_table(0, K_V, 0) == ([1, 2], 5, 0)
    assert m.page_table(0, V_V, 0) == ([4, 5], 5, 0)
    assert m.page_table(1, K_T, 0) == ([6], 3, 1)
    assert m.page_table(1, K_V, 0) == ([1, 2], 5, 0)      # alias of the leader's visual keys
    assert m.page_table(1, V_V, 0) == ([8, 9], 5, 1)
    assert m.page_table(2, V_V, 0) == ([14, 15], 5, 2)
    m.decode_step([0])                       # text 3 -> 4: no page
    assert m.pages_in_use() == 16
    m.decode_step([0])                       # text 4 -> 5: new page for K_T then V_T, layers ascending
    assert m.page_table(0, K_T, 0) == ([0, 16], 5, 0)
    assert m.page_table(0, V_T, 0) == ([3, 17], 5, 0)
    assert m.page_table(1, K_T, 0) == ([6, 18], 5, 1)
    assert m.page_table(1, V_T, 0) == ([7, 19], 5, 1)
    assert m.page_table(2, V_T, 0) == ([13, 21], 5, 2)
    # a second sequence, then free the first: its pages come back first-allocated first
    m.prefill_append([1], [1], [0])
    assert m.page_table(0, K_T, 1) == ([22], 1, 0)
    assert m.page_table(0, K_V, 1) == ([], 0, 0)
    m.free_seq(0)
    assert m.page_table(0, K_T, 0) == ([], 0, -1)
    m.prefill_append([0], [1], [0])
    assert m.page_table(0, K_T, 0) == ([0], 1, 0)
    assert m.page_table(0, V_T, 0) == ([1], 1, 0)


def test_gla_lazy_layer_owns_no_keys():
    m = PagedCacheModel([0, 1], MODE_GLA, page_size=4, n_pages=32, max_seqs=1)
    m.prefill_append([0], [4], [4])
    assert m.page_table(1, K_T, 0) == ([0], 4, 0)
    assert m.page_table(1, K_V, 0) == ([1], 4, 0)
    assert m.page_table(1, V_T, 0) == ([4], 4, 1)
    m.decode_step([0])       # K_T(0), V_T(0), V_T(1) each get a page
    assert m.pages_in_use() == 6 + 3


def test_out_of_pages_leaves_state_unchanged():
    m = PagedCacheModel([0, 1], MODE_VLA_QC, page_size=4, n_pages=7, max_seqs=1)
    m.prefill_append([0], [4], [4])          # 4 + 3 pages
    before = (dict(m.tables), {k: list(v) for k, v in m.length.items()}, list(m.free))
    with pytest.raises(OutOfPages):
        m.decode_step([0])
    assert (dict(m.tables), m.length, m.free) == before


@pytest.mark.parametrize("w", W.WORKLOADS[1:], ids=lambda w: w.name)
@pytest.mark.parametrize("mode", [MODE_VLA_QC, MODE_VLA_EQ8, MODE_GLA])
def test_saving_closed_form_on_the_workloads(w, mode):
    """End of prefill: token-exact saved fraction == n/(2N) (GLA) or |V|/(|V|+|T|) n/(2N) (VLA)."""
    per_layer = 4 * (math.ceil(w.max_tokens / 16) + 2)
    m = PagedCacheModel(w.layer_kind().tolist(), mode, 16, per_layer * w.n_layers * w.batch, w.batch)
    for s in range(w.batch):
        _, kind = w.prompt_layout(s)
        m.prefill_append([s], [int((kind == 0).sum())], [int((kind == 1).sum())])
    saved = Fraction(m.rows_all_full() - m.rows_stored(), m.rows_all_full())
    n, N = len(w.lazy_layers), w.n_layers
    if mode == MODE_GLA:
        assert saved == Fraction(n, 2 * N)
    else:
        assert saved == Fraction(w.n_visual_kept, w.n_prompt) * Fraction(n, 2 * N)


def test_page_counts_at_end_of_decode_match_independent_arithmetic():
    """Pages in use after the last decode step, from ceil() arithmetic written out here."""
    for w in W.WORKLOADS[1:3]:
        per_layer = 4 * (math.ceil(w.max_tokens / 16) + 2)
        m = PagedCacheModel(w.layer_kind().tolist(), MODE_VLA_QC, 16, per_layer * w.n_layers * w.batch, w.batch)
        for s in range(w.batch):
            m.prefill_append([s], [w.n_text_prompt], [w.n_visual_kept])
        for _ in range(w.decode_steps):
            m.decode_step(list(range(w.batch)))
        pt = math.ceil((w.n_text_prompt + w.decode_steps) / 16)
        pv = math.ceil(w.n_visual_kept / 16)
        n = len(w.lazy_layers)
        want = w.batch * ((w.n_layers - n) * 2 * (pt + pv) + n * (2 * pt + pv))
        assert m.pages_in_use() == want
    # the LLaVA-1.5 shape ends at 51 776 pages against 60 416 for an all-ordinary stack
    w = W.get_workload("llava15_7b")
    assert w.batch * (17 * 2 * (23 + 36) + 15 * (2 * 23 + 36)) == 51776
    assert w.batch * 32 * 2 * (23 + 36) == 60416


def test_vanilla_cache_size_matches_table_3():
    """All-ordinary LLaVA-NeXT-7B shape (32 layers, 32 heads of 128, 2-byte K and V) at the
    paper's input length of 2048 tokens, batch 1: the paper's Table 3 prints 1.01 GB."""
    g = _golden()
    m = PagedCacheModel([0] * 32, MODE_VLA_QC, 16, 1 << 16, 1)
    m.prefill_append([0], [128], [int(g["input_length_tokens"]) - 128])
    row_bytes = 32 * 128 * 2
    gib = m.rows_all_full() * row_bytes / 2**30
    assert gib == 1.0
    assert abs(gib - float(g["vanilla_kv_cache_gb"])) < 0.011     # printed to two decimals
    assert m.pages_in_use() * 16 * row_bytes == m.rows_all_full() * row_bytes   # 2048 is page aligned


def test_workload_shapes_follow_the_config_strings():
    tiny, c2, c3, c4, c5 = W.WORKLOADS[:5]
    assert (tiny.n_prompt, tiny.max_tokens) == (672, 688)
    pos, kind = tiny.prompt_layout(0)
    assert kind[64] == 1 and kind[63] == 0 and kind[639] == 1 and kind[640] == 0
    pos, kind = c2.prompt_layout(3)
    assert c2.n_prompt == 675 and kind[35] == 1 and kind[34] == 0 and kind[610] == 1 and kind[611] == 0
    assert c2.lazy_layers == tuple(range(3, 32, 2)) and len(c2.lazy_layers) == 15
    assert c3.n_prompt == 2880 + 128 and c4.n_prompt == 1024 + 96 and len(c4.lazy_layers) == 13
    assert c4.group == 7
    pos, kind = c5.prompt_layout(1)
    assert int((kind == 1).sum()) == 4096 and len(pos) == 4096 + 256
    assert np.all(np.diff(pos) > 0)
    pos_b, _ = c5.prompt_layout(2)
    assert not np.array_equal(pos, pos_b)                    # a different subset per sequence
    assert np.array_equal(pos, c5.prompt_layout(1)[0])       # but reproducible


def test_generator_is_standard_normal_and_identical_in_numpy_and_torch():
    import torch

    w = W.get_workload("tiny")
    kind, k, v = W.prefill_kv_np(w, 0)
    x = W.bf16_bits_to_f64(np.concatenate([k.ravel(), v.ravel()]))
    assert abs(x.mean()) < 5e-3
    assert abs(x.var() - 1.0) < 1e-2
    assert abs(((x - x.mean()) ** 4).mean() / x.var() ** 2 - 3.0) < 5e-2
    assert abs(np.corrcoef(x[:-1], x[1:])[0, 1]) < 5e-3
    _, kt, vt = W.prefill_kv_torch(w, 0, "cpu")
    assert np.array_equal(kt.view(torch.int16).numpy().view(np.uint16), k)
    assert np.array_equal(vt.view(torch.int16).numpy().view(np.uint16), v)
    q, kk, vv = W.decode_qkv_np(w, 5)
    qt, kkt, vvt = W.decode_qkv_torch(w, 5, "cpu")
    for a, b in ((q, qt), (kk, kkt), (vv, vvt)):
        assert np.array_equal(b.view(torch.int16).numpy().view(np.uint16), a)
    # sub-block draws agree with whole-tensor draws (what sampled parity relies on)
    sub = W.decode_qkv_np(w, 5, layers=[1], q_heads=[3], kv_heads=[3])
    assert np.array_equal(sub[0][0, 0, 0], q[1, 0, 3]) and np.array_equal(sub[2][0, 0, 0], vv[1, 0, 3])
    # bf16 helpers: exact round trip and ties-to-even
    bits = np.arange(0, 65536, dtype=np.uint32).astype(np.uint16)
    finite = bits[(bits & 0x7F80) != 0x7F80]
    assert np.array_equal(W.f32_to_bf16_bits(W.bf16_bits_to_f64(finite).astype(np.float32)), finite)
    assert W.f32_to_bf16_bits(np.array([1.0 + 2**-8], np.float32))[0] == 0x3F80      # tie -> even
    assert W.f32_to_bf16_bits(np.array([1.0 + 3 * 2**-8], np.float32))[0] == 0x3F82  # tie -> even (up)
