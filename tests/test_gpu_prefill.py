"""GPU parity of prefill Lazy Attention (qc_prefill_attend) against the fp64 prefill oracle.

Same bars as the decode tests: every element within 2e-2, relative L2 <= 5e-3 per (layer,
token-block); the cache the call leaves behind must be the one qc_prefill_append builds.
"""

import numpy as np
import pytest
import torch

from oracle import prefill_attention as OP
from oracle.lazy_attention import LazyAttentionOracle
from paper_2602_01901_b200 import binding as qc
from paper_2602_01901_b200 import workloads as W
from paper_2602_01901_b200.session import Session, bits_of

from parity_util import MAX_ABS, REL_L2, assert_close, f64

pytestmark = pytest.mark.gpu

MODES = [qc.QC_MODE_VLA_QC, qc.QC_MODE_VLA_EQ8, qc.QC_MODE_GLA]
MODE_IDS = ["vla_qc", "vla_eq8", "gla"]


def _dev(a, device):
    return torch.from_numpy(a.astype(np.int16)).view(torch.bfloat16).to(device).contiguous()


CASES = [
    # (head_dim, group, layer_kind, n_text_before, n_visual, n_text_after)
    (128, 1, [0, 1, 0, 1, 1], 5, 150, 22),      # 177 tokens: three query tiles, ragged tail
    (64, 2, [0, 1, 1], 3, 61, 0),               # exactly 64 tokens, ends on a visual token
    (128, 7, [0, 1], 9, 40, 8),                 # one tile, GQA group of 7
    (64, 1, [0, 0, 1], 0, 130, 3),              # starts with a visual token
    (128, 2, [0, 1, 1, 1, 1, 1, 0], 17, 0, 60),  # text only
]


@pytest.mark.parametrize("mode", MODES, ids=MODE_IDS)
@pytest.mark.parametrize("case", range(len(CASES)))
def test_prefill_attend_small(mode, case):
    D, group, layer_kind, nb, nv, na = CASES[case]
    lazy = tuple(i for i, k in enumerate(layer_kind) if k)
    w = W.Workload(40 + case, f"prefill{case}", len(layer_kind), 2 * group, 2, D, 16, 2, nb, nv, nv, na, 4, lazy)
    s = Session.for_workload(w, lazy_mode=mode, poison_pool=True)
    dec = LazyAttentionOracle(w.n_layers, w.n_q_heads, w.n_kv_heads, D, layer_kind, mode, n_seqs=w.batch)
    for b in range(w.batch):
        kind, k, v = W.prefill_kv_np(w, b)
        q = W.prefill_q_np(w, b)
        out = torch.full((w.n_layers, len(kind), w.n_q_heads, D), float("nan"), dtype=torch.bfloat16, device=s.device)
        s.prefill_attend(b, kind, _dev(q, s.device), _dev(k, s.device), _dev(v, s.device), out)
        ref = OP.prefill_lazy_attention(f64(q), f64(k), f64(v), kind, layer_kind, mode)
        got = bits_of(out)
        for l in range(w.n_layers):
            for t0 in range(0, len(kind), 64):
                assert_close(got[l, t0:t0 + 64], ref[l, t0:t0 + 64], f"case {case} seq {b} layer {l} tokens {t0}..")
        dec.prefill_append(b, kind.tolist(), f64(k), f64(v))
    # the cache is the one qc_prefill_append builds: decoding from it matches the decode oracle
    o = torch.empty((w.n_layers, w.batch, w.n_q_heads, D), dtype=torch.bfloat16, device=s.device)
    for step in range(2):
        qn, kn, vn = W.decode_qkv_np(w, step)
        s.decode_step(list(range(w.batch)), _dev(qn, s.device), _dev(kn, s.device), _dev(vn, s.device), o)
        got = bits_of(o)
        for b in range(w.batch):
            ref, _ = dec.decode_step(b, f64(qn[:, b]), f64(kn[:, b]), f64(vn[:, b]))
            for l in range(w.n_layers):
                assert_close(got[l, b], ref[l], f"decode after prefill: step {step} seq {b} layer {l}")
    assert s.stats().device_error == 0
    s.close()


PAIR_CASES = [
    # (group, layer_kind, n_text_before, n_visual, n_text_after): head_dim 128, two query tiles per CTA
    (1, [0, 1, 0, 1, 1], 5, 150, 22),            # 177 tokens: one pair, second tile ragged
    (7, [0, 1], 9, 40, 8),                       # 57 tokens: the second tile of the pair has no row
    (2, [0, 1, 1, 0], 17, 290, 78),              # 385 tokens: two pairs, the last with one row in its first tile
    (1, [0, 1], 3, 500, 9),                      # 512 tokens: two full pairs
    (2, [0, 1, 1], 40, 0, 260),                  # text only, 300 tokens
    (1, [0, 0, 1], 0, 700, 69),                  # 769 tokens: four pairs, starts with a visual token
]


@pytest.mark.parametrize("mode", MODES, ids=MODE_IDS)
@pytest.mark.parametrize("case", range(len(PAIR_CASES)))
def test_prefill_attend_two_query_tiles_per_cta_small(mode, case):
    """The kernel for long prompts (two query tiles per CTA, 128-key tiles), forced onto short
    prompts so that the oracle checks every row: ragged tails, a pair whose second tile is empty,
    tiles that mix text and visual rows of a VLA lazy layer."""
    group, layer_kind, nb, nv, na = PAIR_CASES[case]
    D = 128
    lazy = tuple(i for i, k in enumerate(layer_kind) if k)
    w = W.Workload(70 + case, f"prefill_pair{case}", len(layer_kind), 2 * group, 2, D, 16, 2, nb, nv, nv, na, 4, lazy)
    s = Session.for_workload(w, lazy_mode=mode, poison_pool=True)
    s.set_option("prefill_pair_min_tokens", 1)
    s.set_option("prefill_shared_scores", 0)
    for b in range(w.batch):
        kind, k, v = W.prefill_kv_np(w, b)
        q = W.prefill_q_np(w, b)
        out = torch.full((w.n_layers, len(kind), w.n_q_heads, D), float("nan"), dtype=torch.bfloat16, device=s.device)
        s.prefill_attend(b, kind, _dev(q, s.device), _dev(k, s.device), _dev(v, s.device), out)
        torch.cuda.synchronize()
        assert s.stats().device_error == 0
        ref = OP.prefill_lazy_attention(f64(q), f64(k), f64(v), kind, layer_kind, mode)
        got = bits_of(out)
        for l in range(w.n_layers):
            for t0 in range(0, len(kind), 64):
                assert_close(got[l, t0:t0 + 64], ref[l, t0:t0 + 64], f"pair case {case} seq {b} layer {l} tokens {t0}..")
    s.close()


@pytest.mark.parametrize("name,mode", [("llava15_7b", qc.QC_MODE_VLA_QC), ("llava15_7b", qc.QC_MODE_GLA),
                                       ("qwen2vl_gqa", qc.QC_MODE_VLA_QC), ("qwen2vl_gqa", qc.QC_MODE_GLA),
                                       ("llava_next_2048_lazy22", qc.QC_MODE_GLA)],
                         ids=["llava15_7b-vla", "llava15_7b-gla", "qwen2vl_gqa-vla", "qwen2vl_gqa-gla",
                              "lazy22-gla"])
def test_prefill_attend_full_size_sampled(name, mode):
    """One full-size prompt (all layers, all heads on the GPU); the oracle checks every row of
    sampled (layer, head) pairs, lazy layers and their leaders included."""
    w = W.get_workload(name)
    s = Session.for_workload(w, lazy_mode=mode)
    seq = 1
    kind, k, v = W.prefill_kv_torch(w, seq, s.device)
    q = W.prefill_q_torch(w, seq, s.device)
    out = torch.empty_like(q)
    s.prefill_attend(0, kind, q, k, v, out)
    torch.cuda.synchronize()
    assert torch.isfinite(out.float()).all()
    kinds = w.layer_kind().tolist()
    leaders = OP.leaders_of(kinds)
    rng = np.random.default_rng(w.seed)
    lz = list(w.lazy_layers)
    samples = [(0, 0), (lz[0], 1), (lz[-1], w.n_q_heads - 1), (w.n_layers - 2, w.n_q_heads // 2)]
    samples += [(int(rng.integers(w.n_layers)), int(rng.integers(w.n_q_heads))) for _ in range(4)]
    worst = 0.0
    for layer, head in samples:
        c = leaders[layer]
        layers = [layer] if c == layer else [c, layer]
        kv = head // w.group
        qn = W.prefill_q_np(w, seq, layers=layers, heads=[head])
        _, kn, vn = W.prefill_kv_np(w, seq, layers=layers, heads=[kv])
        sub_kind = [0] if c == layer else [0, 1]
        ref = OP.prefill_lazy_attention(f64(qn), f64(kn), f64(vn), kind, sub_kind, mode)[-1, :, 0]
        got = bits_of(out[layer, :, head])
        for t0 in range(0, len(kind), 128):
            _, r = assert_close(got[t0:t0 + 128], ref[t0:t0 + 128], f"{name} layer {layer} head {head} tokens {t0}..")
            worst = max(worst, r)
    assert s.stats().device_error == 0
    print(f"{name} mode {mode}: prefill worst rel-L2 {worst:.3e}")
    s.close()


@pytest.mark.parametrize("name,mode,cut", [("llava15_7b", qc.QC_MODE_VLA_QC, 300), ("llava15_7b", qc.QC_MODE_GLA, 64),
                                           ("qwen2vl_gqa", qc.QC_MODE_VLA_QC, 777)],
                         ids=["llava15_7b-vla-300", "llava15_7b-gla-64", "qwen2vl_gqa-vla-777"])
def test_prefill_attend_in_two_chunks_full_size(name, mode, cut):
    """A full-size prompt given as two calls (the cut falls inside the image): the second call's
    key tiles start with the cached text and visual tokens, read from the paged pool by the
    tcgen05 kernel.  Both chunks' rows must equal the oracle's rows of ONE prefill over the whole
    prompt, for sampled (layer, head) pairs, lazy layers and their leaders included."""
    w = W.get_workload(name)
    s = Session.for_workload(w, lazy_mode=mode)
    seq = 2
    kind, k, v = W.prefill_kv_torch(w, seq, s.device)
    q = W.prefill_q_torch(w, seq, s.device)
    T = len(kind)
    out = torch.empty_like(q)
    for a, b in ((0, cut), (cut, T)):
        s.prefill_attend(0, kind[a:b], q[:, a:b].contiguous(), k[:, a:b].contiguous(), v[:, a:b].contiguous(),
                         out_chunk := torch.empty_like(q[:, a:b].contiguous()))
        out[:, a:b] = out_chunk
    torch.cuda.synchronize()
    assert torch.isfinite(out.float()).all()
    kinds = w.layer_kind().tolist()
    leaders = OP.leaders_of(kinds)
    lz = list(w.lazy_layers)
    samples = [(0, 0), (lz[0], 1), (lz[-1], w.n_q_heads - 1), (w.n_layers - 1, w.n_q_heads // 2)]
    for layer, head in samples:
        c = leaders[layer]
        layers = [layer] if c == layer else [c, layer]
        kv = head // w.group
        qn = W.prefill_q_np(w, seq, layers=layers, heads=[head])
        _, kn, vn = W.prefill_kv_np(w, seq, layers=layers, heads=[kv])
        sub_kind = [0] if c == layer else [0, 1]
        ref = OP.prefill_lazy_attention(f64(qn), f64(kn), f64(vn), kind, sub_kind, mode)[-1, :, 0]
        got = bits_of(out[layer, :, head])
        for t0 in range(0, T, 128):
            assert_close(got[t0:t0 + 128], ref[t0:t0 + 128], f"{name} cut {cut} layer {layer} head {head} tokens {t0}..")
    assert s.stats().device_error == 0
    s.close()


@pytest.mark.parametrize("name", ["llava15_7b", "llava_next_2048_lazy22", "qwen2vl_gqa"])
def test_prefill_gla_shared_score_passes_change_no_bit(name):
    """GLA, Eq. 5: the layers of a lazy block attend with the same Q and K, so the kernel computes and
    normalises their scores once per run of up to three layers and applies them to each layer's V.
    That is the same arithmetic in the same order as one pass per layer: identical bits.
    (blocks of two layers in the first workload, of four -- a pass of three and a single -- in the
    second, query groups of seven in the third)"""
    w = W.get_workload(name)
    kind, q = None, None
    outs = []
    for shared in (2, 0):    # 2 = always (the default shares only from 1536 prompt tokens on)
        s = Session.for_workload(w, lazy_mode=qc.QC_MODE_GLA)
        s.set_option("prefill_shared_scores", shared)
        kind, k, v = W.prefill_kv_torch(w, 1, s.device)
        q = W.prefill_q_torch(w, 1, s.device)
        out = torch.full_like(q, float("nan"))
        s.prefill_attend(0, kind, q, k, v, out)
        torch.cuda.synchronize()
        assert s.stats().device_error == 0
        outs.append(out)
        s.close()
    assert torch.isfinite(outs[0].float()).all()
    assert torch.equal(outs[0].view(torch.int16), outs[1].view(torch.int16))


@pytest.mark.parametrize("name", ["llava_next_anyres", "qwen2vl_gqa"])
def test_prefill_attend_repeats_bit_identically(name):
    """The kernel has no atomics and a fixed reduction order, so the same prompt gives the same
    bits every time; a hand-off between its warps that is not ordered shows up here as a
    difference between launches.  Long prompts: many tiles per CTA, both CTAs of an SM busy."""
    w = W.get_workload(name)
    s = Session.for_workload(w)
    kind, k, v = W.prefill_kv_torch(w, 0, s.device)
    q = W.prefill_q_torch(w, 0, s.device)
    first = torch.empty_like(q)
    s.prefill_attend(0, kind, q, k, v, first)
    torch.cuda.synchronize()
    assert torch.isfinite(first.float()).all()
    out = torch.empty_like(q)
    for rep in range(1, 6):
        out.fill_(float("nan"))
        qc.qc_free_seq(s.cache, 0)   # a fresh sequence: the tcgen05 kernel serves prompts that start a sequence
        s.prefill_attend(0, kind, q, k, v, out)
        torch.cuda.synchronize()
        assert torch.equal(out.view(torch.int16), first.view(torch.int16)), f"launch {rep} differs from launch 0"
    assert s.stats().device_error == 0
    s.close()


@pytest.mark.parametrize("mode", MODES, ids=MODE_IDS)
@pytest.mark.parametrize("head_dim,group", [(128, 1), (64, 2), (128, 7)])
def test_prefill_attend_continues_a_cached_sequence(mode, head_dim, group):
    """A later turn: prompt chunk, a few generated tokens, then a second chunk (text and a new
    image).  The second chunk's rows must equal the oracle's rows for one prefill over the whole
    token sequence (chunk 1, generated tokens, chunk 2)."""
    layer_kind = [0, 1, 1, 0, 1]
    lazy = tuple(i for i, k in enumerate(layer_kind) if k)
    w = W.Workload(60 + group, f"turns{group}", len(layer_kind), 2 * group, 2, head_dim, 16, 1, 7, 90, 90, 80, 5, lazy)
    s = Session(w.n_layers, w.n_q_heads, w.n_kv_heads, head_dim, layer_kind, max_seqs=1, max_tokens_per_seq=256,
                n_pages=w.n_layers * 4 * 20, lazy_mode=mode, poison_pool=True)
    kind, k, v = W.prefill_kv_np(w, 0)
    q = W.prefill_q_np(w, 0)
    T1 = 70                       # 7 text + 63 visual: the image is cut in the middle
    dev = s.device
    out1 = torch.empty((w.n_layers, T1, w.n_q_heads, head_dim), dtype=torch.bfloat16, device=dev)
    s.prefill_attend(0, kind[:T1], _dev(q[:, :T1], dev), _dev(k[:, :T1], dev), _dev(v[:, :T1], dev), out1)
    gen_q, gen_k, gen_v = [], [], []
    o = torch.empty((w.n_layers, 1, w.n_q_heads, head_dim), dtype=torch.bfloat16, device=dev)
    for step in range(3):
        qn, kn, vn = W.decode_qkv_np(w, step)
        s.decode_step([0], _dev(qn, dev), _dev(kn, dev), _dev(vn, dev), o)
        gen_q.append(qn[:, 0]), gen_k.append(kn[:, 0]), gen_v.append(vn[:, 0])
    T2 = len(kind) - T1
    out2 = torch.full((w.n_layers, T2, w.n_q_heads, head_dim), float("nan"), dtype=torch.bfloat16, device=dev)
    s.prefill_attend(0, kind[T1:], _dev(q[:, T1:], dev), _dev(k[:, T1:], dev), _dev(v[:, T1:], dev), out2)
    # the oracle sees one sequence: chunk 1, the generated (text) tokens, chunk 2
    cat = lambda a, g, b: np.concatenate([a, np.stack(g, axis=1), b], axis=1)
    q_all, k_all, v_all = cat(q[:, :T1], gen_q, q[:, T1:]), cat(k[:, :T1], gen_k, k[:, T1:]), cat(v[:, :T1], gen_v, v[:, T1:])
    kind_all = np.concatenate([kind[:T1], np.zeros(3, np.uint8), kind[T1:]])
    ref = OP.prefill_lazy_attention(f64(q_all), f64(k_all), f64(v_all), kind_all, layer_kind, mode)
    got1, got2 = bits_of(out1), bits_of(out2)
    for l in range(w.n_layers):
        assert_close(got1[l], ref[l, :T1], f"first chunk layer {l}")
        for t0 in range(0, T2, 64):
            assert_close(got2[l, t0:t0 + 64], ref[l, T1 + 3 + t0: T1 + 3 + t0 + 64], f"second chunk layer {l} tokens {t0}..")
    assert s.stats().device_error == 0
    s.close()
