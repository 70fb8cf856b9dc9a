"""GPU parity: the CUDA library through its C ABI against the fp64 oracle, same seeded inputs.

Bars: every output element within 2e-2 of the oracle and relative L2 error <= 5e-3
(bf16 storage, fp32 accumulation); page tables,
stream lengths, owner layers and Q Cache contents bit-exact.
"""

import math

import numpy as np
import pytest
import torch

from oracle import paging as pg
from oracle.lazy_attention import LazyAttentionOracle
from paper_2602_01901_b200 import binding as qc
from paper_2602_01901_b200 import workloads as W
from paper_2602_01901_b200.session import Session, bits_of

from oracle.lazy_attention import leaders_of as pg_leaders
from parity_util import MAX_ABS, REL_L2, SampledOracle, assert_close, f64, full_oracle, step_schedule

pytestmark = pytest.mark.gpu

MODES = [qc.QC_MODE_VLA_QC, qc.QC_MODE_VLA_EQ8, qc.QC_MODE_GLA]
MODE_IDS = ["vla_qc", "vla_eq8", "gla"]


def _outputs(w, dev):
    out = torch.empty((w.n_layers, w.batch, w.n_q_heads, w.head_dim), dtype=torch.bfloat16, device=dev)
    lse = torch.empty((w.n_layers, w.batch, w.n_q_heads), dtype=torch.float32, device=dev)
    return out, lse


# ------------------------------------------------------------------------------------------
# tiny: every step, every element, every mode (contiguous KV)
# ------------------------------------------------------------------------------------------

@pytest.mark.parametrize("mode", MODES, ids=MODE_IDS)
def test_tiny_every_step(mode):
    w = W.get_workload("tiny")
    s = Session.for_workload(w, lazy_mode=mode, poison_pool=True)
    s.prefill_workload(w)
    o = full_oracle(w, mode)
    out, lse = _outputs(w, s.device)
    ids = list(range(w.batch))
    for step in range(w.decode_steps):
        q, k, v = W.decode_qkv_torch(w, step, s.device)
        s.decode_step(ids, q, k, v, out, lse)
        qn, kn, vn = W.decode_qkv_np(w, step)
        got, got_lse = bits_of(out), lse.cpu().numpy()
        for b in range(w.batch):
            ref, ref_lse = o.decode_step(b, f64(qn[:, b]), f64(kn[:, b]), f64(vn[:, b]))
            for l in range(w.n_layers):
                assert_close(got[l, b], ref[l], f"tiny step {step} layer {l}")
            np.testing.assert_allclose(got_lse[:, b], ref_lse, atol=2e-3, rtol=0)
        # Q Cache: the lazy layer reads exactly the leader's q bits
        assert np.array_equal(s.read_qcache(1)[0], qn[0, 0])
        # appended rows: own text K of the lazy layer (VLA) and V
        pos = w.n_text_prompt + step
        assert np.array_equal(s.read_row(1, qc.QC_STREAM_V_TEXT, 0, pos, 3), vn[1, 0, 3])
        want_k = kn[0, 0, 3] if mode == qc.QC_MODE_GLA else kn[1, 0, 3]   # GLA aliases the leader's text K
        assert np.array_equal(s.read_row(1, qc.QC_STREAM_K_TEXT, 0, pos, 3), want_k)
    # contiguous layout: stream (layer, stream, seq) owns extent ((layer*4 + stream)*max_seqs + seq)
    max_pages = (w.max_tokens + 15) // 16
    ids_, n_tok, owner = s.page_table(1, qc.QC_STREAM_V_VISUAL, 0)
    assert owner == 1 and n_tok == 576
    assert ids_ == [((1 * 4 + 3) * 1 + 0) * max_pages + i for i in range(36)]
    ids_, n_tok, owner = s.page_table(1, qc.QC_STREAM_K_VISUAL, 0)
    assert owner == 0 and ids_[0] == ((0 * 4 + 1) * 1 + 0) * max_pages
    st = s.stats()
    assert st.device_error == 0
    row = w.n_kv_heads * w.head_dim * 2
    assert st.kv_bytes_stored == o.rows_stored() * row and st.kv_bytes_all_full == o.rows_all_full() * row
    s.close()


def _dev(a, device):
    return torch.from_numpy(a.astype(np.int16)).view(torch.bfloat16).to(device).contiguous()


# ------------------------------------------------------------------------------------------
# small paged case: ragged batch, GQA, several lazy-block shapes, split sizes, D in {64, 128}
# ------------------------------------------------------------------------------------------

def _small_workload(head_dim, group, layer_kind, index):
    lazy = tuple(i for i, k in enumerate(layer_kind) if k)
    return W.Workload(index, f"small{index}", len(layer_kind), 2 * group, 2, head_dim, 16, 3, 5, 150, 150, 22, 24, lazy)


SMALL = [
    # (head_dim, group, layer_kind, split_tokens)
    (128, 1, [0, 1, 0, 1, 1], 64),
    (128, 2, [0, 1, 1, 1, 1, 1, 0], 32),     # a block of six: more consumers than one sweep feeds
    (64, 1, [0, 0, 1], 16),
    (128, 4, [0, 1], 512),
    (64, 3, [0, 1, 0, 1], 128),
    (128, 7, [0, 1, 1], 48),                 # the query-group size of the GQA workload
    (64, 12, [0, 1, 1, 0], 80),              # a group wider than one tensor-core tile: two slices per KV head
]


@pytest.mark.parametrize("mode", MODES, ids=MODE_IDS)
@pytest.mark.parametrize("case", range(len(SMALL)))
def test_small_paged_ragged(mode, case):
    head_dim, group, layer_kind, split = SMALL[case]
    w = _small_workload(head_dim, group, layer_kind, 10 + case)
    trunc = [w.n_prompt, 9, 70]      # sequence 1: text only (5 text + 4 visual dropped below), sequence 2: ragged
    s = Session(w.n_layers, w.n_q_heads, w.n_kv_heads, head_dim, layer_kind, max_seqs=4, max_tokens_per_seq=256,
                n_pages=w.n_layers * 4 * 3 * 17, lazy_mode=mode, split_tokens=split, poison_pool=True)
    o = LazyAttentionOracle(w.n_layers, w.n_q_heads, w.n_kv_heads, head_dim, layer_kind, mode, n_seqs=3)
    model = pg.PagedCacheModel(layer_kind, mode, 16, w.n_layers * 4 * 3 * 17, 4)
    seq_ids = [2, 0, 3]              # library sequence ids differ from the batch index on purpose
    for b, sid in enumerate(seq_ids):
        kind, k, v = W.prefill_kv_np(w, b)
        T = trunc[b]
        kind, k, v = kind[:T].copy(), k[:, :T], v[:, :T]
        if b == 1:
            kind[:] = 0              # a sequence without any visual token
        kt = torch.from_numpy(k.astype(np.int16)).view(torch.bfloat16).to(s.device).contiguous()
        vt = torch.from_numpy(v.astype(np.int16)).view(torch.bfloat16).to(s.device).contiguous()
        s.prefill_append([sid], [T], kind, kt, vt)
        o.prefill_append(b, kind.tolist(), f64(k), f64(v))
        model.prefill_append([sid], [int((kind == 0).sum())], [int((kind == 1).sum())])
    _compare_tables(s, model, w.n_layers, seq_ids)
    out = torch.empty((w.n_layers, 3, w.n_q_heads, head_dim), dtype=torch.bfloat16, device=s.device)
    lse = torch.empty((w.n_layers, 3, w.n_q_heads), dtype=torch.float32, device=s.device)
    for step in range(w.decode_steps):
        qn, kn, vn = W.decode_qkv_np(w, step)
        dev = lambda a: torch.from_numpy(a.astype(np.int16)).view(torch.bfloat16).to(s.device).contiguous()
        s.decode_step(seq_ids, dev(qn), dev(kn), dev(vn), out, lse)
        model.decode_step(seq_ids)
        got, got_lse = bits_of(out), lse.cpu().numpy()
        for b in range(3):
            ref, ref_lse = o.decode_step(b, f64(qn[:, b]), f64(kn[:, b]), f64(vn[:, b]))
            for l in range(w.n_layers):
                assert_close(got[l, b], ref[l], f"case {case} step {step} seq {b} layer {l}")
            np.testing.assert_allclose(got_lse[:, b], ref_lse, atol=2e-3, rtol=0)
        if step in (0, 10, 11, w.decode_steps - 1):
            _compare_tables(s, model, w.n_layers, seq_ids)
    st = s.stats()
    assert st.device_error == 0
    assert st.pages_in_use == model.pages_in_use()
    row = w.n_kv_heads * head_dim * 2
    assert st.kv_bytes_stored == model.rows_stored() * row
    assert st.kv_bytes_all_full == model.rows_all_full() * row
    # freeing returns pages in the model's order: the next prefill must pop the same ids
    s_free = seq_ids[0]
    qc.qc_free_seq(s.cache, s_free)
    model.free_seq(s_free)
    kind, k, v = W.prefill_kv_np(w, 0)
    kt = torch.from_numpy(k[:, :40].astype(np.int16)).view(torch.bfloat16).to(s.device).contiguous()
    s.prefill_append([1], [40], kind[:40], kt, kt)
    model.prefill_append([1], [int((kind[:40] == 0).sum())], [int((kind[:40] == 1).sum())])
    _compare_tables(s, model, w.n_layers, [1, seq_ids[1], seq_ids[2], s_free])
    s.close()


def _compare_tables(s, model, n_layers, seq_ids):
    for sid in seq_ids:
        for l in range(n_layers):
            for stream in range(4):
                got = s.page_table(l, stream, sid)
                want = model.page_table(l, stream, sid)
                assert got == (want[0], want[1], want[2]), f"page table layer {l} stream {stream} seq {sid}"


# ------------------------------------------------------------------------------------------
# schedules and entry points that must not change the result
# ------------------------------------------------------------------------------------------

def test_launch_grouping_and_host_entry_give_identical_bits():
    w = _small_workload(128, 1, [0, 1, 0, 0, 1, 1], 20)
    results = []
    for variant in ("one_launch", "per_block", "host_buffers", "per_layer", "per_layer_set_then_host_buffers"):
        s = Session.for_workload(w, lazy_mode=qc.QC_MODE_VLA_QC, split_tokens=64)
        s.prefill_workload(w)
        s.set_option("static_partition", 0)   # same chunks in every variant: the bits can then be compared
        if variant == "per_block":
            s.set_option("layers_per_launch", 1)
        if variant.startswith("per_layer"):
            s.set_option("per_layer_logit_cache", 1)   # (the host-buffer entry point keeps its own launch groups)
        out, lse = _outputs(w, s.device)
        outs = []
        for step in range(6):
            q, k, v = W.decode_qkv_torch(w, step, s.device)
            if variant.endswith("host_buffers"):
                hq, hk, hv = q.cpu().pin_memory(), k.cpu().pin_memory(), v.cpu().pin_memory()
                ho = torch.empty(out.shape, dtype=torch.bfloat16).pin_memory()
                s.decode_step_host(list(range(w.batch)), hq, hk, hv, ho)
                outs.append(ho.view(torch.int16).numpy().copy())
            else:
                s.decode_step(list(range(w.batch)), q, k, v, out, lse)
                outs.append(out.view(torch.int16).cpu().numpy())
        assert s.stats().device_error == 0
        results.append(np.stack(outs))
        s.close()
    for other in results[1:]:
        assert np.array_equal(results[0], other)


@pytest.mark.parametrize("mode", MODES, ids=MODE_IDS)
@pytest.mark.parametrize("case", [0, 1, 4, 5, 6])
def test_per_layer_schedule_with_logit_cache(mode, case):
    """One launch per layer, in layer order; a leader stores the scores its followers share and
    the followers read them instead of the leader's K.  By Eq. 6 (GLA) and the Q Cache rule (VLA_QC)
    those scores ARE the follower's, so the outputs must equal the fused schedule's bit for bit at
    the same split, and the oracle's within tolerance.  Ragged batch: a sequence without visual
    tokens, different lengths, pages that fill up during the steps."""
    head_dim, group, layer_kind, split = SMALL[case]
    w = _small_workload(head_dim, group, layer_kind, 40 + case)
    trunc = [w.n_prompt, 9, 70]
    seq_ids = [2, 0, 3]
    o = LazyAttentionOracle(w.n_layers, w.n_q_heads, w.n_kv_heads, head_dim, layer_kind, mode, n_seqs=3)
    sessions = []
    for per_layer in (False, True):
        s = Session(w.n_layers, w.n_q_heads, w.n_kv_heads, head_dim, layer_kind, max_seqs=4, max_tokens_per_seq=256,
                    n_pages=w.n_layers * 4 * 3 * 17, lazy_mode=mode, split_tokens=split, poison_pool=True)
        s.set_option("static_partition", 0)   # same chunks in both schedules
        if per_layer:
            s.set_option("per_layer_logit_cache", 1)
        sessions.append(s)
    for b, sid in enumerate(seq_ids):
        kind, k, v = W.prefill_kv_np(w, b)
        T = trunc[b]
        kind, k, v = kind[:T].copy(), k[:, :T], v[:, :T]
        if b == 1:
            kind[:] = 0
        for s in sessions:
            s.prefill_append([sid], [T], kind, _dev(k, s.device), _dev(v, s.device))
        o.prefill_append(b, kind.tolist(), f64(k), f64(v))
    outs = [torch.empty((w.n_layers, 3, w.n_q_heads, head_dim), dtype=torch.bfloat16, device=s.device) for s in sessions]
    lses = [torch.empty((w.n_layers, 3, w.n_q_heads), dtype=torch.float32, device=s.device) for s in sessions]
    for step in range(w.decode_steps):
        qn, kn, vn = W.decode_qkv_np(w, step)
        for s, out, lse in zip(sessions, outs, lses):
            s.decode_step(seq_ids, _dev(qn, s.device), _dev(kn, s.device), _dev(vn, s.device), out, lse)
        assert torch.equal(outs[0].view(torch.int16), outs[1].view(torch.int16)), f"step {step}: schedules differ"
        assert torch.equal(lses[0], lses[1]), f"step {step}: log-sum-exp differs"
        got = bits_of(outs[1])
        for b in range(3):
            ref, _ = o.decode_step(b, f64(qn[:, b]), f64(kn[:, b]), f64(vn[:, b]))
            for l in range(w.n_layers):
                assert_close(got[l, b], ref[l], f"per-layer schedule: case {case} step {step} seq {b} layer {l}")
    for s in sessions:
        assert s.stats().device_error == 0
        s.close()


SCHEDULES = {
    # option settings that change how a step is cut into launches and work ranges, never its result
    "one_launch_static_ranges": [("static_partition", 1)],
    "per_block_static_ranges": [("layers_per_launch", 1)],
    "per_layer_logit_cache_static_ranges": [("per_layer_logit_cache", 1)],
    "in_order": [("in_order_launches", 1)],
    "in_order_claimed_items": [("in_order_launches", 1), ("static_partition", 0)],
    "in_order_short_ranges": [("in_order_launches", 1), ("static_min_tiles", 1), ("static_row_cost", 0)],
    "in_order_costly_rows": [("in_order_launches", 1), ("static_row_cost", 5)],
    "in_order_append_at_step_start": [("in_order_launches", 1), ("fold_append", 0)],
    "in_order_merge_in_kernel": [("in_order_launches", 1), ("fused_merge", 1)],
    "one_launch_merge_in_kernel": [("fused_merge", 1)],
}


@pytest.mark.parametrize("schedule", sorted(SCHEDULES))
@pytest.mark.parametrize("mode", MODES, ids=MODE_IDS)
@pytest.mark.parametrize("case", range(len(SMALL)))
def test_schedules_against_the_oracle(mode, case, schedule):
    """Every way of cutting a step into launches and work ranges gives the oracle's result: static
    ranges instead of claimed items, one launch per lazy block, one launch per layer with the logit
    cache, and the in-order schedule in which a leader's launch also sweeps its followers' cached V
    rows (a VLA_QC follower's own launch is its text sweep; a GLA follower's is the merge, which
    adds the new token as one more key, Eq. 6).  Ragged batch: a sequence without visual tokens,
    different lengths, pages that fill up during the steps."""
    head_dim, group, layer_kind, split = SMALL[case]
    w = _small_workload(head_dim, group, layer_kind, 60 + case)
    trunc = [w.n_prompt, 9, 70]
    seq_ids = [2, 0, 3]
    o = LazyAttentionOracle(w.n_layers, w.n_q_heads, w.n_kv_heads, head_dim, layer_kind, mode, n_seqs=3)
    s = Session(w.n_layers, w.n_q_heads, w.n_kv_heads, head_dim, layer_kind, max_seqs=4, max_tokens_per_seq=256,
                n_pages=w.n_layers * 4 * 3 * 17, lazy_mode=mode, split_tokens=split, poison_pool=True)
    for key, value in SCHEDULES[schedule]:
        s.set_option(key, value)
    for b, sid in enumerate(seq_ids):
        kind, k, v = W.prefill_kv_np(w, b)
        T = trunc[b]
        kind, k, v = kind[:T].copy(), k[:, :T], v[:, :T]
        if b == 1:
            kind[:] = 0
        s.prefill_append([sid], [T], kind, _dev(k, s.device), _dev(v, s.device))
        o.prefill_append(b, kind.tolist(), f64(k), f64(v))
    out = torch.empty((w.n_layers, 3, w.n_q_heads, head_dim), dtype=torch.bfloat16, device=s.device)
    lse = torch.empty((w.n_layers, 3, w.n_q_heads), dtype=torch.float32, device=s.device)
    for step in range(w.decode_steps):
        qn, kn, vn = W.decode_qkv_np(w, step)
        s.decode_step(seq_ids, _dev(qn, s.device), _dev(kn, s.device), _dev(vn, s.device), out, lse)
        got, got_lse = bits_of(out), lse.cpu().numpy()
        for b in range(3):
            ref, ref_lse = o.decode_step(b, f64(qn[:, b]), f64(kn[:, b]), f64(vn[:, b]))
            for l in range(w.n_layers):
                assert_close(got[l, b], ref[l], f"{schedule}: case {case} step {step} seq {b} layer {l}")
            np.testing.assert_allclose(got_lse[:, b], ref_lse, atol=2e-3, rtol=0)
    # what the last step left in the cache, whichever launch stored it: the new rows and the Q Cache, bit for bit
    leaders = pg_leaders(layer_kind)
    for b, sid in enumerate(seq_ids):
        _, n_text, _ = s.page_table(0, qc.QC_STREAM_V_TEXT, sid)
        for l in range(w.n_layers):
            assert np.array_equal(s.read_row(l, qc.QC_STREAM_V_TEXT, sid, n_text - 1, 1), vn[l, b, 1])
            owner = l if (layer_kind[l] == 0 or mode != qc.QC_MODE_GLA) else leaders[l]
            assert np.array_equal(s.read_row(l, qc.QC_STREAM_K_TEXT, sid, n_text - 1, 1), kn[owner, b, 1])
            if layer_kind[l]:
                assert np.array_equal(s.read_qcache(l)[sid], qn[leaders[l], b])
    assert s.stats().device_error == 0
    s.close()


def test_split_size_changes_only_rounding():
    w = _small_workload(128, 1, [0, 1], 21)
    o = full_oracle(w, qc.QC_MODE_VLA_QC)
    qn, kn, vn = W.decode_qkv_np(w, 0)
    refs = [o.decode_step(b, f64(qn[:, b]), f64(kn[:, b]), f64(vn[:, b]))[0] for b in range(w.batch)]
    for split in (16, 48, 112, 512):
        s = Session.for_workload(w, split_tokens=16)
        s.set_option("split_tokens", split)
        s.prefill_workload(w)
        out, lse = _outputs(w, s.device)
        q, k, v = W.decode_qkv_torch(w, 0, s.device)
        s.decode_step(list(range(w.batch)), q, k, v, out, lse)
        got = bits_of(out)
        for b in range(w.batch):
            for l in range(w.n_layers):
                assert_close(got[l, b], refs[b][l], f"split {split} seq {b} layer {l}")
        s.close()


# ------------------------------------------------------------------------------------------
# error behaviour: status codes, cache unchanged
# ------------------------------------------------------------------------------------------

def test_errors_leave_the_cache_unchanged():
    w = _small_workload(128, 1, [0, 1], 22)
    # lazy layer 0 is refused at allocation
    with pytest.raises(qc.QcError) as e:
        Session(2, 2, 2, 128, [1, 0], max_seqs=1, max_tokens_per_seq=64, n_pages=64)
    assert e.value.status == qc.QC_ERR_STATE
    # a pool with room for the prompt (177 tokens -> 2 text + 10 visual pages per stream) but not one more page
    prompt_pages = (2 + 10) * 2 + (2 + 2 + 10)
    s = Session(2, 2, 2, 128, [0, 1], max_seqs=2, max_tokens_per_seq=256, n_pages=prompt_pages + 2)
    kind, k, v = W.prefill_kv_np(w, 0)
    kt = torch.from_numpy(k.astype(np.int16)).view(torch.bfloat16).to(s.device).contiguous()
    s.prefill_append([0], [len(kind)], kind, kt, kt)
    out = torch.empty((2, 1, 2, 128), dtype=torch.bfloat16, device=s.device)
    q, kk, vv = (t[:, :1].contiguous() for t in W.decode_qkv_torch(w, 0, s.device))
    # unknown sequence, duplicate ids, bad id
    for ids, status in (([1], qc.QC_ERR_STATE), ([0, 0], qc.QC_ERR_STATE), ([7], qc.QC_ERR_INVALID_ARG)):
        with pytest.raises(qc.QcError) as e:
            s.decode_step(ids, q, kk, vv, out)
        assert e.value.status == status
    before = [s.page_table(l, st, 0) for l in range(2) for st in range(4)]
    # text length 27 -> steps at lengths 27..31 fit the last page; the step at length 32 needs 4 pages, 2 free
    for step in range(5):
        s.decode_step([0], q, kk, vv, out)
    mid = [s.page_table(l, st, 0) for l in range(2) for st in range(4)]
    with pytest.raises(qc.QcError) as e:
        s.decode_step([0], q, kk, vv, out)
    assert e.value.status == qc.QC_ERR_OOM_PAGES
    assert [s.page_table(l, st, 0) for l in range(2) for st in range(4)] == mid
    assert mid[0][1] == before[0][1] + 5
    with pytest.raises(qc.QcError) as e:
        s.prefill_append([1], [len(kind)], kind, kt, kt)
    assert e.value.status == qc.QC_ERR_OOM_PAGES
    assert s.page_table(0, 0, 1) == ([], 0, -1)
    assert s.stats().device_error == 0
    s.close()


# ------------------------------------------------------------------------------------------
# full-size configurations, launched as the benchmark launches them; sampled outputs
# ------------------------------------------------------------------------------------------

def _samples(w, n, rng):
    lazy = list(w.lazy_layers)
    fixed = [(0, 0, 0), (w.n_layers - 1, w.batch - 1, w.n_q_heads - 1), (lazy[0], 0, 1), (lazy[0] - 1, 0, 1),
             (lazy[-1], w.batch - 1, 0), (1, w.batch // 2, w.n_q_heads // 2)]
    out = list(dict.fromkeys(fixed))
    while len(out) < n:
        t = (int(rng.integers(w.n_layers)), int(rng.integers(w.batch)), int(rng.integers(w.n_q_heads)))
        if t not in out:
            out.append(t)
    return out


def test_options_reject_what_they_cannot_take():
    w = _small_workload(128, 1, [0, 1], 24)
    s = Session.for_workload(w, split_tokens=64)
    for key, value in (("no_such_option", 1), ("layers_per_launch", -1), ("layers_per_launch", 3),
                       ("prefill_shared_scores", 3), ("split_tokens", 24), ("split_tokens", 32), ("split_tokens", 1024)):
        with pytest.raises(qc.QcError) as e:
            s.set_option(key, value)
        assert e.value.status == qc.QC_ERR_INVALID_ARG, (key, value)
    for key, value in (("layers_per_launch", 1), ("per_layer_logit_cache", 1), ("per_layer_logit_cache", 0),
                       ("prefill_shared_scores", 2), ("prefill_tcgen05", 0), ("split_tokens", 128), ("split_tokens", 0)):
        s.set_option(key, value)
    s.close()


@pytest.mark.parametrize("mode", MODES, ids=MODE_IDS)
def test_multi_turn_prefill_after_decode(mode):
    """A conversation with a second image: prompt, a few generated tokens, more prompt tokens
    (text and visual) appended to the same sequence, more generated tokens."""
    layer_kind = [0, 1, 1, 0, 1]
    w = _small_workload(128, 2, layer_kind, 23)
    n_pages = w.n_layers * 4 * 2 * 24
    s = Session(w.n_layers, w.n_q_heads, w.n_kv_heads, 128, layer_kind, max_seqs=2, max_tokens_per_seq=384,
                n_pages=n_pages, lazy_mode=mode, split_tokens=64, poison_pool=True)
    o = LazyAttentionOracle(w.n_layers, w.n_q_heads, w.n_kv_heads, 128, layer_kind, mode, n_seqs=2)
    model = pg.PagedCacheModel(layer_kind, mode, 16, n_pages, 2)
    dev = lambda a: torch.from_numpy(a.astype(np.int16)).view(torch.bfloat16).to(s.device).contiguous()
    kinds, ks, vs = zip(*[W.prefill_kv_np(w, b) for b in range(2)])
    out = torch.empty((w.n_layers, 2, w.n_q_heads, 128), dtype=torch.bfloat16, device=s.device)
    step = 0

    def turn(first, last, n_decode):
        nonlocal step
        for b in range(2):
            kd, k, v = kinds[b][first:last], ks[b][:, first:last], vs[b][:, first:last]
            s.prefill_append([b], [last - first], kd, dev(k), dev(v))
            o.prefill_append(b, kd.tolist(), f64(k), f64(v))
            model.prefill_append([b], [int((kd == 0).sum())], [int((kd == 1).sum())])
        for _ in range(n_decode):
            qn, kn, vn = W.decode_qkv_np(w, step, seqs=[0, 1])
            s.decode_step([0, 1], dev(qn), dev(kn), dev(vn), out)
            model.decode_step([0, 1])
            got = bits_of(out)
            for b in range(2):
                ref, _ = o.decode_step(b, f64(qn[:, b]), f64(kn[:, b]), f64(vn[:, b]))
                for l in range(w.n_layers):
                    assert_close(got[l, b], ref[l], f"turn ending at {last}, step {step}, seq {b}, layer {l}")
            step += 1
        _compare_tables(s, model, w.n_layers, [0, 1])

    turn(0, 60, 5)          # 5 text + 55 visual tokens, then 5 generated
    turn(60, 177, 7)        # the rest of the image and the trailing text arrive later
    assert s.stats().device_error == 0
    s.close()


def test_many_short_sequences_and_a_partial_batch():
    """More sequences than travel as a kernel argument (descriptor copy path), ragged lengths, and
    steps that list only some of the active sequences."""
    layer_kind = [0, 1, 0]
    n_seqs, D = 70, 64
    w = W.Workload(24, "many", 3, 4, 2, D, 16, n_seqs, 2, 30, 30, 5, 6, (1,))
    s = Session(3, 4, 2, D, layer_kind, max_seqs=n_seqs, max_tokens_per_seq=64, n_pages=3 * 4 * n_seqs * 4,
                lazy_mode=qc.QC_MODE_VLA_QC, poison_pool=True)
    o = LazyAttentionOracle(3, 4, 2, D, layer_kind, qc.QC_MODE_VLA_QC, n_seqs=n_seqs)
    dev = lambda a: torch.from_numpy(a.astype(np.int16)).view(torch.bfloat16).to(s.device).contiguous()
    for b in range(n_seqs):
        kind, k, v = W.prefill_kv_np(w, b)
        T = 8 + (b * 7) % 29                     # 8..36 tokens: ragged, some without a full page
        s.prefill_append([b], [T], kind[:T], dev(k[:, :T]), dev(v[:, :T]))
        o.prefill_append(b, kind[:T].tolist(), f64(k[:, :T]), f64(v[:, :T]))
    for step, ids in enumerate([list(range(n_seqs)), list(range(0, n_seqs, 3)), list(range(n_seqs))[::-1],
                                [5, 69, 17]]):
        qn, kn, vn = W.decode_qkv_np(w, step, seqs=ids)
        out = torch.empty((3, len(ids), 4, D), dtype=torch.bfloat16, device=s.device)
        s.decode_step(ids, dev(qn), dev(kn), dev(vn), out)
        got = bits_of(out)
        for i, b in enumerate(ids):
            ref, _ = o.decode_step(b, f64(qn[:, i]), f64(kn[:, i]), f64(vn[:, i]))
            for l in range(3):
                assert_close(got[l, i], ref[l], f"step {step} seq {b} layer {l}")
    assert s.stats().device_error == 0
    s.close()


def test_empty_calls_and_the_length_limit():
    """Empty lists are accepted and do nothing; a sequence can grow exactly to max_tokens_per_seq."""
    layer_kind = [0, 1]
    w = W.Workload(25, "edge", 2, 2, 2, 64, 16, 1, 3, 9, 9, 2, 4, (1,))
    s = Session(2, 2, 2, 64, layer_kind, max_seqs=2, max_tokens_per_seq=8, n_pages=2 * 4 * 2 * 2, poison_pool=True)
    o = LazyAttentionOracle(2, 2, 2, 64, layer_kind, qc.QC_MODE_VLA_QC, n_seqs=1)
    dev = lambda a: torch.from_numpy(a.astype(np.int16)).view(torch.bfloat16).to(s.device).contiguous()
    kind, k, v = W.prefill_kv_np(w, 0)                  # 3 text, 9 visual, 2 text
    out = torch.zeros((2, 1, 2, 64), dtype=torch.bfloat16, device=s.device)
    lib = qc.load()
    assert lib.qc_decode_step(s.cache, 0, None, None, None, None, None, None) == qc.QC_OK
    assert lib.qc_prefill_append(s.cache, 0, None, None, None, None, None) == qc.QC_OK
    s.prefill_append([0], [0], [], dev(k[:, :1]), dev(v[:, :1]))        # a listed sequence with no tokens
    assert s.page_table(0, 0, 0)[1] == 0
    with pytest.raises(qc.QcError) as e:                                  # 9 visual tokens exceed the bound of 8
        s.prefill_append([0], [14], kind, dev(k), dev(v))
    assert e.value.status == qc.QC_ERR_INVALID_ARG and s.page_table(0, 1, 0)[1] == 0
    keep = np.r_[0:3, 3:11, 12:14]                                        # 5 text + 8 visual
    s.prefill_append([0], [len(keep)], kind[keep], dev(k[:, keep]), dev(v[:, keep]))
    o.prefill_append(0, kind[keep].tolist(), f64(k[:, keep]), f64(v[:, keep]))
    for step in range(3):                                                 # text length 5 -> 8: the limit
        qn, kn, vn = W.decode_qkv_np(w, step)
        s.decode_step([0], dev(qn), dev(kn), dev(vn), out)
        ref, _ = o.decode_step(0, f64(qn[:, 0]), f64(kn[:, 0]), f64(vn[:, 0]))
        got = bits_of(out)
        for l in range(2):
            assert_close(got[l, 0], ref[l], f"step {step} layer {l}")
    with pytest.raises(qc.QcError) as e:                                  # one token too many
        s.decode_step([0], dev(qn), dev(kn), dev(vn), out)
    assert e.value.status == qc.QC_ERR_INVALID_ARG and s.page_table(0, 0, 0)[1] == 8
    assert s.stats().device_error == 0
    s.close()


FULL_CASES = [
    ("llava15_7b", qc.QC_MODE_VLA_QC, 40),
    ("llava15_7b", qc.QC_MODE_VLA_EQ8, 16),
    ("llava15_7b", qc.QC_MODE_GLA, 16),
    ("llava_next_anyres", qc.QC_MODE_VLA_QC, 32),
    ("qwen2vl_gqa", qc.QC_MODE_VLA_QC, 40),
    ("long_video_pruned", qc.QC_MODE_VLA_QC, 24),
    ("llava_next_2048_lazy22", qc.QC_MODE_VLA_QC, 24),     # blocks of one ordinary + three lazy layers
    ("llava_next_2048_lazy22", qc.QC_MODE_GLA, 16),
    # the per-layer schedule with the logit cache (the configuration bench.py times as per_layer_launches)
    ("llava15_7b", qc.QC_MODE_VLA_QC, 16, "per_layer"),
    ("qwen2vl_gqa", qc.QC_MODE_VLA_QC, 16, "per_layer"),
    ("llava_next_2048_lazy22", qc.QC_MODE_GLA, 16, "per_layer"),
    # the in-order schedule (the configuration bench.py's headline is timed on)
    ("llava15_7b", qc.QC_MODE_VLA_QC, 24, "in_order"),
    ("llava_next_anyres", qc.QC_MODE_VLA_QC, 16, "in_order"),
    ("qwen2vl_gqa", qc.QC_MODE_VLA_QC, 24, "in_order"),
    ("long_video_pruned", qc.QC_MODE_VLA_QC, 16, "in_order"),
    ("llava15_7b", qc.QC_MODE_GLA, 16, "in_order"),
    ("llava_next_2048_lazy22", qc.QC_MODE_GLA, 16, "in_order"),
    ("llava_next_2048_lazy22", qc.QC_MODE_VLA_QC, 16, "in_order"),
    # the host-buffer entry point (four launch groups of lazy blocks, copies overlapped)
    ("llava15_7b", qc.QC_MODE_VLA_QC, 16, "host"),
    ("qwen2vl_gqa", qc.QC_MODE_GLA, 16, "host"),
    ("long_video_pruned", qc.QC_MODE_VLA_QC, 16, "host"),
]


@pytest.mark.parametrize("case", FULL_CASES, ids=["-".join([c[0], MODE_IDS[c[1]]] + list(c[3:])) for c in FULL_CASES])
def test_full_size_sampled(case):
    name, mode, n_samples = case[:3]
    launches = case[3] if len(case) > 3 else "one_launch"
    w = W.get_workload(name)
    rng = np.random.default_rng(w.seed)
    samples = _samples(w, n_samples, rng)
    oracles = [SampledOracle(w, mode, *t) for t in samples]
    schedule = set(step_schedule(w.decode_steps))
    s = Session.for_workload(w, lazy_mode=mode)
    if launches == "per_layer":
        s.set_option("per_layer_logit_cache", 1)
    elif launches == "in_order":
        s.set_option("in_order_launches", 1)
    s.prefill_workload(w)
    model = pg.PagedCacheModel(w.layer_kind().tolist(), mode, 16, s.cfg.n_pages, w.batch)
    for b in range(w.batch):
        model.prefill_append([b], [w.n_text_prompt], [w.n_visual_kept])
    _compare_tables(s, model, w.n_layers, [0, w.batch - 1])
    out, lse = _outputs(w, s.device)
    ids = qc._i32_array(list(range(w.batch)))
    li = torch.tensor([t[0] for t in samples], device=s.device)
    bi = torch.tensor([t[1] for t in samples], device=s.device)
    hi = torch.tensor([t[2] for t in samples], device=s.device)
    worst = (0.0, 0.0)
    if launches == "host":
        h_out = torch.empty(out.shape, dtype=torch.bfloat16).pin_memory()
        h_lse = torch.empty(lse.shape, dtype=torch.float32).pin_memory()
    for step in range(w.decode_steps):
        q, k, v = W.decode_qkv_torch(w, step, s.device)
        if launches == "host":
            s.decode_step_host(ids, q.cpu().pin_memory(), k.cpu().pin_memory(), v.cpu().pin_memory(), h_out, h_lse)
            out.copy_(h_out)
            lse.copy_(h_lse)
        else:
            s.decode_step(ids, q, k, v, out, lse)
        model.decode_step(list(range(w.batch)))
        refs = [o.advance() for o in oracles]
        if step in schedule:
            got = bits_of(out[li, bi, hi])
            got_lse = lse[li, bi, hi].cpu().numpy()
            assert np.all(np.isfinite(f64(bits_of(out)))), f"step {step}: non-finite output somewhere"
            for i, (ref, ref_lse) in enumerate(refs):
                e, r = assert_close(got[i], ref, f"{name} step {step} sample {samples[i]}")
                worst = (max(worst[0], e), max(worst[1], r))
                assert abs(got_lse[i] - ref_lse) <= 2e-3
    st = s.stats()
    assert st.device_error == 0
    assert st.pages_in_use == model.pages_in_use()
    for sid in (0, w.batch // 2, w.batch - 1):
        _compare_tables(s, model, w.n_layers, [sid])
    # Q Cache after the last step: leader's q bits of that step
    lazy_layer = w.lazy_layers[0]
    q_last = W.decode_qkv_np(w, w.decode_steps - 1, layers=[lazy_layer - 1])[0][0]
    assert np.array_equal(s.read_qcache(lazy_layer)[: w.batch], q_last)
    # KV-saving metric: token-exact bytes against the integer model
    row = w.n_kv_heads * w.head_dim * 2
    assert st.kv_bytes_stored == model.rows_stored() * row
    assert st.kv_bytes_all_full == model.rows_all_full() * row
    print(f"{name} mode {mode}: worst max-abs {worst[0]:.3e} (bar {MAX_ABS}), worst rel-L2 {worst[1]:.3e} (bar {REL_L2})")
    s.close()
