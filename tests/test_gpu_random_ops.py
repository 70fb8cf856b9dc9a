"""Random sequences of calls on a small cache, checked after every decode step.

A seeded generator draws what a serving loop does in arbitrary order: start a sequence with a
prompt (any mix of text and visual tokens, including none of one kind), decode a step for a random
subset of the live sequences, append a later turn to a live sequence, free a sequence and reuse
its id.  After every decode step the outputs are compared with the fp64 oracle (one oracle object
per sequence lifetime) and the page tables with the integer model of the allocator.  Each trial
also draws the lazy mode, the layer pattern, the split size and the schedule (one launch per step,
one per lazy block, one per layer with the logit cache).
"""

from __future__ import annotations

import numpy as np
import pytest
import torch

from oracle import paging as pg
from oracle.lazy_attention import LazyAttentionOracle
from paper_2602_01901_b200 import binding as qc
from paper_2602_01901_b200 import workloads as W
from paper_2602_01901_b200.session import Session, bits_of

from parity_util import assert_close, f64

pytestmark = pytest.mark.gpu

PATTERNS = [[0, 1], [0, 1, 1, 0], [0, 0, 1, 1, 1], [0, 1, 0, 1, 1, 1, 1], [0, 0, 0]]
SHAPES = [(128, 1, 2), (64, 2, 2), (128, 7, 1), (64, 1, 4), (128, 4, 2)]   # head_dim, group, kv heads
MAX_SEQS, MAX_TOKENS = 5, 160


def _bits(rng, shape):
    return W.f32_to_bf16_bits(rng.standard_normal(shape).astype(np.float32))


def _dev(a, device):
    return torch.from_numpy(a.astype(np.int16)).view(torch.bfloat16).to(device).contiguous()


@pytest.mark.parametrize("trial", range(30))
def test_random_call_sequences(trial):
    rng = np.random.default_rng(9000 + trial)
    layer_kind = PATTERNS[trial % len(PATTERNS)]
    head_dim, group, hkv = SHAPES[(trial // 2) % len(SHAPES)]
    mode = int(rng.integers(3))
    schedule = ["fused", "per_block", "per_layer", "in_order"][trial % 4]
    split = int(rng.choice([16, 32, 64, 128]))
    n_layers, hq = len(layer_kind), hkv * group
    n_pages = n_layers * 4 * MAX_SEQS * (MAX_TOKENS // 16 + 1)
    s = Session(n_layers, hq, hkv, head_dim, layer_kind, max_seqs=MAX_SEQS, max_tokens_per_seq=MAX_TOKENS,
                n_pages=n_pages, lazy_mode=mode, split_tokens=split, poison_pool=True)
    if schedule == "per_block":
        s.set_option("layers_per_launch", 1)
    elif schedule == "per_layer":
        s.set_option("per_layer_logit_cache", 1)
    elif schedule == "in_order":
        s.set_option("in_order_launches", 1)
    model = pg.PagedCacheModel(layer_kind, mode, 16, n_pages, MAX_SEQS)
    oracles = {}      # live sequence id -> oracle of that lifetime
    lengths = {}      # live sequence id -> tokens held
    what = f"trial {trial} (mode {mode}, {schedule}, split {split}, layers {layer_kind}, D {head_dim}, group {group})"

    def append_tokens(sid, n):
        kind = (rng.random(n) < rng.choice([0.0, 0.5, 0.9, 1.0])).astype(np.uint8)
        k, v = _bits(rng, (n_layers, n, hkv, head_dim)), _bits(rng, (n_layers, n, hkv, head_dim))
        s.prefill_append([sid], [n], kind, _dev(k, s.device), _dev(v, s.device))
        oracles[sid].prefill_append(0, kind.tolist(), f64(k), f64(v))
        model.prefill_append([sid], [int((kind == 0).sum())], [int((kind == 1).sum())])
        lengths[sid] += n

    def check_tables():
        for sid in lengths:
            for l in range(n_layers):
                for stream in range(4):
                    got = s.page_table(l, stream, sid)
                    want = model.page_table(l, stream, sid)
                    assert got == (want[0], want[1], want[2]), f"{what}: page table layer {l} stream {stream} seq {sid}"

    decode_steps = 0
    for op_index in range(60):
        free_ids = [i for i in range(MAX_SEQS) if i not in lengths]
        r = rng.random()
        if free_ids and (not lengths or r < 0.15):
            sid = int(rng.choice(free_ids))
            oracles[sid] = LazyAttentionOracle(n_layers, hq, hkv, head_dim, layer_kind, mode, n_seqs=1)
            lengths[sid] = 0
            append_tokens(sid, int(rng.integers(1, 70)))
        elif r < 0.25 and lengths:
            sid = int(rng.choice(list(lengths)))
            n = int(rng.integers(1, 30))
            if lengths[sid] + n + 8 < MAX_TOKENS:
                append_tokens(sid, n)          # a later turn of a live sequence
        elif r < 0.33 and len(lengths) > 1:
            sid = int(rng.choice(list(lengths)))
            qc.qc_free_seq(s.cache, sid)
            model.free_seq(sid)
            del lengths[sid], oracles[sid]
        else:
            live = [sid for sid in lengths if lengths[sid] + 1 <= MAX_TOKENS]
            if not live:
                continue
            ids = [int(x) for x in rng.permutation(live)[: int(rng.integers(1, len(live) + 1))]]
            n = len(ids)
            q = _bits(rng, (n_layers, n, hq, head_dim))
            k, v = _bits(rng, (n_layers, n, hkv, head_dim)), _bits(rng, (n_layers, n, hkv, head_dim))
            out = torch.empty((n_layers, n, hq, head_dim), dtype=torch.bfloat16, device=s.device)
            lse = torch.empty((n_layers, n, hq), dtype=torch.float32, device=s.device)
            s.decode_step(ids, _dev(q, s.device), _dev(k, s.device), _dev(v, s.device), out, lse)
            model.decode_step(ids)
            got, got_lse = bits_of(out), lse.cpu().numpy()
            for i, sid in enumerate(ids):
                ref, ref_lse = oracles[sid].decode_step(0, f64(q[:, i]), f64(k[:, i]), f64(v[:, i]))
                for l in range(n_layers):
                    assert_close(got[l, i], ref[l], f"{what}: op {op_index} seq {sid} layer {l}")
                np.testing.assert_allclose(got_lse[:, i], ref_lse, atol=2e-3, rtol=0)
                lengths[sid] += 1
            decode_steps += 1
        if op_index % 10 == 9:
            check_tables()
    check_tables()
    st = s.stats()
    assert st.device_error == 0
    assert st.pages_in_use == model.pages_in_use()
    assert decode_steps >= 10, f"{what}: the draw produced too few decode steps to mean anything"
    s.close()
