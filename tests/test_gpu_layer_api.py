"""qc_decode_begin / qc_decode_layer: a decode step issued layer by layer, each call with only that
layer's q/k/v (separately allocated tensors, so that nothing of another layer is within reach),
against the fp64 oracle and against qc_decode_step on a twin cache.  Ragged batch, all modes, MHA
and GQA shapes, blocks with several followers, pages that fill up during the steps."""

import numpy as np
import pytest
import torch

from oracle.lazy_attention import LazyAttentionOracle
from paper_2602_01901_b200 import binding as qc
from paper_2602_01901_b200 import workloads as W
from paper_2602_01901_b200.session import Session, bits_of

from parity_util import MAX_ABS, REL_L2, assert_close, f64

pytestmark = pytest.mark.gpu

MODES = [qc.QC_MODE_VLA_QC, qc.QC_MODE_VLA_EQ8, qc.QC_MODE_GLA]
SHAPES = [
    # (head_dim, group, layer_kind)
    (128, 1, [0, 1, 0, 1, 1]),
    (128, 7, [0, 1, 1]),
    (64, 3, [0, 0, 1, 0]),
    (128, 2, [0, 1, 1, 1, 1, 1, 0]),
]


def _dev(a, device):
    return torch.from_numpy(a.astype(np.int16)).view(torch.bfloat16).to(device).contiguous()


@pytest.mark.parametrize("mode", MODES, ids=["vla_qc", "vla_eq8", "gla"])
@pytest.mark.parametrize("shape", range(len(SHAPES)))
def test_layer_by_layer_step_matches_the_oracle_and_the_step_call(mode, shape):
    head_dim, group, layer_kind = SHAPES[shape]
    lazy = tuple(i for i, k in enumerate(layer_kind) if k)
    w = W.Workload(70 + shape, f"layer{shape}", len(layer_kind), 2 * group, 2, head_dim, 16, 3, 5, 150, 150, 22, 20, lazy)
    trunc, seq_ids = [w.n_prompt, 9, 70], [2, 0, 3]
    o = LazyAttentionOracle(w.n_layers, w.n_q_heads, w.n_kv_heads, head_dim, layer_kind, mode, n_seqs=3)
    sessions = [Session(w.n_layers, w.n_q_heads, w.n_kv_heads, head_dim, layer_kind, max_seqs=4, max_tokens_per_seq=256,
                        n_pages=w.n_layers * 4 * 3 * 17, lazy_mode=mode, poison_pool=True) for _ in range(2)]
    layered, whole = sessions
    for b, sid in enumerate(seq_ids):
        kind, k, v = W.prefill_kv_np(w, b)
        T = trunc[b]
        kind, k, v = kind[:T].copy(), k[:, :T], v[:, :T]
        if b == 1:
            kind[:] = 0
        for s in sessions:
            s.prefill_append([sid], [T], kind, _dev(k, s.device), _dev(v, s.device))
        o.prefill_append(b, kind.tolist(), f64(k), f64(v))
    dev = layered.device
    out_whole = torch.empty((w.n_layers, 3, w.n_q_heads, head_dim), dtype=torch.bfloat16, device=dev)
    for step in range(w.decode_steps):
        qn, kn, vn = W.decode_qkv_np(w, step)
        whole.decode_step(seq_ids, _dev(qn, dev), _dev(kn, dev), _dev(vn, dev), out_whole)
        layered.decode_begin(seq_ids)
        outs, lses = [], []
        for l in range(w.n_layers):
            q_l, k_l, v_l = _dev(qn[l], dev), _dev(kn[l], dev), _dev(vn[l], dev)      # this layer's tensors only
            out_l = torch.empty((3, w.n_q_heads, head_dim), dtype=torch.bfloat16, device=dev)
            lse_l = torch.empty((3, w.n_q_heads), dtype=torch.float32, device=dev)
            layered.decode_layer(l, q_l, k_l, v_l, out_l, lse_l)
            outs.append(out_l)
            lses.append(lse_l)
        torch.cuda.synchronize()
        got = np.stack([bits_of(t) for t in outs])
        got_lse = np.stack([t.cpu().numpy() for t in lses])
        ref_whole = f64(bits_of(out_whole))
        for b in range(3):
            ref, ref_lse = o.decode_step(b, f64(qn[:, b]), f64(kn[:, b]), f64(vn[:, b]))
            for l in range(w.n_layers):
                assert_close(got[l, b], ref[l], f"layer call: shape {shape} step {step} seq {b} layer {l}")
            np.testing.assert_allclose(got_lse[:, b], ref_lse, atol=2e-3, rtol=0)
        diff = f64(got) - ref_whole
        assert float(np.max(np.abs(diff))) <= MAX_ABS
        assert float(np.linalg.norm(diff) / np.linalg.norm(ref_whole)) <= REL_L2
    for s in sessions:
        assert s.stats().device_error == 0
    assert layered.stats().decode_steps == whole.stats().decode_steps == w.decode_steps
    for l in range(w.n_layers):
        for stream in range(4):
            for sid in seq_ids:
                assert layered.page_table(l, stream, sid) == whole.page_table(l, stream, sid)
    for s in sessions:
        s.close()


def test_an_open_step_refuses_everything_but_its_next_layer():
    w = W.Workload(79, "layer_state", 3, 4, 2, 128, 16, 2, 5, 60, 60, 20, 4, (1,))
    s = Session.for_workload(w)
    s.prefill_workload(w)
    dev = s.device
    q, k, v = W.decode_qkv_torch(w, 0, dev)
    out = torch.empty((w.n_layers, w.batch, w.n_q_heads, w.head_dim), dtype=torch.bfloat16, device=dev)
    ids = list(range(w.batch))

    def status_of(fn):
        with pytest.raises(qc.QcError) as e:
            fn()
        return e.value.status

    assert status_of(lambda: s.decode_layer(0, q[0], k[0], v[0], out[0])) == qc.QC_ERR_STATE      # no open step
    s.decode_begin(ids)
    assert status_of(lambda: s.decode_begin(ids)) == qc.QC_ERR_STATE
    assert status_of(lambda: s.decode_step(ids, q, k, v, out)) == qc.QC_ERR_STATE
    assert status_of(lambda: qc.qc_free_seq(s.cache, 0)) == qc.QC_ERR_STATE
    assert status_of(lambda: s.decode_layer(1, q[1], k[1], v[1], out[1])) == qc.QC_ERR_STATE      # out of order
    for l in range(w.n_layers):
        s.decode_layer(l, q[l], k[l], v[l], out[l])
    assert status_of(lambda: s.decode_layer(0, q[0], k[0], v[0], out[0])) == qc.QC_ERR_STATE      # step complete
    q, k, v = W.decode_qkv_torch(w, 1, dev)
    s.decode_step(ids, q, k, v, out)                                                               # usable again
    assert s.stats().device_error == 0 and s.stats().decode_steps == 2
    s.close()
