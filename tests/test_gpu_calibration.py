"""GPU parity of the calibration by-product (qc_layer_similarity) against the fp64 oracle:
head-averaged last-row attention per layer, adjacent-layer Jensen-Shannon divergence (Eq. 3)."""

import math

import numpy as np
import pytest
import torch

from oracle import calibration as OC
from paper_2602_01901_b200 import binding as qc
from paper_2602_01901_b200 import workloads as W
from paper_2602_01901_b200.session import Session

from parity_util import f64

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("head_dim,group,n_layers", [(128, 1, 4), (64, 2, 3), (128, 7, 2)])
def test_layer_similarity_matches_oracle(head_dim, group, n_layers):
    w = W.Workload(50 + group, f"calib{group}", n_layers, 2 * group, 2, head_dim, 16, 3, 5, 150, 150, 22, 2, ())
    s = Session.for_workload(w)
    s.prefill_workload(w)
    dev = s.device
    lens = [w.n_prompt, w.n_prompt, w.n_prompt]
    q_last = np.stack([W.prefill_q_np(w, b)[:, -1] for b in range(w.batch)], axis=1)     # [N, B, Hq, D] bits
    q_dev = torch.from_numpy(q_last.astype(np.int16)).view(torch.bfloat16).to(dev).contiguous()
    max_len = 192
    rows = torch.full((n_layers, w.batch, max_len), float("nan"), dtype=torch.float32, device=dev)
    sim = qc.qc_layer_similarity(s.cache, list(range(w.batch)), q_dev.data_ptr(), rows.data_ptr(), max_len, n_layers)
    got_rows = rows.cpu().numpy()
    ref_rows = []
    for b in range(w.batch):
        kind, k, _ = W.prefill_kv_np(w, b)
        order = np.concatenate([np.nonzero(kind == 0)[0], np.nonzero(kind == 1)[0]])      # text stream, then visual
        per_layer = [OC.last_row_attention(f64(q_last[l, b]), f64(k[l][order]), 1.0 / math.sqrt(head_dim))
                     for l in range(n_layers)]
        ref_rows.append(per_layer)
        for l in range(n_layers):
            np.testing.assert_allclose(got_rows[l, b, : lens[b]], per_layer[l], rtol=2e-4, atol=1e-7)
            assert np.all(got_rows[l, b, lens[b]:] == 0.0)
            assert abs(got_rows[l, b].sum() - 1.0) < 1e-4
    want = OC.adjacent_similarity(ref_rows)
    np.testing.assert_allclose(sim, want, rtol=1e-3, atol=1e-6)
    assert all(0.0 <= x <= math.log(2) for x in sim)
    # Eq. 4 on the measured similarities, library against oracle
    eps = float(np.median(want)) if len(want) else 0.5
    assert qc.qc_lazy_blocks(sim, eps) == OC.lazy_blocks(sim, eps)
    assert s.stats().device_error == 0
    s.close()


def test_layer_similarity_refuses_a_cache_with_lazy_layers_and_short_scratch():
    w = W.Workload(59, "calibx", 2, 2, 2, 128, 16, 1, 3, 20, 20, 4, 2, (1,))
    s = Session.for_workload(w)
    s.prefill_workload(w)
    t = torch.zeros(4096, dtype=torch.float32, device=s.device)
    with pytest.raises(qc.QcError) as e:
        qc.qc_layer_similarity(s.cache, [0], t.data_ptr(), t.data_ptr(), 64, 2)
    assert e.value.status == qc.QC_ERR_STATE
    s.close()
    s = Session.for_workload(w, all_full=True)
    s.prefill_workload(w)
    with pytest.raises(qc.QcError) as e:       # 27 cached tokens do not fit 16 columns
        qc.qc_layer_similarity(s.cache, [0], t.data_ptr(), t.data_ptr(), 16, 2)
    assert e.value.status == qc.QC_ERR_INVALID_ARG
    s.close()
