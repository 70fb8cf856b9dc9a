"""qc_attend_static, the call for users who cannot allocate device memory.

A serving loop with a frozen memory budget, or code running inside another framework's
callback, cannot create a workspace for the library.  qc_attend_static serves them from a
scratch array built into the library.  This test drives it through the C ABI twice in a row
(the second call sees the scratch contents the first one left behind) and checks each result
against the fp64 oracle's softmax attention on the same bits (Eq. 2) and against qc_decode_step
on a one-layer cache fed with the same tensors, within the same tolerances as the other GPU
tests.  It also checks that oversized requests are refused.

The file name sorts last so that a run which stops at the first failure has already run
every other test.
"""

import math

import numpy as np
import pytest
import torch

from oracle.lazy_attention import softmax_attention
from paper_2602_01901_b200 import binding as qc
from paper_2602_01901_b200 import workloads as W
from paper_2602_01901_b200.session import Session, bits_of

from parity_util import MAX_ABS, REL_L2, f64

pytestmark = pytest.mark.gpu


def _to_dev(bits, dev):
    return torch.from_numpy(bits.astype(np.int16)).view(torch.bfloat16).to(dev).contiguous()


@pytest.mark.parametrize("head_dim,n_q,n_kv,n_prompt", [(128, 8, 2, 333), (64, 4, 4, 37)])
def test_static_scratch_entry_point_matches_decode_step(head_dim, n_q, n_kv, n_prompt):
    n_seqs = 3
    w = W.Workload(30, "static", 1, n_q, n_kv, head_dim, 16, n_seqs, 7, n_prompt - 20, n_prompt - 20, 13, 2, ())
    s = Session.for_workload(w)
    s.prefill_workload(w)
    dev = s.device
    stream = torch.cuda.current_stream(dev).cuda_stream
    # the contiguous history the new call reads: prompt rows, then one row per decode step
    hist_k = [W.prefill_kv_np(w, b)[1][0] for b in range(n_seqs)]     # [T][n_kv][D] per sequence
    hist_v = [W.prefill_kv_np(w, b)[2][0] for b in range(n_seqs)]
    out_ref = torch.empty((1, n_seqs, n_q, head_dim), dtype=torch.bfloat16, device=dev)
    out_new = torch.empty((n_seqs, n_q, head_dim), dtype=torch.bfloat16, device=dev)
    for step in range(2):                                             # two calls in a row
        qn, kn, vn = W.decode_qkv_np(w, step)
        s.decode_step(list(range(n_seqs)), _to_dev(qn, dev), _to_dev(kn, dev), _to_dev(vn, dev), out_ref)
        for b in range(n_seqs):
            hist_k[b] = np.concatenate([hist_k[b], kn[0, b][None]])
            hist_v[b] = np.concatenate([hist_v[b], vn[0, b][None]])
        k_all, v_all = _to_dev(np.stack(hist_k), dev), _to_dev(np.stack(hist_v), dev)
        q_all = _to_dev(qn[0], dev)
        out_new.fill_(0)
        qc.qc_attend_static(dev.index, stream, q_all.data_ptr(), k_all.data_ptr(), v_all.data_ptr(),
                            out_new.data_ptr(), n_seqs, k_all.shape[1], n_q, n_kv, head_dim)
        torch.cuda.synchronize()
        ref, got = f64(bits_of(out_ref)[0]), f64(bits_of(out_new))
        assert np.all(np.isfinite(got))
        assert float(np.max(np.abs(got - ref))) <= MAX_ABS
        assert float(np.linalg.norm(got - ref) / np.linalg.norm(ref)) <= REL_L2
        # and against the oracle: plain softmax attention of every head over its whole history
        group = n_q // n_kv
        want = np.empty_like(got)
        for b in range(n_seqs):
            kb, vb = f64(hist_k[b]), f64(hist_v[b])
            for h in range(n_q):
                want[b, h] = softmax_attention([(f64(qn[0, b, h]), kb[:, h // group])], vb[:, h // group],
                                               1.0 / math.sqrt(head_dim))[0]
        assert float(np.max(np.abs(got - want))) <= MAX_ABS
        assert float(np.linalg.norm(got - want) / np.linalg.norm(want)) <= REL_L2
    assert s.stats().device_error == 0
    s.close()


def test_static_scratch_entry_point_refuses_what_does_not_fit():
    dev = torch.device("cuda", 0)
    t = torch.zeros(4096, dtype=torch.bfloat16, device=dev)
    p = t.data_ptr()
    too_many_rows = (qc.QC_STATIC_MAX_ROWS // 32 + 1, 8, 32, 32, 128)       # n_seqs * n_q_heads over the limit
    too_long = (1, qc.QC_STATIC_MAX_TOKENS + 1, 1, 1, 128)
    bad_dim = (1, 8, 1, 1, 96)
    for n_seqs, n_tokens, n_q, n_kv, d in (too_many_rows, too_long, bad_dim):
        with pytest.raises(qc.QcError) as e:
            qc.qc_attend_static(0, 0, p, p, p, p, n_seqs, n_tokens, n_q, n_kv, d)
        assert e.value.status in (qc.QC_ERR_INVALID_ARG, qc.QC_ERR_UNSUPPORTED)
    with pytest.raises(qc.QcError):
        qc.qc_attend_static(0, 0, 0, p, p, p, 1, 8, 1, 1, 128)               # null input
    torch.cuda.synchronize()
