"""The device error path, reached without faulting anything.

A worker of the attention kernel waits for every tile with a bound.  The test hook
``debug_drop_tile`` makes the workers leave out the copy of their first tile, so that wait has
nothing in flight and runs out: a worker records QC_ERR_TIMEOUT in the device error word (and
its mirror in host memory), lets its other copy land and returns; the kernel ends normally.
The host must then see the code in qc_get_stats and refuse further decode steps on that cache,
and the CUDA context must still be usable for a fresh cache.
"""

import numpy as np
import pytest
import torch

from paper_2602_01901_b200 import binding as qc
from paper_2602_01901_b200 import workloads as W
from paper_2602_01901_b200.session import Session, bits_of

from parity_util import assert_close, f64, full_oracle

pytestmark = pytest.mark.gpu


def _workload(group, index):
    return W.Workload(index, f"err{index}", 3, 2 * group, 2, 128, 16, 2, 5, 100, 100, 22, 6, (1,))


@pytest.mark.parametrize("schedule", ["one_launch", "in_order"])
@pytest.mark.parametrize("group", [1, 4], ids=["mha_kernel", "gqa_kernel"])
def test_a_wait_that_runs_out_is_reported_and_nothing_hangs(schedule, group):
    w = _workload(group, 80 + group)
    ids = list(range(w.batch))

    def fresh():
        s = Session.for_workload(w)
        s.prefill_workload(w)
        if schedule == "in_order":
            s.set_option("in_order_launches", 1)
        return s

    s = fresh()
    out = torch.empty((w.n_layers, w.batch, w.n_q_heads, w.head_dim), dtype=torch.bfloat16, device=s.device)
    q, k, v = W.decode_qkv_torch(w, 0, s.device)
    s.decode_step(ids, q, k, v, out)
    assert s.stats().device_error == 0
    s.set_option("debug_drop_tile", 1)
    q, k, v = W.decode_qkv_torch(w, 1, s.device)
    s.decode_step(ids, q, k, v, out)                      # enqueued; the kernel gives up on the device
    assert s.stats().device_error == qc.QC_ERR_TIMEOUT    # (qc_get_stats waits for the stream)
    q, k, v = W.decode_qkv_torch(w, 2, s.device)
    with pytest.raises(qc.QcError) as e:
        s.decode_step(ids, q, k, v, out)
    assert e.value.status == qc.QC_ERR_TIMEOUT
    assert qc.status_string(qc.QC_ERR_TIMEOUT) == "device wait timed out"
    s.close()
    # the context is intact: a new cache computes the right thing
    s = fresh()
    o = full_oracle(w, qc.QC_MODE_VLA_QC)
    for step in range(2):
        q, k, v = W.decode_qkv_torch(w, step, s.device)
        s.decode_step(ids, q, k, v, out)
        qn, kn, vn = W.decode_qkv_np(w, step)
        got = bits_of(out)
        for b in range(w.batch):
            ref, _ = o.decode_step(b, f64(qn[:, b]), f64(kn[:, b]), f64(vn[:, b]))
            for l in range(w.n_layers):
                assert_close(got[l, b], ref[l], f"after the error: step {step} seq {b} layer {l}")
    assert s.stats().device_error == 0
    s.close()


def test_error_codes_have_names_of_their_own():
    names = {qc.status_string(c) for c in (qc.QC_ERR_CUDA, qc.QC_ERR_TIMEOUT, qc.QC_ERR_BAD_PAGE, qc.QC_ERR_PLAN)}
    assert len(names) == 4 and "unknown status" not in names
