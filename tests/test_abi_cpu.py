"""The C-ABI library builds, loads and exports what include/qc.h declares (no GPU needed)."""

import ctypes as C
import os
import re

import pytest

from paper_2602_01901_b200 import binding as qc
from paper_2602_01901_b200 import build as qbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    qbuild.build()
    return qc.load()


def test_every_declared_symbol_is_exported(lib):
    header = open(os.path.join(ROOT, "include", "qc.h")).read()
    declared = set(re.findall(r"\b(qc_[a-z_]+)\s*\(", header))
    assert {"qc_init", "qc_alloc_cache", "qc_prefill_append", "qc_decode_step", "qc_free"} <= declared
    for name in declared:
        assert hasattr(lib, name), f"{name} declared in qc.h but not exported"
    assert declared == set(qc.EXPORTS)


def test_sizes_and_argument_checks_without_a_device(lib):
    cfg = qc.make_config(32, 32, 32, 128, 16, 16, 931, 51776, [0, 0, 0] + [1, 0] * 14 + [1])
    pool, ws = qc.qc_cache_bytes_required(cfg)
    assert pool == 51776 * 32 * 16 * 128 * 2          # pages * [H_kv][16][D] bf16
    assert ws > 0 and ws % 256 == 0
    bad = [
        dict(head_dim=96), dict(page_size=32), dict(n_q_heads=30), dict(max_seqs=0), dict(lazy_mode=3),
        dict(split_tokens=24), dict(n_pages=0),
    ]
    for change in bad:
        args = dict(n_layers=4, n_q_heads=8, n_kv_heads=4, head_dim=128, page_size=16, max_seqs=2,
                    max_tokens_per_seq=100, n_pages=64, layer_kind=[0, 1, 0, 1])
        args.update(change)
        with pytest.raises(qc.QcError) as e:
            qc.qc_cache_bytes_required(qc.make_config(**args))
        assert e.value.status in (qc.QC_ERR_INVALID_ARG, qc.QC_ERR_UNSUPPORTED)
    with pytest.raises(qc.QcError) as e:      # a lazy layer needs a preceding ordinary layer
        qc.qc_cache_bytes_required(qc.make_config(2, 2, 2, 128, 16, 1, 64, 64, [1, 0]))
    assert e.value.status == qc.QC_ERR_STATE
    assert qc.status_string(qc.QC_ERR_OOM_PAGES) == "out of pages"
    # null handles are refused, not dereferenced
    assert lib.qc_decode_step(None, 1, None, None, None, None, None, None) == qc.QC_ERR_INVALID_ARG
    assert lib.qc_get_stats(None, None) == qc.QC_ERR_INVALID_ARG
    assert lib.qc_free(None, None) == qc.QC_OK


def test_no_device_means_an_error_status_not_a_fallback(lib):
    import torch

    if torch.cuda.is_available():
        pytest.skip("a device is present")
    ctx = C.c_void_p()
    assert lib.qc_init(0, None, C.byref(ctx)) == qc.QC_ERR_CUDA
    assert not ctx.value
    from paper_2602_01901_b200.session import Session

    with pytest.raises(RuntimeError):
        Session(2, 2, 2, 128, [0, 1])


def test_lazy_blocks_on_the_host_match_the_oracle(lib):
    from oracle import calibration as OC

    S = [0.30, 0.01, 0.02, 0.40, 0.03, 0.03, 0.03, 0.50]
    for eps, max_block in ((0.05, 0), (0.05, 2), (0.005, 0), (1.0, 0), (0.2, 3)):
        assert qc.qc_lazy_blocks(S, eps, max_block) == OC.lazy_blocks(S, eps, max_block)
    assert qc.qc_lazy_blocks([], 0.5) == [0]
    with pytest.raises(qc.QcError):
        qc.qc_lazy_blocks(S, 0.0)
    with pytest.raises(qc.QcError):
        qc.qc_lazy_blocks(S, 1.5)
