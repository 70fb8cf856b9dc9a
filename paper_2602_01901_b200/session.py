"""Device-memory plumbing around the C ABI: torch owns the pool, the workspace and the stream.

``Session`` allocates the two caller-owned buffers with torch, creates the context and the
cache, and forwards tensors as raw pointers.  All arithmetic runs in the CUDA library.
"""

from __future__ import annotations

from typing import Optional, Sequence

import numpy as np
import torch

from . import binding as qc
from . import workloads as W


class Session:
    def __init__(self, n_layers, n_q_heads, n_kv_heads, head_dim, layer_kind, *, page_size=16, max_seqs=1,
                 max_tokens_per_seq=1024, n_pages=0, lazy_mode=qc.QC_MODE_VLA_QC, split_tokens=0,
                 softmax_scale=0.0, device=0, poison_pool=False):
        if not torch.cuda.is_available():
            raise RuntimeError("a CUDA device is required (no CPU fallback)")
        self.device = torch.device("cuda", device)
        torch.cuda.set_device(self.device)
        self.n_layers, self.hq, self.hkv, self.d = n_layers, n_q_heads, n_kv_heads, head_dim
        self.max_seqs = max_seqs
        self.cfg = qc.make_config(n_layers, n_q_heads, n_kv_heads, head_dim, page_size, max_seqs,
                                  max_tokens_per_seq, n_pages, layer_kind, lazy_mode, split_tokens, softmax_scale)
        pool_bytes, ws_bytes = qc.qc_cache_bytes_required(self.cfg)
        self.pool = torch.empty(pool_bytes, dtype=torch.uint8, device=self.device)
        if poison_pool:   # bf16 NaN pattern: any read of an unwritten row shows up in the output
            self.pool.view(torch.int16).fill_(0x7FC1)
        self.workspace = torch.zeros(ws_bytes, dtype=torch.uint8, device=self.device)
        self.stream = torch.cuda.current_stream(self.device)
        self.ctx = qc.qc_init(device, self.stream.cuda_stream)
        self.cache = qc.qc_alloc_cache(self.ctx, self.cfg, self.pool.data_ptr(), pool_bytes,
                                       self.workspace.data_ptr(), ws_bytes)

    @classmethod
    def for_workload(cls, w: W.Workload, lazy_mode=qc.QC_MODE_VLA_QC, split_tokens=0, device=0,
                     all_full=False, poison_pool=False, slack_pages=0) -> "Session":
        kind = np.zeros(w.n_layers, np.uint8) if all_full else w.layer_kind()
        # room for an all-ordinary cache at the end of decoding: K and V, visual + text streams
        pages_per_tensor = (w.n_visual_kept + 15) // 16 + (w.n_text_prompt + w.decode_steps + 15) // 16
        n_pages = w.n_layers * 2 * w.batch * pages_per_tensor + slack_pages if w.page_size else 0
        return cls(w.n_layers, w.n_q_heads, w.n_kv_heads, w.head_dim, kind.tolist(), page_size=w.page_size,
                   max_seqs=w.batch, max_tokens_per_seq=w.max_tokens, n_pages=n_pages, lazy_mode=lazy_mode,
                   split_tokens=split_tokens, device=device, poison_pool=poison_pool)

    # ---- calls --------------------------------------------------------------------------
    def prefill_append(self, seq_ids: Sequence[int], n_tokens: Sequence[int], kind, k: torch.Tensor, v: torch.Tensor):
        assert k.dtype == torch.bfloat16 and v.dtype == torch.bfloat16 and k.is_contiguous() and v.is_contiguous()
        qc.qc_prefill_append(self.cache, list(seq_ids), list(n_tokens), bytes(bytearray(np.asarray(kind, np.uint8))),
                             k.data_ptr(), v.data_ptr())

    def prefill_attend(self, seq_id: int, kind, q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, out: torch.Tensor):
        for t in (q, k, v, out):
            assert t.dtype == torch.bfloat16 and t.is_contiguous()
        qc.qc_prefill_attend(self.cache, seq_id, bytes(bytearray(np.asarray(kind, np.uint8))), q.data_ptr(),
                             k.data_ptr(), v.data_ptr(), out.data_ptr())

    def decode_step(self, seq_ids, q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, out: torch.Tensor,
                    lse: Optional[torch.Tensor] = None):
        qc.qc_decode_step(self.cache, seq_ids, q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(),
                          lse.data_ptr() if lse is not None else 0)

    def decode_begin(self, seq_ids):
        qc.qc_decode_begin(self.cache, seq_ids)

    def decode_layer(self, layer: int, q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, out: torch.Tensor,
                     lse: Optional[torch.Tensor] = None):
        qc.qc_decode_layer(self.cache, layer, q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(),
                           lse.data_ptr() if lse is not None else 0)

    def decode_step_host(self, seq_ids, q, k, v, out, lse=None):
        qc.qc_decode_step_host(self.cache, seq_ids, q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(),
                               lse.data_ptr() if lse is not None else 0)

    def prefill_workload(self, w: W.Workload, seq_offset: int = 0):
        """Prefill every sequence of a synthetic workload, one sequence per call.  Library
        sequence s holds the generator's sequence ``seq_offset + s``."""
        for s in range(w.batch):
            kind, k, v = W.prefill_kv_torch(w, seq_offset + s, self.device)
            self.prefill_append([s], [len(kind)], kind, k, v)
            del k, v

    def stats(self):
        return qc.qc_get_stats(self.cache)

    def page_table(self, layer, stream, seq):
        return qc.qc_debug_page_table(self.cache, layer, stream, seq)

    def read_qcache(self, layer) -> np.ndarray:
        host = np.empty((self.max_seqs, self.hq, self.d), dtype=np.uint16)
        qc.qc_debug_read_qcache(self.cache, layer, host.ctypes.data)
        return host

    def read_row(self, layer, stream, seq, token, kv_head) -> np.ndarray:
        host = np.empty(self.d, dtype=np.uint16)
        qc.qc_debug_read_row(self.cache, layer, stream, seq, token, kv_head, host.ctypes.data)
        return host

    def set_option(self, key, value):
        qc.qc_set_option(self.cache, key, value)

    def profile(self):
        return qc.qc_get_profile(self.cache)

    def close(self):
        if self.cache is not None:
            qc.qc_free(None, self.cache)
            self.cache = None
        if self.ctx is not None:
            qc.qc_free(self.ctx, None)
            self.ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def bits_of(t: torch.Tensor) -> np.ndarray:
    """bf16 tensor -> uint16 bit patterns on the host."""
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)
