"""Helpers shared by the GPU parity tests: oracle runs on the same seeded inputs."""

from __future__ import annotations

import numpy as np

from oracle.lazy_attention import LAYER_FULL, LAYER_LAZY, LazyAttentionOracle, leaders_of
from paper_2602_01901_b200 import workloads as W

MAX_ABS = 2e-2      # tolerance on every output element (bf16 storage, fp32 accumulate)
REL_L2 = 5e-3       # tolerance on ||gpu - ref|| / ||ref||


def f64(bits):
    return W.bf16_bits_to_f64(bits)


def rel_l2(got: np.ndarray, ref: np.ndarray) -> float:
    return float(np.linalg.norm(got - ref) / np.linalg.norm(ref))


def assert_close(got_bits: np.ndarray, ref: np.ndarray, what: str):
    got = f64(got_bits)
    assert np.all(np.isfinite(got)), f"{what}: non-finite output"
    err = float(np.max(np.abs(got - ref)))
    rl2 = rel_l2(got, ref)
    assert err <= MAX_ABS and rl2 <= REL_L2, f"{what}: max-abs {err:.3e}, rel-L2 {rl2:.3e}"
    return err, rl2


def full_oracle(w: W.Workload, mode: int, layer_kind=None) -> LazyAttentionOracle:
    """Oracle holding the whole workload's prompt (small workloads only)."""
    kind = w.layer_kind().tolist() if layer_kind is None else list(layer_kind)
    o = LazyAttentionOracle(w.n_layers, w.n_q_heads, w.n_kv_heads, w.head_dim, kind, mode, n_seqs=w.batch)
    for s in range(w.batch):
        tk, k, v = W.prefill_kv_np(w, s)
        o.prefill_append(s, tk.tolist(), f64(k), f64(v))
    return o


class SampledOracle:
    """The oracle restricted to one (layer, sequence, query head) of a large workload.

    Only the sampled layer and its leader, one KV head and one query head are generated and
    held, so a full-size configuration costs megabytes instead of gigabytes.  The restricted
    problem is exact: heads, sequences and lazy blocks are independent of one another.
    """

    def __init__(self, w: W.Workload, mode: int, layer: int, seq: int, head: int):
        self.w, self.layer, self.seq, self.head = w, layer, seq, head
        kinds = w.layer_kind().tolist()
        leader = leaders_of(kinds)[layer]
        self.layers = [layer] if leader == layer else [leader, layer]
        self.kv = head // w.group
        sub_kind = [LAYER_FULL] if leader == layer else [LAYER_FULL, LAYER_LAZY]
        self.o = LazyAttentionOracle(len(self.layers), 1, 1, w.head_dim, sub_kind, mode, n_seqs=1)
        tk, k, v = W.prefill_kv_np(w, seq, layers=self.layers, heads=[self.kv])
        self.o.prefill_append(0, tk.tolist(), f64(k), f64(v))
        self.step = 0

    def advance(self):
        """Run the next decode step; returns (out[D], lse) of the sampled (layer, head)."""
        w = self.w
        q, k, v = W.decode_qkv_np(w, self.step, seqs=[self.seq], layers=self.layers, q_heads=[self.head],
                                  kv_heads=[self.kv])
        out, lse = self.o.decode_step(0, f64(q[:, 0]), f64(k[:, 0]), f64(v[:, 0]))
        self.step += 1
        return out[-1, 0], lse[-1, 0]


def step_schedule(n_steps: int):
    """Steps checked on the large workloads: the first ones, a page-boundary crossing, the
    middle and the end."""
    cand = [0, 1, 2, 14, 15, 16, 17, n_steps // 2, n_steps - 2, n_steps - 1]
    return sorted({s for s in cand if 0 <= s < n_steps})
