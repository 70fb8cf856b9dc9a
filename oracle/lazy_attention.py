"""fp64 CPU oracle of Lazy Attention decode with a Q Cache.  TEST INFRASTRUCTURE ONLY.

Only the test-suite, the smoke check and the benchmark's CPU-baseline leg may import this
module; the CUDA library never does, and the two share no code.  Everything here is plain
numpy in float64, one (layer, sequence, head) at a time, with no blocking, fusion or
reordering beyond what the paper's equations state.

What it computes (paper section "Method"):

* Eq. 2 (decode attention of an ordinary layer): the new token's k, v are appended to the
  layer's cache, then ``softmax(q K^T / sqrt(D)) V`` over the whole cache.
* Section "Lazy Attention": a lazy block is one ordinary layer l_c followed by lazy layers;
  the Q Cache holds Q^{l_c}.  Here ``leader[l]`` is the nearest preceding ordinary layer.
* Eq. 6 (GLA decode): Q = Q Cache, K = the leader's K cache (which already holds the
  leader's new key of this step), V = the lazy layer's own V cache plus its new v.
* Eq. 8 (VLA decode): Q = the lazy layer's own q; K = [own text K, leader's visual K, own
  new k]; V = own.  Mode ``VLA_EQ8`` is this equation as printed.
* Mode ``VLA_QC`` (the reading in which decode reads the Q Cache, following the paper's
  description that VLA shares the visual part of the Q cache and K cache): visual keys are
  scored by the Q Cache (leader's query of the same token), text keys by the own query.
* Storage rule (text after Eq. 6 and after Eq. 8, section "Efficiency Analysis"): every
  layer stores all V; ordinary layers store all K; VLA lazy layers store text K only; GLA
  lazy layers store no K.

The token axis is kept as two ordered streams per layer, text (T) and visual (V), which is
the paper's own simplification ("representing them through concatenation").  One softmax
spans both streams.

Parity pins (tests/test_oracle_*.py): closed forms of a hand-worked two-layer example,
zero-query mean, dominant-key limit, lazy == full when the shared Q/K equal the own,
probability rows summing to one, split/merge == single pass, an independent pure-Python
brute force, and a library softmax.  Unpinned: nothing in the paper fixes how far a lazy
layer's output is from full attention on synthetic data ("parity unpinned" for that
quantity only; it is not a result this oracle is used to assert).
"""

from __future__ import annotations

import math
from typing import List, Optional, Sequence, Tuple

import numpy as np

LAYER_FULL = 0
LAYER_LAZY = 1

MODE_VLA_QC = 0
MODE_VLA_EQ8 = 1
MODE_GLA = 2

KIND_TEXT = 0
KIND_VISUAL = 1


# ------------------------------------------------------------------------------------------
# single-head building blocks
# ------------------------------------------------------------------------------------------

def softmax_attention(scored: Sequence[Tuple[np.ndarray, np.ndarray]], values: np.ndarray, scale: float):
    """Eq. 2 for one head: returns (o[D], lse, p[L]).

    ``scored`` lists (query[D], keys[L_i, D]) pairs in key order: ordinary attention passes
    one pair; the lazy modes pass one pair per stream, because different key ranges are
    scored by different queries (Eq. 6, Eq. 8).  ``values`` is [sum L_i, D] in the same
    order.  One softmax spans all keys.
    """
    s = np.concatenate(
        [scale * (np.asarray(k, dtype=np.float64) @ np.asarray(q, dtype=np.float64)) for q, k in scored]
    )
    m = float(np.max(s))
    e = np.exp(s - m)
    denom = float(np.sum(e))
    p = e / denom
    o = p @ np.asarray(values, dtype=np.float64)
    return o, m + math.log(denom), p


def attention_partial(query: np.ndarray, keys: np.ndarray, values: np.ndarray, scale: float):
    """Unnormalised attention over one chunk of keys: (m, l, acc) with
    m = max_j s_j, l = sum_j exp(s_j - m), acc = sum_j exp(s_j - m) v_j."""
    s = scale * (keys.astype(np.float64) @ query.astype(np.float64))
    m = float(np.max(s))
    e = np.exp(s - m)
    return m, float(np.sum(e)), e @ values.astype(np.float64)


def merge_partials(parts: Sequence[Tuple[float, float, np.ndarray]]):
    """Log-sum-exp merge of chunk partials:
    m* = max m_i; l* = sum l_i e^{m_i - m*}; o = sum acc_i e^{m_i - m*} / l*; lse = m* + ln l*."""
    m_star = max(p[0] for p in parts)
    l_star = 0.0
    acc = np.zeros_like(parts[0][2], dtype=np.float64)
    for m, l, a in parts:
        w = math.exp(m - m_star)
        l_star += l * w
        acc = acc + a * w
    return acc / l_star, m_star + math.log(l_star)


def split_attention(query, keys, values, scale, cuts: Sequence[int]):
    """Attention computed chunk by chunk (cut points in key order) and merged."""
    bounds = [0] + [c for c in cuts if 0 < c < keys.shape[0]] + [keys.shape[0]]
    parts = []
    for a, b in zip(bounds[:-1], bounds[1:]):
        if b > a:
            parts.append(attention_partial(query, keys[a:b], values[a:b], scale))
    return merge_partials(parts)


# ------------------------------------------------------------------------------------------
# multi-layer cache state
# ------------------------------------------------------------------------------------------

class _Rows:
    """Ordered list of rows [H_kv, D] (float64), appendable."""

    def __init__(self, h: int, d: int):
        self._buf = np.empty((16, h, d), dtype=np.float64)
        self.n = 0

    def append(self, row: np.ndarray):
        if self.n == self._buf.shape[0]:
            grown = np.empty((2 * self.n,) + self._buf.shape[1:], dtype=np.float64)
            grown[: self.n] = self._buf
            self._buf = grown
        self._buf[self.n] = row
        self.n += 1

    def rows(self) -> np.ndarray:
        return self._buf[: self.n]


def leaders_of(layer_kind: Sequence[int]) -> List[int]:
    """leader[l] = l for an ordinary layer, else the nearest preceding ordinary layer."""
    if len(layer_kind) == 0 or layer_kind[0] != LAYER_FULL:
        raise ValueError("layer 0 must be an ordinary (full) layer")
    out, last = [], 0
    for l, k in enumerate(layer_kind):
        if k == LAYER_FULL:
            last = l
        out.append(last)
    return out


class LazyAttentionOracle:
    """Multi-layer KV cache + Q Cache, decode attention per Eq. 2 / Eq. 6 / Eq. 8."""

    def __init__(self, n_layers: int, n_q_heads: int, n_kv_heads: int, head_dim: int,
                 layer_kind: Sequence[int], mode: int, n_seqs: int, scale: Optional[float] = None):
        if n_q_heads % n_kv_heads:
            raise ValueError("n_q_heads must be a multiple of n_kv_heads")
        if mode not in (MODE_VLA_QC, MODE_VLA_EQ8, MODE_GLA):
            raise ValueError("unknown mode")
        self.N, self.Hq, self.Hkv, self.D = n_layers, n_q_heads, n_kv_heads, head_dim
        self.g = n_q_heads // n_kv_heads
        self.kind = [int(k) for k in layer_kind]
        if len(self.kind) != n_layers:
            raise ValueError("layer_kind length")
        self.leader = leaders_of(self.kind)
        self.mode = mode
        self.scale = 1.0 / math.sqrt(head_dim) if scale is None else float(scale)
        self.n_seqs = n_seqs
        mk = lambda: _Rows(n_kv_heads, head_dim)
        # streams[l][b] = dict of the four streams; None where the layer stores nothing
        self.K_T = [[mk() if self._owns_kt(l) else None for _ in range(n_seqs)] for l in range(n_layers)]
        self.K_V = [[mk() if self._owns_kv(l) else None for _ in range(n_seqs)] for l in range(n_layers)]
        self.V_T = [[mk() for _ in range(n_seqs)] for _ in range(n_layers)]
        self.V_V = [[mk() for _ in range(n_seqs)] for _ in range(n_layers)]
        self.qslot: List[Optional[np.ndarray]] = [None] * n_seqs   # the Q Cache, [H_q, D] per sequence

    # storage rule
    def _owns_kt(self, l: int) -> bool:
        return self.kind[l] == LAYER_FULL or self.mode != MODE_GLA

    def _owns_kv(self, l: int) -> bool:
        return self.kind[l] == LAYER_FULL

    def prefill_append(self, seq: int, kind: Sequence[int], k: np.ndarray, v: np.ndarray):
        """Store the prompt's K/V (Eq. 1: K and V go to the KV cache).

        k, v: [n_layers, T, H_kv, D].  K rows a lazy layer does not keep are dropped.
        """
        T = len(kind)
        for t in range(T):
            for l in range(self.N):
                if kind[t] == KIND_VISUAL:
                    self.V_V[l][seq].append(v[l, t])
                    if self._owns_kv(l):
                        self.K_V[l][seq].append(k[l, t])
                else:
                    self.V_T[l][seq].append(v[l, t])
                    if self._owns_kt(l):
                        self.K_T[l][seq].append(k[l, t])

    def decode_step(self, seq: int, q: np.ndarray, k: Optional[np.ndarray], v: np.ndarray,
                    return_probs: bool = False):
        """One generated (text) token through all layers in ascending order.

        q: [n_layers, H_q, D]; k, v: [n_layers, H_kv, D].  Returns out [n_layers, H_q, D],
        lse [n_layers, H_q] and, if asked, the probability rows as a nested list
        probs[l][h] in (text stream, visual stream) key order.
        """
        out = np.zeros((self.N, self.Hq, self.D), dtype=np.float64)
        lse = np.zeros((self.N, self.Hq), dtype=np.float64)
        probs = []
        for l in range(self.N):
            c = self.leader[l]
            lazy = self.kind[l] == LAYER_LAZY
            # 1. append the new token (always text): V always, K where the layer keeps text K
            self.V_T[l][seq].append(v[l])
            if self._owns_kt(l):
                self.K_T[l][seq].append(k[l])
            # 2. an ordinary layer refreshes the Q Cache
            if not lazy:
                self.qslot[seq] = np.array(q[l], dtype=np.float64)
            # 3. which query scores which keys, and whose keys they are
            own_q = np.asarray(q[l], dtype=np.float64)
            cached_q = self.qslot[seq]
            if not lazy:
                q_text, keys_text = own_q, self.K_T[l][seq].rows()
                q_vis, keys_vis = own_q, self.K_V[l][seq].rows()
            elif self.mode == MODE_GLA:
                q_text, keys_text = cached_q, self.K_T[c][seq].rows()
                q_vis, keys_vis = cached_q, self.K_V[c][seq].rows()
            elif self.mode == MODE_VLA_EQ8:
                q_text, keys_text = own_q, self.K_T[l][seq].rows()
                q_vis, keys_vis = own_q, self.K_V[c][seq].rows()
            else:  # MODE_VLA_QC
                q_text, keys_text = own_q, self.K_T[l][seq].rows()
                q_vis, keys_vis = cached_q, self.K_V[c][seq].rows()
            vals_text = self.V_T[l][seq].rows()
            vals_vis = self.V_V[l][seq].rows()
            if keys_text.shape[0] != vals_text.shape[0] or keys_vis.shape[0] != vals_vis.shape[0]:
                raise RuntimeError("key and value streams differ in length")
            # 4. one joint softmax over both streams, per query head
            layer_probs = []
            for h in range(self.Hq):
                kv = h // self.g
                vals = np.concatenate([vals_text[:, kv], vals_vis[:, kv]], axis=0)
                o, e, p = softmax_attention(
                    [(q_text[h], keys_text[:, kv]), (q_vis[h], keys_vis[:, kv])], vals, self.scale
                )
                out[l, h], lse[l, h] = o, e
                layer_probs.append(p)
            probs.append(layer_probs)
        if return_probs:
            return out, lse, probs
        return out, lse

    # accounting for the KV-saving closed form (section "Efficiency Analysis")
    def rows_stored(self) -> int:
        """K rows + V rows held over all layers and sequences."""
        n = 0
        for l in range(self.N):
            for b in range(self.n_seqs):
                for s in (self.K_T[l][b], self.K_V[l][b], self.V_T[l][b], self.V_V[l][b]):
                    n += 0 if s is None else s.n
        return n

    def rows_all_full(self) -> int:
        """Rows an all-ordinary-layer cache of the same contents would hold."""
        n = 0
        for l in range(self.N):
            for b in range(self.n_seqs):
                n += 2 * (self.V_T[l][b].n + self.V_V[l][b].n)
        return n
