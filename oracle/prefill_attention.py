"""fp64 CPU oracle of prefill-phase attention with Lazy Attention.  TEST INFRASTRUCTURE ONLY.

Only the test-suite, the smoke check and the benchmark's CPU-baseline leg may import this
module; the CUDA library never does, and the two share no code.  Plain numpy in float64, one
(layer, head) at a time, no blocking, fusion or reordering.

What it computes (paper section "Method"), for the prompt of one sequence, T tokens in their
actual order, each tagged text or visual:

* Eq. 1 (ordinary layer): ``A = softmax((Q K^T + M) / sqrt(D))`` with the causal mask M (token
  i sees tokens j <= i), ``O = A V``.
* Eq. 5 (GLA prefill, lazy layer l_i of a block led by l_c): ``Q = Q Cache = Q^{l_c}``,
  ``K = K^{l_c}``, ``V = V^{l_i}``: the attention matrix is the leader's, applied to the own V.
* Eq. 7 (VLA prefill): query rows of text tokens are the layer's own, rows of visual tokens come
  from the Q Cache (the leader's); key rows of text tokens are the own, those of visual tokens
  the leader's; V is the own.  The paper writes the selection as a concatenation "to simplify
  the actual positions"; the mask uses the actual positions.

Both VLA decode readings (Eq. 8 as printed, and the cached query scoring the visual keys)
share this prefill: Eq. 7 is the only prefill form the paper gives for VLA.

Pins (tests/test_oracle_prefill.py): a library causal softmax attention, a hand-worked
three-token example in closed form, lazy == ordinary when the leader's Q/K equal the own, the
leader's probabilities reproduced in GLA, causality, rows summing to one, and agreement of the
last prompt row with the (separately pinned) decode oracle.
"""

from __future__ import annotations

import math
from typing import List, Optional, Sequence

import numpy as np

LAYER_FULL = 0
LAYER_LAZY = 1
MODE_VLA_QC = 0
MODE_VLA_EQ8 = 1
MODE_GLA = 2
KIND_TEXT = 0
KIND_VISUAL = 1


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


def causal_attention(q: np.ndarray, k: np.ndarray, v: np.ndarray, scale: float):
    """Eq. 1 for one head: q, k, v are [T, D]; returns (O [T, D], A [T, T])."""
    T = q.shape[0]
    s = scale * (q.astype(np.float64) @ k.astype(np.float64).T)
    s = np.where(np.arange(T)[None, :] <= np.arange(T)[:, None], s, -np.inf)
    m = s.max(axis=1, keepdims=True)
    e = np.exp(s - m)
    a = e / e.sum(axis=1, keepdims=True)
    return a @ v.astype(np.float64), a


def prefill_lazy_attention(q: np.ndarray, k: np.ndarray, v: np.ndarray, kind: Sequence[int],
                           layer_kind: Sequence[int], mode: int, scale: Optional[float] = None,
                           return_probs: bool = False):
    """Prefill attention of every layer for one prompt.

    q: [n_layers, T, H_q, D]; k, v: [n_layers, T, H_kv, D]; kind: [T] (0 text, 1 visual).
    Returns out [n_layers, T, H_q, D] (and the attention matrices [n_layers][H_q] if asked).
    """
    if mode not in (MODE_VLA_QC, MODE_VLA_EQ8, MODE_GLA):
        raise ValueError("unknown mode")
    N, T, Hq, D = q.shape
    Hkv = k.shape[2]
    if Hq % Hkv:
        raise ValueError("n_q_heads must be a multiple of n_kv_heads")
    g = Hq // Hkv
    scale = 1.0 / math.sqrt(D) if scale is None else float(scale)
    leader = leaders_of([int(x) for x in layer_kind])
    visual = np.asarray(kind) == KIND_VISUAL
    out = np.zeros((N, T, Hq, D), dtype=np.float64)
    probs = []
    for l in range(N):
        c = leader[l]
        if layer_kind[l] == LAYER_FULL:
            take_leader = np.zeros(T, dtype=bool)            # Eq. 1
        elif mode == MODE_GLA:
            take_leader = np.ones(T, dtype=bool)             # Eq. 5: all of Q and K from the block's first layer
        else:
            take_leader = visual                             # Eq. 7: the visual rows of Q and K
        layer_probs = []
        for h in range(Hq):
            kv = h // g
            q_sel = np.where(take_leader[:, None], q[c, :, h], q[l, :, h])
            k_sel = np.where(take_leader[:, None], k[c, :, kv], k[l, :, kv])
            o, a = causal_attention(q_sel, k_sel, v[l, :, kv], scale)
            out[l, :, h] = o
            layer_probs.append(a)
        probs.append(layer_probs)
    if return_probs:
        return out, probs
    return out
