"""fp64 CPU oracle of the layer-similarity calibration.  TEST INFRASTRUCTURE ONLY.

Only the test-suite may import this module; the CUDA library never does, and the two share no
code.  Plain numpy in float64.

What it computes (paper section "Lazy Attention"):

* the last row ``a^l`` of a layer's attention matrix -- the attention of the prompt's last token
  over all prompt tokens -- averaged over the attention heads (the paper analyses the last row
  only, and averages results across heads);
* Eq. 3: ``S(l_m, l_n) = 1/N sum_i JS(a_i^{l_m}, a_i^{l_n})`` over N samples, with
  ``JS(a, b) = 1/2 [KL(a || m) + KL(b || m)]``, ``m = (a + b) / 2`` (natural logarithm, so
  0 <= JS <= ln 2; terms with a zero probability contribute zero);
* Eq. 4: adjacent layers with ``S(l_i, l_{i+1}) < eps`` are merged into a lazy block: the first
  layer of a block stays ordinary, the others become lazy.  ``max_block`` bounds the size of a
  block (the paper keeps blocks small to limit accumulated error; it gives no number).

Pins (tests/test_oracle_calibration.py): closed forms of JS (equal distributions, disjoint
supports, a two-point example), symmetry and the ln 2 bound, SciPy's Jensen-Shannon distance
squared, the last row of the (separately pinned) prefill oracle's attention matrix, and
hand-made similarity vectors for the block construction.
"""

from __future__ import annotations

from typing import List, Sequence

import numpy as np

LAYER_FULL = 0
LAYER_LAZY = 1


def last_row_attention(q_last: np.ndarray, keys: np.ndarray, scale: float) -> np.ndarray:
    """Head-averaged last attention row of one layer.

    q_last: [H_q, D] query of the last prompt token; keys: [L, H_kv, D] every prompt token's key
    (the last token's included).  Returns a [L] distribution.
    """
    Hq, Hkv = q_last.shape[0], keys.shape[1]
    g = Hq // Hkv
    a = np.zeros(keys.shape[0], dtype=np.float64)
    for h in range(Hq):
        s = scale * (keys[:, h // g].astype(np.float64) @ q_last[h].astype(np.float64))
        e = np.exp(s - s.max())
        a += e / e.sum()
    return a / Hq


def kl(a: np.ndarray, b: np.ndarray) -> float:
    """KL(a || b) = sum a ln(a / b), zero-probability terms of a dropped."""
    nz = a > 0
    return float(np.sum(a[nz] * np.log(a[nz] / b[nz])))


def js_divergence(a: np.ndarray, b: np.ndarray) -> float:
    """Eq. 3, second line."""
    m = 0.5 * (np.asarray(a, dtype=np.float64) + np.asarray(b, dtype=np.float64))
    return 0.5 * (kl(np.asarray(a, dtype=np.float64), m) + kl(np.asarray(b, dtype=np.float64), m))


def adjacent_similarity(rows: Sequence[Sequence[np.ndarray]]) -> np.ndarray:
    """Eq. 3, first line, for adjacent layers: rows[i][l] is sample i's a^l.  Returns S[l] =
    mean_i JS(a_i^l, a_i^{l+1}) for l = 0 .. n_layers - 2."""
    n_layers = len(rows[0])
    S = np.zeros(n_layers - 1, dtype=np.float64)
    for sample in rows:
        for l in range(n_layers - 1):
            S[l] += js_divergence(sample[l], sample[l + 1])
    return S / len(rows)


def lazy_blocks(similarity: Sequence[float], eps: float, max_block: int = 0) -> List[int]:
    """Eq. 4: layer l+1 joins the block of layer l when S(l, l+1) < eps (and the block has room).
    Returns layer_kind[n_layers]; the first layer of every block is ordinary."""
    kind = [LAYER_FULL]
    size = 1
    for s in similarity:
        if s < eps and (max_block <= 0 or size < max_block):
            kind.append(LAYER_LAZY)
            size += 1
        else:
            kind.append(LAYER_FULL)
            size = 1
    return kind
