"""Seeded synthetic workloads: shapes, token layouts and the counter-based value generator.

This module is the only code shared by the CUDA path's harness and the CPU oracle's
harness.  It contains no attention arithmetic: it describes the five benchmark shapes
(decoder layers, heads, visual/text token counts, which layers are lazy) and turns an
integer coordinate ``(tensor, layer, sequence, token, head, dim)`` into one bf16 value
drawn from N(0, 1).  The same coordinate gives the same 16 bits in numpy on the host and
in torch on the device, so neither side ever has to ship multi-gigabyte inputs to the
other.

Value recipe.  ``u = splitmix64(coordinate + seed * GOLDEN) >> 48`` selects one of 65 536
equiprobable quantiles of the standard normal, ``Phi^-1((u + 0.5) / 65536)``, rounded to
bf16 (round to nearest even via float32).  splitmix64 is the published 64-bit finaliser of
Steele, Lea and Flood's SplitMix generator.
"""

from __future__ import annotations

import functools
from dataclasses import dataclass
from typing import Tuple

import numpy as np

# ----------------------------------------------------------------------------------------
# shapes
# ----------------------------------------------------------------------------------------

BASE_SEED = 260201901

LAYER_FULL = 0
LAYER_LAZY = 1

KIND_TEXT = 0
KIND_VISUAL = 1

# tensor ids of the generator's coordinate space
T_PREFILL_K = 0
T_PREFILL_V = 1
T_DECODE_Q = 2
T_DECODE_K = 3
T_DECODE_V = 4
T_PRUNE = 5
T_PREFILL_Q = 6


@dataclass(frozen=True)
class Workload:
    """One synthetic decode workload (shape of an MLLM serving batch)."""

    index: int
    name: str
    n_layers: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    page_size: int          # 16, or 0 for contiguous (unpaged) KV
    batch: int
    n_text_before: int      # text tokens in front of the visual span
    n_visual_total: int     # visual tokens produced by the vision tower
    n_visual_kept: int      # visual tokens left after token pruning (== total if none)
    n_text_after: int       # text prompt tokens behind the visual span
    decode_steps: int
    lazy_layers: Tuple[int, ...]

    @property
    def seed(self) -> int:
        return BASE_SEED + self.index

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def n_prompt(self) -> int:
        return self.n_text_before + self.n_visual_kept + self.n_text_after

    @property
    def n_text_prompt(self) -> int:
        return self.n_text_before + self.n_text_after

    @property
    def max_tokens(self) -> int:
        return self.n_prompt + self.decode_steps

    def layer_kind(self) -> np.ndarray:
        kind = np.zeros(self.n_layers, dtype=np.uint8)
        kind[list(self.lazy_layers)] = LAYER_LAZY
        return kind

    def prompt_layout(self, seq: int) -> Tuple[np.ndarray, np.ndarray]:
        """Positions (in the unpruned prompt) and kinds of the tokens given to prefill.

        Text before the visual span, the kept visual tokens in position order, text after.
        With pruning, a seeded subset of exactly ``n_visual_kept`` visual positions is kept
        per sequence; it is the same for every layer.
        """
        first_vis = self.n_text_before
        vis_pos = np.arange(first_vis, first_vis + self.n_visual_total, dtype=np.int64)
        if self.n_visual_kept != self.n_visual_total:
            # rank the visual positions by a hashed key and keep the smallest ones
            key = _splitmix64_np(
                _flat_index_np(T_PRUNE, 0, seq, vis_pos, 0, 0)
                + np.uint64((self.seed * _GOLDEN) & _MASK64)
            )
            order = np.argsort(key, kind="stable")
            vis_pos = np.sort(vis_pos[order[: self.n_visual_kept]])
        before = np.arange(0, first_vis, dtype=np.int64)
        after0 = first_vis + self.n_visual_total
        after = np.arange(after0, after0 + self.n_text_after, dtype=np.int64)
        pos = np.concatenate([before, vis_pos, after])
        kind = np.concatenate(
            [
                np.full(before.size, KIND_TEXT, np.uint8),
                np.full(vis_pos.size, KIND_VISUAL, np.uint8),
                np.full(after.size, KIND_TEXT, np.uint8),
            ]
        )
        return pos, kind


def _odd(lo: int, hi: int) -> Tuple[int, ...]:
    return tuple(range(lo, hi + 1, 2))


WORKLOADS: Tuple[Workload, ...] = (
    Workload(0, "tiny", 2, 8, 8, 64, 0, 1, 64, 576, 576, 32, 16, (1,)),
    Workload(1, "llava15_7b", 32, 32, 32, 128, 16, 16, 35, 576, 576, 64, 256, _odd(3, 31)),
    Workload(2, "llava_next_anyres", 32, 32, 32, 128, 16, 8, 35, 2880, 2880, 93, 512, _odd(3, 31)),
    Workload(3, "qwen2vl_gqa", 28, 28, 4, 128, 16, 32, 35, 1024, 1024, 61, 256, _odd(3, 27)),
    Workload(4, "long_video_pruned", 32, 32, 32, 128, 16, 4, 35, 8192, 4096, 221, 2048, _odd(3, 31)),
    # Beyond the five benchmark shapes: the regime of the paper's efficiency evaluation (7B MHA
    # stack, input length 2048, batch 32, about 35 % of the KV cache saved): 22 of 32 layers lazy,
    # in blocks of one ordinary layer followed by three lazy ones.
    Workload(5, "llava_next_2048_lazy22", 32, 32, 32, 128, 16, 32, 35, 1920, 1920, 93, 256,
             tuple(l for l in range(2, 32) if (l - 2) % 4 != 0)),
)


def get_workload(name_or_index) -> Workload:
    for w in WORKLOADS:
        if w.name == name_or_index or w.index == name_or_index:
            return w
    raise KeyError(name_or_index)


# ----------------------------------------------------------------------------------------
# counter-based generator
# ----------------------------------------------------------------------------------------

_MASK64 = (1 << 64) - 1
_GOLDEN = 0x9E3779B97F4A7C15
_MIX1 = 0xBF58476D1CE4E5B9
_MIX2 = 0x94D049BB133111EB

# coordinate packing (bits): dim 8 | head 8 | token 20 | seq 10 | layer 8 | tensor 4
_SH_HEAD = 8
_SH_TOKEN = 16
_SH_SEQ = 36
_SH_LAYER = 46
_SH_TENSOR = 54


def _flat_index_np(tensor, layer, seq, token, head, dim) -> np.ndarray:
    """Pack a (broadcast) coordinate into one 64-bit counter."""
    u = lambda a: np.asarray(a, dtype=np.uint64)
    return (
        (u(tensor) << np.uint64(_SH_TENSOR))
        + (u(layer) << np.uint64(_SH_LAYER))
        + (u(seq) << np.uint64(_SH_SEQ))
        + (u(token) << np.uint64(_SH_TOKEN))
        + (u(head) << np.uint64(_SH_HEAD))
        + u(dim)
    )


def _splitmix64_np(x: np.ndarray) -> np.ndarray:
    with np.errstate(over="ignore"):
        z = x.astype(np.uint64) + np.uint64(_GOLDEN)
        z = (z ^ (z >> np.uint64(30))) * np.uint64(_MIX1)
        z = (z ^ (z >> np.uint64(27))) * np.uint64(_MIX2)
        z = z ^ (z >> np.uint64(31))
    return z


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bf16 (nearest, ties to even); returns the 16-bit patterns."""
    u = np.asarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    rounded = (u + np.uint64(0x7FFF) + ((u >> np.uint64(16)) & np.uint64(1))) >> np.uint64(16)
    return rounded.astype(np.uint16)


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns to float64."""
    u = np.asarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return u.view(np.float32).astype(np.float64)


@functools.lru_cache(maxsize=1)
def normal_table_bits() -> np.ndarray:
    """65 536 equiprobable N(0,1) quantiles, each rounded to bf16 (uint16 patterns)."""
    from scipy.special import ndtri

    u = (np.arange(65536, dtype=np.float64) + 0.5) / 65536.0
    return f32_to_bf16_bits(ndtri(u).astype(np.float32))


def draw_bits_np(seed: int, tensor, layer, seq, token, head, dim) -> np.ndarray:
    """bf16 bit patterns (uint16) at the broadcast of the given coordinates."""
    idx = _flat_index_np(tensor, layer, seq, token, head, dim)
    with np.errstate(over="ignore"):
        z = _splitmix64_np(idx + np.uint64((seed * _GOLDEN) & _MASK64))
    return normal_table_bits()[(z >> np.uint64(48)).astype(np.int64)]


def _axes(layers, seqs, tokens, heads, head_dim, xp_arange, xp_asarray):
    """Coordinates shaped for a [layers, seqs, tokens, heads, dim] broadcast."""
    l = xp_asarray(layers).reshape(-1, 1, 1, 1, 1)
    s = xp_asarray(seqs).reshape(1, -1, 1, 1, 1)
    t = xp_asarray(tokens).reshape(1, 1, -1, 1, 1)
    h = xp_asarray(heads).reshape(1, 1, 1, -1, 1)
    d = xp_arange(head_dim).reshape(1, 1, 1, 1, -1)
    return l, s, t, h, d


def draw_block_np(seed: int, tensor: int, layers, seqs, tokens, heads, head_dim: int) -> np.ndarray:
    """bf16 bits of shape [len(layers), len(seqs), len(tokens), len(heads), head_dim]."""
    as64 = lambda a: np.asarray(list(a) if isinstance(a, range) else a, dtype=np.int64)
    l, s, t, h, d = _axes(layers, seqs, tokens, heads, head_dim, lambda n: np.arange(n, dtype=np.int64), as64)
    return draw_bits_np(seed, tensor, l, s, t, h, d)


# ---- torch twin (device side of the harness) ---------------------------------------------

def _s64(v: int) -> int:
    v &= _MASK64
    return v - (1 << 64) if v >= (1 << 63) else v


def _lsr_t(z, s: int):
    return (z >> s) & ((1 << (64 - s)) - 1)


def draw_block_torch(seed: int, tensor: int, layers, seqs, tokens, heads, head_dim: int, device):
    """Same values as ``draw_block_np`` as a torch.bfloat16 tensor on ``device``.

    int64 arithmetic wraps modulo 2**64, so the unsigned recipe is reproduced with signed
    constants and masked (logical) right shifts.
    """
    import torch

    as64 = lambda a: torch.as_tensor(np.asarray(list(a) if isinstance(a, range) else a, dtype=np.int64), device=device)
    l, s, t, h, d = _axes(layers, seqs, tokens, heads, head_dim,
                          lambda n: torch.arange(n, dtype=torch.int64, device=device), as64)
    z = ((l << _SH_LAYER) + (s << _SH_SEQ)) + ((t << _SH_TOKEN) + (h << _SH_HEAD) + d)
    z = z + _s64((int(tensor) << _SH_TENSOR) + seed * _GOLDEN + _GOLDEN)
    z = (z ^ _lsr_t(z, 30)) * _s64(_MIX1)
    z = (z ^ _lsr_t(z, 27)) * _s64(_MIX2)
    z = z ^ _lsr_t(z, 31)
    return _table_torch(str(device))[_lsr_t(z, 48)]


@functools.lru_cache(maxsize=4)
def _table_torch(device: str):
    import torch

    bits = normal_table_bits().astype(np.int16)
    return torch.from_numpy(bits).to(device).view(torch.bfloat16)


# ---- whole-tensor helpers in the library's argument layouts -------------------------------

def _all(n):
    return range(n)


def prefill_kv_np(w: Workload, seq: int, layers=None, heads=None):
    """(kind, K bits, V bits) of one sequence's prompt; K, V are [n_layers, T, heads, D]."""
    layers = _all(w.n_layers) if layers is None else layers
    heads = _all(w.n_kv_heads) if heads is None else heads
    pos, kind = w.prompt_layout(seq)
    k = draw_block_np(w.seed, T_PREFILL_K, layers, [seq], pos, heads, w.head_dim)[:, 0]
    v = draw_block_np(w.seed, T_PREFILL_V, layers, [seq], pos, heads, w.head_dim)[:, 0]
    return kind, k, v


def prefill_q_np(w: Workload, seq: int, layers=None, heads=None):
    """Query bits of one sequence's prompt, [n_layers, T, heads, D] (prefill attention only)."""
    layers = _all(w.n_layers) if layers is None else layers
    heads = _all(w.n_q_heads) if heads is None else heads
    pos, _ = w.prompt_layout(seq)
    return draw_block_np(w.seed, T_PREFILL_Q, layers, [seq], pos, heads, w.head_dim)[:, 0]


def prefill_q_torch(w: Workload, seq: int, device):
    """Device twin of ``prefill_q_np`` for all layers and heads (bf16 tensor)."""
    import torch

    pos, _ = w.prompt_layout(seq)
    q = torch.empty((w.n_layers, len(pos), w.n_q_heads, w.head_dim), dtype=torch.bfloat16, device=device)
    for l in range(w.n_layers):
        q[l] = draw_block_torch(w.seed, T_PREFILL_Q, [l], [seq], pos, _all(w.n_q_heads), w.head_dim, device)[0, 0]
    return q


def decode_qkv_np(w: Workload, step: int, seqs=None, layers=None, q_heads=None, kv_heads=None):
    """(q, k, v) bits of one decode step: [n_layers, n_seqs, heads, D] each."""
    seqs = _all(w.batch) if seqs is None else seqs
    layers = _all(w.n_layers) if layers is None else layers
    q_heads = _all(w.n_q_heads) if q_heads is None else q_heads
    kv_heads = _all(w.n_kv_heads) if kv_heads is None else kv_heads
    one = lambda tensor, heads: draw_block_np(w.seed, tensor, layers, seqs, [step], heads, w.head_dim)[:, :, 0]
    return one(T_DECODE_Q, q_heads), one(T_DECODE_K, kv_heads), one(T_DECODE_V, kv_heads)


def prefill_kv_torch(w: Workload, seq: int, device):
    """Device twin of ``prefill_kv_np`` for all layers and heads (bf16 tensors)."""
    import torch

    pos, kind = w.prompt_layout(seq)
    k = torch.empty((w.n_layers, len(pos), w.n_kv_heads, w.head_dim), dtype=torch.bfloat16, device=device)
    v = torch.empty_like(k)
    for l in range(w.n_layers):  # one layer at a time bounds the int64 temporaries
        k[l] = draw_block_torch(w.seed, T_PREFILL_K, [l], [seq], pos, _all(w.n_kv_heads), w.head_dim, device)[0, 0]
        v[l] = draw_block_torch(w.seed, T_PREFILL_V, [l], [seq], pos, _all(w.n_kv_heads), w.head_dim, device)[0, 0]
    return kind, k, v


def decode_qkv_torch(w: Workload, step: int, device, seq_offset: int = 0):
    """Device twin of ``decode_qkv_np`` for the whole batch (bf16 tensors).  ``seq_offset``
    shifts the sequence coordinate: rank r of a multi-GPU run draws sequences r*batch ..."""
    one = lambda tensor, n_heads: draw_block_torch(
        w.seed, tensor, _all(w.n_layers), range(seq_offset, seq_offset + w.batch), [step], _all(n_heads), w.head_dim,
        device
    )[:, :, 0].contiguous()
    return one(T_DECODE_Q, w.n_q_heads), one(T_DECODE_K, w.n_kv_heads), one(T_DECODE_V, w.n_kv_heads)
