"""Integer model of the paged KV allocator.  TEST INFRASTRUCTURE ONLY (see lazy_attention.py).

The paper has no paging; it only fixes WHAT each layer stores (section "Q Cache", text after
Eq. 6 and Eq. 8; section "Efficiency Analysis"): every layer keeps all V, ordinary layers
keep all K, VLA lazy layers keep text K only, GLA lazy layers keep no K.  The page-level
convention below is this build's own and is implemented twice, here in pure Python and in
the CUDA library's host runtime, so that page tables can be compared bit for bit.

Convention.  Pages are numbered 0..P-1.  The free list is a stack that initially pops
0, 1, 2, ...  Each (layer, sequence) has up to four streams, in the fixed order
K_T, K_V, V_T, V_V (text / visual keys, text / visual values).  A stream of n tokens holds
ceil(n / page_size) pages.  ``prefill_append`` walks sequences in call order, layers
ascending, owned streams in the fixed order, and pops as many pages as the new length
needs.  ``decode_step`` walks sequences in call order, layers ascending, K_T (if owned)
then V_T, and pops a page exactly when the stream length before the append is a multiple
of page_size.  ``free_seq`` pushes the sequence's pages back in reverse order of their
allocation.  A call that would exhaust the pool fails and leaves the state unchanged.
A stream a lazy layer does not own is reported as the leader's (an alias) when the mode
reads the leader's keys there, with ``owner_layer = leader``.
"""

from __future__ import annotations

from typing import Dict, List, Sequence, Tuple

LAYER_FULL = 0
LAYER_LAZY = 1
MODE_VLA_QC = 0
MODE_VLA_EQ8 = 1
MODE_GLA = 2

K_T, K_V, V_T, V_V = 0, 1, 2, 3


class OutOfPages(Exception):
    pass


class PagedCacheModel:
    def __init__(self, layer_kind: Sequence[int], mode: int, page_size: int, n_pages: int, max_seqs: int):
        if layer_kind[0] != LAYER_FULL:
            raise ValueError("layer 0 must be ordinary")
        self.kind = list(layer_kind)
        self.N = len(self.kind)
        self.mode = mode
        self.page = page_size
        self.max_seqs = max_seqs
        self.free: List[int] = list(range(n_pages - 1, -1, -1))   # pop() yields 0, 1, 2, ...
        self.leader = []
        last = 0
        for l, k in enumerate(self.kind):
            if k == LAYER_FULL:
                last = l
            self.leader.append(last)
        # length[seq] = (n_text, n_visual); tables[(layer, stream, seq)] = page ids
        self.length: Dict[int, List[int]] = {}
        self.tables: Dict[Tuple[int, int, int], List[int]] = {}
        self.alloc_order: Dict[int, List[int]] = {}

    def owns(self, layer: int, stream: int) -> bool:
        if stream in (V_T, V_V) or self.kind[layer] == LAYER_FULL:
            return True
        if stream == K_T:
            return self.mode != MODE_GLA
        return False   # K_V of a lazy layer

    def _pages_for(self, n_tokens: int) -> int:
        return (n_tokens + self.page - 1) // self.page

    def prefill_append(self, seqs: Sequence[int], n_text: Sequence[int], n_visual: Sequence[int]):
        plan = []   # (seq, layer, stream, n_new_pages)
        need = 0
        for s, nt, nv in zip(seqs, n_text, n_visual):
            old_t, old_v = self.length.get(s, [0, 0])
            for l in range(self.N):
                for stream in (K_T, K_V, V_T, V_V):
                    if not self.owns(l, stream):
                        continue
                    old, add = (old_t, nt) if stream in (K_T, V_T) else (old_v, nv)
                    n_new = self._pages_for(old + add) - self._pages_for(old)
                    if n_new:
                        plan.append((s, l, stream, n_new))
                        need += n_new
        if need > len(self.free):
            raise OutOfPages()
        for s, l, stream, n_new in plan:
            for _ in range(n_new):
                pid = self.free.pop()
                self.tables.setdefault((l, stream, s), []).append(pid)
                self.alloc_order.setdefault(s, []).append(pid)
        for s, nt, nv in zip(seqs, n_text, n_visual):
            cur = self.length.setdefault(s, [0, 0])
            cur[0] += nt
            cur[1] += nv

    def decode_step(self, seqs: Sequence[int]):
        need = 0
        for s in seqs:
            if self.length[s][0] % self.page == 0:
                need += sum(1 for l in range(self.N) for st in (K_T, V_T) if self.owns(l, st))
        if need > len(self.free):
            raise OutOfPages()
        for s in seqs:
            if self.length[s][0] % self.page == 0:
                for l in range(self.N):
                    for stream in (K_T, V_T):
                        if self.owns(l, stream):
                            pid = self.free.pop()
                            self.tables.setdefault((l, stream, s), []).append(pid)
                            self.alloc_order.setdefault(s, []).append(pid)
            self.length[s][0] += 1

    def free_seq(self, seq: int):
        for pid in reversed(self.alloc_order.pop(seq, [])):
            self.free.append(pid)
        for key in [k for k in self.tables if k[2] == seq]:
            del self.tables[key]
        self.length.pop(seq, None)

    def page_table(self, layer: int, stream: int, seq: int):
        """(page ids, n_tokens, owner_layer); owner -1 and no pages for an absent stream."""
        if seq not in self.length:
            return [], 0, -1
        nt, nv = self.length[seq]
        n_tokens = nt if stream in (K_T, V_T) else nv
        owner = layer
        if not self.owns(layer, stream):
            # K_V of any lazy layer, and K_T of a GLA lazy layer, are the leader's
            owner = self.leader[layer]
        return list(self.tables.get((owner, stream, seq), [])), n_tokens, owner

    def pages_in_use(self) -> int:
        return sum(len(v) for v in self.tables.values())

    # token-exact accounting for the KV-saving closed form (section "Efficiency Analysis")
    def rows_stored(self) -> int:
        n = 0
        for s, (nt, nv) in self.length.items():
            for l in range(self.N):
                for stream in (K_T, K_V, V_T, V_V):
                    if self.owns(l, stream):
                        n += nt if stream in (K_T, V_T) else nv
        return n

    def rows_all_full(self) -> int:
        return sum(2 * self.N * (nt + nv) for nt, nv in self.length.values())
