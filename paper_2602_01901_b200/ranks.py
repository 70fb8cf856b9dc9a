"""One process per GPU: the little that the multi-GPU path needs.

Sequences are independent and the Q Cache is per sequence, so N GPUs serve N disjoint
batches with N independent copies of the library and no collective on the data path.
What remains is bookkeeping: which global sequences a rank owns, a barrier around the timed
region, and the maximum of a duration over ranks.  ``torch.distributed`` does the plumbing
(NCCL on GPUs, gloo on CPUs).
"""

from __future__ import annotations

import os
from typing import Optional, Tuple


def owned_sequences(n_global: int, rank: int, world: int) -> range:
    """Contiguous block of global sequence indices owned by ``rank`` (sizes differ by at most one)."""
    if not (0 <= rank < world) or n_global < 0:
        raise ValueError("bad rank / world / count")
    base, extra = divmod(n_global, world)
    start = rank * base + min(rank, extra)
    return range(start, start + base + (1 if rank < extra else 0))


class RankGroup:
    """Rank/world from the launcher's environment, plus barrier and max-over-ranks.

    With WORLD_SIZE unset or 1 nothing is initialised and the reductions are identities.
    """

    def __init__(self, backend: Optional[str] = None, device=None):
        self.rank = int(os.environ.get("RANK", "0"))
        self.world = int(os.environ.get("WORLD_SIZE", "1"))
        self.local_rank = int(os.environ.get("LOCAL_RANK", "0"))
        self.device = device
        self._dist = None
        if self.world > 1:
            import torch
            import torch.distributed as dist

            if backend is None:
                backend = "nccl" if torch.cuda.is_available() else "gloo"
            kwargs = {}
            if backend == "nccl":
                torch.cuda.set_device(self.local_rank)
                self.device = torch.device("cuda", self.local_rank)
                kwargs["device_id"] = self.device
            os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
            dist.init_process_group(backend, rank=self.rank, world_size=self.world, **kwargs)
            self._dist = dist

    def _tensor(self, value: float):
        import torch

        dev = self.device if (self.device is not None and self._dist.get_backend() == "nccl") else "cpu"
        return torch.tensor([value], dtype=torch.float64, device=dev)

    def barrier(self) -> None:
        if self._dist is not None:
            self._dist.barrier()

    def max_over_ranks(self, value: float) -> float:
        if self._dist is None:
            return float(value)
        t = self._tensor(value)
        self._dist.all_reduce(t, op=self._dist.ReduceOp.MAX)
        return float(t.item())

    def sum_over_ranks(self, value: float) -> float:
        if self._dist is None:
            return float(value)
        t = self._tensor(value)
        self._dist.all_reduce(t, op=self._dist.ReduceOp.SUM)
        return float(t.item())

    def throughput(self, units_this_rank: float, seconds_this_rank: float) -> Tuple[float, float]:
        """(whole-job units per second, seconds): all ranks' units over the slowest rank's time."""
        seconds = self.max_over_ranks(seconds_this_rank)
        return self.sum_over_ranks(units_this_rank) / seconds, seconds

    def close(self) -> None:
        if self._dist is not None:
            self._dist.destroy_process_group()
            self._dist = None
