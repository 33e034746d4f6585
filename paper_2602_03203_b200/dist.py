"""One process per GPU: rank discovery, barrier and max-over-ranks for the benchmark.

The path has no exchange step: every (sequence, layer, KV head) segment is
independent, so ranks hold independent replicas (or shards of the sequences)
and no collective sits on the data path.  torch.distributed is used only to
line the ranks up around the timed region and to reduce the timing.
"""
from __future__ import annotations

import os
from typing import List, Sequence

import torch


def shard(items: Sequence, rank: int, world: int) -> List:
    """Contiguous, balanced shard of a list of independent units (sequences or segments)."""
    n = len(items)
    lo = rank * n // world
    hi = (rank + 1) * n // world
    return list(items[lo:hi])


class Ranks:
    def __init__(self, backend: str | None = None):
        self.rank = int(os.environ.get("RANK", "0"))
        self.world = int(os.environ.get("WORLD_SIZE", "1"))
        self.local_rank = int(os.environ.get("LOCAL_RANK", "0"))
        self.backend = backend or ("nccl" if torch.cuda.is_available() else "gloo")
        self._own = False
        if self.world > 1:
            import torch.distributed as dist
            if not dist.is_initialized():
                os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
                os.environ.setdefault("MASTER_PORT", "29500")
                if self.backend == "nccl":
                    torch.cuda.set_device(self.local_rank)
                dist.init_process_group(self.backend, rank=self.rank, world_size=self.world)
                self._own = True

    def _tensor(self, x: float) -> torch.Tensor:
        dev = torch.device("cuda", self.local_rank) if self.backend == "nccl" else torch.device("cpu")
        return torch.tensor([x], dtype=torch.float64, device=dev)

    def barrier(self):
        if self.world > 1:
            import torch.distributed as dist
            dist.barrier()

    def max(self, x: float) -> float:
        if self.world == 1:
            return float(x)
        import torch.distributed as dist
        t = self._tensor(x)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t.item())

    def sum(self, x: float) -> float:
        if self.world == 1:
            return float(x)
        import torch.distributed as dist
        t = self._tensor(x)
        dist.all_reduce(t, op=dist.ReduceOp.SUM)
        return float(t.item())

    def close(self):
        if self._own:
            import torch.distributed as dist
            dist.destroy_process_group()
            self._own = False
