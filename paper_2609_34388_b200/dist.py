"""One process per GPU: rendezvous and the two reductions the benchmark needs.

Requests are independent (each has its own KV pages, rows and accept decision), so ranks process disjoint
batches with a full weight replica and there is no collective on the data path; only timing (max over
ranks) and token counts (sum over ranks) are reduced.
"""
from __future__ import annotations

import os
from dataclasses import dataclass

import torch
import torch.distributed as dist


@dataclass
class DistEnv:
    rank: int = 0
    local_rank: int = 0
    world: int = 1
    backend: str = "nccl"
    initialised: bool = False

    @classmethod
    def from_env(cls, backend: str = "nccl") -> "DistEnv":
        world = int(os.environ.get("WORLD_SIZE", "1"))
        rank = int(os.environ.get("RANK", "0"))
        local = int(os.environ.get("LOCAL_RANK", "0"))
        env = cls(rank, local, world, backend, False)
        if world > 1:
            os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
            os.environ.setdefault("MASTER_PORT", "29500")
            if backend == "nccl":
                torch.cuda.set_device(local)
            dist.init_process_group(backend=backend, rank=rank, world_size=world)
            env.initialised = True
        return env

    def _device(self):
        return torch.device("cuda", self.local_rank) if self.backend == "nccl" else torch.device("cpu")

    def barrier(self) -> None:
        if self.initialised:
            dist.barrier()

    def max_float(self, x: float) -> float:
        if not self.initialised:
            return float(x)
        t = torch.tensor([x], dtype=torch.float64, device=self._device())
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t.item())

    def sum_float(self, x: float) -> float:
        if not self.initialised:
            return float(x)
        t = torch.tensor([x], dtype=torch.float64, device=self._device())
        dist.all_reduce(t, op=dist.ReduceOp.SUM)
        return float(t.item())

    def close(self) -> None:
        if self.initialised:
            dist.destroy_process_group()
            self.initialised = False


def shard_requests(n_req: int, rank: int, world: int):
    """Contiguous, balanced partition of request indices over ranks (strong-scaling helper)."""
    base, rem = divmod(n_req, world)
    lo = rank * base + min(rank, rem)
    return list(range(lo, lo + base + (1 if rank < rem else 0)))
