"""Multi-GPU plumbing of the benchmark: one process per GPU, one independent KV pool per rank.

The repack path has no exchange step: under tensor parallelism every shard owns its pool with
shard-local block ids (Sec. 6 of the paper), data-parallel replicas are independent, and the
token-level plan depends only on tables and masks.  Ranks therefore only meet at barriers and
when the timing is reduced (max over ranks) and the work is summed.
"""
from __future__ import annotations

import dataclasses
import os


@dataclasses.dataclass
class Ranks:
    rank: int = 0
    local_rank: int = 0
    world: int = 1
    _group_ready: bool = False

    @classmethod
    def from_env(cls, expected_world: int | None = None) -> "Ranks":
        world = int(os.environ.get("WORLD_SIZE", "1"))
        rank = int(os.environ.get("RANK", "0"))
        local = int(os.environ.get("LOCAL_RANK", str(rank)))
        if expected_world is not None and expected_world != world:
            if world == 1 and expected_world > 1:
                raise RuntimeError(f"--gpus {expected_world} needs {expected_world} ranks (WORLD_SIZE is unset or 1): "
                                   "launch through torchrun, or let bench.py start its own ranks")
            raise RuntimeError(f"--gpus {expected_world} does not match WORLD_SIZE={world}")
        return cls(rank=rank, local_rank=local, world=world)

    def init(self, backend: str = "nccl") -> None:
        if self.world == 1 or self._group_ready:
            return
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29500")
        if not dist.is_initialized():
            kw = {}
            if backend == "nccl":
                import torch
                kw["device_id"] = torch.device("cuda", self.local_rank)
            dist.init_process_group(backend=backend, rank=self.rank, world_size=self.world, **kw)
        self._backend = backend
        self._group_ready = True

    def _tensor(self, x, dtype):
        import torch
        dev = torch.device("cuda", self.local_rank) if self._backend == "nccl" else torch.device("cpu")
        return torch.tensor([x], dtype=dtype, device=dev)

    def barrier(self) -> None:
        if self.world > 1:
            import torch.distributed as dist
            dist.barrier()

    def max(self, x: float) -> float:
        if self.world == 1:
            return float(x)
        import torch
        import torch.distributed as dist
        t = self._tensor(x, torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t.item())

    def sum(self, x: float) -> float:
        if self.world == 1:
            return float(x)
        import torch
        import torch.distributed as dist
        t = self._tensor(x, torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.SUM)
        return float(t.item())

    def finalize(self) -> None:
        if self.world > 1 and self._group_ready:
            import torch.distributed as dist
            dist.barrier()
            dist.destroy_process_group()
            self._group_ready = False


def job_throughput(ranks: Ranks, units_this_rank: float, seconds_this_rank: float) -> float:
    """Whole-job throughput: the units all ranks processed divided by the slowest rank's time."""
    return ranks.sum(units_this_rank) / ranks.max(seconds_this_rank)
