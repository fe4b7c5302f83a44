"""Host-side plumbing for running N independent replicas of the head, one process per GPU.

The head has no exchange step (positions are independent and the weights are replicated), so there is no
data-path collective: ranks only meet at the timing barrier and to take the maximum elapsed time."""
from __future__ import annotations

import os


def rank_env() -> tuple[int, int, int]:
    """(rank, local_rank, world_size) from the launcher's environment; (0, 0, 1) when launched plainly."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def init_process_group(backend: str):
    import torch.distributed as dist
    rank, _, world = rank_env()
    if world > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29511")
        dist.init_process_group(backend=backend, rank=rank, world_size=world)
    return rank, world


def barrier() -> None:
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized():
        dist.barrier()


def max_over_ranks(value: float, device="cpu") -> float:
    """Every rank contributes its elapsed time; all get the slowest rank's."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_throughput(units_per_rank_per_step: int, steps: int, world: int, max_elapsed_s: float) -> float:
    """Whole-job units per second: every replica processed its own units in the slowest rank's time."""
    return units_per_rank_per_step * steps * world / max_elapsed_s


def replica_seed_offset(rank: int) -> int:
    """Replicas draw different synthetic positions (same weights' distribution, different stream)."""
    return 7919 * rank
