"""Host-side helpers of the multi-GPU launch: sequences are independent, so the
path shards over the batch with no exchange on the data path. What ranks share
is the timing: a barrier on both sides of the timed region and the maximum
over ranks of the measured seconds."""
from __future__ import annotations

import os

import torch
import torch.distributed as dist


def env_rank_world() -> tuple[int, int, int]:
    """(rank, world_size, local_rank) from the launcher's environment."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def init(backend: str, device: torch.device | None = None) -> None:
    if dist.is_initialized():
        return
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    os.environ.setdefault("MASTER_PORT", "29533")
    if backend == "nccl":
        dist.init_process_group(backend, device_id=device)
    else:
        dist.init_process_group(backend)


def barrier(world: int) -> None:
    if world > 1:
        dist.barrier()
    if torch.cuda.is_available():
        torch.cuda.synchronize()


def max_over_ranks(values, world: int, device="cpu") -> list[float]:
    """Element-wise maximum over ranks of a short list of seconds."""
    t = torch.tensor([float(v) for v in values], dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t.tolist()]


def whole_job_rate(units_per_rank: float, world: int, seconds_max: float) -> float:
    """Weak scaling: every rank processes `units_per_rank`; the job rate divides the
    total by the slowest rank's time."""
    return world * units_per_rank / seconds_max
