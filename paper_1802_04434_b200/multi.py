"""Host-side plumbing for running one process per GPU.

The step is elementwise in the parameter index, so it shards over parameters with no exchange: every
rank owns an independent shard (its own g, m, x and word buffers) and runs the same kernels on it.
The only communication is a barrier around the timed region and a max-reduction of the per-rank
device times, both through ``torch.distributed`` (NCCL on GPUs, gloo in the CPU tests).
"""
from __future__ import annotations

import os
from typing import List, Sequence, Tuple

import torch
import torch.distributed as dist


def env_ranks() -> Tuple[int, int, int]:
    """(rank, local_rank, world_size) from the launcher's environment; (0, 0, 1) when run alone."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def init(device: torch.device | None = None) -> Tuple[int, int, int]:
    """Join the process group if there is more than one rank.  NCCL when `device` is a CUDA device."""
    rank, local_rank, world = env_ranks()
    if world > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        if device is not None and device.type == "cuda":
            dist.init_process_group("nccl", device_id=device)
        else:
            dist.init_process_group("gloo")
    return rank, local_rank, world


def finish() -> None:
    if dist.is_initialized():
        dist.destroy_process_group()


def barrier(device: torch.device | None = None) -> None:
    """All ranks have reached this point and (on a GPU) finished their queued work."""
    if dist.is_initialized():
        dist.barrier()
    if device is not None and device.type == "cuda":
        torch.cuda.synchronize(device)


def max_over_ranks(values: Sequence[float], device: torch.device | None = None) -> List[float]:
    """Element-wise maximum of `values` over all ranks (the slowest rank sets the job's time)."""
    if not dist.is_initialized():
        return [float(v) for v in values]
    t = torch.tensor(list(values), dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.tolist()]


def shard_seed(rank: int) -> int:
    """Seed of the rank's shard: distinct ranks draw distinct, reproducible inputs."""
    return int(rank)


def whole_job_rate(units_per_rank: int, steps: int, elapsed_ms_max: float, world: int) -> float:
    """Units per second of the whole job: every rank processed units_per_rank * steps units in
    elapsed_ms_max (the maximum over ranks)."""
    return world * units_per_rank * steps / (elapsed_ms_max * 1e-3)
