"""Host-side plumbing for running one process per GPU.

Two ways to use several GPUs:

* shards: the step is elementwise in the parameter index, so it shards over parameters with no
  exchange: every rank owns an independent shard (its own g, m, x and word buffers, all M simulated
  workers) and runs the same kernels on it.  The only communication is a barrier around the timed
  region and a max-reduction of the per-rank device times.
* workers (`WorkerStep`): Algorithm 3 as the paper states it, one worker per rank, with one exchange
  per step: an all-gather of the packed sign rows.

Both go through ``torch.distributed`` (NCCL on GPUs, gloo in the CPU tests).
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


# ----------------------------------------------------------------------------- one worker per rank

def round_up(n: int, k: int) -> int:
    return (n + k - 1) // k * k


class WorkerStep:
    """Algorithm 3 as a distributed step: every rank is ONE worker.

    Rank r keeps its own gradient g_r, its own momentum m_r and a replica of x.  One step is
      1. worker block: m_r <- beta m_r + (1 - beta) g_r and the 1-bit sign row of it (or of g_r when
         there is no momentum), one launch on this rank's data (M = 1);
      2. the exchange, in place of Algorithm 3's "pull sign(g_m)": an all-gather of the W-word rows, d bits
         up per worker as in Table 1; rank r's row lands in row r of a local [world][ldw] buffer in
         this GPU's own memory;
      3. server block, done by every rank on its local copy of the M rows: the majority vote;
      4. worker block: x <- x - delta sign(vote) on the replica.  All ranks hold the same rows, so they
         compute the same vote and their replicas of x stay identical: no message "down" is needed.

    The kernels only ever read local memory (the gathered rows), with plain loads.  `ops` supplies the
    four compute calls (default: the CUDA binding); the CPU tests pass their own implementation.
    """

    def __init__(self, d: int, device: torch.device, ops=None, group=None, world=None, rank=None):
        if ops is None:
            from . import binding as ops   # the CUDA library; raises if it is missing
        self.ops = ops
        self.d = int(d)
        self.device = torch.device(device)
        self.group = group
        # world / rank default to the process group's; a caller that moves the rows itself (several
        # workers emulated in one process) states them
        if world is None:
            world = dist.get_world_size(group) if dist.is_initialized() else 1
        if rank is None:
            rank = dist.get_rank(group) if dist.is_initialized() else 0
        self.world, self.rank = int(world), int(rank)
        self.ld = round_up(self.d, 4)
        self.words = (self.d + 31) // 32
        self.ldw = round_up(self.words, 4)             # rows stay 16-byte aligned; at most 3 pad words
        self.row = torch.zeros(self.ldw, dtype=torch.int32, device=self.device)
        self.bits = torch.zeros(self.world, self.ldw, dtype=torch.int32, device=self.device)
        self.vote = torch.zeros(self.words, dtype=torch.int32, device=self.device)

    def wire_bytes_sent_per_step(self) -> int:
        """Bytes this rank's row occupies on the wire, once per peer."""
        return self.ldw * 4 * (self.world - 1)

    def pack(self, g: torch.Tensor, m, beta: float) -> None:
        """Worker block, first half: this worker's momentum update and its 1-bit sign row."""
        if m is None:
            self.ops.sign_pack(g, 1, self.d, self.ld, self.row, self.ldw)
        else:
            self.ops.signum_momentum_pack(g, m, 1, self.d, self.ld, beta, self.row, self.ldw)

    def exchange(self) -> None:
        """Gather every rank's row into the local [world][ldw] buffer (row r <- rank r)."""
        if not dist.is_initialized() or dist.get_world_size(self.group) == 1:
            self.bits[self.rank].copy_(self.row)
            return
        try:
            dist.all_gather_into_tensor(self.bits.view(-1), self.row, group=self.group)
        except (RuntimeError, NotImplementedError):
            # a backend without the flat form: one destination view per rank
            dist.all_gather([self.bits[r] for r in range(self.world)], self.row, group=self.group)

    def vote_apply(self, x: torch.Tensor, delta: float) -> None:
        """Server block on the local copy of the M rows, then the worker's update of its replica of x."""
        self.ops.majority_vote(self.bits, self.world, self.d, self.ldw, self.vote)
        self.ops.sign_apply(x, self.vote, self.d, delta)

    def step(self, x: torch.Tensor, g: torch.Tensor, m, beta: float, delta: float, events=None) -> None:
        """One step on this rank's (x replica, g_r [1][ld], m_r [1][ld] or None).  `events`, if given, is a
        list of four CUDA events recorded before the pack, after it, after the exchange and at the end."""
        rec = (lambda i: events[i].record()) if events is not None else (lambda i: None)
        rec(0)
        self.pack(g, m, beta)
        rec(1)
        self.exchange()
        rec(2)
        self.vote_apply(x, delta)
        rec(3)


def all_ranks_equal(t: torch.Tensor, group=None) -> bool:
    """True when every rank holds the same integer tensor (checked by a min and a max reduction)."""
    if not dist.is_initialized():
        return True
    lo, hi = t.clone(), t.clone()
    dist.all_reduce(lo, op=dist.ReduceOp.MIN, group=group)
    dist.all_reduce(hi, op=dist.ReduceOp.MAX, group=group)
    return bool(torch.equal(lo, hi))
