"""Host-side plumbing for running one process per GPU.

Two ways to use several GPUs:

* shards: the step is elementwise in the parameter index, so it shards over parameters with no
  exchange: every rank owns an independent shard (its own g, m, x and word buffers, all M simulated
  workers) and runs the same kernels on it.  The only communication is a barrier around the timed
  region and a max-reduction of the per-rank device times.
* workers (`WorkerStep`): Algorithm 3 as the paper states it, one worker per rank, with one exchange
  per step: an all-gather of the packed sign rows, either as a collective or done by the worker kernel
  itself through peer stores.

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
      2. the exchange, in place of Algorithm 3's "pull sign(g_m)": every rank's W-word row reaches every
         rank, d bits up per worker as in Table 1; rank r's row lands in row r of a [world][ldw] buffer
         in each GPU's own memory;
      3. server block, done by every rank on its local copy of the M rows: the majority vote;
      4. worker block: x <- x - delta sign(vote) on the replica.  All ranks hold the same rows, so they
         compute the same vote and their replicas of x stay identical: no message "down" is needed.

    Two transports for step 2:
      exchange="allgather"  the rows are gathered by `all_gather_into_tensor` (NCCL on GPUs, gloo on CPU);
      exchange="p2p"        steps 1 and 2 are ONE kernel (`signum_momentum_pack_scatter`): the lane that
                            owns a sign word stores it into row r of every rank's rows buffer through
                            peer pointers (torch symmetric memory), so the transfer overlaps the kernel's
                            own g / m stream; a barrier across the ranks follows.  The rows buffers are
                            double-buffered by step parity, so that a fast rank's next scatter cannot
                            overwrite rows a slow rank is still voting on, with one barrier per step.
    Either way the vote kernel only reads this GPU's own memory, with plain loads.  `ops` supplies the
    compute calls (default: the CUDA binding); the CPU tests pass their own implementation.
    """

    def __init__(self, d: int, device: torch.device, ops=None, group=None, world=None, rank=None,
                 exchange: str = "allgather"):
        if ops is None:
            from . import binding as ops   # the CUDA library; raises if it is missing
        if exchange not in ("allgather", "p2p"):
            raise ValueError("exchange must be 'allgather' or 'p2p'")
        self.ops = ops
        self.d = int(d)
        self.device = torch.device(device)
        self.group = group
        self.exchange_kind = exchange
        # world / rank default to the process group's; a caller that moves the rows itself (several
        # workers emulated in one process) states them
        in_group = dist.is_initialized() and world is None
        if world is None:
            world = dist.get_world_size(group) if dist.is_initialized() else 1
        if rank is None:
            rank = dist.get_rank(group) if dist.is_initialized() else 0
        self.world, self.rank = int(world), int(rank)
        self.ld = round_up(self.d, 4)
        self.words = (self.d + 31) // 32
        self.ldw = round_up(self.words, 4)             # rows stay 16-byte aligned; at most 3 pad words
        self.vote = torch.zeros(self.words, dtype=torch.int32, device=self.device)
        self.sync = lambda: None
        if exchange == "allgather":
            self.row = torch.zeros(self.ldw, dtype=torch.int32, device=self.device)
            self.bits = torch.zeros(self.world, self.ldw, dtype=torch.int32, device=self.device)
        else:
            self.parity = 0
            if in_group and self.device.type == "cuda":
                self._rendezvous()
            elif in_group and self.world > 1:
                raise ValueError("exchange='p2p' between processes needs CUDA devices (symmetric memory)")
            else:
                # no group: the rows buffers are ordinary local memory, and `connect` may point several
                # emulated ranks of one process at one another
                self.rows_buf = torch.zeros(2, self.world, self.ldw, dtype=torch.int32, device=self.device)
                self.peer_rows = [[self.rows_buf[k]] for k in (0, 1)] if self.world == 1 else None
            self.bits = self.rows_buf[0]

    def _rendezvous(self) -> None:
        """Rows buffers in symmetric memory: every rank learns every rank's buffer address."""
        import torch.distributed._symmetric_memory as symm_mem
        group = self.group if self.group is not None else dist.group.WORLD
        self.rows_buf = symm_mem.empty((2, self.world, self.ldw), dtype=torch.int32, device=self.device)
        self.rows_buf.zero_()
        self.handle = symm_mem.rendezvous(self.rows_buf, group)
        half = self.world * self.ldw * 4
        self.peer_rows = [[int(self.handle.buffer_ptrs[r]) + k * half for r in range(self.world)] for k in (0, 1)]
        self.sync = lambda: self.handle.barrier(channel=0)
        self.sync()                                    # every rank's zeroing is done before any scatter

    @staticmethod
    def connect(ranks) -> None:
        """Point the emulated ranks of ONE process (exchange="p2p", no process group) at one another."""
        for ws in ranks:
            ws.peer_rows = [[other.rows_buf[k] for other in ranks] for k in (0, 1)]

    def wire_bytes_sent_per_step(self) -> int:
        """Bytes this rank's row occupies on the wire, once per peer."""
        return self.ldw * 4 * (self.world - 1)

    def pack(self, g: torch.Tensor, m, beta: float) -> None:
        """Worker block, first half: this worker's momentum update and its 1-bit sign row.  With the p2p
        transport the same kernel also delivers the row to every rank."""
        if self.exchange_kind == "p2p":
            self.ops.signum_momentum_pack_scatter(g, m, self.d, beta if m is not None else 0.0,
                                                  self.peer_rows[self.parity], self.rank, self.ldw)
        elif m is None:
            self.ops.sign_pack(g, 1, self.d, self.ld, self.row, self.ldw)
        else:
            self.ops.signum_momentum_pack(g, m, 1, self.d, self.ld, beta, self.row, self.ldw)

    def exchange(self) -> None:
        """After this, row r of the local [world][ldw] buffer holds rank r's words, on every rank."""
        if self.exchange_kind == "p2p":
            self.sync()                                # all ranks' scatter kernels have completed
            self.bits = self.rows_buf[self.parity]
            self.parity ^= 1
            return
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
