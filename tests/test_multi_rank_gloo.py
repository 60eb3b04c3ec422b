"""The one-process-per-GPU plumbing on CPU: two gloo ranks run the oracle-free host logic that
bench.py uses at N > 1 -- independent shards per rank, barrier, max over ranks, whole-job rate."""
import os
import socket

import torch
import torch.multiprocessing as mp

from paper_1802_04434_b200 import multi
from paper_1802_04434_b200 import workloads as wl


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out_dir):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    r, lr, w = multi.init(torch.device("cpu"))
    assert (r, lr, w) == (rank, rank, world)
    cfg = wl.small_signum(d=4096, M=3)
    cfg.seed = multi.shard_seed(r)
    g = cfg.g(0)
    multi.barrier()
    # a made-up device time per rank: rank 1 is the slow one
    elapsed, kernel = multi.max_over_ranks([10.0 + 5.0 * r, 9.0 + r])
    rate = multi.whole_job_rate(cfg.d, 7, elapsed, w)
    torch.save({"g_sum": float(g.double().sum()), "elapsed": elapsed, "kernel": kernel, "rate": rate},
               os.path.join(out_dir, "rank%d.pt" % r))
    multi.barrier()
    multi.finish()


def test_two_gloo_ranks_shard_and_reduce(tmp_path):
    world, port = 2, _free_port()
    mp.spawn(_rank_main, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    res = [torch.load(tmp_path / ("rank%d.pt" % r)) for r in range(world)]
    assert res[0]["g_sum"] != res[1]["g_sum"]                       # independent shards
    for r in res:
        assert r["elapsed"] == 15.0 and r["kernel"] == 10.0         # the slowest rank, on every rank
        assert abs(r["rate"] - 2 * 4096 * 7 / 15e-3) < 1e-6 * r["rate"]
    # a rank's shard is reproducible from its seed alone
    cfg = wl.small_signum(d=4096, M=3)
    cfg.seed = multi.shard_seed(1)
    assert float(cfg.g(0).double().sum()) == res[1]["g_sum"]


def test_single_process_needs_no_group():
    assert multi.max_over_ranks([3.0, 4.0]) == [3.0, 4.0]
    assert multi.whole_job_rate(100, 10, 2.0, 1) == 100 * 10 / 2e-3
    multi.barrier()
