"""Algorithm 3 with one worker per rank (`multi.WorkerStep`): the host-side logic of the exchange.

CPU part (not gpu): two gloo ranks, compute calls served by the oracle -- rank r's row must land in row
r on every rank, pad words stay as initialised, every rank ends with the same vote and the same x, and
the result equals the single-process step over the M = 2 stacked gradients.
GPU part: the ranks' worker steps run one after another on cuda:0 through the CUDA library, the rows
are moved between the emulated ranks by plain copies, and words, vote, x and every m row must match
`oracle.signsgd_step` bit for bit.
"""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.multiprocessing as mp

HERE = os.path.dirname(os.path.abspath(__file__))
if HERE not in sys.path:
    sys.path.insert(0, HERE)

import oracle
from paper_1802_04434_b200 import multi
from paper_1802_04434_b200 import workloads as wl


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def worker_inputs(world, d, steps, seed, momentum=True):
    """x0 [d], g [steps][world][ld], m0 [world][ld]: the same on whoever calls with the same arguments."""
    r = np.random.default_rng(seed)
    ld = multi.round_up(d, 4)
    x0 = r.standard_normal(d).astype(np.float32)
    g = np.zeros((steps, world, ld), dtype=np.float32)
    g[:, :, :d] = r.standard_normal((steps, world, d)).astype(np.float32)
    g[:, :, :d][r.random((steps, world, d)) < 0.05] = 0.0
    m0 = np.zeros((world, ld), dtype=np.float32)
    if momentum:
        m0[:, :d] = 0.1 * r.standard_normal((world, d)).astype(np.float32)
    return x0, g, m0


def reference_run(x0, g, m0, d, beta, delta, momentum=True):
    """The single-process step of the oracle over the stacked rows; returns per-step (bits, vote) and final x, m."""
    steps, world, ld = g.shape
    x, m = x0.copy(), (m0.copy().reshape(-1) if momentum else None)
    ldw = multi.round_up(oracle.words(d), 4)
    out = []
    for k in range(steps):
        b, v = oracle.signsgd_step(x, g[k].reshape(-1), m, world, d, beta, delta, ld=ld, ldw=ldw)
        out.append((b.reshape(world, ldw), v))
    return out, x, m


def _rank_main(rank, world, port, out_dir, d, steps, beta, delta):
    sys.path.insert(0, HERE)
    import oracle_ops
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    multi.init(torch.device("cpu"))
    x0, g, m0 = worker_inputs(world, d, steps, seed=7)
    x = torch.from_numpy(x0.copy())
    m = torch.from_numpy(m0[rank:rank + 1].copy())            # this worker's own momentum only
    ws = multi.WorkerStep(d, torch.device("cpu"), ops=oracle_ops)
    assert (ws.world, ws.rank) == (world, rank)
    ws.bits.fill_(0x5A5A5A5A)                                   # every word of the gather buffer must be replaced
    hist = []
    for k in range(steps):
        ws.step(x, torch.from_numpy(g[k, rank:rank + 1].copy()), m, beta, delta)
        hist.append((ws.bits.clone(), ws.vote.clone()))
    same = multi.all_ranks_equal(ws.vote)
    torch.save({"x": x, "m": m, "hist": hist, "same": same, "sent": ws.wire_bytes_sent_per_step()},
               os.path.join(out_dir, "rank%d.pt" % rank))
    multi.barrier()
    multi.finish()


@pytest.mark.parametrize("d", [1000, 4099])
def test_two_gloo_ranks_run_algorithm3_one_worker_each(tmp_path, d):
    world, steps, beta, delta = 2, 3, 0.9, 1e-3
    mp.spawn(_rank_main, args=(world, _free_port(), str(tmp_path), d, steps, beta, delta), nprocs=world, join=True)
    res = [torch.load(tmp_path / ("rank%d.pt" % r)) for r in range(world)]
    x0, g, m0 = worker_inputs(world, d, steps, seed=7)
    ref, x_ref, m_ref = reference_run(x0, g, m0, d, beta, delta)
    W = oracle.words(d)
    ldw = multi.round_up(W, 4)
    for r in range(world):
        assert res[r]["same"] and res[r]["sent"] == ldw * 4 * (world - 1)
        for k in range(steps):
            bits, vote = res[r]["hist"][k]
            got = bits.numpy().view(np.uint32)
            assert np.array_equal(got[:, :W], ref[k][0][:, :W]), "rank %d step %d: row r must hold rank r's words" % (r, k)
            assert np.all(got[:, W:] == 0)                      # pad words: the senders' zeros, never garbage
            assert np.array_equal(vote.numpy().view(np.uint32), ref[k][1])
        assert np.array_equal(res[r]["x"].numpy().view(np.uint32), x_ref.view(np.uint32))   # replicas stay identical
        ld = multi.round_up(d, 4)
        assert np.array_equal(res[r]["m"].numpy().reshape(-1).view(np.uint32), m_ref[r * ld:(r + 1) * ld].view(np.uint32))
    # Table 1: d bits up per worker -- the row on the wire is ceil(d/32) words, padded to a multiple of 4
    assert ldw * 32 - d < 128


def test_single_process_worker_step_needs_no_group():
    import oracle_ops
    d = 777
    x0, g, m0 = worker_inputs(1, d, 2, seed=3)
    ws = multi.WorkerStep(d, torch.device("cpu"), ops=oracle_ops)
    x, m = torch.from_numpy(x0.copy()), torch.from_numpy(m0.copy())
    for k in range(2):
        ws.step(x, torch.from_numpy(g[k].copy()), m, 0.9, 1e-3)
    ref, x_ref, m_ref = reference_run(x0, g, m0, d, 0.9, 1e-3)
    assert np.array_equal(x.numpy().view(np.uint32), x_ref.view(np.uint32))
    assert np.array_equal(ws.vote.numpy().view(np.uint32), ref[-1][1])     # M = 1: the vote is the row


@pytest.mark.gpu
@pytest.mark.parametrize("world,d,momentum", [(2, 100_003, True), (8, 1_000_003, True), (8, 70_001, False),
                                             (3, 4_200_000, True)])
def test_emulated_ranks_on_one_gpu_match_the_oracle(world, d, momentum):
    """Every emulated rank owns its buffers on cuda:0; the rows travel by plain device copies (the
    stand-in for the all-gather), so each rank's vote kernel reads only its own gathered copy."""
    from paper_1802_04434_b200 import binding as B
    B.lib()
    dev = torch.device("cuda", 0)
    steps, beta, delta = 2, (0.9 if momentum else 0.0), 1e-3
    x0, g, m0 = worker_inputs(world, d, steps, seed=world * 31 + d, momentum=momentum)
    ranks = [multi.WorkerStep(d, dev, world=world, rank=r) for r in range(world)]
    xs = [torch.from_numpy(x0.copy()).to(dev) for _ in range(world)]
    ms = [torch.from_numpy(m0[r:r + 1].copy()).to(dev) if momentum else None for r in range(world)]
    ref, x_ref, m_ref = reference_run(x0, g, m0, d, beta, delta, momentum)
    W = oracle.words(d)
    for k in range(steps):
        gk = [torch.from_numpy(g[k, r:r + 1].copy()).to(dev) for r in range(world)]
        for r, ws in enumerate(ranks):
            ws.pack(gk[r], ms[r], beta)
        for ws in ranks:                                       # the exchange: row r of everyone <- rank r's row
            for r, src in enumerate(ranks):
                ws.bits[r].copy_(src.row)
        for r, ws in enumerate(ranks):
            ws.vote_apply(xs[r], delta)
        torch.cuda.synchronize()
        for r, ws in enumerate(ranks):
            got = ws.bits.cpu().numpy().view(np.uint32)
            assert np.array_equal(got[:, :W], ref[k][0][:, :W]) and np.all(got[:, W:] == 0)
            assert np.array_equal(ws.vote.cpu().numpy().view(np.uint32), ref[k][1])
    ld = multi.round_up(d, 4)
    for r in range(world):
        assert np.array_equal(xs[r].cpu().numpy().view(np.uint32), x_ref.view(np.uint32))
        if momentum:
            assert np.array_equal(ms[r].cpu().numpy().reshape(-1).view(np.uint32),
                                  m_ref[r * ld:(r + 1) * ld].view(np.uint32))
