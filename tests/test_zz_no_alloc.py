"""The no-allocation step: for callers that cannot obtain device memory (a framework has reserved it
all, or cudaMalloc's device-wide synchronisation is not acceptable where they run), the library keeps
the packed sign rows and the vote in a fixed internal array.  Its x and m must equal those of the
ordinary step and of the CPU oracle, call after call, although the internal array is reused and never
cleared.

Collected last on purpose (file name), so that a run that stops at the first failure has already run
every other test.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_1802_04434_b200 import binding as B
from paper_1802_04434_b200 import workloads as wl

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def same_bits(t: torch.Tensor, ref: np.ndarray) -> bool:
    return np.array_equal(t.detach().cpu().numpy().reshape(-1).view(np.uint32), ref.reshape(-1).view(np.uint32))


def run_pair(cfg, steps=2):
    M, d, ld, ldw, W = cfg.M, cfg.d, cfg.ld, cfg.ldw, cfg.words
    shared = cfg.shared(DEV)
    xa, xb = cfg.x0(DEV), cfg.x0(DEV)
    ma = cfg.m0(DEV) if cfg.momentum_buffer else None
    mb = cfg.m0(DEV) if cfg.momentum_buffer else None
    x_ref = xa.cpu().numpy().copy()
    m_ref = ma.cpu().numpy().reshape(-1).copy() if ma is not None else None
    bits = torch.zeros(M, ldw, dtype=torch.int32, device=DEV)
    vote = torch.zeros(W, dtype=torch.int32, device=DEV)
    for k in range(steps):                              # consecutive calls reuse the internal array
        g = cfg.g(k, DEV, shared)
        B.signsgd_step(xa, g, ma, M, d, ld, cfg.beta, cfg.delta, bits, ldw, vote)
        B.signsgd_step_noalloc(xb, g, mb, M, d, ld, cfg.beta, cfg.delta)
        oracle.signsgd_step(x_ref, g.cpu().numpy().reshape(-1), m_ref, M, d, cfg.beta, cfg.delta, ld=ld, ldw=ldw)
        torch.cuda.synchronize()
        # same kernels, same order of operations: bit-identical, which is inside the 1-ulp bound
        assert torch.equal(xa.view(torch.int32), xb.view(torch.int32)), "x differs at call %d" % k
        assert same_bits(xb, x_ref), "x differs from the oracle's at call %d" % k
        if ma is not None:
            assert torch.equal(ma.view(torch.int32), mb.view(torch.int32)), "m differs at call %d" % k
            assert same_bits(mb, m_ref), "m differs from the oracle's at call %d" % k
        assert not torch.equal(xa, cfg.x0(DEV))         # the step did move x


def test_noalloc_step_matches_ordinary_step_on_two_calls_in_a_row():
    run_pair(wl.small_signum(d=1_000_000, M=3))


def test_noalloc_step_after_a_differently_shaped_call():
    # leftovers of a wider, shorter problem stay in the array; the next call must not see them
    run_pair(wl.sweep_point(40_001, 31))
    run_pair(wl.small_signum(d=300_003, M=2))
    run_pair(wl.tie_zero_stress(d=1 << 18, M=8))        # beta = 0, no momentum buffer
    # more than 8 workers (worker + vote + apply kernels) with a row length that is not a multiple of
    # four words, right after calls that left non-zero words everywhere in the array: the vote reads
    # the stale padding words of every row and must mask them
    assert oracle.words(70_033) % 4 != 0
    run_pair(wl.sweep_point(70_033, 16))


def test_noalloc_step_rejects_problems_beyond_its_capacity():
    # Buffers have the full size the arguments describe, so that a regression of the capacity check
    # would show up as a changed canary, not as an out-of-bounds access.
    M, d = 7, 1 << 25                                   # (7 + 1) * 2^20 words = twice the capacity
    assert (M + 1) * (d // 32) > B.NOALLOC_SCRATCH_WORDS
    x = torch.full((d,), 3.25, device=DEV)
    g = torch.full((M, d), -1.5, device=DEV)
    with pytest.raises(B.SignSGDError) as e:
        B.signsgd_step_noalloc(x, g, None, M, d, d, 0.0, 1e-4)
    assert e.value.status == 6 and "scratch" in str(e.value)
    torch.cuda.synchronize()
    assert float(x.min()) == 3.25 == float(x.max()) and float(g.min()) == -1.5 == float(g.max())
    del x, g
    # the largest problem that fits is accepted: (M + 1) * W4 == capacity
    M, d = 3, 32 * (B.NOALLOC_SCRATCH_WORDS // 4)
    cfg = wl.sweep_point(d, M)
    xs, g, m = cfg.x0(DEV), cfg.g(0, DEV), cfg.m0(DEV)
    B.signsgd_step_noalloc(xs, g, m, M, d, cfg.ld, 0.9, 1e-4)
    torch.cuda.synchronize()
