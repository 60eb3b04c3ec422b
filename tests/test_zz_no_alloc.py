"""The no-allocation step: for callers that cannot obtain device memory (a framework has reserved it
all, or cudaMalloc's device-wide synchronisation is not acceptable where they run), the library keeps
the packed sign rows and the vote in a fixed internal array.  Its x and m must equal those of the
ordinary step, call after call, although the internal array is reused and never cleared.

Collected last on purpose (file name), so that a run that stops at the first failure has already run
every other test.
"""
import pytest
import torch

from paper_1802_04434_b200 import binding as B
from paper_1802_04434_b200 import workloads as wl

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def run_pair(cfg, steps=2):
    M, d, ld, ldw, W = cfg.M, cfg.d, cfg.ld, cfg.ldw, cfg.words
    shared = cfg.shared(DEV)
    xa, xb = cfg.x0(DEV), cfg.x0(DEV)
    ma = cfg.m0(DEV) if cfg.momentum_buffer else None
    mb = cfg.m0(DEV) if cfg.momentum_buffer else None
    bits = torch.zeros(M, ldw, dtype=torch.int32, device=DEV)
    vote = torch.zeros(W, dtype=torch.int32, device=DEV)
    for k in range(steps):                              # consecutive calls reuse the internal array
        g = cfg.g(k, DEV, shared)
        B.signsgd_step(xa, g, ma, M, d, ld, cfg.beta, cfg.delta, bits, ldw, vote)
        B.signsgd_step_noalloc(xb, g, mb, M, d, ld, cfg.beta, cfg.delta)
        torch.cuda.synchronize()
        # same kernels, same order of operations: bit-identical, which is inside the 1-ulp bound
        assert torch.equal(xa.view(torch.int32), xb.view(torch.int32)), "x differs at call %d" % k
        if ma is not None:
            assert torch.equal(ma.view(torch.int32), mb.view(torch.int32)), "m differs at call %d" % k
        assert not torch.equal(xa, cfg.x0(DEV))         # the step did move x


def test_noalloc_step_matches_ordinary_step_on_two_calls_in_a_row():
    run_pair(wl.small_signum(d=1_000_000, M=3))


def test_noalloc_step_after_a_differently_shaped_call():
    # leftovers of a wider, shorter problem stay in the array; the next call must not see them
    run_pair(wl.sweep_point(40_001, 31))
    run_pair(wl.small_signum(d=300_003, M=2))
    run_pair(wl.tie_zero_stress(d=1 << 18, M=8))        # beta = 0, no momentum buffer


def test_noalloc_step_rejects_problems_beyond_its_capacity():
    M, d = 7, 1 << 25                                   # (7 + 1) * 2^20 words = twice the capacity
    assert (M + 1) * (d // 32) > B.NOALLOC_SCRATCH_WORDS
    x = torch.zeros(16, device=DEV)
    with pytest.raises(B.SignSGDError) as e:
        B.lib().ssgd_signsgd_step_noalloc.restype           # symbol present
        B._check(B.lib().ssgd_signsgd_step_noalloc(x.data_ptr(), x.data_ptr(), x.data_ptr(), M, d, d,
                                                   0.9, 1e-4, None), "ssgd_signsgd_step_noalloc")
    assert e.value.status == 6 and "scratch" in str(e.value)
    assert float(x.abs().max()) == 0.0
    # the largest problem that fits is accepted: (M + 1) * W4 == capacity
    M, d = 3, 32 * (B.NOALLOC_SCRATCH_WORDS // 4)
    cfg = wl.sweep_point(d, M)
    xs, g, m = cfg.x0(DEV), cfg.g(0, DEV), cfg.m0(DEV)
    B.signsgd_step_noalloc(xs, g, m, M, d, cfg.ld, 0.9, 1e-4)
    torch.cuda.synchronize()
