"""Host-side checks of the C ABI that need no GPU: the library loads, exports every
symbol the header declares, and rejects bad arguments before launching anything."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "signsgd.h")


@pytest.fixture(scope="module")
def L():
    from paper_1802_04434_b200 import _build, binding
    _build.build()
    return binding.lib()


def declared_symbols():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ssgd_[a-z0-9_]+)\s*\(", text)))


def test_header_declares_the_expected_calls():
    names = declared_symbols()
    for n in ("ssgd_sign_pack", "ssgd_signum_momentum_pack", "ssgd_majority_vote", "ssgd_sign_apply",
              "ssgd_signsgd_step", "ssgd_words", "ssgd_status_str"):
        assert n in names


def test_library_exports_every_declared_symbol(L):
    for n in declared_symbols():
        assert hasattr(L, n), n


def test_words(L):
    for d in (0, 1, 31, 32, 33, 25_557_056, 335_141_888, 2**40 + 1):
        assert L.ssgd_words(d) == -(-d // 32)


def test_status_strings(L):
    seen = {L.ssgd_status_str(i) for i in range(6)}
    assert len(seen) == 6 and all(s for s in seen)


A = 0x10000          # a fake, 16-byte aligned address: these calls must fail before touching it
OK, NULL, ALIGN, SIZE, ARG = 0, 1, 2, 3, 4


def test_sign_pack_argument_checks(L):
    f = L.ssgd_sign_pack
    assert f(None, 1, 64, 64, A, 4, None) == NULL
    assert f(A, 1, 64, 64, None, 4, None) == NULL
    assert f(A + 4, 1, 64, 64, A, 4, None) == ALIGN
    assert f(A, 1, 64, 64, A + 8, 4, None) == ALIGN
    assert f(A, 1, 64, 66, A, 4, None) == ALIGN            # ld not a multiple of 4
    assert f(A, 1, 64, 64, A, 2, None) == ALIGN            # ldw not a multiple of 4
    assert f(A, 0, 64, 64, A, 4, None) == SIZE             # M = 0
    assert f(A, 1025, 64, 64, A, 4, None) == SIZE          # M above the maximum
    assert f(A, 1, 64, 60, A, 4, None) == SIZE             # ld < d
    assert f(A, 1, 160, 160, A, 4, None) == SIZE           # ldw < W = 5
    assert f(A, 4, 2**62, 2**62, A, 2**57, None) == SIZE   # M * ld overflows
    assert f(A, 1, 0, 0, A, 0, None) == OK                 # d = 0: nothing to do


def test_momentum_pack_argument_checks(L):
    f = L.ssgd_signum_momentum_pack
    assert f(A, None, 1, 64, 64, 0.9, A, 4, None) == NULL
    assert f(A, A + 4, 1, 64, 64, 0.9, A, 4, None) == ALIGN
    for beta in (1.0, 1.5, -0.1, float("nan"), float("inf")):
        assert f(A, A, 1, 64, 64, beta, A, 4, None) == ARG
    assert f(A, A, 1, 0, 0, 0.0, A, 0, None) == OK


def test_vote_argument_checks(L):
    f = L.ssgd_majority_vote
    assert f(None, 3, 64, 4, A, None) == NULL
    assert f(A, 3, 64, 4, None, None) == NULL
    assert f(A, 3, 64, 4, A + 4, None) == ALIGN
    assert f(A, 3, 64, 6, A, None) == ALIGN
    assert f(A, 0, 64, 4, A, None) == SIZE
    assert f(A, 3, 640, 16, A, None) == SIZE               # W = 20 > ldw
    assert f(A, 3, 0, 0, A, None) == OK


def test_staged_vote_argument_checks(L):
    for f in (L.ssgd_majority_vote_staged, L.ssgd_majority_vote_staged_wait_selftest):
        assert f(None, 3, 64, 4, A, A, None) == NULL
        assert f(A, 3, 64, 4, A, None, None) == NULL           # the status word is required
        assert f(A, 3, 64, 4, A, A + 2, None) == ALIGN
        assert f(A, 3, 64, 6, A, A, None) == ALIGN
        assert f(A, 0, 64, 4, A, A, None) == SIZE
        assert f(A, 3, 0, 0, A, A, None) == OK
    assert L.ssgd_majority_vote_staged_wait_selftest(A, 3, 1 << 20, 1 << 15, A, A, None) == SIZE


def test_apply_argument_checks(L):
    f = L.ssgd_sign_apply
    assert f(None, A, 64, 0.1, None) == NULL
    assert f(A, None, 64, 0.1, None) == NULL
    assert f(A + 4, A, 64, 0.1, None) == ALIGN
    for delta in (float("nan"), float("inf"), float("-inf")):
        assert f(A, A, 64, delta, None) == ARG
    assert f(A, A, 0, 0.1, None) == OK


def test_step_argument_checks(L):
    f = L.ssgd_signsgd_step
    assert f(None, A, A, 1, 64, 64, 0.9, 0.1, A, 4, A, None) == NULL
    assert f(A, A, None, 1, 64, 64, 0.9, 0.1, A, 4, A, None) == NULL     # m required when beta > 0
    assert f(A, A, None, 1, 0, 0, 0.0, 0.1, A, 0, A, None) == OK         # m optional when beta = 0
    assert f(A, A, A, 1, 64, 64, 1.0, 0.1, A, 4, A, None) == ARG
    assert f(A, A, A, 1, 64, 64, 0.9, float("nan"), A, 4, A, None) == ARG
    assert f(A, A, A, 2000, 64, 64, 0.9, 0.1, A, 4, A, None) == SIZE
    h = L.ssgd_signsgd_step_host
    assert h(A, None, A, 1, 64, 64, 0.9, 0.1, A, A, 4, A, None, None) == NULL
    assert h(A, A, A, 1, 64, 64, 0.9, 0.1, A + 4, A, 4, A, None, None) == ALIGN


def test_noalloc_step_rejects_before_touching_the_device(L):
    # capacity and range checks come before the first CUDA call, so fake pointers are safe here
    f = L.ssgd_signsgd_step_noalloc
    assert f(A, A, A, 0, 64, 64, 0.9, 0.1, None) == SIZE
    assert f(A, A, A, 1025, 64, 64, 0.9, 0.1, None) == SIZE
    assert f(A, A, A, 7, 1 << 25, 1 << 25, 0.9, 0.1, None) == 6           # (7 + 1) * 2^20 words > 4 Mi
    assert f(A, A, A, 3, 32 * (1 << 20) + 1, 32 * (1 << 20) + 4, 0.9, 0.1, None) == 6
    assert b"scratch" in L.ssgd_status_str(6)


def test_pack_scatter_argument_checks(L):
    f = L.ssgd_signum_momentum_pack_scatter
    rows = (ctypes.c_void_p * 3)(A, A + 0x1000, A + 0x2000)
    assert f(None, A, 64, 0.9, rows, 3, 0, 4, None) == NULL
    assert f(A, A, 64, 0.9, None, 3, 0, 4, None) == NULL
    assert f(A, None, 64, 0.9, rows, 3, 0, 4, None) == NULL            # m required when beta > 0
    assert f(A, A + 4, 64, 0.9, rows, 3, 0, 4, None) == ALIGN
    assert f(A, A, 64, 1.0, rows, 3, 0, 4, None) == ARG
    assert f(A, A, 64, 0.9, rows, 0, 0, 4, None) == SIZE               # no destination
    assert f(A, A, 64, 0.9, rows, 65, 0, 4, None) == SIZE              # more than SSGD_MAX_PEERS
    assert f(A, A, 64, 0.9, rows, 3, 1024, 4, None) == SIZE            # row index out of range
    assert f(A, A, 640, 0.9, rows, 3, 0, 16, None) == SIZE             # ldw < W
    assert f(A, A, 64, 0.9, rows, 3, 0, 6, None) == ALIGN
    bad = (ctypes.c_void_p * 3)(A, None, A)
    assert f(A, A, 64, 0.9, bad, 3, 0, 4, None) == NULL
    odd = (ctypes.c_void_p * 3)(A, A + 8, A)
    assert f(A, A, 64, 0.9, odd, 3, 0, 4, None) == ALIGN
    assert f(A, None, 0, 0.0, rows, 3, 5, 0, None) == OK               # d = 0; m optional when beta = 0


def test_warmup_steps_is_host_arithmetic(L):
    assert L.ssgd_warmup_steps(0.9) == 54          # the value Theorem 3 prints for beta = 0.9
    assert L.ssgd_warmup_steps(0.0) == 1
    assert L.ssgd_warmup_steps(1.0) == 0 and L.ssgd_warmup_steps(float("nan")) == 0
    # the launch-shape query answers 0 for sizes out of range (and, with no device, for everything)
    assert L.ssgd_step_is_fused(0, 1000, 1) == 0 and L.ssgd_step_is_fused(1025, 1000, 0) == 0
    assert L.ssgd_step_is_fused(3, 0, 1) == 0
    w = L.ssgd_signsgd_warmup_step
    assert w(A, A, None, 1, 64, 64, 0.9, 0.1, A, 4, A, None) == NULL     # m is required
    assert w(A, A, A, 1, 0, 0, 0.9, 0.1, A, 0, A, None) == OK
    assert L.ssgd_signum_warmup_pack(A, A, 1, 64, 64, 1.0, A, 4, None) == ARG


def test_good_scheme_argument_checks(L):
    assert [L.ssgd_count_planes(M) for M in (1, 2, 3, 4, 7, 8, 1024)] == [1, 2, 2, 3, 3, 4, 11]
    assert L.ssgd_count_planes(0) == 0 and L.ssgd_count_planes(1025) == 0
    c = L.ssgd_vote_counts
    assert c(None, 3, 64, 4, A, 4, None) == NULL
    assert c(A, 3, 64, 4, A + 4, 4, None) == ALIGN
    assert c(A, 3, 64, 4, A, 2, None) == ALIGN
    assert c(A, 3, 640, 20, A, 16, None) == SIZE            # ldc < W
    assert c(A, 0, 64, 4, A, 4, None) == SIZE
    assert c(A, 3, 0, 0, A, 0, None) == OK
    a = L.ssgd_sum_apply
    assert a(None, A, 3, 64, 4, 0.1, None) == NULL
    assert a(A, A, 0, 64, 4, 0.1, None) == SIZE
    assert a(A, A, 3, 64, 4, float("inf"), None) == ARG
    assert a(A, A, 3, 0, 0, 0.1, None) == OK


def test_abstention_argument_checks(L):
    t = L.ssgd_ternary_pack
    assert t(None, A, 1, 64, 64, 0.9, 0.1, A, A, 4, None) == NULL
    assert t(A, None, 1, 64, 64, 0.9, 0.1, A, A, 4, None) == NULL        # m required when beta > 0
    assert t(A, None, 1, 0, 0, 0.0, 0.1, A, A, 0, None) == OK
    assert t(A, A, 1, 64, 64, 0.9, -0.1, A, A, 4, None) == ARG           # tau < 0
    assert t(A, A, 1, 64, 64, 0.9, float("nan"), A, A, 4, None) == ARG
    assert t(A, A, 1, 64, 64, 0.9, 0.1, A + 4, A, 4, None) == ALIGN
    q = L.ssgd_quorum_vote
    assert q(A, None, 3, 64, 4, 1, A, A, None) == NULL
    assert q(A, A, 0, 64, 4, 1, A, A, None) == SIZE
    assert q(A, A, 3, 0, 0, 1, A, A, None) == OK
    a = L.ssgd_ternary_apply
    assert a(A, A, None, 64, 0.1, None) == NULL
    assert a(A, A, A, 64, float("inf"), None) == ARG
    assert a(A, A, A, 0, 0.1, None) == OK


def test_statistics_argument_checks(L):
    w = L.ssgd_welford_update
    assert w(None, 1, A, A, 64, None) == NULL
    assert w(A, 0, A, A, 64, None) == ARG                 # samples count from 1
    assert w(A, (1 << 24) + 1, A, A, 64, None) == ARG
    assert w(A + 4, 1, A, A, 64, None) == ALIGN
    assert w(A, 1, A, A, 0, None) == OK
    assert L.ssgd_density_sums(None, 64, 0, A, None) == NULL
    assert L.ssgd_density_sums(A, 64, 0, A + 8, None) == ALIGN
    f = L.ssgd_density_from_sums
    assert f(4.0, 4.0, 4) == 1.0 and f(2.0, 4.0, 4) == 0.25 and f(0.0, 0.0, 4) == 0.0 and f(1.0, 1.0, 0) == 0.0


def test_binding_refuses_to_run_without_the_library(monkeypatch, tmp_path):
    from paper_1802_04434_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", str(tmp_path / "missing.so"))
    with pytest.raises(ImportError):
        binding.words(64)
