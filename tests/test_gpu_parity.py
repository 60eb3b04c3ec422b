"""GPU parity: every entry point of the C ABI against the CPU oracle, element by
element on the same seeded inputs.

Acceptance bound: packed sign words and vote words bit-exact; m and x within
1 ulp of fp32 (|diff| <= 1.2e-7 * |value|).  Both sides evaluate the momentum as the same two
correctly rounded fp32 operations and the apply step as one correctly rounded
add, so the tests below demand equality of the fp32 bit patterns, which is
stricter; a sign bit may therefore never differ either.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_1802_04434_b200 import binding as B
from paper_1802_04434_b200 import workloads as wl

pytestmark = pytest.mark.gpu

DEV = "cuda:0"
CANARY_WORD = -559038737  # 0xDEADBEEF as int32
CANARY_F = 12345.678


def u32(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().numpy().view(np.uint32)


def f32(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().numpy()


def assert_same_f32(a: np.ndarray, b: np.ndarray, what: str):
    """Bit-identical fp32 (NaN payloads aside); reports the 1-ulp acceptance bound on failure."""
    ai, bi = a.view(np.uint32), b.view(np.uint32)
    same = (ai == bi) | (np.isnan(a) & np.isnan(b))
    if not same.all():
        bad = np.flatnonzero(~same)
        i = bad[0]
        rel = abs(float(a[i]) - float(b[i])) / max(abs(float(b[i])), 1e-45)
        raise AssertionError("%s: %d of %d elements differ, first at %d: gpu %r oracle %r (rel %.3g; "
                             "acceptance bound 1.2e-7)" % (what, bad.size, a.size, i, a[i], b[i], rel))


def rand_inputs(M, d, ld, seed, special=False):
    r = np.random.default_rng(seed)
    g = (r.standard_normal((M, ld)) * 10.0 ** r.integers(-3, 2, (M, ld))).astype(np.float32)
    m = (r.standard_normal((M, ld)) * 10.0 ** r.integers(-3, 2, (M, ld))).astype(np.float32)
    x = r.standard_normal(max(d, 1)).astype(np.float32)
    g[r.random((M, ld)) < 0.03] = 0.0
    if special and d >= 16:
        vals = np.array([0.0, -0.0, np.nan, np.inf, -np.inf, 1e-45, -1e-45, 1e-39, -1e-39,
                         3.4e38, -3.4e38, 1.17549435e-38], dtype=np.float32)
        for w in range(M):
            idx = r.choice(d, size=min(d, 24), replace=False)
            g[w, idx] = r.choice(vals, size=idx.size)
            idx = r.choice(d, size=min(d, 24), replace=False)
            m[w, idx] = r.choice(vals, size=idx.size)
    return g, m, x


SMALL_D = [1, 2, 31, 32, 33, 127, 128, 129, 511, 512, 513, 4095, 4096, 4097, 5000, 16389, 100003]
SMALL_M = [1, 2, 3, 4, 7, 8, 15, 16, 31, 32, 33]


@pytest.mark.parametrize("d", SMALL_D)
def test_sign_pack_and_momentum_pack_small(d):
    for M in (1, 3, 8):
        ld = wl.round_up(d, 4) + 4
        W = oracle.words(d)
        ldw = wl.round_up(W, 4) + 4
        g, m, _ = rand_inputs(M, d, ld, seed=d * 31 + M, special=True)
        gd = torch.from_numpy(g).to(DEV)
        # sign_pack
        bits = torch.full((M, ldw), CANARY_WORD, dtype=torch.int32, device=DEV)
        B.sign_pack(gd, M, d, ld, bits, ldw)
        ref = oracle.sign_pack(g.reshape(-1), M, d, ld=ld, ldw=ldw).reshape(M, ldw)
        got = u32(bits)
        assert np.array_equal(got[:, :W], ref[:, :W])
        assert np.all(got[:, W:] == np.uint32(0xDEADBEEF))      # row padding never written
        # signum_momentum_pack
        for beta in (0.9, 0.0):
            md = torch.from_numpy(m).to(DEV)
            bits.fill_(CANARY_WORD)
            B.signum_momentum_pack(gd, md, M, d, ld, beta, bits, ldw)
            m_ref = m.copy().reshape(-1)
            ref = oracle.signum_momentum_pack(g.reshape(-1), m_ref, M, d, beta, ld=ld, ldw=ldw).reshape(M, ldw)
            got_m = f32(md)
            assert_same_f32(got_m.reshape(-1), m_ref, "m (d=%d M=%d beta=%g)" % (d, M, beta))
            assert np.array_equal(got_m[:, d:].view(np.uint32), m[:, d:].view(np.uint32))
            got = u32(bits)
            assert np.array_equal(got[:, :W], ref[:, :W])
            assert np.all(got[:, W:] == np.uint32(0xDEADBEEF))


@pytest.mark.parametrize("M", SMALL_M + [64, 100, 255, 256, 1000, 1024])
def test_majority_vote_small(M):
    for d in (1, 33, 128, 1000, 4097, 40000 if M <= 64 else 3000):
        r = np.random.default_rng(M * 1000 + d)
        W = oracle.words(d)
        ldw = wl.round_up(W, 4) + (4 if M % 2 else 0)
        p = r.random(d) if M > 2 else np.full(d, 0.5)           # per-element bias: spans all counts
        s = (r.random((M, d)) < p).astype(np.uint8)
        rows = np.zeros((M, ldw), dtype=np.uint32)
        for w in range(M):
            rows[w, :W] = oracle.pack_bits(s[w])
        rows[:, W:] = r.integers(0, 2**32, size=(M, ldw - W), dtype=np.uint32)  # garbage in row padding
        vote = torch.full((W + 4,), CANARY_WORD, dtype=torch.int32, device=DEV)
        B.majority_vote(torch.from_numpy(rows.view(np.int32)).to(DEV), M, d, ldw, vote)
        ref = oracle.majority_vote(rows.reshape(-1), M, d, ldw=ldw)
        got = u32(vote)
        assert np.array_equal(got[:W], ref), "M=%d d=%d" % (M, d)
        assert np.all(got[W:] == np.uint32(0xDEADBEEF))


@pytest.mark.parametrize("M,d", [(5, (1 << 25) + 37), (7, (1 << 25) + 37), (7, 5_000_003), (4, 3_000_001),
                                 (13, (1 << 24) + 4099), (31, 5_000_003), (63, 2_000_003), (64, 2_000_003),
                                 (100, 1_000_003), (64, 5_000_003), (100, 5_000_003), (16, 3_000_001),
                                 (16, 1_500_001)])
def test_majority_vote_long_vectors(M, d):
    """The vote kernels (the one for exactly 2 .. 7 rows; the general one with its remaining rows as one guarded
    batch, M = 8 .. 127, or in batches of 4, 2, 1; the one that spreads 13 and more rows over the warps of a CTA
    while the vector is short: both sides of its threshold for M = 16, 64, 100) on launches many CTAs per SM deep
    and on shorter ones, with a ragged last word and garbage in the row padding."""
    r = np.random.default_rng(M * 7919 + d % 1000)
    W = oracle.words(d)
    ldw = wl.round_up(W, 4) + 8
    rows = r.integers(0, 2**32, size=(M, ldw), dtype=np.uint32)
    # a band of elements where the count sits at the threshold: exactly ceil(M/2) and ceil(M/2) - 1 set bits
    T = (M + 1) // 2
    for j, ones in ((3, T), (W // 2, T - 1), (W - 2, T)):
        rows[:, j] = 0
        rows[:ones, j] = 0xFFFFFFFF
    vote = torch.full((W + 4,), CANARY_WORD, dtype=torch.int32, device=DEV)
    B.majority_vote(torch.from_numpy(rows.view(np.int32)).to(DEV), M, d, ldw, vote)
    ref = oracle.majority_vote(rows.reshape(-1), M, d, ldw=ldw)
    got = u32(vote)
    assert got[3] == 0xFFFFFFFF and got[W // 2] == 0 and ref[3] == 0xFFFFFFFF and ref[W // 2] == 0
    assert np.array_equal(got[:W], ref), "M=%d d=%d" % (M, d)
    assert np.all(got[W:] == np.uint32(0xDEADBEEF))


@pytest.mark.parametrize("M", [1, 2, 3, 7, 8, 9, 16, 17, 31, 33, 100, 1024])
def test_majority_vote_staged_through_shared_memory(M):
    # the second kernel design (rows staged by bulk copies, 8 rows per mbarrier phase): same words
    for d in (1, 33, 4097, 32768, 32768 + 5, 100_003 if M <= 100 else 40_000, 1_000_003 if M <= 17 else 70_001):
        r = np.random.default_rng(M * 1000 + d)
        W = oracle.words(d)
        ldw = wl.round_up(W, 4) + (4 if M % 2 else 0)
        s = (r.random((M, d)) < r.random(d)).astype(np.uint8) if M * d <= 20_000_000 else \
            (r.random((M, d), dtype=np.float32) < 0.5).astype(np.uint8)
        rows = np.zeros((M, ldw), dtype=np.uint32)
        for w in range(M):
            rows[w, :W] = oracle.pack_bits(s[w])
        rows[:, W:] = r.integers(0, 2**32, size=(M, ldw - W), dtype=np.uint32)   # garbage in row padding
        vote = torch.full((W + 4,), CANARY_WORD, dtype=torch.int32, device=DEV)
        status = torch.zeros(1, dtype=torch.int32, device=DEV)
        B.majority_vote_staged(torch.from_numpy(rows.view(np.int32)).to(DEV), M, d, ldw, vote, status)
        ref = oracle.majority_vote(rows.reshape(-1), M, d, ldw=ldw)
        got = u32(vote)
        assert int(status.item()) == 0
        assert np.array_equal(got[:W], ref), "M=%d d=%d" % (M, d)
        assert np.all(got[W:] == np.uint32(0xDEADBEEF))


def test_staged_vote_bounded_waits_run_out_and_report():
    """Every wait in the staged kernel has an iteration limit.  The self-test entry arms each phase for more
    bytes than its copies deliver, so the waits must run out: the call returns, the status word says so, the
    output is untouched, and the device is fine afterwards."""
    M, d = 19, 20_000
    W = oracle.words(d)
    ldw = wl.round_up(W, 4)
    bits = torch.randint(-2**31, 2**31 - 1, (M, ldw), dtype=torch.int32, device=DEV)
    vote = torch.full((W,), CANARY_WORD, dtype=torch.int32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    L = B.lib()
    rc = L.ssgd_majority_vote_staged_wait_selftest(bits.data_ptr(), M, d, ldw, vote.data_ptr(), status.data_ptr(),
                                                   torch.cuda.current_stream().cuda_stream)
    assert rc == 0
    torch.cuda.synchronize()
    assert int(status.item()) == 1
    assert np.all(u32(vote) == np.uint32(0xDEADBEEF))
    assert L.ssgd_majority_vote_staged_wait_selftest(bits.data_ptr(), M, 1 << 20, 1 << 15, vote.data_ptr(),
                                                     status.data_ptr(), None) == 3          # larger sizes refused
    status.zero_()
    B.majority_vote_staged(bits, M, d, ldw, vote, status)                                    # and it still works
    ref = torch.zeros(W, dtype=torch.int32, device=DEV)
    B.majority_vote(bits, M, d, ldw, ref)
    torch.cuda.synchronize()
    assert int(status.item()) == 0 and torch.equal(vote, ref)


def test_majority_vote_ignores_garbage_padding_bits():
    # padding bits of the last word are the caller's to keep 0; the vote masks them anyway
    M, d = 3, 40
    rows = np.full((M, 4), 0xFFFFFFFF, dtype=np.uint32)
    vote = torch.zeros(4, dtype=torch.int32, device=DEV)
    B.majority_vote(torch.from_numpy(rows.view(np.int32)).to(DEV), M, d, 4, vote)
    assert u32(vote)[:2].tolist() == [0xFFFFFFFF, 0xFF]


@pytest.mark.parametrize("d", SMALL_D)
def test_sign_apply_small(d):
    r = np.random.default_rng(d)
    W = oracle.words(d)
    x = np.full(d + 7, CANARY_F, dtype=np.float32)
    x[:d] = (r.standard_normal(d) * 10.0 ** r.integers(-6, 3, d)).astype(np.float32)
    vote = oracle.pack_bits(r.integers(0, 2, d, dtype=np.uint8))
    for delta in (1e-4, 0.37):
        xd = torch.from_numpy(x).to(DEV)
        B.sign_apply(xd, torch.from_numpy(vote.view(np.int32)).to(DEV), d, delta)
        ref = x[:d].copy()
        oracle.sign_apply(ref, vote, d, delta)
        got = f32(xd)
        assert_same_f32(got[:d], ref, "x (d=%d)" % d)
        assert np.all(got[d:] == np.float32(CANARY_F))


@pytest.mark.parametrize("M", SMALL_M)
def test_whole_step_small(M):
    # 33 .. 70001: one launch whose warps take different rows (2 <= M <= 32); 400003: past that kernel's range for
    # every M, i.e. the fused kernel's smallest tile with a ragged span (M <= 8) or worker + vote + apply.
    # Row strides longer than the rows, canaries behind every output.
    for d in (33, 1000, 4097, 70001, 400_003):
        for beta, with_m in ((0.9, True), (0.0, True), (0.0, False)):
            shape = B.lib().ssgd_step_is_fused(M, d, 1 if with_m else 0)
            if d < 400_003:
                assert shape == (2 if 2 <= M <= 32 else (1 if M == 1 else 0)), (M, d, shape)
            else:
                assert shape == (1 if M <= 8 else 0), (M, d, shape)
            ld, W = wl.round_up(d, 4) + 4, oracle.words(d)
            ldw = wl.round_up(W, 4) + 4
            g, m, x = rand_inputs(M, d, ld, seed=M * 77 + d, special=True)
            x = np.concatenate([x, np.full(8, CANARY_F, dtype=np.float32)])
            gd, md, xd = (torch.from_numpy(a).to(DEV) for a in (g, m, x))
            bits = torch.full((M, ldw), CANARY_WORD, dtype=torch.int32, device=DEV)
            vote = torch.full((W + 4,), CANARY_WORD, dtype=torch.int32, device=DEV)
            B.signsgd_step(xd, gd, md if with_m else None, M, d, ld, beta, 1e-3, bits, ldw, vote)
            m_ref, x_ref = m.copy().reshape(-1), x[:d].copy()
            b_ref, v_ref = oracle.signsgd_step(x_ref, g.reshape(-1), m_ref if with_m else None, M, d,
                                               beta, 1e-3, ld=ld, ldw=ldw)
            what = "M=%d d=%d beta=%g m=%s" % (M, d, beta, with_m)
            check_rows(bits, b_ref, M, ldw, W, "bits " + what)
            assert np.array_equal(u32(vote)[:W], v_ref), what
            assert np.all(u32(vote)[W:] == np.uint32(0xDEADBEEF)), what
            gx = f32(xd)
            assert_same_f32(gx[:d], x_ref, "x " + what)
            assert np.all(gx[d:] == np.float32(CANARY_F)), what
            if with_m:
                assert_same_f32(f32(md).reshape(-1), m_ref, "m " + what)       # includes the untouched elements >= d


@pytest.mark.parametrize("seed", range(48))
def test_whole_step_random_shapes(seed):
    """Seeded random problems across the launch forms of the step (row-parallel, fused with either tile, worker +
    vote + apply): random worker count, length, row strides and mode (Signum, sign-only, warm-up), two steps each,
    everything compared with the oracle, canaries behind every output."""
    r = np.random.default_rng(1000 + seed)
    M = int(r.choice([1, 2, 3, 4, 5, 6, 7, 8, 9, 12, 15, 16, 17, 24, 31, 32, 33, 40]))
    d = int(10 ** r.uniform(0.0, 5.6)) if seed % 4 else int(r.choice([65_535, 65_537, 131_073, 262_145, 151_553, 303_105]))
    mode = ("signum", "sign_only", "warmup")[seed % 3]
    ld = wl.round_up(d, 4) + 4 * int(r.integers(0, 3))
    W = oracle.words(d)
    ldw = wl.round_up(W, 4) + 4 * int(r.integers(0, 3))
    beta = 0.0 if mode == "sign_only" else float(r.choice([0.5, 0.9, 0.99]))
    delta = float(r.choice([1e-4, 1e-2, 0.5]))
    g0, m, x = rand_inputs(M, d, ld, seed=seed, special=True)
    x = np.concatenate([x[:d], np.full(8, CANARY_F, dtype=np.float32)])
    with_m = mode != "sign_only"
    md = torch.from_numpy(m).to(DEV) if with_m else None
    xd = torch.from_numpy(x).to(DEV)
    m_ref = m.copy().reshape(-1) if with_m else None
    x_ref = x[:d].copy()
    for k in range(2):
        g = g0 if k == 0 else rand_inputs(M, d, ld, seed=seed + 500)[0]
        bits = torch.full((M, ldw), CANARY_WORD, dtype=torch.int32, device=DEV)
        vote = torch.full((W + 4,), CANARY_WORD, dtype=torch.int32, device=DEV)
        gd = torch.from_numpy(g).to(DEV)
        if mode == "warmup":
            B.signsgd_warmup_step(xd, gd, md, M, d, ld, beta, delta, bits, ldw, vote)
            b_ref, v_ref = oracle.signsgd_warmup_step(x_ref, g.reshape(-1), m_ref, M, d, beta, delta, ld=ld, ldw=ldw)
        else:
            B.signsgd_step(xd, gd, md, M, d, ld, beta, delta, bits, ldw, vote)
            b_ref, v_ref = oracle.signsgd_step(x_ref, g.reshape(-1), m_ref, M, d, beta, delta, ld=ld, ldw=ldw)
        what = "seed=%d M=%d d=%d %s step %d" % (seed, M, d, mode, k)
        check_rows(bits, b_ref, M, ldw, W, "bits " + what)
        assert np.array_equal(u32(vote)[:W], v_ref), what
        assert np.all(u32(vote)[W:] == np.uint32(0xDEADBEEF)), what
        gx = f32(xd)
        assert_same_f32(gx[:d], x_ref, "x " + what)
        assert np.all(gx[d:] == np.float32(CANARY_F)), what
        if with_m:
            assert_same_f32(f32(md).reshape(-1), m_ref, "m " + what)


# Odd vector lengths large enough that the launchers pick their largest tiles (16 and 32 elements per
# thread: from about 64 Mi elements with a momentum, 32 Mi without), so that those instantiations meet a
# ragged last tile, a last word with pad bits, and rows whose stride exceeds d.
BIG_ODD_D = [5_000_003, (1 << 23) + 4099]


def big_inputs(M, d, ld, seed, with_m=True):
    r = np.random.default_rng(seed)
    g = r.standard_normal((M, ld), dtype=np.float32)
    g[:, ::97] = 0.0
    g[:, 5::1013] *= np.float32(1e-3)
    m = (0.3 * r.standard_normal((M, ld), dtype=np.float32)) if with_m else None
    x = r.standard_normal(d + 8, dtype=np.float32)
    x[d:] = CANARY_F
    return g, m, x


def check_rows(bits, ref, M, ldw, W, what):
    got = u32(bits)
    assert np.array_equal(got[:, :W], ref.reshape(M, ldw)[:, :W]), what
    assert np.all(got[:, W:] == np.uint32(0xDEADBEEF)), what + ": row padding written"


@pytest.mark.parametrize("d", BIG_ODD_D)
@pytest.mark.parametrize("M", [1, 3, 7])
def test_sign_pack_large_odd_d(d, M):
    ld, W = wl.round_up(d, 4) + 8, oracle.words(d)
    ldw = wl.round_up(W, 4) + 4
    g, _, _ = big_inputs(M, d, ld, seed=d % 1000 + M, with_m=False)
    bits = torch.full((M, ldw), CANARY_WORD, dtype=torch.int32, device=DEV)
    B.sign_pack(torch.from_numpy(g).to(DEV), M, d, ld, bits, ldw)
    check_rows(bits, oracle.sign_pack(g.reshape(-1), M, d, ld=ld, ldw=ldw), M, ldw, W, "sign_pack d=%d M=%d" % (d, M))


@pytest.mark.parametrize("d", BIG_ODD_D)
@pytest.mark.parametrize("M,beta,with_m", [(1, 0.0, False), (8, 0.0, False), (16, 0.9, True), (5, 0.9, True), (12, 0.0, False),
                                           (9, 0.0, False), (17, 0.0, False), (32, 0.0, False), (33, 0.0, False)])
def test_whole_step_large_odd_d(d, M, beta, with_m):
    # both launch shapes of the step occur here for the same M: without a momentum, 9 to 32 workers run as the
    # one fused kernel on the longer vector and as worker + vote + apply kernels on the shorter one
    if not with_m and 8 < M <= 32:
        assert B.step_is_fused(M, d, False) == (d > 7_500_000)
    assert B.step_is_fused(M, d, with_m) == (M <= 8 or (not with_m and M <= 32 and d > 7_500_000))
    ld, W = wl.round_up(d, 4) + 8, oracle.words(d)
    ldw = wl.round_up(W, 4) + 4
    g, m, x = big_inputs(M, d, ld, seed=d % 1000 + 7 * M, with_m=with_m)
    gd, xd = torch.from_numpy(g).to(DEV), torch.from_numpy(x).to(DEV)
    md = torch.from_numpy(m).to(DEV) if with_m else None
    bits = torch.full((M, ldw), CANARY_WORD, dtype=torch.int32, device=DEV)
    vote = torch.full((W + 4,), CANARY_WORD, dtype=torch.int32, device=DEV)
    B.signsgd_step(xd, gd, md, M, d, ld, beta, 1e-3, bits, ldw, vote)
    x_ref = x[:d].copy()
    m_ref = m.copy().reshape(-1) if with_m else None
    b_ref, v_ref = oracle.signsgd_step(x_ref, g.reshape(-1), m_ref, M, d, beta, 1e-3, ld=ld, ldw=ldw)
    check_rows(bits, b_ref, M, ldw, W, "bits d=%d M=%d" % (d, M))
    assert np.array_equal(u32(vote)[:W], v_ref) and np.all(u32(vote)[W:] == np.uint32(0xDEADBEEF))
    gx = f32(xd)
    assert_same_f32(gx[:d], x_ref, "x")
    assert np.all(gx[d:] == np.float32(CANARY_F))
    if with_m:
        gm = f32(md)
        assert_same_f32(gm.reshape(-1), m_ref, "m")                 # includes the untouched elements >= d
        assert np.array_equal(gm[:, d:].view(np.uint32), m[:, d:].view(np.uint32))


@pytest.mark.parametrize("d", BIG_ODD_D)
@pytest.mark.parametrize("M", [7, 16])
def test_warmup_large_odd_d(d, M):
    ld, W = wl.round_up(d, 4) + 8, oracle.words(d)
    ldw = wl.round_up(W, 4) + 4
    g, m, x = big_inputs(M, d, ld, seed=d % 1000 + 3 * M)
    gd = torch.from_numpy(g).to(DEV)
    md = torch.from_numpy(m).to(DEV)
    bits = torch.full((M, ldw), CANARY_WORD, dtype=torch.int32, device=DEV)
    B.signum_warmup_pack(gd, md, M, d, ld, 0.9, bits, ldw)
    m_ref = m.copy().reshape(-1)
    check_rows(bits, oracle.signum_warmup_pack(g.reshape(-1), m_ref, M, d, 0.9, ld=ld, ldw=ldw), M, ldw, W, "warm-up pack")
    assert_same_f32(f32(md).reshape(-1), m_ref, "m after warm-up pack")
    md, xd = torch.from_numpy(m).to(DEV), torch.from_numpy(x).to(DEV)
    bits.fill_(CANARY_WORD)
    vote = torch.full((W + 4,), CANARY_WORD, dtype=torch.int32, device=DEV)
    B.signsgd_warmup_step(xd, gd, md, M, d, ld, 0.9, 1e-3, bits, ldw, vote)
    m_ref, x_ref = m.copy().reshape(-1), x[:d].copy()
    b_ref, v_ref = oracle.signsgd_warmup_step(x_ref, g.reshape(-1), m_ref, M, d, 0.9, 1e-3, ld=ld, ldw=ldw)
    check_rows(bits, b_ref, M, ldw, W, "warm-up step bits")
    assert np.array_equal(u32(vote)[:W], v_ref) and np.all(u32(vote)[W:] == np.uint32(0xDEADBEEF))
    gx = f32(xd)
    assert_same_f32(gx[:d], x_ref, "x")
    assert np.all(gx[d:] == np.float32(CANARY_F))
    assert_same_f32(f32(md).reshape(-1), m_ref, "m")


@pytest.mark.parametrize("M,d", [(100, 40_001), (1000, 5_000), (1024, 4_097)])
def test_whole_step_many_workers(M, d):
    # grid rows up to the worker limit, ten and eleven counter planes in the vote
    ld, W = wl.round_up(d, 4), oracle.words(d)
    ldw = wl.round_up(W, 4)
    g, m, x = rand_inputs(M, d, ld, seed=M + d)
    gd, md, xd = (torch.from_numpy(a).to(DEV) for a in (g, m, x))
    bits = torch.zeros(M, ldw, dtype=torch.int32, device=DEV)
    vote = torch.zeros(W, dtype=torch.int32, device=DEV)
    B.signsgd_step(xd, gd, md, M, d, ld, 0.9, 1e-3, bits, ldw, vote)
    m_ref, x_ref = m.copy().reshape(-1), x.copy()
    b_ref, v_ref = oracle.signsgd_step(x_ref, g.reshape(-1), m_ref, M, d, 0.9, 1e-3, ld=ld, ldw=ldw)
    assert np.array_equal(u32(bits).reshape(-1), b_ref) and np.array_equal(u32(vote), v_ref)
    assert_same_f32(f32(xd), x_ref, "x")
    assert_same_f32(f32(md).reshape(-1), m_ref, "m")
    with pytest.raises(B.SignSGDError):
        B.signsgd_step(xd, gd, md, 1025, 4, 4, 0.9, 1e-3, bits, 4, vote)       # beyond the worker limit


def test_empty_input_launches_nothing():
    z = torch.zeros(4, dtype=torch.float32, device=DEV)
    b = torch.full((4,), CANARY_WORD, dtype=torch.int32, device=DEV)
    B.sign_pack(z, 1, 0, 0, b, 0)
    B.signum_momentum_pack(z, z.clone(), 1, 0, 0, 0.9, b, 0)
    B.majority_vote(b, 1, 0, 0, b.clone())
    B.sign_apply(z, b, 0, 0.1)
    B.signsgd_step(z, z.clone(), z.clone(), 1, 0, 0, 0.9, 0.1, b, 0, b.clone())
    torch.cuda.synchronize()
    assert np.all(u32(b) == np.uint32(0xDEADBEEF)) and float(z.abs().max()) == 0.0


# ------------------------------------------------------------------ the named configurations

def run_config_full(cfg, check_every_step=True):
    """Run cfg.steps steps on the GPU and in the oracle on identical inputs; compare everything."""
    M, d, ld, ldw, W = cfg.M, cfg.d, cfg.ld, cfg.ldw, cfg.words
    shared = cfg.shared(DEV)
    xd = cfg.x0(DEV)
    md = cfg.m0(DEV) if cfg.momentum_buffer else None
    x_ref = f32(xd).copy()
    m_ref = f32(md).reshape(-1).copy() if md is not None else None
    bits = torch.zeros(M, ldw, dtype=torch.int32, device=DEV)
    vote = torch.zeros(W, dtype=torch.int32, device=DEV)
    for k in range(cfg.steps):
        gd = cfg.g(k, DEV, shared)
        B.signsgd_step(xd, gd, md, M, d, ld, cfg.beta, cfg.delta, bits, ldw, vote)
        g_host = f32(gd).reshape(-1)
        b_ref, v_ref = oracle.signsgd_step(x_ref, g_host, m_ref, M, d, cfg.beta, cfg.delta, ld=ld, ldw=ldw)
        if check_every_step or k == cfg.steps - 1:
            assert np.array_equal(u32(bits).reshape(-1), b_ref), "bits, step %d" % k
            assert np.array_equal(u32(vote), v_ref), "vote, step %d" % k
            assert_same_f32(f32(xd), x_ref, "x, step %d" % k)
            if md is not None:
                assert_same_f32(f32(md).reshape(-1), m_ref, "m, step %d" % k)
    return f32(gd), v_ref


def test_config1_small_signum_five_steps():
    run_config_full(wl.small_signum())


def test_config2_resnet50_layout():
    cfg = wl.resnet50_signum()
    _, v_ref = run_config_full(cfg)
    # padding elements between tensors hold g = 0, so they vote +1 on both sides
    votes = oracle.unpack_bits(v_ref, cfg.d)
    end = cfg.segments[-1][0] + cfg.segments[-1][1]
    assert end < cfg.d and votes[end:].all()


def test_config2_per_tensor_slices_of_the_wire_words():
    """Every tensor of the bucketed vector starts on a word boundary, so a tensor's own sign words are a plain
    slice of the row: packing one tensor alone (a call on that slice) gives exactly the words the whole-vector
    call wrote at the tensor's word offset."""
    cfg = wl.resnet50_signum()
    M, d, ld, ldw = cfg.M, cfg.d, cfg.ld, cfg.ldw
    gd = cfg.g(0, DEV)
    bits = torch.zeros(M, ldw, dtype=torch.int32, device=DEV)
    B.sign_pack(gd, M, d, ld, bits, ldw)
    whole = u32(bits)
    picks = [0, 1, 2, 57, 159, 160]                       # stem conv, two batch-norm vectors, a mid conv, fc weight, fc bias
    for t in picks:
        off, size = cfg.segments[t]
        assert off % 32 == 0
        W_t = oracle.words(size)
        ldw_t = wl.round_up(W_t, 4)
        ld_t = wl.round_up(size, 4)
        g_t = torch.zeros(M, ld_t, device=DEV)
        g_t[:, :size] = gd[:, off:off + size]
        b_t = torch.zeros(M, ldw_t, dtype=torch.int32, device=DEV)
        B.sign_pack(g_t, M, size, ld_t, b_t, ldw_t)
        mine = whole[:, off // 32:off // 32 + W_t].copy()
        if size % 32:                                     # the slice's last word also holds the pad elements (g = 0: bit 1)
            mine[:, -1] &= np.uint32((1 << (size % 32)) - 1)
        assert np.array_equal(u32(b_t)[:, :W_t], mine), "tensor %d" % t
        ref = oracle.sign_pack(np.ascontiguousarray(f32(g_t)).reshape(-1), M, size, ld=ld_t, ldw=ldw_t).reshape(M, ldw_t)
        assert np.array_equal(u32(b_t)[:, :W_t], ref[:, :W_t])


def test_config3_ties_and_zeros():
    cfg = wl.tie_zero_stress()
    g, v_ref = run_config_full(cfg)
    g = g[:, :cfg.d]
    votes = oracle.unpack_bits(v_ref, cfg.d).astype(bool)
    P = (~(g < 0)).sum(axis=0)
    tie = 2 * P == cfg.M
    assert tie.mean() > 0.30 and votes[tie].all()            # every tie resolves to +1
    # the same inputs through the fused momentum kernel with beta = 0 give the same words
    gd = cfg.g(0, DEV)
    md = torch.randn(cfg.M, cfg.ld, device=DEV)
    b1 = torch.zeros(cfg.M, cfg.ldw, dtype=torch.int32, device=DEV)
    b2 = torch.zeros_like(b1)
    B.sign_pack(gd, cfg.M, cfg.d, cfg.ld, b1, cfg.ldw)
    B.signum_momentum_pack(gd, md, cfg.M, cfg.d, cfg.ld, 0.0, b2, cfg.ldw)
    assert torch.equal(b1, b2) and torch.equal(md, gd)


def sampled_chunk_parity(cfg, n_chunks, chunk, seed):
    """Full-size run on the GPU; the oracle recomputes `n_chunks` slices of `chunk` elements from
    host copies of the very same inputs.  Plus properties that hold at any size, checked in full
    with plain torch reductions."""
    M, d, ld, ldw, W = cfg.M, cfg.d, cfg.ld, cfg.ldw, cfg.words
    shared = cfg.shared(DEV)
    xd = cfg.x0(DEV)
    md = cfg.m0(DEV)
    if cfg.beta > 0:
        cfg.g(1000, DEV, shared, out=md)                  # a non-trivial starting momentum
        md.mul_(0.5)
    gd = cfg.g(0, DEV, shared)
    r = np.random.default_rng(seed)
    starts = sorted(set([0, (d - chunk) // 32 * 32] +
                        [int(o) * 32 for o in r.integers(0, (d - chunk) // 32, n_chunks - 2)]))
    x0_s = [f32(xd[o:o + chunk]).copy() for o in starts]
    m0_s = [f32(md[:, o:o + chunk]).copy() for o in starts]
    bits = torch.zeros(M, ldw, dtype=torch.int32, device=DEV)
    vote = torch.zeros(W, dtype=torch.int32, device=DEV)
    x_before_sum = xd.double().sum().item()
    B.signsgd_step(xd, gd, md, M, d, ld, cfg.beta, cfg.delta, bits, ldw, vote)
    torch.cuda.synchronize()
    for o, x_ref, m_ref in zip(starts, x0_s, m0_s):
        n = min(chunk, d - o)
        g_s = np.ascontiguousarray(f32(gd[:, o:o + n]))
        m_flat = np.ascontiguousarray(m_ref).reshape(-1)
        b_ref, v_ref = oracle.signsgd_step(x_ref, g_s.reshape(-1), m_flat, M, n, cfg.beta, cfg.delta)
        wn = oracle.words(n)
        assert np.array_equal(u32(bits[:, o // 32:o // 32 + wn]).reshape(-1), b_ref), "bits @%d" % o
        assert np.array_equal(u32(vote[o // 32:o // 32 + wn]), v_ref), "vote @%d" % o
        assert_same_f32(f32(xd[o:o + n]), x_ref, "x @%d" % o)
        assert_same_f32(f32(md[:, o:o + n]).reshape(-1), m_flat, "m @%d" % o)
    # any-size properties: popcount of each packed row = number of non-negative momenta;
    # popcount of the vote tells how far sum(x) moved
    pops = [int(_popcount(bits[w, :W])) for w in range(M)]
    nonneg = [int((~(md[w, :d] < 0)).sum().item()) for w in range(M)]
    assert pops == nonneg
    pv = int(_popcount(vote))
    moved = x_before_sum - xd.double().sum().item()
    assert abs(moved - cfg.delta * (2 * pv - d)) <= 1e-3 * cfg.delta * d + 1e-6


def _popcount(t: torch.Tensor) -> int:
    v = t.to(torch.int64) & 0xFFFFFFFF
    total = 0
    for sh in range(0, 32, 8):
        b = (v >> sh) & 0xFF
        b = (b & 0x55) + ((b >> 1) & 0x55)
        b = (b & 0x33) + ((b >> 2) & 0x33)
        b = (b & 0x0F) + ((b >> 4) & 0x0F)
        total += int(b.sum().item())
    return total


def test_config4_bert_large_full_size_sampled():
    free, _ = torch.cuda.mem_get_info()
    cfg = wl.bert_large_signum()
    need = 2 * cfg.M * cfg.ld * 4 + 4 * cfg.d * 4 + (8 << 30)
    if free < need:
        pytest.skip("needs %.0f GB of free device memory" % (need / 2**30))
    sampled_chunk_parity(cfg, n_chunks=24, chunk=1 << 20, seed=4)


@pytest.mark.parametrize("d,M", [(1 << 10, 31), (1 << 13, 15), (1 << 16, 7), (1 << 20, 3), (1 << 22, 1),
                                 (1 << 24, 7), (1 << 24, 31)])
def test_config5_sweep_points_full_parity(d, M):
    run_config_full(wl.sweep_point(d, M))


@pytest.mark.parametrize("d,M", [(1 << 26, 7), (1 << 28, 3), (1 << 28, 31)])
def test_config5_large_sweep_points_sampled(d, M):
    free, _ = torch.cuda.mem_get_info()
    need = 2 * M * d * 4 + 6 * d * 4 + (8 << 30)
    if free < need:
        pytest.skip("needs %.0f GB of free device memory" % (need / 2**30))
    sampled_chunk_parity(wl.sweep_point(d, M), n_chunks=16, chunk=1 << 20, seed=d % 1000 + M)


def test_host_buffer_step_matches_device_step():
    cfg = wl.small_signum(d=300_001, M=5)
    M, d, ld, ldw, W = cfg.M, cfg.d, cfg.ld, cfg.ldw, cfg.words
    g_host = cfg.g(0).pin_memory()
    x1, x2 = cfg.x0(DEV), cfg.x0(DEV)
    m1 = torch.randn(M, ld, device=DEV) * 0.1
    m2 = m1.clone()
    bits1 = torch.zeros(M, ldw, dtype=torch.int32, device=DEV)
    bits2, vote1 = torch.zeros_like(bits1), torch.zeros(W, dtype=torch.int32, device=DEV)
    vote2 = torch.zeros_like(vote1)
    stage = torch.empty(M, ld, device=DEV)
    vote_host = torch.zeros(W, dtype=torch.int32).pin_memory()
    B.signsgd_step(x1, g_host.to(DEV), m1, M, d, ld, cfg.beta, cfg.delta, bits1, ldw, vote1)
    B.signsgd_step_host(x2, g_host, m2, M, d, ld, cfg.beta, cfg.delta, stage, bits2, ldw, vote2, vote_host)
    torch.cuda.synchronize()
    assert torch.equal(x1, x2) and torch.equal(m1, m2) and torch.equal(bits1, bits2)
    assert torch.equal(vote1.cpu(), vote_host)


@pytest.mark.parametrize("M,d,beta", [(5, 8_000_003, 0.9), (12, 6_000_007, 0.9), (3, 24_000_001, 0.0)])
def test_host_buffer_step_in_column_slabs(M, d, beta):
    """Transfers of 128 MB and more are cut into column slabs that a second stream copies while the step runs on
    the slabs before them.  Two calls in a row with different gradients through the SAME staging buffer (the second
    call's copies must wait for the first call's kernels), against two device steps; x starts from a canary tail."""
    ld, W = wl.round_up(d, 4) + 4, oracle.words(d)
    ldw = wl.round_up(W, 4) + 4
    gen = torch.Generator().manual_seed(M * 1000 + d % 997)
    g_host = [torch.randn(M, ld, generator=gen).pin_memory() for _ in range(2)]
    x0 = torch.randn(d + 8, generator=gen)
    x0[d:] = CANARY_F
    with_m = beta != 0.0
    xs, ms, bs, vs = [], [], [], []
    for _ in range(2):
        xs.append(x0.to(DEV))
        ms.append(torch.zeros(M, ld, device=DEV) if with_m else None)
        bs.append(torch.full((M, ldw), CANARY_WORD, dtype=torch.int32, device=DEV))
        vs.append(torch.full((W + 4,), CANARY_WORD, dtype=torch.int32, device=DEV))
    stage = torch.full((M, ld), float("nan"), device=DEV)
    vote_host = [torch.zeros(W, dtype=torch.int32).pin_memory() for _ in range(2)]
    votes_dev = []
    for k in range(2):
        B.signsgd_step(xs[0], g_host[k].to(DEV), ms[0], M, d, ld, beta, 1e-3, bs[0], ldw, vs[0])
        votes_dev.append(vs[0][:W].clone())
    for k in range(2):                                   # back to back, no synchronisation in between
        B.signsgd_step_host(xs[1], g_host[k], ms[1], M, d, ld, beta, 1e-3, stage, bs[1], ldw, vs[1], vote_host[k])
    torch.cuda.synchronize()
    assert torch.equal(xs[0].view(torch.int32), xs[1].view(torch.int32))
    assert torch.equal(bs[0], bs[1]) and torch.equal(vs[0], vs[1])
    if with_m:
        assert torch.equal(ms[0].view(torch.int32), ms[1].view(torch.int32))
    for k in range(2):
        assert torch.equal(votes_dev[k].cpu(), vote_host[k]), "voted words of call %d" % k
    assert np.all(u32(vs[1])[W:] == np.uint32(0xDEADBEEF)) and np.all(f32(xs[1])[d:] == np.float32(CANARY_F))
    assert np.all(u32(bs[1])[:, W:] == np.uint32(0xDEADBEEF))


def test_resume_from_copied_state_is_bit_identical():
    cfg = wl.small_signum(d=50_000, M=3)
    M, d, ld, ldw, W = cfg.M, cfg.d, cfg.ld, cfg.ldw, cfg.words
    mu = cfg.shared(DEV)
    gs = [cfg.g(k, DEV, mu) for k in range(5)]
    bits = torch.zeros(M, ldw, dtype=torch.int32, device=DEV)
    vote = torch.zeros(W, dtype=torch.int32, device=DEV)
    xa, ma = cfg.x0(DEV), cfg.m0(DEV)
    for k in range(5):
        B.signsgd_step(xa, gs[k], ma, M, d, ld, cfg.beta, cfg.delta, bits, ldw, vote)
    xb, mb = cfg.x0(DEV), cfg.m0(DEV)
    for k in range(2):
        B.signsgd_step(xb, gs[k], mb, M, d, ld, cfg.beta, cfg.delta, bits, ldw, vote)
    xb, mb = xb.cpu().to(DEV), mb.cpu().to(DEV)             # state leaves and re-enters the device
    for k in range(2, 5):
        B.signsgd_step(xb, gs[k], mb, M, d, ld, cfg.beta, cfg.delta, bits, ldw, vote)
    assert torch.equal(xa, xb) and torch.equal(ma, mb)


@pytest.mark.parametrize("M,d", [(12, 600_007), (16, 3_000_017), (9, 20_011), (5, 300_001)])
def test_step_on_a_side_stream_beside_other_work(M, d):
    """The step on a stream of its own while the default stream is busy with unrelated kernels: its kernels
    (vote and apply are programmatic dependents of the kernel before them on THAT stream) must order among
    themselves alone.  Several steps back to back, then one comparison with the oracle."""
    ld, W = wl.round_up(d, 4), oracle.words(d)
    ldw = wl.round_up(W, 4)
    steps = 3
    gs = [big_inputs(M, d, ld, seed=100 * k + M)[0] for k in range(steps)]
    _, m, x = big_inputs(M, d, ld, seed=M + 17)
    gd = [torch.from_numpy(g).to(DEV) for g in gs]
    md, xd = torch.from_numpy(m).to(DEV), torch.from_numpy(x[:d].copy()).to(DEV)
    bits = torch.zeros(M, ldw, dtype=torch.int32, device=DEV)
    vote = torch.zeros(W, dtype=torch.int32, device=DEV)
    between, beside = torch.randn(1 << 22, device=DEV), torch.randn(1 << 24, device=DEV)
    side = torch.cuda.Stream(device=DEV)
    torch.cuda.synchronize()
    with torch.cuda.stream(side):
        for k in range(steps):
            between.mul_(1.0001)                    # a foreign kernel on the side stream between two steps
            B.signsgd_step(xd, gd[k], md, M, d, ld, 0.9, 1e-3, bits, ldw, vote, side)
    for _ in range(20):
        beside.add_(1.0)                            # the default stream, unordered with the side stream
    torch.cuda.synchronize()
    m_ref, x_ref = m.copy().reshape(-1), x[:d].copy()
    for k in range(steps):
        b_ref, v_ref = oracle.signsgd_step(x_ref, gs[k].reshape(-1), m_ref, M, d, 0.9, 1e-3, ld=ld, ldw=ldw)
    assert np.array_equal(u32(bits).reshape(-1), b_ref)
    assert np.array_equal(u32(vote), v_ref)
    assert_same_f32(f32(xd), x_ref, "x")
    assert_same_f32(f32(md).reshape(-1), m_ref, "m")


@pytest.mark.parametrize("M,d", [(5, 300_001), (12, 600_007)])
def test_step_replayed_from_a_cuda_graph(M, d):
    """The step entry point allocates nothing and never synchronises, so a caller can capture it into a CUDA
    graph (one fused kernel for M = 5; worker + tail + vote + apply launches for M = 12) and replay it."""
    cfg = wl.small_signum(d=d, M=M)
    ld, ldw, W = cfg.ld, cfg.ldw, cfg.words
    mu = cfg.shared(DEV)
    xd, md = cfg.x0(DEV), cfg.m0(DEV)
    gd = cfg.g(0, DEV, mu)
    bits = torch.zeros(M, ldw, dtype=torch.int32, device=DEV)
    vote = torch.zeros(W, dtype=torch.int32, device=DEV)
    x_ref, m_ref = f32(xd).copy(), f32(md).reshape(-1).copy()
    B.signsgd_step(xd.clone(), gd, md.clone(), M, d, ld, cfg.beta, cfg.delta, bits, ldw, vote)   # warm-up outside the capture
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        B.signsgd_step(xd, gd, md, M, d, ld, cfg.beta, cfg.delta, bits, ldw, vote)
    for k in range(3):                                   # three replays = three steps on fresh gradients
        gd.copy_(cfg.g(k, DEV, mu))
        graph.replay()
        torch.cuda.synchronize()
        b_ref, v_ref = oracle.signsgd_step(x_ref, f32(gd).reshape(-1), m_ref, M, d, cfg.beta, cfg.delta, ld=ld, ldw=ldw)
        assert np.array_equal(u32(bits).reshape(-1), b_ref) and np.array_equal(u32(vote), v_ref)
        assert_same_f32(f32(xd), x_ref, "x, replay %d" % k)
        assert_same_f32(f32(md).reshape(-1), m_ref, "m, replay %d" % k)


# ------------------------------------------------------------------ Theorem 3 warm-up

def test_warmup_length_matches_oracle():
    for beta in (0.0, 0.3, 0.5, 0.8, 0.9, 0.95, 0.99, 0.999):
        assert B.warmup_steps(beta) == oracle.warmup_steps(beta)
    assert B.warmup_steps(0.9) == 54
    assert B.warmup_steps(1.0) == 0 and B.warmup_steps(float("nan")) == 0


@pytest.mark.parametrize("M,d", [(1, 1000), (3, 4097), (7, 100003), (8, 1 << 20), (16, 70001), (33, 5000)])
def test_warmup_pack_and_step(M, d):
    ld, W = wl.round_up(d, 4), oracle.words(d)
    ldw = wl.round_up(W, 4)
    g, m, x = rand_inputs(M, d, ld, seed=M + d, special=True)
    with np.errstate(over="ignore"):
        m *= 3.0
    gd, md = torch.from_numpy(g).to(DEV), torch.from_numpy(m).to(DEV)
    bits = torch.zeros(M, ldw, dtype=torch.int32, device=DEV)
    B.signum_warmup_pack(gd, md, M, d, ld, 0.9, bits, ldw)
    m_ref = m.copy().reshape(-1)
    b_ref = oracle.signum_warmup_pack(g.reshape(-1), m_ref, M, d, 0.9, ld=ld, ldw=ldw)
    assert np.array_equal(u32(bits).reshape(-1), b_ref)
    assert_same_f32(f32(md).reshape(-1), m_ref, "m")
    # whole step
    md, xd = torch.from_numpy(m).to(DEV), torch.from_numpy(x).to(DEV)
    vote = torch.zeros(W, dtype=torch.int32, device=DEV)
    B.signsgd_warmup_step(xd, gd, md, M, d, ld, 0.9, 1e-3, bits, ldw, vote)
    m_ref, x_ref = m.copy().reshape(-1), x.copy()
    b_ref, v_ref = oracle.signsgd_warmup_step(x_ref, g.reshape(-1), m_ref, M, d, 0.9, 1e-3, ld=ld, ldw=ldw)
    assert np.array_equal(u32(bits).reshape(-1), b_ref) and np.array_equal(u32(vote), v_ref)
    assert_same_f32(f32(xd), x_ref, "x")
    assert_same_f32(f32(md).reshape(-1), m_ref, "m")


def test_warmup_then_signum_schedule():
    """Theorem 3's schedule on the small workload: warm-up steps first, Signum steps after."""
    cfg = wl.small_signum(d=100_000, M=3)
    M, d, ld, ldw, W = cfg.M, cfg.d, cfg.ld, cfg.ldw, cfg.words
    mu = cfg.shared(DEV)
    xd, md = cfg.x0(DEV), cfg.m0(DEV)
    x_ref, m_ref = f32(xd).copy(), f32(md).reshape(-1).copy()
    bits = torch.zeros(M, ldw, dtype=torch.int32, device=DEV)
    vote = torch.zeros(W, dtype=torch.int32, device=DEV)
    C = 3                                      # a short warm-up keeps the test fast
    for k in range(6):
        gd = cfg.g(k, DEV, mu)
        gh = f32(gd).reshape(-1)
        if k < C:
            B.signsgd_warmup_step(xd, gd, md, M, d, ld, cfg.beta, cfg.delta, bits, ldw, vote)
            b_ref, v_ref = oracle.signsgd_warmup_step(x_ref, gh, m_ref, M, d, cfg.beta, cfg.delta, ld=ld, ldw=ldw)
        else:
            B.signsgd_step(xd, gd, md, M, d, ld, cfg.beta, cfg.delta, bits, ldw, vote)
            b_ref, v_ref = oracle.signsgd_step(x_ref, gh, m_ref, M, d, cfg.beta, cfg.delta, ld=ld, ldw=ldw)
        assert np.array_equal(u32(bits).reshape(-1), b_ref) and np.array_equal(u32(vote), v_ref)
        assert_same_f32(f32(xd), x_ref, "x step %d" % k)
        assert_same_f32(f32(md).reshape(-1), m_ref, "m step %d" % k)


# ------------------------------------------------------------------ the "(good)" scheme of Sec. 4

@pytest.mark.parametrize("M", [1, 2, 3, 7, 8, 15, 16, 31, 33, 255, 1024])
def test_vote_counts_and_sum_apply(M):
    for d in (1, 33, 1000, 4097, 100003 if M <= 33 else 5000):
        r = np.random.default_rng(M * 7 + d)
        W = oracle.words(d)
        ldw, ldc = wl.round_up(W, 4), wl.round_up(W, 4) + 4
        NPc = M.bit_length()
        assert B.count_planes(M) == NPc
        s = (r.random((M, d)) < r.random(d)).astype(np.uint8)
        rows = np.zeros((M, ldw), dtype=np.uint32)
        for w in range(M):
            rows[w, :W] = oracle.pack_bits(s[w])
        counts = torch.full((NPc, ldc), CANARY_WORD, dtype=torch.int32, device=DEV)
        B.vote_counts(torch.from_numpy(rows.view(np.int32)).to(DEV), M, d, ldw, counts, ldc)
        ref = oracle.vote_count_planes(rows.reshape(-1), M, d, ldw=ldw, ldc=ldc).reshape(NPc, ldc)
        got = u32(counts)
        assert np.array_equal(got[:, :W], ref[:, :W]), "M=%d d=%d" % (M, d)
        assert np.all(got[:, W:] == np.uint32(0xDEADBEEF))
        x = np.full(d + 5, CANARY_F, dtype=np.float32)
        x[:d] = (r.standard_normal(d) * 10.0 ** r.integers(-4, 2, d)).astype(np.float32)
        xd = torch.from_numpy(x).to(DEV)
        clean = counts.clone()
        clean[:, W:] = 0
        B.sum_apply(xd, clean, M, d, ldc, 2e-3)
        x_ref = x[:d].copy()
        oracle.sum_apply(x_ref, ref.reshape(-1).copy(), M, d, 2e-3, ldc=ldc)
        gx = f32(xd)
        assert_same_f32(gx[:d], x_ref, "x (M=%d d=%d)" % (M, d))
        assert np.all(gx[d:] == np.float32(CANARY_F))


@pytest.mark.parametrize("seed", range(32))
def test_vote_and_count_planes_random_shapes(seed):
    """Seeded random worker counts (1 .. 1024, every kernel form: one row, 2 .. 7 rows, guarded and plain tails,
    up to eleven planes), lengths and row strides; random words with garbage in the row padding; vote and count
    planes against the oracle, canaries behind both outputs."""
    r = np.random.default_rng(7000 + seed)
    M = int(r.choice([1, 2, 3, 4, 5, 6, 7, 8, 9, 13, 16, 31, 32, 63, 64, 127, 128, 300, 1024])) if seed % 2 else int(r.integers(1, 130))
    d = int(10 ** r.uniform(0.0, 5.3 if M <= 130 else 4.0))
    W = oracle.words(d)
    ldw, ldc = wl.round_up(W, 4) + 4 * int(r.integers(0, 3)), wl.round_up(W, 4) + 4 * int(r.integers(0, 3))
    rows = r.integers(0, 2**32, size=(M, ldw), dtype=np.uint32)
    rows[:, W - 1] &= np.uint32((1 << (d - 32 * (W - 1))) - 1 if d % 32 else 0xFFFFFFFF)   # pad bits 0, as the pack calls write them
    bd = torch.from_numpy(rows.view(np.int32)).to(DEV)
    vote = torch.full((W + 4,), CANARY_WORD, dtype=torch.int32, device=DEV)
    B.majority_vote(bd, M, d, ldw, vote)
    ref = oracle.majority_vote(rows.reshape(-1), M, d, ldw=ldw)
    assert np.array_equal(u32(vote)[:W], ref), "vote seed=%d M=%d d=%d" % (seed, M, d)
    assert np.all(u32(vote)[W:] == np.uint32(0xDEADBEEF))
    NPc = M.bit_length()
    counts = torch.full((NPc, ldc), CANARY_WORD, dtype=torch.int32, device=DEV)
    B.vote_counts(bd, M, d, ldw, counts, ldc)
    cref = oracle.vote_count_planes(rows.reshape(-1), M, d, ldw=ldw, ldc=ldc).reshape(NPc, ldc)
    got = u32(counts)
    assert np.array_equal(got[:, :W], cref[:, :W]), "counts seed=%d M=%d d=%d" % (seed, M, d)
    assert np.all(got[:, W:] == np.uint32(0xDEADBEEF))


# ------------------------------------------------------------------ majority vote with abstention

@pytest.mark.parametrize("M", [1, 2, 3, 7, 8, 16, 33, 255, 1024])
def test_abstention_path(M):
    for d in (1, 33, 1000, 4097, 70001 if M <= 33 else 3000):
        ld, W = wl.round_up(d, 4), oracle.words(d)
        ldw = wl.round_up(W, 4)
        g, m, x = rand_inputs(M, d, ld, seed=M * 13 + d, special=True)
        for beta, with_m, tau, Q in ((0.9, True, 0.05, 2), (0.0, False, 0.3, 0), (0.9, True, 0.0, 0), (0.0, False, 1.0, M // 2 + 1)):
            gd, xd = torch.from_numpy(g).to(DEV), torch.from_numpy(x).to(DEV)
            md = torch.from_numpy(m).to(DEV) if with_m else None
            sb = torch.full((M, ldw), CANARY_WORD, dtype=torch.int32, device=DEV)
            ab = torch.full((M, ldw), CANARY_WORD, dtype=torch.int32, device=DEV)
            B.ternary_pack(gd, md, M, d, ld, beta, tau, sb, ab, ldw)
            m_ref = m.copy().reshape(-1) if with_m else None
            sb_ref, ab_ref = oracle.ternary_pack(g.reshape(-1), m_ref, M, d, beta, tau, ld=ld, ldw=ldw)
            got_s, got_a = u32(sb), u32(ab)
            assert np.array_equal(got_s[:, :W], sb_ref.reshape(M, ldw)[:, :W])
            assert np.array_equal(got_a[:, :W], ab_ref.reshape(M, ldw)[:, :W])
            assert np.all(got_s[:, W:] == np.uint32(0xDEADBEEF)) and np.all(got_a[:, W:] == np.uint32(0xDEADBEEF))
            if with_m:
                assert_same_f32(f32(md).reshape(-1), m_ref, "m")
            sb[:, W:] = 0
            ab[:, W:] = 0
            vs = torch.full((W + 4,), CANARY_WORD, dtype=torch.int32, device=DEV)
            va = torch.full((W + 4,), CANARY_WORD, dtype=torch.int32, device=DEV)
            B.quorum_vote(sb, ab, M, d, ldw, Q, vs, va)
            vs_ref, va_ref = oracle.quorum_vote(u32(sb).reshape(-1).copy(), u32(ab).reshape(-1).copy(), M, d, Q, ldw=ldw)
            assert np.array_equal(u32(vs)[:W], vs_ref) and np.array_equal(u32(va)[:W], va_ref), (M, d, Q)
            assert np.all(u32(vs)[W:] == np.uint32(0xDEADBEEF)) and np.all(u32(va)[W:] == np.uint32(0xDEADBEEF))
            B.ternary_apply(xd, vs, va, d, 1e-3)
            x_ref = x.copy()
            oracle.ternary_apply(x_ref, vs_ref, va_ref, d, 1e-3)
            assert_same_f32(f32(xd), x_ref, "x")


@pytest.mark.parametrize("M,d,with_m", [(8, 1_000_003, True), (3, 2_500_003, False)])
def test_abstention_path_large_odd_d(M, d, with_m):
    # large enough for the interior-only ternary pack kernel and its tail launch; rows longer than d
    ld, W = wl.round_up(d, 4) + 8, oracle.words(d)
    ldw = wl.round_up(W, 4) + 4
    g, m, x = big_inputs(M, d, ld, seed=M * 17 + d % 1000, with_m=with_m)
    beta, tau, Q = (0.9, 0.2, 2) if with_m else (0.0, 0.5, 1)
    gd, xd = torch.from_numpy(g).to(DEV), torch.from_numpy(x).to(DEV)
    md = torch.from_numpy(m).to(DEV) if with_m else None
    sb = torch.full((M, ldw), CANARY_WORD, dtype=torch.int32, device=DEV)
    ab = torch.full((M, ldw), CANARY_WORD, dtype=torch.int32, device=DEV)
    B.ternary_pack(gd, md, M, d, ld, beta, tau, sb, ab, ldw)
    m_ref = m.copy().reshape(-1) if with_m else None
    sb_ref, ab_ref = oracle.ternary_pack(g.reshape(-1), m_ref, M, d, beta, tau, ld=ld, ldw=ldw)
    check_rows(sb, sb_ref, M, ldw, W, "sign plane")
    check_rows(ab, ab_ref, M, ldw, W, "active plane")
    if with_m:
        gm = f32(md)
        assert_same_f32(gm.reshape(-1), m_ref, "m")
        assert np.array_equal(gm[:, d:].view(np.uint32), m[:, d:].view(np.uint32))
    sb[:, W:] = 0
    ab[:, W:] = 0
    vs = torch.full((W + 4,), CANARY_WORD, dtype=torch.int32, device=DEV)
    va = torch.full((W + 4,), CANARY_WORD, dtype=torch.int32, device=DEV)
    B.quorum_vote(sb, ab, M, d, ldw, Q, vs, va)
    vs_ref, va_ref = oracle.quorum_vote(u32(sb).reshape(-1).copy(), u32(ab).reshape(-1).copy(), M, d, Q, ldw=ldw)
    assert np.array_equal(u32(vs)[:W], vs_ref) and np.array_equal(u32(va)[:W], va_ref)
    B.ternary_apply(xd, vs, va, d, 1e-3)
    x_ref = x[:d].copy()
    oracle.ternary_apply(x_ref, vs_ref, va_ref, d, 1e-3)
    gx = f32(xd)
    assert_same_f32(gx[:d], x_ref, "x")
    assert np.all(gx[d:] == np.float32(CANARY_F))


# ------------------------------------------------------------------ Section 3: density and Welford

@pytest.mark.parametrize("d", [1, 3, 1000, 4099, 1 << 20, (1 << 22) + 5])
def test_welford_and_density(d):
    r = np.random.default_rng(d)
    n = 5
    g = (0.3 + r.standard_normal((n, d))).astype(np.float32)
    mean_d = torch.zeros(d, device=DEV)
    m2_d = torch.zeros(d, device=DEV)
    mean, m2 = np.zeros(d, dtype=np.float32), np.zeros(d, dtype=np.float32)
    for k in range(n):
        B.welford_update(torch.from_numpy(g[k]).to(DEV), k + 1, mean_d, m2_d, d)
        oracle.welford_update(g[k], k + 1, mean, m2)
    assert_same_f32(f32(mean_d), mean, "mean")
    assert_same_f32(f32(m2_d), m2, "m2")
    # the density is an fp64 sum of exactly representable terms in a different order than the
    # oracle's: relative error is bounded by d * 2^-53, far inside 1e-11
    phi_ref, l1, l2 = oracle.density(mean)
    phi = B.density(mean_d, d)
    assert abs(phi - phi_ref) <= 1e-11 * max(phi_ref, 1e-300)
    # the noise density phi(sigma) from the variances: the root form, against the oracle's
    phi_s_ref, _, l2s = oracle.density_of_root(m2)
    phi_s = B.density(m2_d, d, root=True)
    assert abs(phi_s - phi_s_ref) <= 1e-11 * phi_s_ref if l2s > 0 else phi_s == 0.0


def test_density_of_dense_and_one_hot_vectors_gpu():
    d = 1 << 20
    dense = torch.full((d,), -0.75, device=DEV)
    assert abs(B.density(dense, d) - 1.0) < 1e-12
    one_hot = torch.zeros(d, device=DEV)
    one_hot[12345] = 4.0
    assert abs(B.density(one_hot, d) - 1.0 / d) < 1e-18
    assert B.density(torch.zeros(8, device=DEV), 8) == 0.0
    # the same end points for a vector of variances through the root form
    assert abs(B.density(torch.full((d,), 6.25, device=DEV), d, root=True) - 1.0) < 1e-12
    assert abs(B.density(one_hot, d, root=True) - 1.0 / d) < 1e-18
