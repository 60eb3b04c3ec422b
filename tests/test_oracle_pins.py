"""Pins for the CPU oracle: everything here checks ``oracle/`` against something
other than itself -- brute force written in Python integers, exact rational
arithmetic, closed forms in extended precision, bitwise identities, the bounds
and the worked numbers printed in the paper (tests/golden/paper_values.txt).
"""
import itertools
import math
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle
from exact import f32_to_fraction, round_f32, ulp_distance

GOLDEN = {}
with open(os.path.join(os.path.dirname(__file__), "golden", "paper_values.txt")) as fh:
    for line in fh:
        line = line.strip()
        if line and not line.startswith("#"):
            k, v = [t.strip() for t in line.split("=")]
            GOLDEN[k] = float(v)


def rng(seed):
    return np.random.default_rng(seed)


def py_pack(bits):
    """Packing written with a Python big integer: bit i of the integer = element i."""
    n = 0
    for i, b in enumerate(bits):
        if b:
            n |= 1 << i
    W = (len(bits) + 31) // 32
    return [(n >> (32 * j)) & 0xFFFFFFFF for j in range(W)]


# ---------------------------------------------------------------- sign + packing

def test_sign_rule_special_values():
    # sign(0) -> +1, -0.0 -> +1, NaN -> +1, infinities and denormals by their sign.
    v = np.array([0.0, -0.0, np.nan, np.inf, -np.inf, 1e-45, -1e-45, 1.0, -1.0,
                  np.float32(-1.17549435e-38), np.float32(3.4e38)], dtype=np.float32)
    expect = [1, 1, 1, 1, 0, 1, 0, 1, 0, 0, 1]
    assert oracle.sign_unpacked(v).tolist() == expect


def test_words_is_ceil_d_over_32():
    for d in list(range(0, 200)) + [2**24 - 1, 2**24, 2**24 + 1, 335_141_888]:
        assert oracle.words(d) == -(-d // 32)


@pytest.mark.parametrize("d", list(range(0, 131)))
def test_pack_every_length_against_bigint(d):
    r = rng(d)
    s = r.integers(0, 2, size=d, dtype=np.uint8)
    w = oracle.pack_bits(s)
    assert w.tolist() == py_pack(s.tolist())
    # padding bits of the last word are zero, round trip is the identity
    if d % 32:
        assert int(w[-1]) >> (d % 32) == 0
    assert oracle.unpack_bits(w, d).tolist() == s.tolist()


def test_pack_bit_order_is_lsb_first():
    for i in (0, 1, 31, 32, 33, 63, 64, 95):
        s = np.zeros(96, dtype=np.uint8)
        s[i] = 1
        w = oracle.pack_bits(s)
        expect = [0, 0, 0]
        expect[i // 32] = 1 << (i % 32)
        assert w.tolist() == expect


def test_popcount_equals_number_of_nonnegative_entries():
    r = rng(7)
    M, d = 5, 1003
    g = r.standard_normal((M, d)).astype(np.float32)
    g[r.random((M, d)) < 0.05] = 0.0
    bits = oracle.sign_pack(g.reshape(-1).copy(), M, d, ld=d).reshape(M, -1)
    for w in range(M):
        pop = sum(bin(int(v)).count("1") for v in bits[w])
        assert pop == int(np.count_nonzero(~(g[w] < 0)))


def test_row_strides_and_padding_untouched():
    r = rng(11)
    M, d, ld, ldw = 3, 70, 76, 8
    g = r.standard_normal((M, ld)).astype(np.float32)
    m = r.standard_normal((M, ld)).astype(np.float32)
    m_before = m.copy()
    bits = oracle.signum_momentum_pack(g.reshape(-1), m.reshape(-1), M, d, 0.9, ld=ld, ldw=ldw)
    bits = bits.reshape(M, ldw)
    assert np.array_equal(m[:, d:], m_before[:, d:])          # beyond d: not written
    assert not np.array_equal(m[:, :d], m_before[:, :d])
    assert np.all(bits[:, 3:] == 0)                           # W = 3 words per row
    for w in range(M):
        assert bits[w, :3].tolist() == py_pack((~(m[w, :d] < 0)).tolist())


# ---------------------------------------------------------------- majority vote

@pytest.mark.parametrize("M", list(range(1, 13)))
def test_vote_truth_table_all_patterns(M):
    """Every one of the 2^M vote patterns: the decoder of the repetition code R_M
    (Sec. 2; proof of Theorem 2) with the tie rule -> +1."""
    d = 2 ** M
    rows = []
    for w in range(M):
        rows.append(py_pack([(e >> w) & 1 for e in range(d)]))
    W = len(rows[0])
    bits = np.array(rows, dtype=np.uint32).reshape(-1)
    vote = oracle.majority_vote(bits, M, d, ldw=W)
    counts = oracle.vote_counts(bits, M, d, ldw=W)
    exp_counts = [bin(e).count("1") for e in range(d)]
    assert counts.tolist() == exp_counts
    # Algorithm 3 literally: sign of the sum of +-1 votes, sign(0) = +1
    exp = []
    for e in range(d):
        total = sum(1 if (e >> w) & 1 else -1 for w in range(M))
        exp.append(1 if total >= 0 else 0)
    assert vote.tolist() == py_pack(exp)
    # threshold form: P >= ceil(M/2)
    assert exp == [1 if p >= (M + 1) // 2 else 0 for p in exp_counts]


def test_vote_M3_is_bitwise_majority():
    r = rng(3)
    W = 257
    a, b, c = (r.integers(0, 2**32, size=W, dtype=np.uint32) for _ in range(3))
    bits = np.concatenate([a, b, c])
    vote = oracle.majority_vote(bits, 3, W * 32, ldw=W)
    assert np.array_equal(vote, (a & b) | (a & c) | (b & c))


def test_vote_M1_is_the_vector_itself_and_matches_sign_of_g():
    r = rng(4)
    d = 1000
    g = r.standard_normal(d).astype(np.float32)
    bits = oracle.sign_pack(g, 1, d)
    vote = oracle.majority_vote(bits, 1, d)
    assert np.array_equal(vote, bits)
    assert oracle.unpack_bits(vote, d).tolist() == (~(g < 0)).astype(int).tolist()


def test_vote_M2_tie_goes_positive():
    # one worker says +, the other -: sum of signs is 0 -> +1
    bits = np.array([0b01, 0b10], dtype=np.uint32)
    vote = oracle.majority_vote(bits, 2, 2, ldw=1)
    assert vote.tolist() == [0b11]
    bits = np.array([0b00, 0b10], dtype=np.uint32)
    assert oracle.majority_vote(bits, 2, 2, ldw=1).tolist() == [0b10]


@pytest.mark.parametrize("M", [2, 3, 4, 7, 8, 15, 16, 31, 32, 33, 100])
def test_vote_invariant_to_worker_permutation(M):
    r = rng(M)
    d = 777
    g = r.standard_normal((M, d)).astype(np.float32)
    bits = oracle.sign_pack(g.reshape(-1).copy(), M, d)
    perm = r.permutation(M)
    bits_p = oracle.sign_pack(g[perm].reshape(-1).copy(), M, d)
    assert np.array_equal(oracle.majority_vote(bits, M, d), oracle.majority_vote(bits_p, M, d))


@pytest.mark.parametrize("M", [1, 3, 4, 7, 8, 16])
def test_negating_all_gradients_negates_vote_away_from_zeros_and_ties(M):
    r = rng(100 + M)
    d = 2000
    g = r.standard_normal((M, d)).astype(np.float32)
    g[r.random((M, d)) < 0.03] = 0.0
    v_pos = oracle.unpack_bits(oracle.majority_vote(oracle.sign_pack(g.reshape(-1).copy(), M, d), M, d), d)
    v_neg = oracle.unpack_bits(oracle.majority_vote(oracle.sign_pack((-g).reshape(-1).copy(), M, d), M, d), d)
    P = np.count_nonzero(g > 0, axis=0)
    clean = np.all(g != 0, axis=0) & (2 * P != M)
    assert clean.sum() > d // 4
    assert np.array_equal(v_pos[clean], 1 - v_neg[clean])
    # and at a clean element the vote is the sign of the integer sum of signs
    assert np.array_equal(v_pos[clean], (np.sign(g).sum(axis=0)[clean] > 0).astype(np.uint8))


def test_vote_large_M_against_numpy_counts():
    r = rng(9)
    for M in (64, 255, 256, 1000, 1024):
        d = 333
        s = r.integers(0, 2, size=(M, d), dtype=np.uint8)
        bits = np.concatenate([np.array(py_pack(row.tolist()), dtype=np.uint32) for row in s])
        vote = oracle.unpack_bits(oracle.majority_vote(bits, M, d), d)
        assert np.array_equal(vote, (2 * s.sum(axis=0, dtype=np.int64) >= M).astype(np.uint8))


def test_remark3_skewed_law_drives_vote_to_wrong_sign():
    """Remark 3 of Sec. 4: X = 50 w.p. 0.1, -1 w.p. 0.9 has positive mean, yet a
    majority over more workers picks the negative sign more and more often."""
    hi, plo = GOLDEN["remark3_value_hi"], GOLDEN["remark3_prob_lo"]
    lo = GOLDEN["remark3_value_lo"]
    assert GOLDEN["remark3_prob_hi"] * hi + plo * lo > 0
    r = rng(33)
    d = 20000
    frac_neg = []
    for M in (1, 5, 25):
        g = np.where(r.random((M, d)) < plo, lo, hi).astype(np.float32)
        v = oracle.unpack_bits(oracle.majority_vote(oracle.sign_pack(g.reshape(-1).copy(), M, d), M, d), d)
        frac_neg.append(1.0 - v.mean())
    assert abs(frac_neg[0] - 0.9) < 0.02
    assert frac_neg[0] < frac_neg[1] < frac_neg[2] and frac_neg[2] > 0.999


def test_gaussian_sign_error_under_lemma1_and_vote_error_under_eq_section():
    """Lemma 1: per-worker sign failure q <= q~(S); proof of Theorem 2(b):
    P[vote wrong] <= 1 / (sqrt(M) S).  Checked on Gaussian noise (unimodal, symmetric)."""
    r = rng(5)
    d = 200_000
    for S in (0.25, 0.5, 1.0, 1.5, 2.5):
        mu = -S  # true gradient negative, sigma = 1
        if S > GOLDEN["lemma1_switch_S"]:
            qb = GOLDEN["lemma1_tail_coeff"] / S**2
        else:
            qb = 0.5 - S * GOLDEN["lemma1_slope"]
        for M in (1, 3, 7, 15):
            g = (mu + r.standard_normal((M, d))).astype(np.float32)
            bits = oracle.sign_pack(g.reshape(-1).copy(), M, d).reshape(M, -1)
            q_emp = np.mean([oracle.unpack_bits(bits[w], d).mean() for w in range(M)])
            exact_q = 0.5 * math.erfc(S / math.sqrt(2))
            assert abs(q_emp - exact_q) < 5 * math.sqrt(exact_q / (M * d)) + 1e-4
            assert q_emp <= qb
            vote_err = oracle.unpack_bits(oracle.majority_vote(bits.reshape(-1), M, d), d).mean()
            assert vote_err <= 1.0 / (math.sqrt(M) * S)
            # exact binomial tail for odd M: the vote really is a majority
            k0 = (M + 1) // 2
            tail = sum(math.comb(M, k) * exact_q**k * (1 - exact_q)**(M - k) for k in range(k0, M + 1))
            assert abs(vote_err - tail) < 5 * math.sqrt(tail / d) + 1e-4


def test_table1_wire_size():
    # d bits up and d bits down per worker: 2*M*d bits per iteration (Table 1).
    for M, d in ((3, 1_000_000), (7, 25_557_056), (16, 335_141_888)):
        W = oracle.words(d)
        assert d % 32 == 0
        up_bits = M * W * 32
        down_bits = M * W * 32          # the same W-word vote goes to each of M workers
        assert up_bits + down_bits == GOLDEN["table1_signsgd_vote_bits_per_Md"] * M * d
        assert 2 * 32 * M * d == GOLDEN["table1_sgd_bits_per_Md"] * M * d


# ---------------------------------------------------------------- momentum

def test_momentum_is_two_correctly_rounded_operations():
    """m_new = RN( beta*m + RN((1-beta)*g) ), checked in exact rational arithmetic,
    including elements built to cancel almost completely."""
    r = rng(21)
    for beta in (0.9, 0.99, 0.5, 0.123, 0.0):
        beta32 = np.float32(beta)
        omb = round_f32(Fraction(1) - f32_to_fraction(beta32))
        n = 400
        g = (r.standard_normal(n) * 10.0 ** r.integers(-6, 3, n)).astype(np.float32)
        m = (r.standard_normal(n) * 10.0 ** r.integers(-6, 3, n)).astype(np.float32)
        if beta > 0:
            # near-cancellation: m ~ -(1-beta) g / beta, perturbed by a few ulp
            k = n // 2
            mc = (-(np.float64(omb) * g[:k].astype(np.float64)) / np.float64(beta32)).astype(np.float32)
            m[:k] = np.nextafter(mc, np.float32(np.inf) * r.choice([-1, 1], k).astype(np.float32))
        g[0], m[0] = np.float32(1e-40), np.float32(-1e-41)          # subnormals
        expect = []
        for gi, mi in zip(g.tolist(), m.tolist()):
            t = round_f32(Fraction(omb) * Fraction(gi))
            expect.append(round_f32(f32_to_fraction(beta32) * Fraction(mi) + Fraction(t)))
        got = m.copy()
        oracle.momentum(g, got, float(beta32))
        assert got.tolist() == expect


def test_constant_gradient_closed_form():
    # m_0 = 0, constant g: m_K = (1 - beta^K) g  (bias-corrected form, Sec. on Signum analysis)
    r = rng(22)
    d, K, beta = 500, 60, np.float32(0.9)
    g = r.standard_normal(d).astype(np.float32)
    m = np.zeros(d, dtype=np.float32)
    for _ in range(K):
        oracle.momentum(g, m, float(beta))
    ref = (1.0 - np.longdouble(beta) ** K) * g.astype(np.longdouble)
    assert np.all(np.abs(m.astype(np.longdouble) - ref) <= 4e-7 * np.abs(ref))


def test_general_gradient_ema_closed_form_and_sign_of_bias_corrected_momentum():
    # m_K = (1-beta) sum_t beta^t g_{K-1-t}; the paper's analysis form divides by
    # (1 - beta^K) > 0, which cannot change the sign.
    r = rng(23)
    d, K, beta = 300, 40, np.float32(0.9)
    gs = r.standard_normal((K, d)).astype(np.float32)
    m = np.zeros(d, dtype=np.float32)
    for k in range(K):
        oracle.momentum(gs[k], m, float(beta))
    b = np.longdouble(beta)
    omb = np.longdouble(np.float32(1.0) - beta)
    ref = sum(omb * b ** t * gs[K - 1 - t].astype(np.longdouble) for t in range(K))
    scale = sum(omb * b ** t * np.abs(gs[K - 1 - t]).astype(np.longdouble) for t in range(K))
    assert np.all(np.abs(m.astype(np.longdouble) - ref) <= 3e-7 * scale)
    safe = np.abs(ref) > 1e-5 * scale
    bias_corrected = ref / (1 - b ** K)
    s = oracle.sign_unpacked(m)
    assert np.array_equal(s[safe], (bias_corrected[safe] > 0).astype(np.uint8))


def test_signum_with_beta_zero_is_signsgd():
    r = rng(24)
    M, d = 4, 999
    g = r.standard_normal((M, d)).astype(np.float32)
    g[r.random((M, d)) < 0.02] = 0.0
    m = r.standard_normal((M, d)).astype(np.float32)
    flat_g = g.reshape(-1).copy()
    flat_m = m.reshape(-1).copy()
    b_signum = oracle.signum_momentum_pack(flat_g, flat_m, M, d, 0.0)
    b_sign = oracle.sign_pack(flat_g, M, d)
    assert np.array_equal(b_signum, b_sign)
    assert np.array_equal(flat_m, flat_g)


def test_sign_is_taken_after_the_momentum_update():
    # m = +1, g very negative: old momentum positive, new momentum negative.
    g = np.array([-100.0], dtype=np.float32)
    m = np.array([1.0], dtype=np.float32)
    bits = oracle.signum_momentum_pack(g, m, 1, 1, 0.9)
    assert m[0] < 0 and bits.tolist() == [0]


# ---------------------------------------------------------------- apply + whole step

def test_sign_apply_is_one_correctly_rounded_add_per_element():
    r = rng(31)
    d = 777
    x = (r.standard_normal(d) * 10.0 ** r.integers(-8, 4, d)).astype(np.float32)
    s = r.integers(0, 2, size=d, dtype=np.uint8)
    vote = np.array(py_pack(s.tolist()), dtype=np.uint32)
    for delta in (1e-4, 1e-3, 0.5):
        d32 = np.float32(delta)
        got = x.copy()
        oracle.sign_apply(got, vote, d, float(d32))
        expect = [round_f32(Fraction(xi) - Fraction(float(d32)) if si else Fraction(xi) + Fraction(float(d32)))
                  for xi, si in zip(x.tolist(), s.tolist())]
        assert got.tolist() == expect
        # every coordinate moves by delta up to one rounding (l-infinity steepest descent)
        big = np.abs(x) < 1.0
        assert np.all(np.abs(np.abs(got[big].astype(np.float64) - x[big]) - float(d32)) <= 2.0 ** -24)


def test_sign_apply_leaves_elements_beyond_d_alone():
    x = np.arange(40, dtype=np.float32)
    vote = np.array([0xFFFFFFFF, 0xFFFFFFFF], dtype=np.uint32)
    oracle.sign_apply(x, vote, 33, 0.5)
    assert np.array_equal(x[33:], np.arange(33, 40, dtype=np.float32))
    assert np.array_equal(x[:33], np.arange(33, dtype=np.float32) - 0.5)


def test_constant_vote_walks_x_by_K_delta():
    d, K, delta = 64, 100, np.float32(1e-3)
    x0 = np.linspace(-1, 1, d).astype(np.float32)
    x = x0.copy()
    g = np.ones(d, dtype=np.float32)
    for _ in range(K):
        oracle.signsgd_step(x, g, None, 1, d, 0.0, float(delta))
    assert np.all(np.abs((x0.astype(np.float64) - x) - K * float(delta)) <= K * 2.0 ** -24)


def test_step_is_the_composition_of_its_parts():
    r = rng(41)
    M, d, beta, delta = 5, 1234, 0.9, 1e-4
    g = r.standard_normal((M, d)).astype(np.float32).reshape(-1)
    m = (0.1 * r.standard_normal((M, d))).astype(np.float32).reshape(-1)
    x = r.standard_normal(d).astype(np.float32)
    m1, x1 = m.copy(), x.copy()
    bits, vote = oracle.signsgd_step(x1, g, m1, M, d, beta, delta)
    m2, x2 = m.copy(), x.copy()
    b2 = oracle.signum_momentum_pack(g, m2, M, d, beta)
    v2 = oracle.majority_vote(b2, M, d)
    oracle.sign_apply(x2, v2, d, delta)
    assert np.array_equal(bits, b2) and np.array_equal(vote, v2)
    assert np.array_equal(m1, m2) and np.array_equal(x1, x2)
    # numpy restatement of the vote on unpacked momenta
    mm = m2.reshape(M, d)
    exp_vote = (2 * np.count_nonzero(~(mm < 0), axis=0) >= M)
    assert oracle.unpack_bits(vote, d).astype(bool).tolist() == exp_vote.tolist()
    assert np.array_equal(x1, np.where(exp_vote, x - np.float32(delta), x + np.float32(delta)))


def test_resume_from_copied_state_is_bit_identical():
    r = rng(42)
    M, d, beta, delta = 3, 500, 0.9, 1e-4
    gs = [r.standard_normal(M * d).astype(np.float32) for _ in range(5)]
    x = r.standard_normal(d).astype(np.float32)
    m = np.zeros(M * d, dtype=np.float32)
    xa, ma = x.copy(), m.copy()
    for k in range(5):
        oracle.signsgd_step(xa, gs[k], ma, M, d, beta, delta)
    xb, mb = x.copy(), m.copy()
    for k in range(2):
        oracle.signsgd_step(xb, gs[k], mb, M, d, beta, delta)
    xb, mb = np.array(xb.tolist(), dtype=np.float32), np.array(mb.tolist(), dtype=np.float32)
    for k in range(2, 5):
        oracle.signsgd_step(xb, gs[k], mb, M, d, beta, delta)
    assert np.array_equal(xa, xb) and np.array_equal(ma, mb)


def test_single_worker_algorithms_1_and_2():
    # Algorithm 1: x <- x - delta sign(g);  Algorithm 2 with M = 1.
    g = np.array([0.3, -0.2, 0.0, -0.0, 5.0], dtype=np.float32)
    x = np.zeros(5, dtype=np.float32)
    oracle.signsgd_step(x, g, None, 1, 5, 0.0, 0.25)
    assert x.tolist() == [-0.25, 0.25, -0.25, -0.25, -0.25]
    m = np.array([1.0, 1.0, -1.0, 0.0, -100.0], dtype=np.float32)
    x = np.zeros(5, dtype=np.float32)
    oracle.signsgd_step(x, g, m, 1, 5, 0.5, 0.25)
    # m_new = 0.5 m + 0.5 g = [0.65, 0.4, -0.5, 0, -47.5]
    assert m.tolist() == [np.float32(0.65), np.float32(0.4), -0.5, 0.0, -47.5]
    assert x.tolist() == [-0.25, -0.25, 0.25, -0.25, 0.25]


# ---------------------------------------------------------------- Theorem 3 warm-up

def warmup_conditions(beta32, C):
    """The two inequalities of Theorem 3's C(beta), in exact rational arithmetic."""
    b = f32_to_fraction(beta32)
    first = Fraction(C, 2) * b ** C <= 1 / (1 - b * b) * Fraction(1, C + 1)
    second = b ** (C + 1) <= Fraction(1, 2)
    return first, second


def test_warmup_length_is_54_at_beta_0_9_as_printed():
    assert oracle.warmup_steps(0.9) == int(GOLDEN["warmup_C_beta_0.9"]) == 54
    b = np.float32(0.9)
    assert warmup_conditions(b, 54) == (True, True)
    assert warmup_conditions(b, 53)[0] is False          # 53 fails the first inequality
    assert all(warmup_conditions(b, C) != (True, True) for C in range(1, 54))


@pytest.mark.parametrize("beta", [0.0, 0.1, 0.5, 0.75, 0.8, 0.95, 0.99, 0.995])
def test_warmup_length_is_the_least_integer_satisfying_both_conditions(beta):
    b = np.float32(beta)
    C = oracle.warmup_steps(float(b))
    assert C >= 1 and warmup_conditions(b, C) == (True, True)
    assert all(warmup_conditions(b, c) != (True, True) for c in range(1, C))


def test_warmup_length_rejects_bad_beta():
    for beta in (1.0, 1.5, -0.1, float("nan")):
        assert oracle.warmup_steps(beta) == 0


def test_warmup_pack_sends_sign_of_gradient_and_keeps_signum_momentum():
    r = rng(51)
    M, d = 4, 1500
    g = r.standard_normal((M, d)).astype(np.float32).reshape(-1)
    m0 = (r.standard_normal((M, d)) * 3).astype(np.float32).reshape(-1)   # momentum often disagrees with g
    m_w, m_s = m0.copy(), m0.copy()
    bits_w = oracle.signum_warmup_pack(g, m_w, M, d, 0.9)
    bits_s = oracle.signum_momentum_pack(g, m_s, M, d, 0.9)
    assert np.array_equal(m_w, m_s)                                       # momentum accumulates as normal
    assert np.array_equal(bits_w, oracle.sign_pack(g, M, d))              # but the update uses sign(g)
    assert not np.array_equal(bits_w, bits_s)
    # whole step: x moves by the vote over sign(g)
    x = r.standard_normal(d).astype(np.float32)
    x1, m1 = x.copy(), m0.copy()
    b1, v1 = oracle.signsgd_warmup_step(x1, g, m1, M, d, 0.9, 1e-3)
    x2 = x.copy()
    b2, v2 = oracle.signsgd_step(x2, g, None, M, d, 0.0, 1e-3)
    assert np.array_equal(b1, b2) and np.array_equal(v1, v2) and np.array_equal(x1, x2)
    assert np.array_equal(m1, m_s)


# ---------------------------------------------------------------- the "(good)" scheme

@pytest.mark.parametrize("M", [1, 2, 3, 4, 7, 8, 15, 16, 31, 32, 100, 1024])
def test_count_planes_hold_the_integer_sum_of_signs(M):
    r = rng(60 + M)
    d = 500
    assert oracle.count_planes(M) == M.bit_length()
    s = (r.random((M, d)) < r.random(d)).astype(np.uint8)
    bits = np.concatenate([np.array(py_pack(row.tolist()), dtype=np.uint32) for row in s])
    planes = oracle.vote_count_planes(bits, M, d).reshape(M.bit_length(), -1)
    P = s.sum(axis=0, dtype=np.int64)
    for p in range(M.bit_length()):
        assert planes[p].tolist() == py_pack(((P >> p) & 1).tolist())
    # the sign of the sum is the majority vote, the tie (sum = 0) voting +1
    vote = oracle.unpack_bits(oracle.majority_vote(bits, M, d), d)
    assert np.array_equal(vote, (2 * P - M >= 0).astype(np.uint8))


def test_sum_apply_is_x_minus_delta_times_sum_rounded_once():
    r = rng(61)
    M, d = 7, 600
    s = r.integers(0, 2, size=(M, d), dtype=np.uint8)
    bits = np.concatenate([np.array(py_pack(row.tolist()), dtype=np.uint32) for row in s])
    planes = oracle.vote_count_planes(bits, M, d)
    x = (r.standard_normal(d) * 10.0 ** r.integers(-5, 2, d)).astype(np.float32)
    delta = np.float32(3e-3)
    got = x.copy()
    oracle.sum_apply(got, planes, M, d, float(delta))
    S = 2 * s.sum(axis=0, dtype=np.int64) - M
    expect = [round_f32(Fraction(xi) - Fraction(float(delta)) * int(si)) for xi, si in zip(x.tolist(), S.tolist())]
    assert got.tolist() == expect
    # M = 1: the sum of one sign is that sign, so the update is Algorithm 1's
    one = oracle.vote_count_planes(bits[:oracle.words(d)].copy(), 1, d)
    xa, xb = x.copy(), x.copy()
    oracle.sum_apply(xa, one, 1, d, float(delta))
    oracle.sign_apply(xb, bits[:oracle.words(d)].copy(), d, float(delta))
    assert np.array_equal(xa, xb)


# ---------------------------------------------------------------- vote with abstention
# (the paper gives this scheme in words only; these tests pin the oracle to the stated definition:
#  abstain when |v| < tau; decided when |P - N| >= max(Q, 1); sign of P - N)

def test_abstention_rule_on_listed_values():
    v = np.array([0.5, -0.5, 0.09, -0.09, 0.1, -0.1, 0.0, -0.0, np.nan, np.inf, -np.inf], dtype=np.float32)
    sb, ab = oracle.ternary_pack(v, None, 1, v.size, 0.0, float(np.float32(0.1)))
    assert oracle.unpack_bits(sb, v.size).tolist() == [1, 0, 1, 0, 1, 0, 1, 1, 1, 1, 0]
    assert oracle.unpack_bits(ab, v.size).tolist() == [1, 1, 0, 0, 1, 1, 0, 0, 1, 1, 1]
    sb0, ab0 = oracle.ternary_pack(v, None, 1, v.size, 0.0, 0.0)       # tau = 0 never abstains
    assert np.array_equal(sb0, oracle.sign_pack(v, 1, v.size)) and oracle.unpack_bits(ab0, v.size).all()


@pytest.mark.parametrize("M", [1, 2, 3, 4, 5, 6])
def test_quorum_vote_all_ternary_patterns(M):
    pats = list(itertools.product((-1, 0, 1), repeat=M))
    d = len(pats)
    sb = np.concatenate([np.array(py_pack([1 if p[w] > 0 else 0 for p in pats]), dtype=np.uint32) for w in range(M)])
    ab = np.concatenate([np.array(py_pack([1 if p[w] != 0 else 0 for p in pats]), dtype=np.uint32) for w in range(M)])
    for Q in (0, 1, 2, 3, M, M + 1, 50):
        vs, va = oracle.quorum_vote(sb, ab, M, d, Q)
        exp_a = [1 if abs(sum(p)) >= max(Q, 1) else 0 for p in pats]
        exp_s = [1 if (abs(sum(p)) >= max(Q, 1) and sum(p) > 0) else 0 for p in pats]
        assert va.tolist() == py_pack(exp_a) and vs.tolist() == py_pack(exp_s), (M, Q)


def test_abstention_with_tau0_q0_equals_one_bit_path_away_from_ties():
    r = rng(71)
    M, d = 7, 3000
    g = r.standard_normal((M, d)).astype(np.float32).reshape(-1)
    m = (0.2 * r.standard_normal((M, d))).astype(np.float32).reshape(-1)
    x = r.standard_normal(d).astype(np.float32)
    m1, x1 = m.copy(), x.copy()
    bits, vote = oracle.signsgd_step(x1, g, m1, M, d, 0.9, 1e-3)
    m2, x2 = m.copy(), x.copy()
    sb, ab = oracle.ternary_pack(g, m2, M, d, 0.9, 0.0)
    vs, va = oracle.quorum_vote(sb, ab, M, d, 0)
    oracle.ternary_apply(x2, vs, va, d, 1e-3)
    assert np.array_equal(sb, bits) and np.array_equal(m1, m2)
    assert oracle.unpack_bits(va, d).all()                     # odd M, nobody abstains: always decided
    assert np.array_equal(vs, vote) and np.array_equal(x1, x2)


def test_ternary_apply_moves_only_decided_elements():
    r = rng(72)
    d = 500
    x = r.standard_normal(d).astype(np.float32)
    s = r.integers(0, 2, d, dtype=np.uint8)
    a = r.integers(0, 2, d, dtype=np.uint8)
    got = x.copy()
    oracle.ternary_apply(got, np.array(py_pack((s & a).tolist()), dtype=np.uint32),
                         np.array(py_pack(a.tolist()), dtype=np.uint32), d, 0.25)
    expect = [round_f32(Fraction(xi) + (0 if not ai else (Fraction(-1, 4) if si else Fraction(1, 4))))
              for xi, si, ai in zip(x.tolist(), s.tolist(), a.tolist())]
    assert got.tolist() == expect


def test_abstention_shrinks_wrong_decisions_on_noisy_small_gradients():
    # workers that abstain when unsure and a server that wants a margin decide less often, and when
    # they do decide they are wrong less often than the plain majority: the point of the scheme
    r = rng(73)
    M, d = 15, 100_000
    mu = np.float32(-0.2)
    g = (mu + r.standard_normal((M, d))).astype(np.float32).reshape(-1)
    plain = oracle.unpack_bits(oracle.majority_vote(oracle.sign_pack(g, M, d), M, d), d)
    sb, ab = oracle.ternary_pack(g, None, M, d, 0.0, 0.5)
    vs, va = oracle.quorum_vote(sb, ab, M, d, 3)
    vs, va = oracle.unpack_bits(vs, d).astype(bool), oracle.unpack_bits(va, d).astype(bool)
    assert 0.2 < va.mean() < 0.9
    assert vs[va].mean() < plain.mean()          # true sign is negative: a set bit is a wrong decision


# ---------------------------------------------------------------- Section 3: density and Welford

def test_density_of_dense_and_one_hot_vectors():
    # Sec. 3 gives the two end points of phi: 1 when every component has the same magnitude, 1/d for a one-hot vector
    d = 1000
    r = rng(81)
    dense = (3.0 * r.choice([-1.0, 1.0], d)).astype(np.float32)
    assert abs(oracle.density(dense)[0] - 1.0) < 1e-12
    one_hot = np.zeros(d, dtype=np.float32)
    one_hot[17] = -2.5
    assert abs(oracle.density(one_hot)[0] - 1.0 / d) < 1e-15
    assert oracle.density(np.zeros(5, dtype=np.float32))[0] == 0.0
    # a Gaussian vector: E|z| = sqrt(2/pi), E z^2 = 1, so phi -> 2/pi
    z = r.standard_normal(400_000).astype(np.float32)
    phi, l1, l2 = oracle.density(z)
    assert abs(phi - 2 / math.pi) < 5e-3
    assert abs(l1 - float(np.abs(z.astype(np.float64)).sum())) < 1e-9 * l1
    assert abs(l2 - float((z.astype(np.float64) ** 2).sum())) < 1e-9 * l2
    # k equal non-zeros out of d: phi = k / d
    v = np.zeros(d, dtype=np.float32)
    v[:250] = 0.5
    assert abs(oracle.density(v)[0] - 0.25) < 1e-12


def test_density_of_root_on_vectors_of_variances():
    # Sec. 3's end points for the noise vector sigma, given as variances sigma^2:
    # every component equally noisy -> 1; noise on one component only -> 1/d
    d = 1000
    assert abs(oracle.density_of_root(np.full(d, 6.25, dtype=np.float32))[0] - 1.0) < 1e-12
    one = np.zeros(d, dtype=np.float32)
    one[3] = 1e4                                    # e.g. the toy problem: noise on a single coordinate
    assert abs(oracle.density_of_root(one)[0] - 1.0 / d) < 1e-15
    assert oracle.density_of_root(np.zeros(4, dtype=np.float32))[0] == 0.0
    v = np.zeros(d, dtype=np.float32)
    v[:250] = 0.49
    assert abs(oracle.density_of_root(v)[0] - 0.25) < 1e-9
    # perfect squares: the roots are exact integers, so the sums are exact small integers
    r = rng(84)
    k = r.integers(0, 200, 5000)
    sq = (k * k).astype(np.float32)
    phi, l1, l2 = oracle.density_of_root(sq)
    assert l1 == float(k.sum()) and l2 == float((k * k).sum())
    assert phi == float(k.sum()) ** 2 / (5000 * float((k * k).sum()))
    # half-normal scale mixture: sigma_i = |z_i| has phi -> 2/pi, from v = z^2
    z = r.standard_normal(400_000)
    assert abs(oracle.density_of_root((z * z).astype(np.float32))[0] - 2 / math.pi) < 5e-3


def test_welford_matches_two_pass_mean_and_variance():
    r = rng(82)
    n, d = 40, 3000
    g = (1.5 + 2.0 * r.standard_normal((n, d))).astype(np.float32)
    mean = np.zeros(d, dtype=np.float32)
    m2 = np.zeros(d, dtype=np.float32)
    for k in range(n):
        oracle.welford_update(g[k], k + 1, mean, m2)
    g64 = g.astype(np.float64)
    assert np.allclose(mean, g64.mean(axis=0), rtol=0, atol=2e-6)
    assert np.allclose(m2 / (n - 1), g64.var(axis=0, ddof=1), rtol=2e-5)
    # the noise density needs no division: phi(sigma) = phi(sqrt(m2))
    sigma = np.sqrt(m2 / np.float32(n - 1)).astype(np.float32)
    assert abs(oracle.density(sigma)[0] - oracle.density(np.sqrt(m2).astype(np.float32))[0]) < 1e-6


def test_welford_update_rounding_sequence():
    r = rng(83)
    d = 300
    g = r.standard_normal(d).astype(np.float32)
    mean = r.standard_normal(d).astype(np.float32)
    m2 = np.abs(r.standard_normal(d)).astype(np.float32)
    n = 7
    expect_mean, expect_m2 = [], []
    for gi, mu, s in zip(g.tolist(), mean.tolist(), m2.tolist()):
        d1 = round_f32(Fraction(gi) - Fraction(mu))
        q = round_f32(Fraction(d1) / n)
        mu2 = round_f32(Fraction(mu) + Fraction(q))
        d2 = round_f32(Fraction(gi) - Fraction(mu2))
        expect_mean.append(mu2)
        expect_m2.append(round_f32(Fraction(d1) * Fraction(d2) + Fraction(s)))
    oracle.welford_update(g, n, mean, m2)
    assert mean.tolist() == expect_mean and m2.tolist() == expect_m2
    # first sample: mean becomes the sample, m2 stays 0
    mean0, m20 = np.zeros(d, dtype=np.float32), np.zeros(d, dtype=np.float32)
    oracle.welford_update(g, 1, mean0, m20)
    assert np.array_equal(mean0, g) and not m20.any()
