// CPU oracle for the signSGD / Signum / majority-vote step (Bernstein et al.,
// "signSGD: Compressed Optimisation for Non-Convex Problems", Algorithms 1-3).
//
// TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition that the
// CUDA library is checked against.  It shares no code, header, table or helper
// with the CUDA sources, and the product never calls it: only the test-suite,
// the smoke check and the benchmark's cpu-baseline leg load this library.
//
// Everything is written as scalar loops over *unpacked* values (one byte per
// sign), with packing into words kept in a separate trivial loop, so that an
// arithmetic mistake and a packing mistake show up in different tests.
//
// Conventions the paper leaves open and this oracle fixes (each is pinned by a
// test against brute force or a closed form):
//   * sign(v) is encoded in one bit as  bit = !(v < 0): zero, -0.0 and NaN all
//     count as +1, so that "1-bit" (Sec. 1, Table 1) holds without a third symbol.
//   * an even-M tie, sum_m sign(g_m) = 0 in Algorithm 3, resolves to +1;
//     equivalently vote = [P >= ceil(M/2)] with P the number of +1 votes.
//   * word j of a packed row holds elements 32j .. 32j+31, least significant
//     bit first; bits at positions >= d are 0.
//   * momentum (Algorithm 2, second step) is evaluated in fp32 as
//         omb = fl(1 - beta);  t = fl(omb * g);  m <- fma(beta, m, t)
//     i.e. two roundings per element, the last one a fused multiply-add.
//   * each worker keeps its own momentum and sends sign(m_new)  (Algorithm 2
//     run per worker, feeding Algorithm 3's server); beta = 0 gives Algorithm 3
//     as printed.
//
// All pointers are HOST pointers.  Parity status: every function below is
// pinned by tests that do not call back into this file (brute force in Python,
// closed forms in extended precision, invariants, bitwise MAJ3) -- except that
// the three abstention functions (ssgd_ternary_pack_ref, ssgd_quorum_vote_ref,
// ssgd_ternary_apply_ref) are "parity unpinned" against the paper, which gives
// their scheme in words without thresholds; they are pinned to the definition
// stated above them.

#include <cmath>
#include <cstddef>
#include <cstdint>
#include <cstdlib>
#include <vector>

extern "C" {

// Number of 32-bit words that hold d one-bit signs (Table 1: d bits per vector).
size_t ssgd_words_ref(size_t d) { return d / 32 + (d % 32 != 0 ? 1 : 0); }

// sign(.) of Algorithms 1-3 on one row, unpacked: s[i] = 1 for +1, 0 for -1.
void ssgd_sign_unpacked_ref(const float* v, size_t d, uint8_t* s) {
  for (size_t i = 0; i < d; ++i) {
    s[i] = (v[i] < 0.0f) ? 0 : 1;
  }
}

// The 1-bit wire format: LSB-first words, padding bits zero.
void ssgd_pack_bits_ref(const uint8_t* s, size_t d, uint32_t* words) {
  const size_t W = ssgd_words_ref(d);
  for (size_t j = 0; j < W; ++j) words[j] = 0u;
  for (size_t i = 0; i < d; ++i) {
    if (s[i]) words[i / 32] |= (uint32_t(1) << (i % 32));
  }
}

void ssgd_unpack_bits_ref(const uint32_t* words, size_t d, uint8_t* s) {
  for (size_t i = 0; i < d; ++i) {
    s[i] = uint8_t((words[i / 32] >> (i % 32)) & 1u);
  }
}

// Algorithm 1 / Algorithm 3 worker side: every worker w sends sign(g_w).
void ssgd_sign_pack_ref(const float* g, size_t M, size_t d, size_t ld,
                        uint32_t* bits, size_t ldw) {
  std::vector<uint8_t> s(d);
  for (size_t w = 0; w < M; ++w) {
    ssgd_sign_unpacked_ref(g + w * ld, d, s.data());
    ssgd_pack_bits_ref(s.data(), d, bits + w * ldw);
  }
}

// Algorithm 2, second step, on one row, in place: m <- beta m + (1-beta) g.
void ssgd_momentum_ref(const float* g, float* m, size_t d, float beta) {
  const float omb = 1.0f - beta;
  for (size_t i = 0; i < d; ++i) {
    const float t = omb * g[i];
    m[i] = std::fmaf(beta, m[i], t);
  }
}

// Algorithm 2 per worker, then the sign of the *new* momentum is what is sent.
void ssgd_signum_momentum_pack_ref(const float* g, float* m, size_t M, size_t d,
                                   size_t ld, float beta, uint32_t* bits,
                                   size_t ldw) {
  std::vector<uint8_t> s(d);
  for (size_t w = 0; w < M; ++w) {
    ssgd_momentum_ref(g + w * ld, m + w * ld, d, beta);
    ssgd_sign_unpacked_ref(m + w * ld, d, s.data());
    ssgd_pack_bits_ref(s.data(), d, bits + w * ldw);
  }
}

// Theorem 3's warm-up length: C(beta) = min C in Z+ such that
//   (C/2) beta^C <= 1/(1 - beta^2) * 1/(C + 1)   and   beta^(C+1) <= 1/2.
// Each candidate is tested directly from this definition, in extended precision.
size_t ssgd_warmup_steps_ref(float beta) {
  if (!(beta >= 0.0f && beta < 1.0f)) return 0;
  const long double b = (long double)beta;
  for (size_t C = 1;; ++C) {
    const long double lhs = ((long double)C / 2.0L) * std::pow(b, (long double)C);
    const long double rhs = 1.0L / (1.0L - b * b) * 1.0L / ((long double)C + 1.0L);
    if (lhs <= rhs && std::pow(b, (long double)C + 1.0L) <= 0.5L) return C;
  }
}

// Theorem 3, warm-up iterations: the momentum is accumulated as in Algorithm 2,
// but the sign that is sent is that of the stochastic gradient.
void ssgd_signum_warmup_pack_ref(const float* g, float* m, size_t M, size_t d,
                                 size_t ld, float beta, uint32_t* bits,
                                 size_t ldw) {
  std::vector<uint8_t> s(d);
  for (size_t w = 0; w < M; ++w) {
    ssgd_momentum_ref(g + w * ld, m + w * ld, d, beta);
    ssgd_sign_unpacked_ref(g + w * ld, d, s.data());
    ssgd_pack_bits_ref(s.data(), d, bits + w * ldw);
  }
}

// Algorithm 3 server side on unpacked signs: count the +1 votes per element.
void ssgd_vote_counts_ref(const uint32_t* bits, size_t M, size_t d, size_t ldw,
                          int32_t* P) {
  std::vector<uint8_t> s(d);
  for (size_t i = 0; i < d; ++i) P[i] = 0;
  for (size_t w = 0; w < M; ++w) {
    ssgd_unpack_bits_ref(bits + w * ldw, d, s.data());
    for (size_t i = 0; i < d; ++i) P[i] += s[i];
  }
}

// Algorithm 3 server side: sign[ sum_m sign(g_m) ].  With P positive votes the
// sum is P - (M - P) = 2P - M; it is >= 0 (tie counts as +1) iff 2P >= M.
void ssgd_majority_vote_ref(const uint32_t* bits, size_t M, size_t d,
                            size_t ldw, uint32_t* vote) {
  std::vector<int32_t> P(d);
  std::vector<uint8_t> s(d);
  ssgd_vote_counts_ref(bits, M, d, ldw, P.data());
  for (size_t i = 0; i < d; ++i) {
    const long long sum = 2LL * P[i] - (long long)M;
    s[i] = (sum < 0) ? 0 : 1;
  }
  ssgd_pack_bits_ref(s.data(), d, vote);
}

// Algorithm 3 worker side (also the last line of Algorithms 1 and 2):
// x <- x - delta * sign(vote).
void ssgd_sign_apply_ref(float* x, const uint32_t* vote, size_t d, float delta) {
  std::vector<uint8_t> s(d);
  ssgd_unpack_bits_ref(vote, d, s.data());
  for (size_t i = 0; i < d; ++i) {
    if (s[i]) x[i] = x[i] - delta;
    else      x[i] = x[i] + delta;
  }
}

// One whole step of Algorithm 3 with Signum workers.  beta == 0 is Algorithm 3
// as printed (workers send sign(g)); m may then be NULL.
void ssgd_signsgd_step_ref(float* x, const float* g, float* m, size_t M,
                           size_t d, size_t ld, float beta, float delta,
                           uint32_t* bits, size_t ldw, uint32_t* vote) {
  if (beta == 0.0f && m == nullptr) {
    ssgd_sign_pack_ref(g, M, d, ld, bits, ldw);
  } else {
    ssgd_signum_momentum_pack_ref(g, m, M, d, ld, beta, bits, ldw);
  }
  ssgd_majority_vote_ref(bits, M, d, ldw, vote);
  ssgd_sign_apply_ref(x, vote, d, delta);
}

// ---- the "(good)" scheme of Section 4: x <- x - delta * sum_m sign(g_m) --------
// The server's answer is the count P of +1 votes per element (sum of signs =
// 2P - M), sent bit-sliced: plane p holds bit p of every count, packed like a
// sign vector.

size_t ssgd_count_planes_ref(size_t M) {
  size_t n = 0;
  while ((M >> n) != 0) ++n;   // bits needed for the values 0..M
  return n;
}

void ssgd_vote_count_planes_ref(const uint32_t* bits, size_t M, size_t d,
                                size_t ldw, uint32_t* counts, size_t ldc) {
  std::vector<int32_t> P(d);
  std::vector<uint8_t> s(d);
  ssgd_vote_counts_ref(bits, M, d, ldw, P.data());
  const size_t planes = ssgd_count_planes_ref(M);
  for (size_t p = 0; p < planes; ++p) {
    for (size_t i = 0; i < d; ++i) s[i] = uint8_t((P[i] >> p) & 1);
    ssgd_pack_bits_ref(s.data(), d, counts + p * ldc);
  }
}

void ssgd_sum_apply_ref(float* x, const uint32_t* counts, size_t M, size_t d,
                        size_t ldc, float delta) {
  const size_t planes = ssgd_count_planes_ref(M);
  std::vector<uint8_t> s(d);
  std::vector<int32_t> P(d, 0);
  for (size_t p = 0; p < planes; ++p) {
    ssgd_unpack_bits_ref(counts + p * ldc, d, s.data());
    for (size_t i = 0; i < d; ++i) P[i] += int32_t(s[i]) << p;
  }
  for (size_t i = 0; i < d; ++i) {
    const float sum_of_signs = float(2 * P[i] - int32_t(M));
    x[i] = std::fmaf(-delta, sum_of_signs, x[i]);   // x - delta * sum, rounded once
  }
}

// ---- majority vote with abstention (Discussion section) ------------------------
// The paper gives the scheme in words only (Discussion section): a worker that
// doubts the sign of the true gradient sends 0 instead of +-1, and the server
// answers 0 when the cast votes do not reach a quorum.  No thresholds are given,
// so the two used here are a definition of this code base, not the paper's:
// a worker is unsure when |v| < tau; quorum is reached when |P - N| >= max(Q, 1),
// P / N being the numbers of +1 / -1 votes cast.  (Parity with the paper is
// therefore unpinned for these three functions; they are pinned to this
// definition by brute force.)

void ssgd_ternary_pack_ref(const float* g, float* m, size_t M, size_t d, size_t ld,
                           float beta, float tau, uint32_t* sign_bits,
                           uint32_t* active_bits, size_t ldw) {
  std::vector<uint8_t> s(d), a(d);
  for (size_t w = 0; w < M; ++w) {
    const float* v = g + w * ld;
    if (m != nullptr) {
      ssgd_momentum_ref(g + w * ld, m + w * ld, d, beta);
      v = m + w * ld;
    }
    ssgd_sign_unpacked_ref(v, d, s.data());
    for (size_t i = 0; i < d; ++i) a[i] = (std::fabs(v[i]) < tau) ? 0 : 1;
    ssgd_pack_bits_ref(s.data(), d, sign_bits + w * ldw);
    ssgd_pack_bits_ref(a.data(), d, active_bits + w * ldw);
  }
}

void ssgd_quorum_vote_ref(const uint32_t* sign_bits, const uint32_t* active_bits,
                          size_t M, size_t d, size_t ldw, size_t quorum,
                          uint32_t* vote_sign, uint32_t* vote_active) {
  std::vector<uint8_t> s(d), a(d), vs(d), va(d);
  std::vector<int32_t> diff(d, 0);   // P - N
  for (size_t w = 0; w < M; ++w) {
    ssgd_unpack_bits_ref(sign_bits + w * ldw, d, s.data());
    ssgd_unpack_bits_ref(active_bits + w * ldw, d, a.data());
    for (size_t i = 0; i < d; ++i) {
      if (a[i]) diff[i] += s[i] ? 1 : -1;
    }
  }
  const long long Q = quorum < 1 ? 1 : (long long)quorum;
  for (size_t i = 0; i < d; ++i) {
    const long long margin = diff[i] < 0 ? -(long long)diff[i] : (long long)diff[i];
    va[i] = margin >= Q ? 1 : 0;
    vs[i] = (va[i] && diff[i] > 0) ? 1 : 0;
  }
  ssgd_pack_bits_ref(vs.data(), d, vote_sign);
  ssgd_pack_bits_ref(va.data(), d, vote_active);
}

void ssgd_ternary_apply_ref(float* x, const uint32_t* vote_sign,
                            const uint32_t* vote_active, size_t d, float delta) {
  std::vector<uint8_t> s(d), a(d);
  ssgd_unpack_bits_ref(vote_sign, d, s.data());
  ssgd_unpack_bits_ref(vote_active, d, a.data());
  for (size_t i = 0; i < d; ++i) {
    if (!a[i]) continue;           // the server answered 0: no move
    if (s[i]) x[i] = x[i] - delta;
    else      x[i] = x[i] + delta;
  }
}

// ---- Section 3: density of a vector and Welford's mean / variance ---------------

// phi(v) = |v|_1^2 / (d |v|_2^2); the two norms are returned too (fp64 sums).
double ssgd_density_ref(const float* v, size_t d, double* l1_out, double* l2sq_out) {
  double l1 = 0.0, l2sq = 0.0;
  for (size_t i = 0; i < d; ++i) {
    l1 += std::fabs((double)v[i]);
    l2sq += (double)v[i] * (double)v[i];
  }
  if (l1_out) *l1_out = l1;
  if (l2sq_out) *l2sq_out = l2sq;
  if (d == 0 || !(l2sq > 0.0)) return 0.0;
  return l1 * l1 / ((double)d * l2sq);
}

// Density of the element-wise square root of a non-negative vector, phi(sqrt(v)):
// Section 3 measures phi(sigma) of the noise vector sigma, whose squares (the
// per-component variances, up to a common factor that cancels in phi) are what a
// variance estimator holds.  |sqrt(v)|_1 = sum sqrt(v_i), |sqrt(v)|_2^2 = sum v_i.
double ssgd_density_of_root_ref(const float* v, size_t d, double* l1_out, double* l2sq_out) {
  double l1 = 0.0, l2sq = 0.0;
  for (size_t i = 0; i < d; ++i) {
    l1 += std::sqrt((double)v[i]);
    l2sq += (double)v[i];
  }
  if (l1_out) *l1_out = l1;
  if (l2sq_out) *l2sq_out = l2sq;
  if (d == 0 || !(l2sq > 0.0)) return 0.0;
  return l1 * l1 / ((double)d * l2sq);
}

// Welford's update with the n-th sample (n counts from 1), per element, in fp32:
// the textbook recurrence  mean_n = mean_{n-1} + (g - mean_{n-1}) / n,
// M2_n = M2_{n-1} + (g - mean_{n-1}) (g - mean_n), the last line as one fma.
void ssgd_welford_update_ref(const float* g, size_t n, float* mean, float* m2, size_t d) {
  const float nf = (float)n;
  for (size_t i = 0; i < d; ++i) {
    const float d1 = g[i] - mean[i];
    mean[i] = mean[i] + d1 / nf;
    const float d2 = g[i] - mean[i];
    m2[i] = std::fmaf(d1, d2, m2[i]);
  }
}

// One whole warm-up step: Theorem 3's warm-up on every worker, then Algorithm 3.
void ssgd_signsgd_warmup_step_ref(float* x, const float* g, float* m, size_t M,
                                  size_t d, size_t ld, float beta, float delta,
                                  uint32_t* bits, size_t ldw, uint32_t* vote) {
  ssgd_signum_warmup_pack_ref(g, m, M, d, ld, beta, bits, ldw);
  ssgd_majority_vote_ref(bits, M, d, ldw, vote);
  ssgd_sign_apply_ref(x, vote, d, delta);
}

}  // extern "C"
