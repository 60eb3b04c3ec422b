// Calls every function of the CPU oracle on tiny problems with heap buffers of exactly the
// documented sizes, so that AddressSanitizer / UndefinedBehaviorSanitizer see any access outside
// them, any misaligned or overflowing arithmetic.  Built and run by test_host_sanitizers.py.
#include <cmath>
#include <cstddef>
#include <cstdint>
#include <cstdio>
#include <vector>

extern "C" {
size_t ssgd_words_ref(size_t d);
void ssgd_sign_unpacked_ref(const float* v, size_t d, uint8_t* s);
void ssgd_pack_bits_ref(const uint8_t* s, size_t d, uint32_t* words);
void ssgd_unpack_bits_ref(const uint32_t* words, size_t d, uint8_t* s);
void ssgd_sign_pack_ref(const float* g, size_t M, size_t d, size_t ld, uint32_t* bits, size_t ldw);
void ssgd_momentum_ref(const float* g, float* m, size_t d, float beta);
void ssgd_signum_momentum_pack_ref(const float* g, float* m, size_t M, size_t d, size_t ld, float beta,
                                   uint32_t* bits, size_t ldw);
size_t ssgd_warmup_steps_ref(float beta);
void ssgd_signum_warmup_pack_ref(const float* g, float* m, size_t M, size_t d, size_t ld, float beta,
                                 uint32_t* bits, size_t ldw);
void ssgd_vote_counts_ref(const uint32_t* bits, size_t M, size_t d, size_t ldw, int32_t* P);
void ssgd_majority_vote_ref(const uint32_t* bits, size_t M, size_t d, size_t ldw, uint32_t* vote);
void ssgd_sign_apply_ref(float* x, const uint32_t* vote, size_t d, float delta);
void ssgd_signsgd_step_ref(float* x, const float* g, float* m, size_t M, size_t d, size_t ld, float beta,
                           float delta, uint32_t* bits, size_t ldw, uint32_t* vote);
size_t ssgd_count_planes_ref(size_t M);
void ssgd_vote_count_planes_ref(const uint32_t* bits, size_t M, size_t d, size_t ldw, uint32_t* counts,
                                size_t ldc);
void ssgd_sum_apply_ref(float* x, const uint32_t* counts, size_t M, size_t d, size_t ldc, float delta);
void ssgd_ternary_pack_ref(const float* g, float* m, size_t M, size_t d, size_t ld, float beta, float tau,
                           uint32_t* sign_bits, uint32_t* active_bits, size_t ldw);
void ssgd_quorum_vote_ref(const uint32_t* sign_bits, const uint32_t* active_bits, size_t M, size_t d,
                          size_t ldw, size_t quorum, uint32_t* vote_sign, uint32_t* vote_active);
void ssgd_ternary_apply_ref(float* x, const uint32_t* vote_sign, const uint32_t* vote_active, size_t d,
                            float delta);
double ssgd_density_ref(const float* v, size_t d, double* l1_out, double* l2sq_out);
double ssgd_density_of_root_ref(const float* v, size_t d, double* l1_out, double* l2sq_out);
void ssgd_welford_update_ref(const float* g, size_t n, float* mean, float* m2, size_t d);
void ssgd_signsgd_warmup_step_ref(float* x, const float* g, float* m, size_t M, size_t d, size_t ld,
                                  float beta, float delta, uint32_t* bits, size_t ldw, uint32_t* vote);
}

static uint32_t lcg_state = 12345u;
static float next_value() {
  lcg_state = lcg_state * 1664525u + 1013904223u;
  const int k = int(lcg_state >> 24) - 128;
  return k == 0 ? 0.0f : float(k) / 37.0f;   // exact zeros occur
}

// a buffer of exactly n elements on the heap (n == 0 gives a valid pointer to nothing)
template <typename T>
struct Tight {
  T* p;
  size_t n;
  explicit Tight(size_t n_) : p(new T[n_ == 0 ? 1 : n_]), n(n_) {
    if (n_ == 0) { delete[] p; p = new T[0]; }
  }
  ~Tight() { delete[] p; }
  Tight(const Tight&) = delete;
  Tight& operator=(const Tight&) = delete;
};

static void fill(Tight<float>& t) { for (size_t i = 0; i < t.n; ++i) t.p[i] = next_value(); }

static int run_case(size_t M, size_t d) {
  const size_t W = ssgd_words_ref(d);
  if (W != (d + 31) / 32) return 1;
  const size_t ld = d, ldw = W;            // the tightest strides the functions accept
  Tight<float> g(M * ld), m(M * ld), x(d), mean(d), m2(d);
  Tight<uint32_t> bits(M * ldw), act(M * ldw), vote(W), vs(W), va(W);
  Tight<uint8_t> s(d);
  Tight<int32_t> P(d);
  fill(g); fill(m); fill(x);
  for (size_t i = 0; i < d; ++i) { mean.p[i] = 0.0f; m2.p[i] = 0.0f; }

  ssgd_sign_unpacked_ref(g.p, d, s.p);
  ssgd_pack_bits_ref(s.p, d, vote.p);
  ssgd_unpack_bits_ref(vote.p, d, s.p);
  ssgd_sign_pack_ref(g.p, M, d, ld, bits.p, ldw);
  ssgd_momentum_ref(g.p, m.p, d, 0.9f);
  ssgd_signum_momentum_pack_ref(g.p, m.p, M, d, ld, 0.9f, bits.p, ldw);
  ssgd_signum_warmup_pack_ref(g.p, m.p, M, d, ld, 0.5f, bits.p, ldw);
  ssgd_vote_counts_ref(bits.p, M, d, ldw, P.p);
  ssgd_majority_vote_ref(bits.p, M, d, ldw, vote.p);
  ssgd_sign_apply_ref(x.p, vote.p, d, 1e-3f);
  ssgd_signsgd_step_ref(x.p, g.p, m.p, M, d, ld, 0.9f, 1e-3f, bits.p, ldw, vote.p);
  ssgd_signsgd_step_ref(x.p, g.p, nullptr, M, d, ld, 0.0f, 1e-3f, bits.p, ldw, vote.p);
  ssgd_signsgd_warmup_step_ref(x.p, g.p, m.p, M, d, ld, 0.9f, 1e-3f, bits.p, ldw, vote.p);

  const size_t planes = ssgd_count_planes_ref(M);
  Tight<uint32_t> counts(planes * W);
  ssgd_vote_count_planes_ref(bits.p, M, d, ldw, counts.p, W);
  ssgd_sum_apply_ref(x.p, counts.p, M, d, W, 1e-3f);

  ssgd_ternary_pack_ref(g.p, m.p, M, d, ld, 0.9f, 0.25f, bits.p, act.p, ldw);
  ssgd_ternary_pack_ref(g.p, nullptr, M, d, ld, 0.0f, 0.25f, bits.p, act.p, ldw);
  for (size_t q = 0; q <= M + 1; ++q) ssgd_quorum_vote_ref(bits.p, act.p, M, d, ldw, q, vs.p, va.p);
  ssgd_ternary_apply_ref(x.p, vs.p, va.p, d, 1e-3f);

  double l1 = 0, l2 = 0;
  const double phi = ssgd_density_ref(g.p, d, &l1, &l2);
  ssgd_density_ref(g.p, d, nullptr, nullptr);
  for (size_t n = 1; n <= 3; ++n) ssgd_welford_update_ref(g.p, n, mean.p, m2.p, d);
  const double phi_r = ssgd_density_of_root_ref(m2.p, d, &l1, &l2);
  if (!(phi >= 0.0 && phi <= 1.0 + 1e-12) || !(phi_r >= 0.0 && phi_r <= 1.0 + 1e-12)) return 2;
  for (size_t i = 0; i < d; ++i)
    if (std::isnan(x.p[i])) return 3;
  return 0;
}

int main() {
  const size_t ds[] = {0, 1, 31, 32, 33, 130};
  const size_t Ms[] = {1, 2, 3, 8};
  for (size_t d : ds)
    for (size_t M : Ms) {
      const int rc = run_case(M, d);
      if (rc != 0) {
        std::printf("case M=%zu d=%zu failed with %d\n", M, d, rc);
        return rc;
      }
    }
  if (ssgd_warmup_steps_ref(0.9f) != 54 || ssgd_warmup_steps_ref(1.0f) != 0) return 4;
  std::printf("sanitizer driver: all cases ran\n");
  return 0;
}
