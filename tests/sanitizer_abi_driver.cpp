// Calls the host side of every entry point of the CUDA library with arguments that must be rejected (or
// accepted as empty) before anything touches the device, under AddressSanitizer / UndefinedBehavior-
// Sanitizer: the argument checks' own arithmetic (products, roundings, shifts) is what is under test.
// The pointers are fake, 16-byte aligned addresses; no call here may reach a launch.  Built and run by
// test_host_sanitizers.py on a machine without a GPU.
#include <cmath>
#include <cstdint>
#include <cstdio>
#include <limits>

#include "signsgd.h"

static int failures = 0;
#define EXPECT(call, want)                                                          \
  do {                                                                              \
    const int got_ = (int)(call);                                                   \
    if (got_ != (int)(want)) {                                                      \
      std::printf("line %d: %s returned %d, expected %d\n", __LINE__, #call, got_, (int)(want)); \
      ++failures;                                                                   \
    }                                                                               \
  } while (0)

int main() {
  float* F = reinterpret_cast<float*>(0x10000);
  uint32_t* U = reinterpret_cast<uint32_t*>(0x20000);
  double* D = reinterpret_cast<double*>(0x30000);
  const float nan = std::numeric_limits<float>::quiet_NaN(), inf = std::numeric_limits<float>::infinity();
  const size_t huge = ~(size_t)0;

  EXPECT(ssgd_words(0), 0);
  EXPECT(ssgd_words(33), 2);
  EXPECT(ssgd_words(huge) == huge / 32 + 1, 1);
  for (int s = -1; s <= 8; ++s)
    if (ssgd_status_str((ssgd_status)s) == nullptr) ++failures;

  EXPECT(ssgd_sign_pack(nullptr, 1, 64, 64, U, 4, nullptr), SSGD_ERR_NULL);
  EXPECT(ssgd_sign_pack(F + 1, 1, 64, 64, U, 4, nullptr), SSGD_ERR_ALIGN);
  EXPECT(ssgd_sign_pack(F, 1, 64, 66, U, 4, nullptr), SSGD_ERR_ALIGN);
  EXPECT(ssgd_sign_pack(F, 0, 64, 64, U, 4, nullptr), SSGD_ERR_SIZE);
  EXPECT(ssgd_sign_pack(F, 1, huge, huge - 3, U, 4, nullptr), SSGD_ERR_SIZE);
  EXPECT(ssgd_sign_pack(F, 1024, (size_t)1 << 62, (size_t)1 << 62, U, (size_t)1 << 57, nullptr), SSGD_ERR_SIZE);
  EXPECT(ssgd_sign_pack(F, 1, 0, 0, U, 0, nullptr), SSGD_OK);

  EXPECT(ssgd_signum_momentum_pack(F, nullptr, 1, 64, 64, 0.9f, U, 4, nullptr), SSGD_ERR_NULL);
  EXPECT(ssgd_signum_momentum_pack(F, F, 1, 64, 64, 1.0f, U, 4, nullptr), SSGD_ERR_ARG);
  EXPECT(ssgd_signum_momentum_pack(F, F, 1, 64, 64, nan, U, 4, nullptr), SSGD_ERR_ARG);
  EXPECT(ssgd_signum_momentum_pack(F, F, 1, 64, 64, -inf, U, 4, nullptr), SSGD_ERR_ARG);
  EXPECT(ssgd_signum_momentum_pack(F, F, 3, 0, 0, 0.5f, U, 0, nullptr), SSGD_OK);
  EXPECT(ssgd_signum_warmup_pack(F, F, 1, 64, 64, 2.0f, U, 4, nullptr), SSGD_ERR_ARG);
  EXPECT(ssgd_signum_warmup_pack(F, F, 1, 0, 0, 0.9f, U, 0, nullptr), SSGD_OK);

  EXPECT(ssgd_majority_vote(U, 1025, 64, 4, U, nullptr), SSGD_ERR_SIZE);
  EXPECT(ssgd_majority_vote(U, 3, 640, 16, U, nullptr), SSGD_ERR_SIZE);
  EXPECT(ssgd_majority_vote(U, 3, 64, 6, U, nullptr), SSGD_ERR_ALIGN);
  EXPECT(ssgd_majority_vote(U, 1024, 0, 0, U, nullptr), SSGD_OK);

  EXPECT(ssgd_sign_apply(F, nullptr, 64, 0.1f, nullptr), SSGD_ERR_NULL);
  EXPECT(ssgd_sign_apply(F, U, huge, 0.1f, nullptr), SSGD_ERR_SIZE);
  EXPECT(ssgd_sign_apply(F, U, 64, inf, nullptr), SSGD_ERR_ARG);
  EXPECT(ssgd_sign_apply(F, U, 0, 0.1f, nullptr), SSGD_OK);

  EXPECT(ssgd_signsgd_step(F, F, nullptr, 1, 64, 64, 0.9f, 0.1f, U, 4, U, nullptr), SSGD_ERR_NULL);
  EXPECT(ssgd_signsgd_step(F, F, F, 2000, 64, 64, 0.9f, 0.1f, U, 4, U, nullptr), SSGD_ERR_SIZE);
  EXPECT(ssgd_signsgd_step(F, F, F, 1, 64, 64, 0.9f, nan, U, 4, U, nullptr), SSGD_ERR_ARG);
  EXPECT(ssgd_signsgd_step(F, F, nullptr, 1, 0, 0, 0.0f, 0.1f, U, 0, U, nullptr), SSGD_OK);
  EXPECT(ssgd_signsgd_warmup_step(F, F, nullptr, 1, 64, 64, 0.9f, 0.1f, U, 4, U, nullptr), SSGD_ERR_NULL);
  EXPECT(ssgd_signsgd_warmup_step(F, F, F, 1, 0, 0, 0.9f, 0.1f, U, 0, U, nullptr), SSGD_OK);
  EXPECT(ssgd_signsgd_step_host(F, nullptr, F, 1, 64, 64, 0.9f, 0.1f, F, U, 4, U, nullptr, nullptr), SSGD_ERR_NULL);
  EXPECT(ssgd_signsgd_step_host(F, F, F, 1, 0, 0, 0.9f, 0.1f, F, U, 0, U, nullptr, nullptr), SSGD_OK);
  EXPECT(ssgd_signsgd_step_noalloc(F, F, F, 0, 64, 64, 0.9f, 0.1f, nullptr), SSGD_ERR_SIZE);
  EXPECT(ssgd_signsgd_step_noalloc(F, F, F, 7, (size_t)1 << 25, (size_t)1 << 25, 0.9f, 0.1f, nullptr), SSGD_ERR_SCRATCH);
  EXPECT(ssgd_signsgd_step_noalloc(F, F, F, 1024, huge - 200, huge - 203, 0.9f, 0.1f, nullptr), SSGD_ERR_SCRATCH);
  EXPECT(ssgd_signsgd_step_noalloc(F, F, F, 1, huge - 100, huge - 103, 0.9f, 0.1f, nullptr), SSGD_ERR_SIZE);

  uint32_t* rows[3] = {U, U + 1024, U + 2048};
  uint32_t* rows_null[3] = {U, nullptr, U};
  EXPECT(ssgd_signum_momentum_pack_scatter(F, F, 64, 0.9f, rows, 65, 0, 4, nullptr), SSGD_ERR_SIZE);
  EXPECT(ssgd_signum_momentum_pack_scatter(F, F, 64, 0.9f, rows, 3, 1024, 4, nullptr), SSGD_ERR_SIZE);
  EXPECT(ssgd_signum_momentum_pack_scatter(F, F, 64, 0.9f, rows, 3, 1023, huge / 4 * 4, nullptr), SSGD_ERR_SIZE);
  EXPECT(ssgd_signum_momentum_pack_scatter(F, F, 64, 0.9f, rows_null, 3, 0, 4, nullptr), SSGD_ERR_NULL);
  EXPECT(ssgd_signum_momentum_pack_scatter(F, nullptr, 0, 0.0f, rows, 3, 7, 0, nullptr), SSGD_OK);

  EXPECT(ssgd_warmup_steps(0.9f), 54);
  EXPECT(ssgd_warmup_steps(0.0f), 1);
  EXPECT(ssgd_warmup_steps(nan), 0);
  EXPECT(ssgd_warmup_steps(0.999f) > 1000, 1);
  EXPECT(ssgd_count_planes(1024), 11);
  EXPECT(ssgd_count_planes(0), 0);
  EXPECT(ssgd_count_planes(huge), 0);
  EXPECT(ssgd_vote_counts(U, 3, 640, 20, U, 16, nullptr), SSGD_ERR_SIZE);
  EXPECT(ssgd_vote_counts(U, 3, 0, 0, U, 0, nullptr), SSGD_OK);
  EXPECT(ssgd_sum_apply(F, U, 0, 64, 4, 0.1f, nullptr), SSGD_ERR_SIZE);
  EXPECT(ssgd_sum_apply(F, U, 3, 0, 0, 0.1f, nullptr), SSGD_OK);

  EXPECT(ssgd_ternary_pack(F, F, 1, 64, 64, 0.9f, -0.1f, U, U, 4, nullptr), SSGD_ERR_ARG);
  EXPECT(ssgd_ternary_pack(F, nullptr, 1, 0, 0, 0.0f, 0.1f, U, U, 0, nullptr), SSGD_OK);
  EXPECT(ssgd_quorum_vote(U, U, 0, 64, 4, 1, U, U, nullptr), SSGD_ERR_SIZE);
  EXPECT(ssgd_quorum_vote(U, U, 3, 0, 0, huge, U, U, nullptr), SSGD_OK);
  EXPECT(ssgd_ternary_apply(F, U, nullptr, 64, 0.1f, nullptr), SSGD_ERR_NULL);
  EXPECT(ssgd_ternary_apply(F, U, U, 0, 0.1f, nullptr), SSGD_OK);

  EXPECT(ssgd_welford_update(F, 0, F, F, 64, nullptr), SSGD_ERR_ARG);
  EXPECT(ssgd_welford_update(F, ((size_t)1 << 24) + 1, F, F, 64, nullptr), SSGD_ERR_ARG);
  EXPECT(ssgd_welford_update(F, 1, F, F, 0, nullptr), SSGD_OK);
  EXPECT(ssgd_density_sums(nullptr, 64, 0, D, nullptr), SSGD_ERR_NULL);
  EXPECT(ssgd_density_sums(F, 64, 0, reinterpret_cast<double*>(0x30008), nullptr), SSGD_ERR_ALIGN);
  EXPECT(ssgd_density_from_sums(4.0, 4.0, 4) == 1.0, 1);
  EXPECT(ssgd_density_from_sums(0.0, 0.0, 4) == 0.0, 1);
  EXPECT(ssgd_density_from_sums(1.0, 1.0, 0) == 0.0, 1);

  std::printf(failures ? "abi sanitizer driver: %d failures\n" : "abi sanitizer driver: all checks passed%.0d\n", failures);
  return failures ? 1 : 0;
}
