// Launchers of the direct (register-load) vote kernels (general, exact row count, rows split over warps), for the
// translation units that vote: the step entry points and the count-plane variant.  Unnamed namespace: one copy per
// including unit.
#ifndef SSGD_VOTE_LAUNCH_H_
#define SSGD_VOTE_LAUNCH_H_

#include "host_common.h"

namespace {

template <int NP, bool COUNTS, int MROWS>
void launch_vote_exact(const uint32_t* bits, size_t d, size_t W, size_t ldw, uint32_t* out, size_t ldc,
                       unsigned grid, unsigned start, cudaStream_t s) {
  launch_kernel(vote_exact_kernel<NP, COUNTS, MROWS>, grid, kThreads, 0, s, true, bits, (unsigned long long)d,
                (unsigned long long)W, (unsigned long long)ldw, out, (unsigned long long)ldc, start);
}

template <int NP, bool COUNTS>
void launch_vote_np(const uint32_t* bits, size_t M, size_t d, size_t W, size_t ldw, uint32_t* out,
                    size_t ldc, unsigned grid, bool guarded, bool split, bool pdl, cudaStream_t s) {
  const unsigned start = COUNTS ? 0u : vote_start_value(M, NP);
  const unsigned long long d64 = d, W64 = W, ldw64 = ldw, ldc64 = ldc;
  if constexpr (NP == 2) {          // M = 2, 3 (as a vote and as a count)
    if (M == 2) launch_vote_exact<NP, COUNTS, 2>(bits, d, W, ldw, out, ldc, grid, start, s);
    else launch_vote_exact<NP, COUNTS, 3>(bits, d, W, ldw, out, ldc, grid, start, s);
  } else if constexpr (NP == 3) {   // M = 4 .. 7
    switch (M) {
      case 4: launch_vote_exact<NP, COUNTS, 4>(bits, d, W, ldw, out, ldc, grid, start, s); break;
      case 5: launch_vote_exact<NP, COUNTS, 5>(bits, d, W, ldw, out, ldc, grid, start, s); break;
      case 6: launch_vote_exact<NP, COUNTS, 6>(bits, d, W, ldw, out, ldc, grid, start, s); break;
      default: launch_vote_exact<NP, COUNTS, 7>(bits, d, W, ldw, out, ldc, grid, start, s); break;
    }
  } else {
    if constexpr (NP >= 4) {           // 13 rows and more have four planes and more
      if (split) {
        launch_kernel(vote_split_kernel<NP, COUNTS>, (unsigned)(((W64 + 3) / 4 + 31) / 32), kThreads, 0, s, pdl, bits,
                      (unsigned)M, d64, W64, ldw64, out, ldc64, start);
        return;
      }
    }
    if constexpr (NP >= kGuardedMinPlanes && NP <= kGuardedMaxPlanes) {   // the only ones vote_guarded() picks
      if (guarded) {
        launch_kernel(vote_kernel<NP, COUNTS, true>, grid, kThreads, 0, s, pdl, bits, (unsigned)M, d64, W64, ldw64,
                      out, ldc64, start);
        return;
      }
    }
    launch_kernel(vote_kernel<NP, COUNTS, false>, grid, kThreads, 0, s, pdl, bits, (unsigned)M, d64, W64, ldw64,
                  out, ldc64, start);
  }
}

// planes that hold a count in 0..M: the bit length of M
unsigned count_planes(size_t M) {
  unsigned n = 0;
  while ((M >> n) != 0) ++n;
  return n;
}

template <bool COUNTS>
ssgd_status launch_vote_any(const uint32_t* bits, size_t M, size_t d, size_t ldw, uint32_t* out,
                            size_t ldc, cudaStream_t s) {
  const bool pdl = true;   // the vote kernels begin with pdl_wait()
  DeviceInfo di;
  if (!device_info(&di)) return SSGD_ERR_CUDA;
  const size_t W = ssgd_words(d);
  const unsigned long long chunks = (W + 3) / 4;
  const unsigned long long ctas = (chunks + kThreads - 1) / kThreads;
  const unsigned grid = grid_for(ctas);
  const unsigned planes = COUNTS ? count_planes(M) : vote_planes(M);
  const bool g = vote_guarded(planes);
  const bool sp = vote_split(M, chunks, di.sms);
  switch (planes) {
#define SSGD_VOTE_CASE(n) \
  case n: launch_vote_np<n, COUNTS>(bits, M, d, W, ldw, out, ldc, grid, g, sp, pdl, s); break;
    SSGD_VOTE_CASE(1) SSGD_VOTE_CASE(2) SSGD_VOTE_CASE(3) SSGD_VOTE_CASE(4) SSGD_VOTE_CASE(5) SSGD_VOTE_CASE(6)
    SSGD_VOTE_CASE(7) SSGD_VOTE_CASE(8) SSGD_VOTE_CASE(9) SSGD_VOTE_CASE(10) SSGD_VOTE_CASE(11)
#undef SSGD_VOTE_CASE
    default: return SSGD_ERR_SIZE;
  }
  return launch_status();
}

}  // namespace

#endif  // SSGD_VOTE_LAUNCH_H_
