// Launchers of the direct (register-load) vote kernel, for the translation units that vote: the step
// entry points and the count-plane variant.  Unnamed namespace: one copy per including unit.
#ifndef SSGD_VOTE_LAUNCH_H_
#define SSGD_VOTE_LAUNCH_H_

#include "host_common.h"

namespace {

template <int NP, bool COUNTS>
void launch_vote_np(const uint32_t* bits, size_t M, size_t d, size_t W, size_t ldw, uint32_t* out,
                    size_t ldc, unsigned grid, cudaStream_t s) {
  const unsigned start = COUNTS ? 0u : vote_start_value(M, NP);
  vote_kernel<NP, COUNTS><<<grid, kThreads, 0, s>>>(bits, (unsigned)M, d, W, ldw, out, ldc, start);
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
  const size_t W = ssgd_words(d);
  const unsigned long long chunks = (W + 3) / 4;
  const unsigned grid = grid_for((chunks + kThreads - 1) / kThreads);
  switch (COUNTS ? count_planes(M) : vote_planes(M)) {
    case 1: launch_vote_np<1, COUNTS>(bits, M, d, W, ldw, out, ldc, grid, s); break;
    case 2: launch_vote_np<2, COUNTS>(bits, M, d, W, ldw, out, ldc, grid, s); break;
    case 3: launch_vote_np<3, COUNTS>(bits, M, d, W, ldw, out, ldc, grid, s); break;
    case 4: launch_vote_np<4, COUNTS>(bits, M, d, W, ldw, out, ldc, grid, s); break;
    case 5: launch_vote_np<5, COUNTS>(bits, M, d, W, ldw, out, ldc, grid, s); break;
    case 6: launch_vote_np<6, COUNTS>(bits, M, d, W, ldw, out, ldc, grid, s); break;
    case 7: launch_vote_np<7, COUNTS>(bits, M, d, W, ldw, out, ldc, grid, s); break;
    case 8: launch_vote_np<8, COUNTS>(bits, M, d, W, ldw, out, ldc, grid, s); break;
    case 9: launch_vote_np<9, COUNTS>(bits, M, d, W, ldw, out, ldc, grid, s); break;
    case 10: launch_vote_np<10, COUNTS>(bits, M, d, W, ldw, out, ldc, grid, s); break;
    case 11: launch_vote_np<11, COUNTS>(bits, M, d, W, ldw, out, ldc, grid, s); break;
    default: return SSGD_ERR_SIZE;
  }
  return launch_status();
}

}  // namespace

#endif  // SSGD_VOTE_LAUNCH_H_
