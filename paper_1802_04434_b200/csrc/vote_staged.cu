// Majority vote (Algorithm 3, server block) with the worker rows STAGED THROUGH
// SHARED MEMORY by bulk asynchronous copies -- the alternative design to the
// register-load vote kernel that ssgd_majority_vote uses.  It computes exactly the
// same words.  It exists so that the comparison between the two designs can be
// re-measured from this source tree (sweep.py times both); the step entry points
// do not use it, because on B200 it is not faster: every word is read once, by
// one thread, so shared memory has no reuse to serve, and the direct kernel
// already runs in the time of a plain device copy of the same bytes.
//
// One CTA owns a tile of 1024 consecutive words (one 128-bit chunk per thread) and
// walks the M rows in groups of 8.  For every group one elected thread arms an
// mbarrier with the group's byte count and issues one bulk copy per row (4 KB,
// global -> this CTA's shared memory only, completion counted on the mbarrier); the groups
// are double-buffered, so the copies of group i + 1 fly while group i is counted.
// All threads wait for the group's mbarrier phase, read their 128-bit chunk of
// each row from shared memory and fold it into the same bit-sliced carry-save
// counter as the direct kernel.
//
// Every wait is bounded: a thread that does not see its phase complete within the
// iteration limit reports it, the CTA agrees on the failure at its next barrier,
// gives its outstanding copies one more bounded wait, sets bit 0 of *status and
// returns without writing output.  No wait here depends on another CTA.

#include "host_common.h"

namespace {

constexpr int kStageRows = 8;                 // rows per group = per mbarrier phase
constexpr int kStages = 2;                    // groups in flight
constexpr int kTileWords = kThreads * 4;      // 1024 words = 4 KB per row and tile
constexpr unsigned kSpinLimit = 1u << 20;     // polls before giving up: some 0.1 s, a legitimate wait is microseconds
constexpr size_t kStagedSmemBytes = (size_t)kStages * kStageRows * kTileWords * sizeof(uint32_t);

__device__ __forceinline__ unsigned smem_addr(const void* p) {
  return (unsigned)__cvta_generic_to_shared(p);
}

__device__ __forceinline__ void mbar_init(unsigned bar, unsigned count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}

__device__ __forceinline__ void mbar_expect_tx(unsigned bar, unsigned bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}

// global -> shared bulk copy of `bytes` (a multiple of 16; both addresses 16-byte aligned), completion
// reported to the mbarrier as transferred bytes.  The destination is this CTA's own shared memory.
__device__ __forceinline__ void bulk_load(unsigned dst, const void* src, unsigned bytes, unsigned bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar)
               : "memory");
}

// true once the phase with the given parity has completed; false if it has not within the limit.
// The poll is the non-blocking test_wait, so that the limit is a number of instructions, not of
// hardware-defined suspensions.
__device__ __forceinline__ bool mbar_wait(unsigned bar, unsigned parity) {
  for (unsigned it = 0; it < kSpinLimit; ++it) {
    unsigned done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(bar), "r"(parity)
        : "memory");
    if (done) return true;
  }
  return false;
}

template <int NP>
__global__ void __launch_bounds__(kThreads)
vote_staged_kernel(const uint32_t* __restrict__ bits, unsigned M, unsigned long long d, unsigned long long W,
                   unsigned long long ldw, uint32_t* __restrict__ vote, unsigned start_value,
                   unsigned* __restrict__ status, unsigned starve_bytes) {
  extern __shared__ __align__(128) uint32_t stage[];   // [kStages][kStageRows][kTileWords]
  __shared__ __align__(8) unsigned long long bars[kStages];

  const unsigned long long chunks = (W + 3) / 4;
  const unsigned long long word0 = (unsigned long long)blockIdx.x * kTileWords;       // first word of the tile
  const unsigned long long left = chunks * 4 - word0;                                // words left in the row, padded to 4
  const unsigned tile_bytes = (unsigned)((left < (unsigned long long)kTileWords ? left : kTileWords) * sizeof(uint32_t));
  const unsigned groups = (M + kStageRows - 1) / kStageRows;
  const unsigned bar0 = smem_addr(&bars[0]);
  const unsigned stage0 = smem_addr(stage);

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) mbar_init(bar0 + 8u * s, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();

  // the elected thread arms the slot's mbarrier and issues one bulk copy per row of the group
  auto issue = [&](unsigned group) {
    const unsigned slot = group % kStages;
    const unsigned first = group * kStageRows;
    const unsigned rows = M - first < (unsigned)kStageRows ? M - first : (unsigned)kStageRows;
    const unsigned bar = bar0 + 8u * slot;
    // the slot's earlier reads (generic proxy) are ordered before the copies' writes (async proxy)
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    mbar_expect_tx(bar, rows * tile_bytes + starve_bytes);   // starve_bytes is 0 except in the self-test
    for (unsigned r = 0; r < rows; ++r)
      bulk_load(stage0 + (slot * kStageRows + r) * (unsigned)(kTileWords * sizeof(uint32_t)),
                bits + (unsigned long long)(first + r) * ldw + word0, tile_bytes, bar);
  };

  Counter<NP> cnt;
#pragma unroll
  for (int p = 0; p < NP; ++p) {
    const unsigned f = ((start_value >> p) & 1u) ? 0xFFFFFFFFu : 0u;
    cnt.c[p] = W4{f, f, f, f};
  }

  if (threadIdx.x == 0) issue(0);
  unsigned issued = 1;
  bool failed = false;
  for (unsigned g = 0; g < groups; ++g) {
    // slot (g + 1) % kStages was last read in iteration g - 1, which ended with a CTA barrier
    if (threadIdx.x == 0 && g + 1 < groups) issue(g + 1);
    if (g + 1 < groups) issued = g + 2;
    const unsigned slot = g % kStages;
    const bool ok = mbar_wait(bar0 + 8u * slot, (g / kStages) & 1u);
    if (__syncthreads_or(ok ? 0 : 1)) {   // the CTA leaves together
      failed = true;
      break;
    }
    const unsigned first = g * kStageRows;
    const unsigned rows = M - first < (unsigned)kStageRows ? M - first : (unsigned)kStageRows;
    const uint32_t* mine = stage + (size_t)slot * kStageRows * kTileWords + threadIdx.x * 4;
    W4 a[kStageRows];
#pragma unroll
    for (int r = 0; r < kStageRows; ++r) {
      if ((unsigned)r < rows) {
        const uint4 v = *reinterpret_cast<const uint4*>(mine + (size_t)r * kTileWords);
        a[r] = W4{v.x, v.y, v.z, v.w};
      } else {
        a[r] = W4{0u, 0u, 0u, 0u};
      }
    }
    if (NP >= 4 && rows == (unsigned)kStageRows) {
      cnt.add8(a);
    } else {
#pragma unroll
      for (int r = 0; r < kStageRows; ++r)
        if ((unsigned)r < rows) cnt.template add<0>(a[r]);
    }
    __syncthreads();   // everyone is done with this slot before it is filled again
  }

  if (failed) {
    // copies may still be on their way into this CTA's shared memory: give each armed phase one more
    // bounded wait before the CTA gives the memory up, then report
    for (unsigned g = 0; g < issued; ++g)
      if (g + kStages >= issued) (void)mbar_wait(bar0 + 8u * (g % kStages), (g / kStages) & 1u);
    if (threadIdx.x == 0) atomicOr(status, 1u);
    return;
  }
  const unsigned long long q = (unsigned long long)blockIdx.x * kThreads + threadIdx.x;
  if (q < chunks) store_plane_words(vote, q, d, cnt.c[NP - 1]);
}

template <int NP>
ssgd_status launch_staged_np(const uint32_t* bits, size_t M, size_t d, size_t ldw, uint32_t* vote,
                             unsigned* status, unsigned starve_bytes, cudaStream_t s) {
  const size_t W = ssgd_words(d);
  const unsigned long long tiles = (W + kTileWords - 1) / kTileWords;
  if (tiles > kMaxGrid) return SSGD_ERR_SIZE;
  auto kernel = vote_staged_kernel<NP>;
  if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kStagedSmemBytes) != cudaSuccess)
    return SSGD_ERR_CUDA;
  kernel<<<(unsigned)tiles, kThreads, kStagedSmemBytes, s>>>(bits, (unsigned)M, d, W, ldw, vote,
                                                             vote_start_value(M, NP), status, starve_bytes);
  return launch_status();
}

ssgd_status staged_vote(const uint32_t* bits, size_t M, size_t d, size_t ldw, uint32_t* vote, unsigned* status,
                        unsigned starve_bytes, void* stream) {
  if (!bits || !vote || !status) return SSGD_ERR_NULL;
  if (!aligned16(bits) || !aligned16(vote) || (reinterpret_cast<uintptr_t>(status) & 3u) != 0) return SSGD_ERR_ALIGN;
  const ssgd_status st = check_rows(M, d, 0, ldw, false);
  if (st != SSGD_OK || d == 0) return st;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  switch (vote_planes(M)) {
    case 1: return launch_staged_np<1>(bits, M, d, ldw, vote, status, starve_bytes, s);
    case 2: return launch_staged_np<2>(bits, M, d, ldw, vote, status, starve_bytes, s);
    case 3: return launch_staged_np<3>(bits, M, d, ldw, vote, status, starve_bytes, s);
    case 4: return launch_staged_np<4>(bits, M, d, ldw, vote, status, starve_bytes, s);
    case 5: return launch_staged_np<5>(bits, M, d, ldw, vote, status, starve_bytes, s);
    case 6: return launch_staged_np<6>(bits, M, d, ldw, vote, status, starve_bytes, s);
    case 7: return launch_staged_np<7>(bits, M, d, ldw, vote, status, starve_bytes, s);
    case 8: return launch_staged_np<8>(bits, M, d, ldw, vote, status, starve_bytes, s);
    case 9: return launch_staged_np<9>(bits, M, d, ldw, vote, status, starve_bytes, s);
    case 10: return launch_staged_np<10>(bits, M, d, ldw, vote, status, starve_bytes, s);
    case 11: return launch_staged_np<11>(bits, M, d, ldw, vote, status, starve_bytes, s);
  }
  return SSGD_ERR_SIZE;
}

}  // namespace

extern "C" ssgd_status ssgd_majority_vote_staged(const uint32_t* bits, size_t M, size_t d, size_t ldw,
                                                 uint32_t* vote, unsigned* status, void* stream) {
  return staged_vote(bits, M, d, ldw, vote, status, 0u, stream);
}

// The same launch with every mbarrier phase armed for 16 bytes more than its copies deliver, so that no
// phase ever completes: all copies still arrive (nothing is left in flight), every wait runs into its
// limit, and the kernel must come back with bit 0 of *status set and the output untouched.
extern "C" ssgd_status ssgd_majority_vote_staged_wait_selftest(const uint32_t* bits, size_t M, size_t d,
                                                               size_t ldw, uint32_t* vote, unsigned* status,
                                                               void* stream) {
  if (d > 32768) return SSGD_ERR_SIZE;   // one tile is enough to exercise the path; keeps the run short
  return staged_vote(bits, M, d, ldw, vote, status, 16u, stream);
}
