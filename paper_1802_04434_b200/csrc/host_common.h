// Host-side helpers shared by the entry points: argument checks, launch shapes,
// plane counts.  Unnamed namespace: one copy per translation unit.
#ifndef SSGD_HOST_COMMON_H_
#define SSGD_HOST_COMMON_H_

#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

#include "signsgd.h"
#include "device_common.cuh"

namespace {

struct DeviceInfo {
  int sms;
};

bool device_info(DeviceInfo* out) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return false;
  static int cached_sms[64] = {0};   // filled on first use; any thread stores the same value
  if (dev < 0 || dev >= 64) return false;
  int sms = __atomic_load_n(&cached_sms[dev], __ATOMIC_RELAXED);
  if (sms == 0) {
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
      return false;
    __atomic_store_n(&cached_sms[dev], sms, __ATOMIC_RELAXED);
  }
  out->sms = sms;
  return true;
}

// Arguments of one whole step (ssgd_signsgd_step and its warm-up form).
struct StepArgs {
  const float* g;
  float* m;
  float* x;
  uint32_t* bits;
  uint32_t* vote;
  size_t M, d, ld, ldw;
  float beta, delta;
};

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

inline bool mul_overflows(size_t a, size_t b) { return b != 0 && a > SIZE_MAX / b; }

ssgd_status check_rows(size_t M, size_t d, size_t ld, size_t ldw, bool need_ld) {
  if (M < 1 || M > SSGD_MAX_WORKERS) return SSGD_ERR_SIZE;
  if (d > SIZE_MAX - 31) return SSGD_ERR_SIZE;
  const size_t W = ssgd_words(d);
  if (need_ld) {
    if (ld % 4 != 0) return SSGD_ERR_ALIGN;
    if (ld < d || mul_overflows(M, ld) || mul_overflows(M * ld, sizeof(float))) return SSGD_ERR_SIZE;
  }
  if (ldw % 4 != 0) return SSGD_ERR_ALIGN;
  if (ldw < W || mul_overflows(M, ldw) || mul_overflows(M * ldw, sizeof(uint32_t))) return SSGD_ERR_SIZE;
  return SSGD_OK;
}

inline bool beta_ok(float beta) { return beta >= 0.0f && beta < 1.0f; }  // false for NaN

ssgd_status launch_status() { return cudaGetLastError() == cudaSuccess ? SSGD_OK : SSGD_ERR_CUDA; }

// Kernel launch with the programmatic-serialization attribute (see pdl_wait in device_common.cuh), for
// kernels that begin with pdl_wait(); pdl = false gives an ordinary launch.
template <typename... KArgs, typename... Args>
void launch_kernel(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, bool pdl,
                   Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl ? 1 : 0;
  (void)cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);   // errors are read by launch_status()
}

// One tile per CTA; the kernels keep a grid-stride loop for grids beyond the limit.
constexpr unsigned long long kMaxGrid = 0x7FFFFFFFull;
unsigned grid_for(unsigned long long ctas) { return (unsigned)(ctas < kMaxGrid ? ctas : kMaxGrid); }

// Tile choice.  A thread handles 4 * unroll elements of one row, a CTA a tile of kThreads * 4 * unroll.
// Large tiles give each thread more independent loads in flight and suit long streams; small tiles give a
// short launch more CTAs to spread over the SMs.  The crossovers below were measured on B200 (148 SMs) by
// forcing every tile size over d = 2^14 .. 2^27 and M = 1 .. 16, and are stated in tiles per SM.
inline unsigned long long tile_count(unsigned long long elements_per_row, unsigned long long rows, int unroll) {
  const unsigned long long tile = (unsigned long long)kThreads * 4 * unroll;
  return ((elements_per_row + tile - 1) / tile) * rows;
}

// Worker kernel.  With a momentum: the interior-only 4096-element tiles win from about 64 Mi elements on
// (2-4 % over 1024-element tiles), below that the 1024-element tiles win by 1-5 %; 2048 is never best.
// Sign-only (one array): 8192-element tiles from about 32 Mi elements, 2048 from about 1.5 Mi, else 1024.
inline int worker_unroll(unsigned long long d, unsigned long long rows, int sms, bool momentum) {
  if (momentum) return tile_count(d, rows, 4) >= 112ull * sms ? 4 : 1;
  if (tile_count(d, rows, 8) >= 24ull * sms) return 8;
  return tile_count(d, rows, 2) >= 5ull * sms ? 2 : 1;
}

// Fused step kernel (a CTA walks all rows of its columns): the larger tile as soon as it still gives
// three CTAs per SM (17-40 % faster than the next smaller tile at d = 2^20 .. 2^21, equal from 2^22 on).
inline int fused_unroll(unsigned long long d, int sms, bool momentum) {
  if (!momentum && tile_count(d, 1, 4) >= 3ull * sms) return 4;
  return tile_count(d, 1, 2) >= 3ull * sms ? 2 : 1;
}

// Apply kernel: interior-only 2048-element tiles once they fill the machine 8 CTAs deep (no measurable
// difference between the tile sizes below that).
inline int apply_unroll(unsigned long long d, int sms) { return tile_count(d, 1, 2) >= 8ull * sms ? 2 : 1; }

// Vote kernel: the remaining rows after the batches of eight come as one guarded batch (see vote_kernel)
// with four to six planes (M = 8 .. 127: 5-20 % faster at every size measured).  With more planes the
// kernel makes eight and more round trips anyway and the guarded form would go from 64 to 72-80
// registers.  One plane is one row; two and three planes (M = 2 .. 7) have a kernel of their own.
constexpr int kGuardedMinPlanes = 4;
constexpr int kGuardedMaxPlanes = 6;
inline bool vote_guarded(unsigned planes) {
  return planes >= (unsigned)kGuardedMinPlanes && planes <= (unsigned)kGuardedMaxPlanes;
}

// Vote of many rows on a short vector: the kernel that spreads the rows over the warps of a CTA (one CTA
// per 32 chunks of four words), from 13 rows on, while its grid is at most 4 CTAs per SM (13 .. 23 rows:
// d up to 2^21 on 148 SMs) or 8 CTAs per SM (24 rows and more: d up to 2^22); measured crossovers on B200.
inline bool vote_split(size_t M, unsigned long long chunks, int sms) {
  if (M < 13) return false;
  return (chunks + 31) / 32 <= (M >= 24 ? 8ull : 4ull) * (unsigned long long)sms;
}

unsigned vote_planes(size_t M) {
  unsigned L = 0;
  while ((M / 2) >= (size_t(1) << L)) ++L;  // smallest L with floor(M/2) < 2^L
  return L + 1;
}

// counter start value 2^(NP-1) - ceil(M/2), see the vote kernel
unsigned vote_start_value(size_t M, unsigned planes) {
  return (1u << (planes - 1)) - (unsigned)((M + 1) / 2);
}

}  // namespace

#endif  // SSGD_HOST_COMMON_H_
