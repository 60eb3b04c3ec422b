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

// One tile per CTA; the kernels keep a grid-stride loop for grids beyond the limit.
constexpr unsigned long long kMaxGrid = 0x7FFFFFFFull;
unsigned grid_for(unsigned long long ctas) { return (unsigned)(ctas < kMaxGrid ? ctas : kMaxGrid); }

// Elements per thread: 4 * unroll.  Large inputs take the largest unroll allowed
// (eight 128-bit loads in flight per thread in the worker step); smaller ones
// shrink the tile so that the launch still fills the machine with a few CTAs per SM.
int pick_unroll(unsigned long long elements_per_row, unsigned long long rows, int sms, int max_unroll = 4) {
  const unsigned long long want = 8ull * sms;                  // CTAs
  for (int u = max_unroll; u > 1; u /= 2) {
    const unsigned long long tile = (unsigned long long)kThreads * 4 * u;
    if (((elements_per_row + tile - 1) / tile) * rows >= want) return u;
  }
  return 1;
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
