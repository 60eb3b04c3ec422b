// Gradient statistics of Section 3: the density phi(v) = |v|_1^2 / (d |v|_2^2)
// of a vector, and Welford's single-pass mean / variance over gradient samples
// (how the paper measures the true gradient g and its noise vector sigma).
// See include/signsgd.h for the contract of each call.

#include "host_common.h"

namespace {

// One sample folded into the running mean and sum of squared deviations
// (Welford's update), per element, with this rounding sequence in fp32:
//   d1 = g - mean;  mean' = mean + d1 / n;  d2 = g - mean';  m2' = fma(d1, d2, m2).
__device__ __forceinline__ void welford1(float g, float n, float& mean, float& m2) {
  const float d1 = __fsub_rn(g, mean);
  mean = __fadd_rn(mean, __fdiv_rn(d1, n));
  const float d2 = __fsub_rn(g, mean);
  m2 = __fmaf_rn(d1, d2, m2);
}

__global__ void __launch_bounds__(kThreads)
welford_kernel(const float* __restrict__ g, float* __restrict__ mean, float* __restrict__ m2,
               unsigned long long d, float n) {
  const unsigned long long stride = (unsigned long long)gridDim.x * kThreads * 4;
  for (unsigned long long e = ((unsigned long long)blockIdx.x * kThreads + threadIdx.x) * 4; e < d; e += stride) {
    if (e + 4 <= d) {
      const float4 gv = ld128(g + e);
      float4 mu = ld128(mean + e);
      float4 s = ld128(m2 + e);
      welford1(gv.x, n, mu.x, s.x);
      welford1(gv.y, n, mu.y, s.y);
      welford1(gv.z, n, mu.z, s.z);
      welford1(gv.w, n, mu.w, s.w);
      st128(mean + e, mu);
      st128(m2 + e, s);
    } else {
      for (unsigned long long i = e; i < d; ++i) welford1(g[i], n, mean[i], m2[i]);
    }
  }
}

// sums[0] += sum_i |t_i|, sums[1] += sum_i t_i^2 with t = v, or t = sqrt(v) when
// ROOT (then sums[1] is sum_i v_i): all that phi needs.  Accumulated in fp64:
// per thread, then per warp by shuffles, per CTA through shared memory, and one
// atomic add per CTA and quantity.
constexpr int kDensityUnroll = 4;   // 128-bit loads in flight per thread

template <bool ROOT>
__device__ __forceinline__ void density_term(float t, double& l1, double& l2) {
  const double td = (double)t;
  if (ROOT) {
    l1 += sqrt(td);
    l2 += td;
  } else {
    l1 += fabs(td);
    l2 = fma(td, td, l2);
  }
}

template <bool ROOT>
__global__ void __launch_bounds__(kThreads)
density_sums_kernel(const float* __restrict__ v, unsigned long long d, double* __restrict__ sums) {
  constexpr unsigned long long TILE = (unsigned long long)kThreads * 4 * kDensityUnroll;
  double l1 = 0.0, l2 = 0.0;
  for (unsigned long long t0 = (unsigned long long)blockIdx.x * TILE; t0 < d; t0 += (unsigned long long)gridDim.x * TILE) {
    if (t0 + TILE <= d) {
      float4 q[kDensityUnroll];
#pragma unroll
      for (int u = 0; u < kDensityUnroll; ++u) q[u] = ld128(v + t0 + (unsigned long long)u * kThreads * 4 + threadIdx.x * 4);
#pragma unroll
      for (int u = 0; u < kDensityUnroll; ++u) {
        density_term<ROOT>(q[u].x, l1, l2);
        density_term<ROOT>(q[u].y, l1, l2);
        density_term<ROOT>(q[u].z, l1, l2);
        density_term<ROOT>(q[u].w, l1, l2);
      }
    } else {
      for (unsigned long long i = t0 + threadIdx.x; i < d; i += kThreads) density_term<ROOT>(v[i], l1, l2);
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    l1 += __shfl_xor_sync(0xFFFFFFFFu, l1, o);
    l2 += __shfl_xor_sync(0xFFFFFFFFu, l2, o);
  }
  __shared__ double part[2][kThreads / 32];
  const unsigned lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
  if (lane == 0) {
    part[0][warp] = l1;
    part[1][warp] = l2;
  }
  __syncthreads();
  if (threadIdx.x < 2) {
    double s = 0.0;
#pragma unroll
    for (int w = 0; w < kThreads / 32; ++w) s += part[threadIdx.x][w];
    atomicAdd(sums + threadIdx.x, s);
  }
}

}  // namespace

extern "C" {

ssgd_status ssgd_welford_update(const float* g, size_t n, float* mean, float* m2, size_t d, void* stream) {
  if (!g || !mean || !m2) return SSGD_ERR_NULL;
  if (!aligned16(g) || !aligned16(mean) || !aligned16(m2)) return SSGD_ERR_ALIGN;
  if (d > SIZE_MAX - 31) return SSGD_ERR_SIZE;
  if (n < 1 || n > ((size_t)1 << 24)) return SSGD_ERR_ARG;   // n must be exact in fp32
  if (d == 0) return SSGD_OK;
  const unsigned long long ctas = ((d + 3) / 4 + kThreads - 1) / kThreads;
  welford_kernel<<<grid_for(ctas), kThreads, 0, static_cast<cudaStream_t>(stream)>>>(g, mean, m2, d, (float)n);
  return launch_status();
}

ssgd_status ssgd_density_sums(const float* v, size_t d, int root, double* sums, void* stream) {
  if (!v || !sums) return SSGD_ERR_NULL;
  if (!aligned16(v) || !aligned16(sums)) return SSGD_ERR_ALIGN;
  if (d > SIZE_MAX - 31) return SSGD_ERR_SIZE;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (cudaMemsetAsync(sums, 0, 2 * sizeof(double), s) != cudaSuccess) return SSGD_ERR_CUDA;
  if (d == 0) return SSGD_OK;
  const unsigned long long tile = (unsigned long long)kThreads * 4 * kDensityUnroll;
  const unsigned long long ctas = (d + tile - 1) / tile;
  if (root)
    density_sums_kernel<true><<<grid_for(ctas), kThreads, 0, s>>>(v, d, sums);
  else
    density_sums_kernel<false><<<grid_for(ctas), kThreads, 0, s>>>(v, d, sums);
  return launch_status();
}

double ssgd_density_from_sums(double l1, double l2_squared, size_t d) {
  if (d == 0 || !(l2_squared > 0.0)) return 0.0;
  return l1 * l1 / ((double)d * l2_squared);
}

}  // extern "C"
