// The whole step (Algorithm 3: worker step of every row, majority vote, apply) for SHORT vectors, as one
// kernel whose warps work on different rows at the same time.  Unnamed namespace: included by the unit
// that holds the step entry points.
//
// fused_step_kernel walks the M rows of its columns one after another, which is right for long vectors
// (few concurrent streams, many loads in flight per thread) but makes a short launch a chain of M + 1
// dependent round trips to memory; the three-kernel form pays three launches instead.  Here a CTA owns
// 128 columns (four words) and its eight warps take the rows w, w + 8, w + 16, ... of those columns, RIF
// rows per warp in flight at once (1, 2 or 4: enough for all M <= 8, 16, 32 rows), so that a step with up
// to 32 workers is ONE launch and ONE round trip for g and m (x is fetched at the same time).  Each warp
// keeps the bit-sliced count of its own rows; the eight partial counts meet in shared memory, and the
// first warp adds them (a ripple-carry addition over the planes), writes the voted words and updates x.
// Per parameter it moves what fused_step_kernel moves: 12.125 M + 8.125 bytes (4.125 M + 8.125 without a
// momentum).  Each thread has only two to eight 128-bit loads in flight, so it is the slower kernel as
// soon as bandwidth matters; the host uses it below a measured number of tiles (see step_rows_max_tiles).
// The launch bounds hold the register allocation to 48 / 64 / 85 registers for RIF = 1 / 2 / 4 (5 / 4 / 3
// resident CTAs per SM; 128 registers for the six-plane form, M = 32, which would spill at 85), which is
// what its range on the middling sizes depends on.
#ifndef SSGD_STEP_ROWS_CUH_
#define SSGD_STEP_ROWS_CUH_

#include "host_common.h"

namespace {

constexpr int kRowsKernelMaxWorkers = 32;   // rows per CTA at most: 8 warps x 4 rows in flight
constexpr int kRowsKernelMaxPlanes = 6;     // planes needed for M <= 32

// Four consecutive elements starting at e, those at or beyond d read as 0 / are not written.
__device__ __forceinline__ float4 load4_below(const float* p, unsigned long long e, unsigned long long d) {
  return make_float4(e < d ? p[0] : 0.0f, e + 1 < d ? p[1] : 0.0f, e + 2 < d ? p[2] : 0.0f, e + 3 < d ? p[3] : 0.0f);
}
__device__ __forceinline__ void store4_below(float* p, unsigned long long e, unsigned long long d, const float4& v) {
  if (e < d) p[0] = v.x;
  if (e + 1 < d) p[1] = v.y;
  if (e + 2 < d) p[2] = v.z;
  if (e + 3 < d) p[3] = v.w;
}

template <int MODE, int NP, int RIF>
__global__ void __launch_bounds__(kThreads, RIF <= 1 ? 5 : (RIF == 2 ? 4 : (NP >= 6 ? 2 : 3)))
step_rows_kernel(const float* __restrict__ g, float* __restrict__ m, float* __restrict__ x,
                 uint32_t* __restrict__ bits, uint32_t* __restrict__ vote, unsigned M,
                 unsigned long long d, unsigned long long ld, unsigned long long ldw, float beta,
                 float omb, float delta, unsigned start_value) {
  constexpr bool MOMENTUM = MODE != kSignSGD;
  constexpr bool SIGN_OF_G = MODE != kSignum;
  constexpr unsigned kWarps = kThreads / 32;
  __shared__ unsigned part[kWarps][NP][4];   // partial counts: [warp][plane][word of the tile]
  pdl_launch_dependents();
  pdl_wait();
  const unsigned lane = threadIdx.x & 31u;
  const unsigned warp = threadIdx.x >> 5;
  const unsigned group = lane >> 3;          // which of the tile's four words this lane's bits go to
  const unsigned sub = lane & 7u;
  const unsigned long long c0 = (unsigned long long)blockIdx.x * 128;   // first column of the tile
  const unsigned long long e = c0 + lane * 4;                          // this lane's first column
  const bool interior = c0 + 128 <= d;                                 // uniform over the CTA
  const bool own_word = sub == 0 && c0 + 32ull * group < d;            // this lane stores its group's word
  // bits of this lane's nibble that belong to elements below d
  const unsigned valid = interior ? 0xFu
                                  : ((e < d ? 1u : 0u) | (e + 1 < d ? 2u : 0u) | (e + 2 < d ? 4u : 0u) | (e + 3 < d ? 8u : 0u));
  float4 xv = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
  if (warp == 0) xv = interior ? ld128(x + e) : load4_below(x + e, e, d);   // early: needed after the vote

  Counter1<NP> cnt;
  cnt.init(0u);
  for (unsigned r0 = warp; r0 < M; r0 += kWarps * RIF) {
    float4 gv[RIF], mv[RIF];
#pragma unroll
    for (int k = 0; k < RIF; ++k) {
      const unsigned r = r0 + kWarps * k;
      if (r < M) {                                                     // uniform over the warp
        const float* gp = g + (unsigned long long)r * ld + e;
        gv[k] = interior ? ld128(gp) : load4_below(gp, e, d);
        if (MOMENTUM) {
          const float* mp = m + (unsigned long long)r * ld + e;
          mv[k] = interior ? ld128(mp) : load4_below(mp, e, d);
        }
      }
    }
#pragma unroll
    for (int k = 0; k < RIF; ++k) {
      const unsigned r = r0 + kWarps * k;
      if (r < M) {
        float4 v = gv[k];
        if (MOMENTUM) {
          v = momentum_update4(beta, omb, mv[k], v);
          float* mp = m + (unsigned long long)r * ld + e;
          if (interior) st128(mp, v);
          else store4_below(mp, e, d, v);
        }
        const unsigned word = assemble_word(sign_nibble(SIGN_OF_G ? gv[k] : v) & valid, lane);
        if (own_word) bits[(unsigned long long)r * ldw + (c0 >> 5) + group] = word;
        cnt.template add<0>(word);
      }
    }
  }
  if (sub == 0) {
#pragma unroll
    for (int p = 0; p < NP; ++p) part[warp][p][group] = cnt.c[p];
  }
  __syncthreads();
  if (warp != 0) return;

  // total = start value + the eight partial counts, plane by plane with a rippling carry.  The host sizes
  // NP so that the total stays below 2^NP; its top plane is the voted bit (see vote_kernel).
  Counter1<NP> total;
  total.init(start_value);
#pragma unroll
  for (unsigned w = 0; w < kWarps; ++w) {
    unsigned carry = 0u;
#pragma unroll
    for (int p = 0; p < NP; ++p) {
      const unsigned a = part[w][p][group];
      const unsigned sum = xor3(total.c[p], a, carry);
      carry = maj3(total.c[p], a, carry);
      total.c[p] = sum;
    }
  }
  const unsigned voted = total.top();   // bits at positions >= d: every row has 0 there, the count stays below the threshold
  if (own_word) vote[(c0 >> 5) + group] = voted;
  const float4 xn = apply4(xv, voted >> (4u * sub), delta, -delta);
  if (interior) st128(x + e, xn);
  else store4_below(x + e, e, d, xn);
}

// Tiles (of 128 columns) up to which the row-parallel kernel is the faster form of the step, stated per SM
// of the device.  Measured on B200 (148 SMs; 512 tiles are d = 2^16) against fused_step_kernel (M <= 8)
// and against worker + vote + apply, with and without a momentum (the crossovers agree), d = 2^10 .. 2^21:
//   one worker: never (the fused kernel is then a single round trip itself);
//   M = 2 up to d = 2^16; M = 3 .. 5 up to 2^17; M = 6 .. 8 up to 2^18; M = 9 .. 16 up to 2^17;
//   M = 17 .. 32 up to 2^16.
// Examples, us per step, this kernel against the other form: M = 8, d = 2^16: 4.1 / 10.8; M = 3, d = 2^15:
// 2.1 / 3.0; M = 16, d = 2^16: 5.3 / 7.8; M = 31, d = 2^14: 4.9 / 7.9.  One size further up it loses: each
// thread has too few loads in flight to compete once bandwidth matters (M = 7, d = 2^20: 26 / 17).
inline unsigned long long step_rows_max_tiles(size_t M, int sms) {
  unsigned per_sm;
  if (M <= 1) per_sm = 0;
  else if (M == 2) per_sm = 4;
  else if (M <= 5) per_sm = 8;
  else if (M <= 8) per_sm = 16;
  else if (M <= 16) per_sm = 8;
  else per_sm = 4;
  return (unsigned long long)per_sm * (unsigned long long)sms;
}

inline bool step_uses_rows_kernel(size_t M, size_t d, int sms) {
  return M <= (size_t)kRowsKernelMaxWorkers && (d + 127) / 128 <= step_rows_max_tiles(M, sms);
}

template <int MODE, int NP, int RIF>
void launch_step_rows_np(const StepArgs& a, cudaStream_t s) {
  const unsigned tiles = (unsigned)((a.d + 127) / 128);
  launch_kernel(step_rows_kernel<MODE, NP, RIF>, tiles, kThreads, 0, s, true, a.g, a.m, a.x, a.bits, a.vote,
                (unsigned)a.M, (unsigned long long)a.d, (unsigned long long)a.ld, (unsigned long long)a.ldw, a.beta,
                1.0f - a.beta, a.delta, vote_start_value(a.M, NP));
}

template <int MODE>
ssgd_status launch_step_rows(const StepArgs& a, cudaStream_t s) {
  static_assert(kRowsKernelMaxWorkers / 2 < (1 << (kRowsKernelMaxPlanes - 1)), "planes cover the worker limit");
  // planes 2..4 <=> M = 2 .. 15, 5 <=> M = 16 .. 31, 6 <=> M = 32; rows in flight per warp = ceil(M / 8) rounded up to
  // 1, 2 or 4.  One worker (one plane) never takes this kernel (step_rows_max_tiles).
  switch (vote_planes(a.M)) {
    case 2: launch_step_rows_np<MODE, 2, 1>(a, s); break;
    case 3: launch_step_rows_np<MODE, 3, 1>(a, s); break;
    case 4:
      if (a.M <= 8) launch_step_rows_np<MODE, 4, 1>(a, s);
      else launch_step_rows_np<MODE, 4, 2>(a, s);
      break;
    case 5:
      if (a.M <= 16) launch_step_rows_np<MODE, 5, 2>(a, s);
      else launch_step_rows_np<MODE, 5, 4>(a, s);
      break;
    case 6: launch_step_rows_np<MODE, 6, 4>(a, s); break;
    default: return SSGD_ERR_SIZE;
  }
  return launch_status();
}

}  // namespace

#endif  // SSGD_STEP_ROWS_CUH_
