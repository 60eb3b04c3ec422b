// sm_100a kernels and C ABI for the signSGD / Signum / majority-vote step
// (Algorithms 1-3 of Bernstein et al., "signSGD: Compressed Optimisation for
// Non-Convex Problems").  See include/signsgd.h for the contract of each call.
//
// Every kernel here streams its operands once and is bound by HBM bandwidth:
//   worker kernel   12.125 B per parameter per worker (g read, m read + write,
//                   1/8 B of sign bits written); 4.125 B for the sign-only form
//   vote kernel     (M + 1) / 8 B per parameter
//   apply kernel    8.125 B per parameter
//   fused step      12.125 M + 8.125 B per parameter (the three above in one
//                   launch; the sign words are not read back)
// No step is a contraction, so there is no tensor-core work.  The design rules
// that measurement on B200 settled: 128-bit coalesced accesses, eight independent
// loads in flight per thread, one tile per CTA (the hardware's CTA scheduler
// balances DRAM channels better than a persistent grid-stride loop did), default
// caching on loads and streaming stores, 64-bit indexing (M * d exceeds 2^32).
// Staging tiles through shared memory with bulk asynchronous copies was tried for
// the worker kernel and was 15-25 % slower than direct register loads: there is
// no reuse for shared memory to serve, only an extra hop.

#include "host_common.h"
#include "vote_launch.h"
#include "step_rows.cuh"

namespace {

// ---------------------------------------------------------------------------
// worker step: [momentum update +] sign + 1-bit pack, all M rows in one launch.
// Grid: x = tile within the row, y = row; one tile per CTA, consecutive CTAs on
// consecutive tiles of a row.  A warp owns a span of 128 * UNROLL consecutive
// elements of one row.

// One span that crosses the end of its row: element-wise guards, padding bits
// stay 0, and nothing at or beyond d is written.
template <int MODE, int UNROLL>
__device__ __forceinline__ void worker_ragged_span(const float* __restrict__ gr, float* __restrict__ mr,
                                                   uint32_t* __restrict__ br, unsigned long long d,
                                                   unsigned long long e0, float beta, float omb) {
  constexpr bool MOMENTUM = MODE != kSignSGD;
  constexpr bool SIGN_OF_G = MODE != kSignum;
  const unsigned lane = threadIdx.x & 31u;
#pragma unroll 1
  for (int u = 0; u < UNROLL; ++u) {
    const unsigned long long e = e0 + u * 128 + lane * 4;
    unsigned nib = 0;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      if (e + k < d) {
        const float gk = gr[e + k];
        float v = gk;
        if (MOMENTUM) {
          v = momentum_update(beta, omb, mr[e + k], gk);
          mr[e + k] = v;
        }
        nib |= sign_bit(SIGN_OF_G ? gk : v) << k;
      }
    }
    const unsigned word = assemble_word(nib, lane);
    const unsigned long long first = e0 + u * 128 + (lane >> 3) * 32;  // first element of the word
    if ((lane & 7u) == 0 && first < d) br[u * 4 + (lane >> 3)] = word;
  }
}

// RAGGED = true: the kernel also handles the span that crosses the end of the row
// (used for the small tiles, where one launch matters more than the last per cent
// of bandwidth).  RAGGED = false: such a span is left to worker_tail_kernel, and
// this kernel is nothing but the interior path.  Measured on B200 at d = 335 M,
// M = 16: with the guarded path compiled into the same kernel the interior path
// gets a different register allocation (40 or 48 registers instead of 52, hence
// 6 or 5 resident CTAs per SM instead of 4) and streams 1.5-2.5 % slower.
template <int MODE, int UNROLL, bool RAGGED>
__global__ void __launch_bounds__(kThreads, 1)
worker_pack_kernel(const float* __restrict__ g, float* __restrict__ m,
                   uint32_t* __restrict__ bits, unsigned long long d,
                   unsigned long long ld, unsigned long long ldw, float beta, float omb) {
  constexpr bool MOMENTUM = MODE != kSignSGD;
  constexpr bool SIGN_OF_G = MODE != kSignum;
  constexpr unsigned long long TILE = (unsigned long long)kThreads * 4 * UNROLL;
  constexpr unsigned SPAN = 128 * UNROLL;
  pdl_launch_dependents();
  pdl_wait();
  const unsigned lane = threadIdx.x & 31u;
  const unsigned warp = threadIdx.x >> 5;
  const unsigned long long row = blockIdx.y;
  // first element of this warp's span, within the row
  const unsigned long long e0 = (unsigned long long)blockIdx.x * TILE + (unsigned long long)warp * SPAN;
  if (e0 + SPAN > d) {   // uniform over the warp; nothing below synchronises across warps
    if (RAGGED && e0 < d)
      worker_ragged_span<MODE, UNROLL>(g + row * ld, MOMENTUM ? m + row * ld : nullptr,
                                       bits + row * ldw + (e0 >> 5), d, e0, beta, omb);
    return;
  }
  // interior: no bounds checks, all loads issued before any use
  const float* gr = g + row * ld + e0 + lane * 4;
  float* mr = MOMENTUM ? m + row * ld + e0 + lane * 4 : nullptr;
  float4 gv[UNROLL], mv[UNROLL];
#pragma unroll
  for (int u = 0; u < UNROLL; ++u) gv[u] = ld128(gr + u * 128);
  if (MOMENTUM) {
#pragma unroll
    for (int u = 0; u < UNROLL; ++u) mv[u] = ld128(mr + u * 128);
  }
  unsigned mine = 0;
#pragma unroll
  for (int u = 0; u < UNROLL; ++u) {
    float4 v = gv[u];
    if (MOMENTUM) {
      v = momentum_update4(beta, omb, mv[u], v);
      st128(mr + u * 128, v);
    }
    const unsigned word = assemble_word(sign_nibble(SIGN_OF_G ? gv[u] : v), lane);
    if ((lane & 7u) == (unsigned)u) mine = word;
  }
  if ((lane & 7u) < (unsigned)UNROLL) bits[row * ldw + (e0 >> 5) + own_word_index<UNROLL>(lane)] = mine;
}

// The last, partial span of every row, for the launches whose main kernel is
// interior-only: one warp per row.
template <int MODE, int UNROLL>
__global__ void __launch_bounds__(32)
worker_tail_kernel(const float* __restrict__ g, float* __restrict__ m, uint32_t* __restrict__ bits,
                   unsigned long long d, unsigned long long ld, unsigned long long ldw, float beta,
                   float omb) {
  constexpr unsigned SPAN = 128 * UNROLL;
  const unsigned long long row = blockIdx.x;
  const unsigned long long e0 = d / SPAN * SPAN;
  if (e0 >= d) return;
  worker_ragged_span<MODE, UNROLL>(g + row * ld, MODE != kSignSGD ? m + row * ld : nullptr,
                                   bits + row * ldw + (e0 >> 5), d, e0, beta, omb);
}

// ---------------------------------------------------------------------------
// apply: x <- x -/+ delta by the voted bit.  Thread layout as in the worker
// kernel: lane l of a warp holds elements 4l..4l+3 of a 128-element step, whose
// four bits sit at position 4(l%8) of word l/8 of that step.

// One span that crosses the end of x: element-wise, nothing at or beyond d is touched.
template <int UNROLL>
__device__ __forceinline__ void apply_ragged_span(float* __restrict__ x, const uint32_t* __restrict__ vote,
                                                  unsigned long long d, unsigned long long e0, float delta) {
  const unsigned lane = threadIdx.x & 31u;
  const float minus = -delta;
#pragma unroll 1
  for (int u = 0; u < UNROLL; ++u) {
    const unsigned long long e = e0 + u * 128 + lane * 4;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      if (e + k < d) {
        const unsigned bit = (vote[(e + k) >> 5] >> ((e + k) & 31u)) & 1u;
        x[e + k] = __fadd_rn(x[e + k], bit ? minus : delta);
      }
    }
  }
}

// RAGGED as in the worker kernel: true = the kernel also handles the span that
// crosses the end of x; false = interior only, the last partial span goes to
// apply_tail_kernel (measured at d = 2^26 .. 2^28: 6.84-6.90 TB/s against 6.70
// with the guarded path and a grid-stride loop compiled in).
template <int UNROLL, bool RAGGED>
__global__ void __launch_bounds__(kThreads, 1)
apply_kernel(float* __restrict__ x, const uint32_t* __restrict__ vote, unsigned long long d, float delta) {
  pdl_launch_dependents();
  pdl_wait();
  constexpr unsigned long long TILE = (unsigned long long)kThreads * 4 * UNROLL;
  constexpr unsigned SPAN = 128 * UNROLL;
  const unsigned lane = threadIdx.x & 31u;
  const unsigned warp = threadIdx.x >> 5;
  const unsigned long long e0 = (unsigned long long)blockIdx.x * TILE + (unsigned long long)warp * SPAN;
  if (e0 + SPAN > d) {
    if (RAGGED && e0 < d) apply_ragged_span<UNROLL>(x, vote, d, e0, delta);
    return;
  }
  const float minus = -delta;
  const uint32_t* vw = vote + (e0 >> 5);
  float* xr = x + e0 + lane * 4;
  float4 xv[UNROLL];
  unsigned wv[UNROLL];
#pragma unroll
  for (int u = 0; u < UNROLL; ++u) {
    xv[u] = ld128(xr + u * 128);
    wv[u] = __ldg(vw + u * 4 + (lane >> 3));
  }
#pragma unroll
  for (int u = 0; u < UNROLL; ++u)
    st128(xr + u * 128, apply4(xv[u], wv[u] >> (4u * (lane & 7u)), delta, minus));
}

template <int UNROLL>
__global__ void __launch_bounds__(32)
apply_tail_kernel(float* __restrict__ x, const uint32_t* __restrict__ vote, unsigned long long d, float delta) {
  constexpr unsigned SPAN = 128 * UNROLL;
  const unsigned long long e0 = d / SPAN * SPAN;
  if (e0 < d) apply_ragged_span<UNROLL>(x, vote, d, e0, delta);
}

// ---------------------------------------------------------------------------
// fused step: one launch does the worker step for all M rows, the vote and the
// apply on a tile of columns, so that the sign words are never read back from
// memory and x is touched by the CTA that voted on it.  Per parameter it moves
// 12.125 M + 8.125 bytes (g and m of every row, the M sign words and the vote
// word written out as the wire data, x read and written).
//
// A CTA owns columns [tile * TILE, (tile + 1) * TILE) and walks the M rows.  For
// every row each warp does what the worker kernel does on its span; the lane
// that keeps "its" word (see own_word_index) stores it to the row's sign words
// and folds it into a private bit-sliced counter.  After the last row the top
// plane of that counter is the voted word; it is stored and handed back to the
// eight lanes of its group by shuffles for the update of x.
//
// Measured on B200: with few workers (M <= 8) this beats the three separate
// kernels (one launch, no second pass over the words); with many workers the
// 2M + 1 concurrent row streams cost 1-5 % of DRAM efficiency against the worker
// kernel's two, so the step entry point then uses the three kernels.

constexpr int kFusedMaxWorkers = 8;           // rows walked by one CTA at most, with a momentum
constexpr int kFusedMaxWorkersSignOnly = 32;  // ... without one, on long vectors (see step_is_fused)
constexpr int kFusedMaxPlanes = 4;            // planes needed for M <= 8
constexpr int kFusedMaxPlanesSignOnly = 6;    // ... for M <= 32

template <int MODE, int UNROLL, int NP>
__device__ __forceinline__ void fused_row(const float* __restrict__ gr, float* __restrict__ mr,
                                          uint32_t* __restrict__ brow, float beta, float omb,
                                          unsigned lane, unsigned sub, unsigned long long my_word,
                                          Counter1<NP>& cnt) {
  constexpr bool MOMENTUM = MODE != kSignSGD;
  constexpr bool SIGN_OF_G = MODE != kSignum;
  float4 gv[UNROLL], mv[UNROLL];
#pragma unroll
  for (int u = 0; u < UNROLL; ++u) gv[u] = ld128(gr + u * 128);
  if (MOMENTUM) {
#pragma unroll
    for (int u = 0; u < UNROLL; ++u) mv[u] = ld128(mr + u * 128);
  }
  unsigned mine = 0;
#pragma unroll
  for (int u = 0; u < UNROLL; ++u) {
    float4 v = gv[u];
    if (MOMENTUM) {
      v = momentum_update4(beta, omb, mv[u], v);
      st128(mr + u * 128, v);
    }
    const unsigned word = assemble_word(sign_nibble(SIGN_OF_G ? gv[u] : v), lane);
    if (sub == (unsigned)u) mine = word;
  }
  if (sub < (unsigned)UNROLL) brow[my_word] = mine;
  cnt.template add<0>(mine);
}

// The span that crosses the end of the vector: the same walk with element-wise
// guards.  Bits at positions >= d stay 0 in every row, so they count 0 votes and
// the voted word has them 0 as well (the threshold is at least 1).  Kept out of
// line so that the interior path's register allocation is not affected.
template <int MODE, int UNROLL, int NP>
__device__ __noinline__ void fused_ragged_span(const float* __restrict__ g, float* __restrict__ m,
                                               float* __restrict__ x, uint32_t* __restrict__ bits,
                                               uint32_t* __restrict__ vote, unsigned M,
                                               unsigned long long d, unsigned long long ld,
                                               unsigned long long ldw, float beta, float omb, float delta,
                                               unsigned start_value, unsigned long long e0) {
  constexpr bool MOMENTUM = MODE != kSignSGD;
  constexpr bool SIGN_OF_G = MODE != kSignum;
  const unsigned lane = threadIdx.x & 31u;
  const unsigned sub = lane & 7u;
  const float minus = -delta;
  const unsigned long long my_word = (e0 >> 5) + own_word_index<UNROLL>(lane);
  const bool have_word = sub < (unsigned)UNROLL && my_word * 32 < d;   // its first element is below d
  Counter1<NP> cnt;
  cnt.init(start_value);
  for (unsigned row = 0; row < M; ++row) {
    const float* gr = g + (unsigned long long)row * ld;
    float* mr = MOMENTUM ? m + (unsigned long long)row * ld : nullptr;
    unsigned mine = 0;
#pragma unroll 1
    for (int u = 0; u < UNROLL; ++u) {
      const unsigned long long e = e0 + u * 128 + lane * 4;
      unsigned nib = 0;
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        if (e + k < d) {
          const float gk = gr[e + k];
          float v = gk;
          if (MOMENTUM) {
            v = momentum_update(beta, omb, mr[e + k], gk);
            mr[e + k] = v;
          }
          nib |= sign_bit(SIGN_OF_G ? gk : v) << k;
        }
      }
      const unsigned word = assemble_word(nib, lane);
      if (sub == (unsigned)u) mine = word;
    }
    if (have_word) bits[(unsigned long long)row * ldw + my_word] = mine;
    cnt.template add<0>(mine);
  }
  const unsigned voted = cnt.top();
  if (have_word) vote[my_word] = voted;
#pragma unroll 1
  for (int u = 0; u < UNROLL; ++u) {
    const unsigned vw = __shfl_sync(0xFFFFFFFFu, voted, (lane & 24u) + u);
    const unsigned long long e = e0 + u * 128 + lane * 4;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      if (e + k < d) x[e + k] = __fadd_rn(x[e + k], ((vw >> (4u * sub + k)) & 1u) ? minus : delta);
    }
  }
}

// UNROLL == 1 is the form for vectors too short to fill the machine with larger tiles (see fused_unroll).
// There a CTA's walk down its rows is a chain of dependent round trips to memory that nothing else hides,
// so that form fetches x at the start and the NEXT row's g and m before it works on the current row
// (56-64 registers, four resident CTAs per SM).  Measured on B200 at d = 2^17 .. 2^19: 14-17 % faster for
// one worker (3.1 -> 2.6 us at 2^18), 0-12 % for 2 .. 8, up to 23 % without a momentum, never slower; with
// the larger tiles (d >= 2^20) the same prefetch costs 5-35 % (fewer resident CTAs), so they do without.
template <int MODE, int UNROLL, int NP>
__global__ void __launch_bounds__(kThreads, UNROLL == 1 ? 4 : 5)
fused_step_kernel(const float* __restrict__ g, float* __restrict__ m, float* __restrict__ x,
                  uint32_t* __restrict__ bits, uint32_t* __restrict__ vote, unsigned M,
                  unsigned long long d, unsigned long long ld, unsigned long long ldw,
                  float beta, float omb, float delta, unsigned start_value) {
  constexpr bool MOMENTUM = MODE != kSignSGD;
  constexpr unsigned long long TILE = (unsigned long long)kThreads * 4 * UNROLL;
  constexpr unsigned SPAN = 128 * UNROLL;
  const unsigned lane = threadIdx.x & 31u;
  const unsigned warp = threadIdx.x >> 5;
  const unsigned sub = lane & 7u;
  pdl_launch_dependents();
  pdl_wait();
  const unsigned long long e0 = (unsigned long long)blockIdx.x * TILE + (unsigned long long)warp * SPAN;
  if (e0 >= d) return;   // uniform over the warp; nothing below synchronises across warps
  if (e0 + SPAN > d) {
    fused_ragged_span<MODE, UNROLL, NP>(g, m, x, bits, vote, M, d, ld, ldw, beta, omb, delta,
                                            start_value, e0);
    return;
  }
  Counter1<NP> cnt;
  cnt.init(start_value);
  const unsigned long long my_word = (e0 >> 5) + own_word_index<UNROLL>(lane);
  const unsigned long long off = e0 + lane * 4;
  if constexpr (UNROLL == 1) {
    constexpr bool SIGN_OF_G = MODE != kSignum;
    float4 gv = ld128(g + off);
    float4 mv = MOMENTUM ? ld128(m + off) : gv;
    const float4 xv = ld128(x + off);
    for (unsigned row = 0; row < M; ++row) {
      float4 gn = gv, mn = mv;
      if (row + 1 < M) {                                   // the next row's loads go out before this row's work
        gn = ld128(g + (unsigned long long)(row + 1) * ld + off);
        if (MOMENTUM) mn = ld128(m + (unsigned long long)(row + 1) * ld + off);
      }
      float4 v = gv;
      if (MOMENTUM) {
        v = momentum_update4(beta, omb, mv, gv);
        st128(m + (unsigned long long)row * ld + off, v);
      }
      const unsigned word = assemble_word(sign_nibble(SIGN_OF_G ? gv : v), lane);
      if (sub == 0) bits[(unsigned long long)row * ldw + my_word] = word;
      cnt.template add<0>(word);
      gv = gn;
      mv = mn;
    }
    const unsigned voted = cnt.top();                      // every lane of a group holds its group's word
    if (sub == 0) vote[my_word] = voted;
    st128(x + off, apply4(xv, voted >> (4u * sub), delta, -delta));
  } else {
    for (unsigned row = 0; row < M; ++row) {
      fused_row<MODE, UNROLL, NP>(g + (unsigned long long)row * ld + off,
                                      MOMENTUM ? m + (unsigned long long)row * ld + off : nullptr,
                                      bits + (unsigned long long)row * ldw, beta, omb, lane, sub, my_word, cnt);
    }
    const unsigned voted = cnt.top();
    if (sub < (unsigned)UNROLL) vote[my_word] = voted;
    const float minus = -delta;
    float4 xv[UNROLL];
#pragma unroll
    for (int u = 0; u < UNROLL; ++u) xv[u] = ld128(x + off + u * 128);
#pragma unroll
    for (int u = 0; u < UNROLL; ++u) {
      const unsigned vw = __shfl_sync(0xFFFFFFFFu, voted, (lane & 24u) + u);  // owner of step u in my group
      st128(x + off + u * 128, apply4(xv[u], vw >> (4u * sub), delta, minus));
    }
  }
}

// ---------------------------------------------------------------------------
// host side

ssgd_status launch_vote(const uint32_t* bits, size_t M, size_t d, size_t ldw, uint32_t* vote,
                        cudaStream_t s) {
  return launch_vote_any<false>(bits, M, d, ldw, vote, 0, s);
}

constexpr size_t kWorkerSharedHint = 36 * 1024;   // below the 48 KB that need no opt-in

template <int MODE, int UNROLL>
bool launch_worker_u(const float* g, float* m, size_t M, size_t d, size_t ld, float beta,
                     uint32_t* bits, size_t ldw, cudaStream_t s) {
  constexpr unsigned long long TILE = (unsigned long long)kThreads * 4 * UNROLL;
  constexpr bool SPLIT = UNROLL >= 4;    // large inputs: interior-only main kernel + a tail launch if needed
  const unsigned long long tiles_per_row = (d + TILE - 1) / TILE;
  if (tiles_per_row > kMaxGrid) return false;     // beyond any device's memory
  const float omb = 1.0f - beta;
  // The interior-only kernels ask for 36 KB of dynamic shared memory per CTA that they never touch.
  // With four resident CTAs that moves 144 KB of the SM's L1 / shared-memory array to the shared side;
  // measured on B200 (d = 335 M, M = 16, five runs on different boards) the stream is then 0.7-1.3 %
  // faster than with the whole array as L1, while 170 KB and more on the shared side is slower.
  const size_t smem = SPLIT ? kWorkerSharedHint : 0;
  launch_kernel(worker_pack_kernel<MODE, UNROLL, !SPLIT>, dim3((unsigned)tiles_per_row, (unsigned)M), kThreads, smem, s,
                true, g, m, bits, (unsigned long long)d, (unsigned long long)ld, (unsigned long long)ldw, beta, omb);
  if constexpr (SPLIT) {
    if (d % (128 * UNROLL) != 0)
      worker_tail_kernel<MODE, UNROLL><<<(unsigned)M, 32, 0, s>>>(g, m, bits, d, ld, ldw, beta, omb);
  }
  return true;
}

template <int MODE>
ssgd_status launch_worker(const float* g, float* m, size_t M, size_t d, size_t ld, float beta,
                          uint32_t* bits, size_t ldw, cudaStream_t s) {
  DeviceInfo di;
  if (!device_info(&di)) return SSGD_ERR_CUDA;
  bool ok;
  if constexpr (MODE == kSignSGD) {
    // one array to load: twice the elements per thread keep as many loads in flight
    switch (worker_unroll(d, M, di.sms, false)) {
      case 8: ok = launch_worker_u<kSignSGD, 8>(g, m, M, d, ld, beta, bits, ldw, s); break;
      case 2: ok = launch_worker_u<kSignSGD, 2>(g, m, M, d, ld, beta, bits, ldw, s); break;
      default: ok = launch_worker_u<kSignSGD, 1>(g, m, M, d, ld, beta, bits, ldw, s); break;
    }
  } else {
    ok = worker_unroll(d, M, di.sms, true) == 4 ? launch_worker_u<MODE, 4>(g, m, M, d, ld, beta, bits, ldw, s)
                                                : launch_worker_u<MODE, 1>(g, m, M, d, ld, beta, bits, ldw, s);
  }
  return ok ? launch_status() : SSGD_ERR_SIZE;
}

template <int UNROLL, bool SPLIT>
bool launch_apply_u(float* x, const uint32_t* vote, size_t d, float delta, cudaStream_t s) {
  constexpr unsigned long long TILE = (unsigned long long)kThreads * 4 * UNROLL;
  const unsigned long long tiles = (d + TILE - 1) / TILE;
  if (tiles > kMaxGrid) return false;     // beyond any device's memory
  launch_kernel(apply_kernel<UNROLL, !SPLIT>, (unsigned)tiles, kThreads, 0, s, true, x, vote,
                (unsigned long long)d, delta);
  if constexpr (SPLIT) {
    if (d % (128 * UNROLL) != 0) apply_tail_kernel<UNROLL><<<1, 32, 0, s>>>(x, vote, d, delta);
  }
  return true;
}

ssgd_status launch_apply(float* x, const uint32_t* vote, size_t d, float delta, cudaStream_t s) {
  DeviceInfo di;
  if (!device_info(&di)) return SSGD_ERR_CUDA;
  // 2048-element tiles, interior-only, once they fill the machine 8 CTAs deep; below that the smallest
  // tile with the guarded path inline (one launch)
  const bool ok = apply_unroll(d, di.sms) == 2 ? launch_apply_u<2, true>(x, vote, d, delta, s)
                                               : launch_apply_u<1, false>(x, vote, d, delta, s);
  return ok ? launch_status() : SSGD_ERR_SIZE;
}

template <int MODE, int UNROLL, int NP>
void launch_fused_mun(const StepArgs& a, cudaStream_t s) {
  constexpr unsigned long long TILE = (unsigned long long)kThreads * 4 * UNROLL;
  const unsigned long long tiles = (a.d + TILE - 1) / TILE;
  launch_kernel(fused_step_kernel<MODE, UNROLL, NP>, (unsigned)tiles, kThreads, 0, s, true, a.g, a.m, a.x, a.bits,
                a.vote, (unsigned)a.M, (unsigned long long)a.d, (unsigned long long)a.ld, (unsigned long long)a.ldw,
                a.beta, 1.0f - a.beta, a.delta, vote_start_value(a.M, NP));
}

template <int MODE, int UNROLL>
bool launch_fused_mu(const StepArgs& a, cudaStream_t s) {
  switch (vote_planes(a.M)) {
    case 1: launch_fused_mun<MODE, UNROLL, 1>(a, s); return true;
    case 2: launch_fused_mun<MODE, UNROLL, 2>(a, s); return true;
    case 3: launch_fused_mun<MODE, UNROLL, 3>(a, s); return true;
    case 4: launch_fused_mun<MODE, UNROLL, 4>(a, s); return true;
  }
  if constexpr (MODE == kSignSGD && UNROLL == 4) {   // more than eight workers: sign-only, long vectors
    switch (vote_planes(a.M)) {
      case 5: launch_fused_mun<MODE, UNROLL, 5>(a, s); return true;
      case 6: launch_fused_mun<MODE, UNROLL, 6>(a, s); return true;
    }
  }
  return false;
}

// Whether the step runs as the fused kernel.  Up to eight workers: always (if the vector fits one grid
// of tiles).  Nine to 32 workers: only without a momentum and on long vectors -- there the worker
// kernel is a read-only stream and the x update rides along with it: measured on B200 at d >= 2^23 the
// fused kernel is 8-13 % faster for M = 9 .. 12 and 2-3 % for M = 16 .. 31, while on shorter vectors,
// and with a momentum at any size, the three kernels win by up to 5 %.
template <int MODE>
bool step_is_fused(size_t M, size_t d, int sms) {
  static_assert(kFusedMaxWorkers / 2 < (1 << (kFusedMaxPlanes - 1)), "planes cover the fused worker limit");
  static_assert(kFusedMaxWorkersSignOnly / 2 < (1 << (kFusedMaxPlanesSignOnly - 1)), "... and the sign-only one");
  const int unroll = fused_unroll(d, sms, MODE != kSignSGD);
  if (tile_count(d, 1, unroll) > kMaxGrid) return false;
  if (M <= (size_t)kFusedMaxWorkers) return true;
  return MODE == kSignSGD && M <= (size_t)kFusedMaxWorkersSignOnly && unroll == 4 &&
         tile_count(d, 1, 4) >= 12ull * sms;
}

template <int MODE>
ssgd_status launch_fused(const StepArgs& a, cudaStream_t s, bool* launched) {
  *launched = false;
  DeviceInfo di;
  if (!device_info(&di)) return SSGD_ERR_CUDA;
  if (!step_is_fused<MODE>(a.M, a.d, di.sms)) return SSGD_OK;
  // Elements per thread and row: 8 with a momentum (two arrays to load: four 128-bit loads in flight),
  // 16 without (one array), less for short vectors (see fused_unroll).
  const int unroll = fused_unroll(a.d, di.sms, MODE != kSignSGD);
  bool ok;
  if (MODE == kSignSGD && unroll == 4) ok = launch_fused_mu<kSignSGD, 4>(a, s);
  else if (unroll == 2) ok = launch_fused_mu<MODE, 2>(a, s);
  else ok = launch_fused_mu<MODE, 1>(a, s);
  if (!ok) return SSGD_ERR_SIZE;
  *launched = true;
  return launch_status();
}

// One whole step in the given worker mode: the row-parallel kernel for short vectors, the fused kernel
// where it applies, otherwise worker, vote and apply kernels on the same stream.
template <int MODE>
ssgd_status run_step(const StepArgs& a, cudaStream_t s) {
  DeviceInfo di;
  if (!device_info(&di)) return SSGD_ERR_CUDA;
  // short vectors: one launch whose warps work on different rows at once (step_rows.cuh)
  if (step_uses_rows_kernel(a.M, a.d, di.sms)) return launch_step_rows<MODE>(a, s);
  bool launched = false;
  ssgd_status st = launch_fused<MODE>(a, s, &launched);
  if (st != SSGD_OK || launched) return st;
  st = launch_worker<MODE>(a.g, a.m, a.M, a.d, a.ld, a.beta, a.bits, a.ldw, s);
  if (st != SSGD_OK) return st;
  // programmatic dependent launches: vote and apply are each brought onto the SMs while the kernel before
  // them drains (see pdl_wait)
  st = launch_vote(a.bits, a.M, a.d, a.ldw, a.vote, s);
  if (st != SSGD_OK) return st;
  return launch_apply(a.x, a.vote, a.d, a.delta, s);
}

// argument checks shared by the entry points -------------------------------

ssgd_status check_sign_pack(const float* g, size_t M, size_t d, size_t ld, const uint32_t* bits,
                            size_t ldw) {
  if (!g || !bits) return SSGD_ERR_NULL;
  if (!aligned16(g) || !aligned16(bits)) return SSGD_ERR_ALIGN;
  return check_rows(M, d, ld, ldw, true);
}

ssgd_status check_momentum_pack(const float* g, const float* m, size_t M, size_t d, size_t ld,
                                float beta, const uint32_t* bits, size_t ldw) {
  if (!g || !m || !bits) return SSGD_ERR_NULL;
  if (!aligned16(g) || !aligned16(m) || !aligned16(bits)) return SSGD_ERR_ALIGN;
  const ssgd_status st = check_rows(M, d, ld, ldw, true);
  if (st != SSGD_OK) return st;
  return beta_ok(beta) ? SSGD_OK : SSGD_ERR_ARG;
}

ssgd_status check_vote(const uint32_t* bits, size_t M, size_t d, size_t ldw, const uint32_t* vote) {
  if (!bits || !vote) return SSGD_ERR_NULL;
  if (!aligned16(bits) || !aligned16(vote)) return SSGD_ERR_ALIGN;
  return check_rows(M, d, 0, ldw, false);
}

ssgd_status check_apply(const float* x, const uint32_t* vote, size_t d, float delta) {
  if (!x || !vote) return SSGD_ERR_NULL;
  if (!aligned16(x) || !aligned16(vote)) return SSGD_ERR_ALIGN;
  if (d > SIZE_MAX - 31) return SSGD_ERR_SIZE;
  return isfinite(delta) ? SSGD_OK : SSGD_ERR_ARG;
}

ssgd_status check_step(const float* x, const float* g, const float* m, size_t M, size_t d, size_t ld,
                       float beta, float delta, const uint32_t* bits_ws, size_t ldw,
                       const uint32_t* vote_ws) {
  if (!x || !g || !bits_ws || !vote_ws) return SSGD_ERR_NULL;
  if (!beta_ok(beta)) return SSGD_ERR_ARG;
  if (!m && beta != 0.0f) return SSGD_ERR_NULL;
  ssgd_status st = m ? check_momentum_pack(g, m, M, d, ld, beta, bits_ws, ldw)
                     : check_sign_pack(g, M, d, ld, bits_ws, ldw);
  if (st != SSGD_OK) return st;
  st = check_vote(bits_ws, M, d, ldw, vote_ws);
  if (st != SSGD_OK) return st;
  return check_apply(x, vote_ws, d, delta);
}

}  // namespace

// ---------------------------------------------------------------------------
// C ABI

extern "C" {

size_t ssgd_words(size_t d) { return d / 32 + (d % 32 != 0 ? 1 : 0); }

const char* ssgd_status_str(ssgd_status s) {
  switch (s) {
    case SSGD_OK: return "ok";
    case SSGD_ERR_NULL: return "a required pointer is NULL";
    case SSGD_ERR_ALIGN: return "pointer not 16-byte aligned or row stride not a multiple of 4";
    case SSGD_ERR_SIZE: return "worker count out of range, row stride too short, or size overflow";
    case SSGD_ERR_ARG: return "beta outside [0,1) or delta not finite";
    case SSGD_ERR_CUDA: return "CUDA runtime error";
    case SSGD_ERR_SCRATCH: return "problem exceeds the built-in scratch capacity of the no-allocation call";
  }
  return "unknown status";
}

ssgd_status ssgd_sign_pack(const float* g, size_t M, size_t d, size_t ld, uint32_t* bits,
                           size_t ldw, void* stream) {
  const ssgd_status st = check_sign_pack(g, M, d, ld, bits, ldw);
  if (st != SSGD_OK || d == 0) return st;
  return launch_worker<kSignSGD>(g, nullptr, M, d, ld, 0.0f, bits, ldw, static_cast<cudaStream_t>(stream));
}

ssgd_status ssgd_signum_momentum_pack(const float* g, float* m, size_t M, size_t d, size_t ld,
                                      float beta, uint32_t* bits, size_t ldw, void* stream) {
  const ssgd_status st = check_momentum_pack(g, m, M, d, ld, beta, bits, ldw);
  if (st != SSGD_OK || d == 0) return st;
  return launch_worker<kSignum>(g, m, M, d, ld, beta, bits, ldw, static_cast<cudaStream_t>(stream));
}

ssgd_status ssgd_majority_vote(const uint32_t* bits, size_t M, size_t d, size_t ldw,
                               uint32_t* vote, void* stream) {
  const ssgd_status st = check_vote(bits, M, d, ldw, vote);
  if (st != SSGD_OK || d == 0) return st;
  return launch_vote(bits, M, d, ldw, vote, static_cast<cudaStream_t>(stream));
}

ssgd_status ssgd_sign_apply(float* x, const uint32_t* vote, size_t d, float delta, void* stream) {
  const ssgd_status st = check_apply(x, vote, d, delta);
  if (st != SSGD_OK || d == 0) return st;
  return launch_apply(x, vote, d, delta, static_cast<cudaStream_t>(stream));
}

ssgd_status ssgd_signsgd_step(float* x, const float* g, float* m, size_t M, size_t d, size_t ld,
                              float beta, float delta, uint32_t* bits_ws, size_t ldw,
                              uint32_t* vote_ws, void* stream) {
  const ssgd_status st = check_step(x, g, m, M, d, ld, beta, delta, bits_ws, ldw, vote_ws);
  if (st != SSGD_OK || d == 0) return st;
  const StepArgs a{g, m, x, bits_ws, vote_ws, M, d, ld, ldw, beta, delta};
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  return m ? run_step<kSignum>(a, s) : run_step<kSignSGD>(a, s);
}

int ssgd_step_is_fused(size_t M, size_t d, int momentum) {
  DeviceInfo di;
  if (M < 1 || M > SSGD_MAX_WORKERS || d == 0 || !device_info(&di)) return 0;
  if (step_uses_rows_kernel(M, d, di.sms)) return 2;
  return (momentum ? step_is_fused<kSignum>(M, d, di.sms) : step_is_fused<kSignSGD>(M, d, di.sms)) ? 1 : 0;
}

size_t ssgd_warmup_steps(float beta) {
  if (!beta_ok(beta)) return 0;
  // C(beta) of Theorem 3: the least positive integer C with
  //   (C / 2) beta^C <= 1 / ((1 - beta^2) (C + 1))   and   beta^(C + 1) <= 1 / 2.
  const double b = (double)beta;
  const double rhs = 1.0 / (1.0 - b * b);
  double bc = b;  // beta^C
  for (size_t C = 1; C != 0; ++C, bc *= b) {
    if (0.5 * (double)C * bc * ((double)C + 1.0) <= rhs && bc * b <= 0.5) return C;
  }
  return 0;
}

ssgd_status ssgd_signum_warmup_pack(const float* g, float* m, size_t M, size_t d, size_t ld,
                                    float beta, uint32_t* bits, size_t ldw, void* stream) {
  const ssgd_status st = check_momentum_pack(g, m, M, d, ld, beta, bits, ldw);
  if (st != SSGD_OK || d == 0) return st;
  return launch_worker<kSignumWarmup>(g, m, M, d, ld, beta, bits, ldw, static_cast<cudaStream_t>(stream));
}

ssgd_status ssgd_signsgd_warmup_step(float* x, const float* g, float* m, size_t M, size_t d,
                                     size_t ld, float beta, float delta, uint32_t* bits_ws,
                                     size_t ldw, uint32_t* vote_ws, void* stream) {
  if (!m) return SSGD_ERR_NULL;
  const ssgd_status st = check_step(x, g, m, M, d, ld, beta, delta, bits_ws, ldw, vote_ws);
  if (st != SSGD_OK || d == 0) return st;
  const StepArgs a{g, m, x, bits_ws, vote_ws, M, d, ld, ldw, beta, delta};
  return run_step<kSignumWarmup>(a, static_cast<cudaStream_t>(stream));
}

ssgd_status ssgd_signsgd_step_host(float* x, const float* g_host, float* m, size_t M, size_t d,
                                   size_t ld, float beta, float delta, float* g_stage,
                                   uint32_t* bits_ws, size_t ldw, uint32_t* vote_ws,
                                   uint32_t* vote_host, void* stream) {
  if (!g_host) return SSGD_ERR_NULL;
  ssgd_status st = check_step(x, g_stage, m, M, d, ld, beta, delta, bits_ws, ldw, vote_ws);
  if (st != SSGD_OK || d == 0) return st;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const size_t vote_bytes = ssgd_words(d) * sizeof(uint32_t);

  // The step is elementwise in the parameter index, so a slab of columns can be stepped as soon as it
  // has arrived.  Large transfers are therefore cut into column slabs that a second stream copies while
  // `stream` computes on the slabs before them; the host link stays busy throughout and only the last
  // slab's kernels are left over at the end.  Slab starts are multiples of 4096 parameters (whole words,
  // 16-byte aligned rows).  Small transfers, and calls under stream capture, take one copy and one step.
  constexpr size_t kSlabBytes = size_t(64) << 20;
  constexpr size_t kMaxSlabs = 32;
  const size_t total = M * d * sizeof(float);
  size_t slabs = total / kSlabBytes;
  if (slabs > kMaxSlabs) slabs = kMaxSlabs;
  cudaStreamCaptureStatus capturing = cudaStreamCaptureStatusNone;
  if (cudaStreamIsCapturing(s, &capturing) != cudaSuccess) return SSGD_ERR_CUDA;
  if (slabs < 2 || capturing != cudaStreamCaptureStatusNone) {
    if (cudaMemcpyAsync(g_stage, g_host, M * ld * sizeof(float), cudaMemcpyHostToDevice, s) != cudaSuccess)
      return SSGD_ERR_CUDA;
    st = ssgd_signsgd_step(x, g_stage, m, M, d, ld, beta, delta, bits_ws, ldw, vote_ws, stream);
    if (st != SSGD_OK) return st;
    if (vote_host && cudaMemcpyAsync(vote_host, vote_ws, vote_bytes, cudaMemcpyDeviceToHost, s) != cudaSuccess)
      return SSGD_ERR_CUDA;
    return SSGD_OK;
  }

  const size_t width = ((d + slabs - 1) / slabs + 4095) / 4096 * 4096;   // parameters per slab
  cudaStream_t copier = nullptr;
  cudaEvent_t ready[kMaxSlabs + 1] = {};                                  // [slabs]: `stream`'s earlier work
  size_t events = 0;
  bool ok = cudaStreamCreateWithFlags(&copier, cudaStreamNonBlocking) == cudaSuccess;
  for (; ok && events <= slabs; ++events)
    ok = cudaEventCreateWithFlags(&ready[events], cudaEventDisableTiming) == cudaSuccess;
  // the copies may not overwrite g_stage before what `stream` already holds has run
  ok = ok && cudaEventRecord(ready[slabs], s) == cudaSuccess &&
       cudaStreamWaitEvent(copier, ready[slabs], 0) == cudaSuccess;
  st = SSGD_OK;
  size_t k = 0;
  for (size_t off = 0; ok && st == SSGD_OK && off < d; off += width, ++k) {
    const size_t w = d - off < width ? d - off : width;
    ok = cudaMemcpy2DAsync(g_stage + off, ld * sizeof(float), g_host + off, ld * sizeof(float), w * sizeof(float), M,
                           cudaMemcpyHostToDevice, copier) == cudaSuccess &&
         cudaEventRecord(ready[k], copier) == cudaSuccess && cudaStreamWaitEvent(s, ready[k], 0) == cudaSuccess;
    if (ok)
      st = ssgd_signsgd_step(x + off, g_stage + off, m ? m + off : nullptr, M, w, ld, beta, delta, bits_ws + off / 32,
                             ldw, vote_ws + off / 32, stream);
  }
  if (ok && st == SSGD_OK && vote_host)
    ok = cudaMemcpyAsync(vote_host, vote_ws, vote_bytes, cudaMemcpyDeviceToHost, s) == cudaSuccess;
  // events and the stream may be destroyed while their work is still queued: the runtime releases them
  // once it has completed
  for (size_t e = 0; e < events; ++e) (void)cudaEventDestroy(ready[e]);
  if (copier) (void)cudaStreamDestroy(copier);
  if (st != SSGD_OK) return st;
  if (!ok) {
    (void)cudaGetLastError();
    return SSGD_ERR_CUDA;
  }
  return SSGD_OK;
}

}  // extern "C"

// ---------------------------------------------------------------------------
// The step for callers that cannot allocate: its word workspaces live in a fixed
// array in device memory instead of caller-provided buffers.
//
// `noalloc_scratch` below is a device symbol.  Inside host code its name is only
// a stand-in that the runtime maps to the real array, never a pointer a kernel
// could use, so the host asks the runtime for the device address once per device
// and hands that address to the launches.

namespace {

static __device__ __align__(256) uint32_t noalloc_scratch[SSGD_NOALLOC_SCRATCH_WORDS];

constexpr int kMaxDevices = 64;
uint32_t* noalloc_scratch_addr[kMaxDevices];  // device address per device, filled on first use

// Device address of the scratch array on the current device, or nullptr on error.
uint32_t* noalloc_scratch_on_current_device() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
  uint32_t* p = __atomic_load_n(&noalloc_scratch_addr[dev], __ATOMIC_ACQUIRE);
  if (p) return p;
  void* sym = nullptr;
  if (cudaGetSymbolAddress(&sym, noalloc_scratch) != cudaSuccess || sym == nullptr) {
    (void)cudaGetLastError();
    return nullptr;
  }
  p = static_cast<uint32_t*>(sym);
  __atomic_store_n(&noalloc_scratch_addr[dev], p, __ATOMIC_RELEASE);  // same value from any thread
  return p;
}

}  // namespace

extern "C" ssgd_status ssgd_signsgd_step_noalloc(float* x, const float* g, float* m, size_t M,
                                                 size_t d, size_t ld, float beta, float delta,
                                                 void* stream) {
  if (M < 1 || M > SSGD_MAX_WORKERS || d > SIZE_MAX - 127) return SSGD_ERR_SIZE;
  const size_t W4 = (ssgd_words(d) + 3) / 4 * 4;              // row stride: keeps rows 16-byte aligned
  if (W4 > SSGD_NOALLOC_SCRATCH_WORDS / (M + 1)) return SSGD_ERR_SCRATCH;
  uint32_t* scratch = noalloc_scratch_on_current_device();
  if (!scratch) return SSGD_ERR_CUDA;
  uint32_t* bits_ws = scratch;                                 // [M][W4]
  uint32_t* vote_ws = scratch + M * W4;                        // [W4]
  return ssgd_signsgd_step(x, g, m, M, d, ld, beta, delta, bits_ws, W4, vote_ws, stream);
}
