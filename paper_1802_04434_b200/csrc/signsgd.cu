// sm_100a kernels and C ABI for the signSGD / Signum / majority-vote step
// (Algorithms 1-3 of Bernstein et al., "signSGD: Compressed Optimisation for
// Non-Convex Problems").  See include/signsgd.h for the contract of each call.
//
// Every kernel here streams its operands once and is bound by HBM bandwidth:
//   worker kernel   12.125 B per parameter per worker (g read, m read + write,
//                   1/8 B of sign bits written); 4.125 B for the sign-only form
//   vote kernel     (M + 1) / 8 B per parameter
//   apply kernel    8.125 B per parameter
// so the design rules are: 128-bit coalesced accesses, many independent loads
// in flight per thread, streaming cache hints (nothing is re-read), grids sized
// in whole waves of the SM count, and 64-bit indexing (M * d exceeds 2^32).

#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

#include "signsgd.h"

namespace {

// ---------------------------------------------------------------------------
// small device helpers

// 128-bit accesses.  Loads use the default caching path and stores the streaming
// one: measured on B200 this pair, with one tile per CTA, streams faster than a
// device-to-device copy, while evict-first loads and persistent grids were 8-10 %
// slower.
__device__ __forceinline__ float4 ld128(const float* p) {
  return *reinterpret_cast<const float4*>(p);
}
__device__ __forceinline__ void st128(float* p, float4 v) {
  __stcs(reinterpret_cast<float4*>(p), v);
}

// sign(.) of Algorithms 1-3 in one bit: +0, -0 and NaN all count as +1.
__device__ __forceinline__ unsigned sign_bit(float v) { return (v < 0.0f) ? 0u : 1u; }

__device__ __forceinline__ unsigned sign_nibble(const float4& v) {
  return sign_bit(v.x) | (sign_bit(v.y) << 1) | (sign_bit(v.z) << 2) | (sign_bit(v.w) << 3);
}

// Algorithm 2, second step, as two correctly rounded fp32 operations.  Written
// with explicit intrinsics so that the compiler can neither contract nor split them.
__device__ __forceinline__ float momentum_update(float beta, float omb, float m, float g) {
  return __fmaf_rn(beta, m, __fmul_rn(omb, g));
}
__device__ __forceinline__ float4 momentum_update4(float beta, float omb, const float4& m, const float4& g) {
  return make_float4(momentum_update(beta, omb, m.x, g.x), momentum_update(beta, omb, m.y, g.y),
                     momentum_update(beta, omb, m.z, g.z), momentum_update(beta, omb, m.w, g.w));
}

// Algorithm 3, worker block: four parameters move by -delta or +delta according
// to four voted bits (bit set = sign +1 = subtract delta).
__device__ __forceinline__ float4 apply4(const float4& x, unsigned nib, float delta, float minus) {
  return make_float4(__fadd_rn(x.x, (nib & 1u) ? minus : delta), __fadd_rn(x.y, (nib & 2u) ? minus : delta),
                     __fadd_rn(x.z, (nib & 4u) ? minus : delta), __fadd_rn(x.w, (nib & 8u) ? minus : delta));
}

// A warp holds 128 consecutive elements, lane l the four elements 4l..4l+3.
// Lane l's four sign bits are bits 4(l%8)..4(l%8)+3 of word l/8, so an OR over
// each group of eight lanes assembles the four canonical words; every lane of a
// group receives its group's word.
__device__ __forceinline__ unsigned assemble_word(unsigned nibble, unsigned lane) {
  const unsigned group_mask = 0xFFu << (lane & 24u);
  return __reduce_or_sync(group_mask, nibble << (4u * (lane & 7u)));
}

// Tiling shared by the worker, apply and fused kernels: a CTA of kThreads threads
// owns a tile of kThreads * 4 * UNROLL consecutive elements of one row, a warp
// 128 * UNROLL consecutive elements of it ("span"), so that a warp's words are
// consecutive too: its span covers words (e0 / 32) + 4u + j for unroll step u and
// lane group j = lane / 8.
constexpr int kThreads = 256;

// What a worker sends, and whether it keeps a momentum:
//   kSignSGD       bit = sign(g)                       (Algorithm 1 / Algorithm 3 as printed)
//   kSignum        m <- beta m + (1-beta) g, bit = sign(m)            (Algorithm 2)
//   kSignumWarmup  m updated as in kSignum, bit = sign(g): the first C(beta)
//                  iterations of Theorem 3, which accumulate the momentum as
//                  normal but step with the sign of the stochastic gradient
constexpr int kSignSGD = 0;
constexpr int kSignum = 1;
constexpr int kSignumWarmup = 2;

// Within a group of eight lanes all lanes hold the same assembled word.  Lane
// (lane % 8) == u keeps the word of unroll step u ("its" word), so that after the
// UNROLL steps the 4 * UNROLL words of the span sit in 4 * UNROLL distinct lanes
// and can be stored, or counted, once each.
template <int UNROLL>
__device__ __forceinline__ unsigned long long own_word_index(unsigned lane) {
  return (unsigned long long)(lane & 7u) * 4u + (lane >> 3);   // valid for lane % 8 < UNROLL
}

// ---------------------------------------------------------------------------
// worker kernel: [momentum update +] sign + 1-bit pack, all M rows in one launch.
// Tiles are numbered row-major over (row, tile in row), one tile per CTA.

template <int MODE, int UNROLL>
__global__ void __launch_bounds__(kThreads)
worker_pack_kernel(const float* __restrict__ g, float* __restrict__ m,
                   uint32_t* __restrict__ bits, unsigned long long d,
                   unsigned long long ld, unsigned long long ldw,
                   unsigned long long tiles_per_row, unsigned long long total_tiles,
                   float beta, float omb) {
  constexpr bool MOMENTUM = MODE != kSignSGD;
  constexpr bool SIGN_OF_G = MODE != kSignum;
  constexpr unsigned long long TILE = (unsigned long long)kThreads * 4 * UNROLL;
  constexpr unsigned SPAN = 128 * UNROLL;
  const unsigned lane = threadIdx.x & 31u;
  const unsigned warp = threadIdx.x >> 5;

  for (unsigned long long t = blockIdx.x; t < total_tiles; t += gridDim.x) {
    const unsigned long long row = t / tiles_per_row;
    const unsigned long long tile = t - row * tiles_per_row;
    // first element of this warp's span, within the row
    const unsigned long long e0 = tile * TILE + (unsigned long long)warp * SPAN;
    if (e0 >= d) continue;
    const float* gr = g + row * ld;
    float* mr = MOMENTUM ? m + row * ld : nullptr;
    uint32_t* br = bits + row * ldw + (e0 >> 5);
    unsigned mine = 0;

    if (e0 + SPAN <= d) {
      // interior: no bounds checks, all loads issued before any use
      float4 gv[UNROLL], mv[UNROLL];
#pragma unroll
      for (int u = 0; u < UNROLL; ++u) gv[u] = ld128(gr + e0 + u * 128 + lane * 4);
      if (MOMENTUM) {
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) mv[u] = ld128(mr + e0 + u * 128 + lane * 4);
      }
#pragma unroll
      for (int u = 0; u < UNROLL; ++u) {
        float4 v = gv[u];
        if (MOMENTUM) {
          v = momentum_update4(beta, omb, mv[u], v);
          st128(mr + e0 + u * 128 + lane * 4, v);
        }
        const unsigned word = assemble_word(sign_nibble(SIGN_OF_G ? gv[u] : v), lane);
        if ((lane & 7u) == (unsigned)u) mine = word;
      }
      if ((lane & 7u) < (unsigned)UNROLL) br[own_word_index<UNROLL>(lane)] = mine;
    } else {
      // ragged end of the row: element-wise guards, padding bits stay 0, and
      // nothing at or beyond d is written
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
  }
}

// ---------------------------------------------------------------------------
// majority vote: bit-sliced vertical counter
//
// The count of set bits per parameter is kept as NP bit-planes (plane p holds
// bit p of 32 counters per word), and rows are folded in with carry-save adders
// (3 words in, sum + carry out: one XOR3 and one MAJ3 per word), eight rows per
// block, so the cost is about two logic operations per input word.
//
// The comparison with the threshold T = ceil(M/2) is folded into the counter's
// start value: with L = NP - 1 chosen so that floor(M/2) < 2^L, the counter
// starts at 2^L - T and can reach at most 2^L - T + M < 2^(L+1); its top plane
// is then exactly [P >= T], the voted bit (ties, 2P = M, included).

struct W4 {
  unsigned x, y, z, w;
};
__device__ __forceinline__ W4 ld_words(const uint32_t* p) {
  const uint4 v = *reinterpret_cast<const uint4*>(p);
  return W4{v.x, v.y, v.z, v.w};
}
__device__ __forceinline__ unsigned xor3(unsigned a, unsigned b, unsigned c) { return a ^ b ^ c; }
__device__ __forceinline__ unsigned maj3(unsigned a, unsigned b, unsigned c) {
  return (a & b) | (c & (a | b));
}
// carry-save adder on 4 words: lo <- a ^ b ^ lo, returns the carries
__device__ __forceinline__ W4 csa(W4& lo, const W4& a, const W4& b) {
  W4 hi{maj3(lo.x, a.x, b.x), maj3(lo.y, a.y, b.y), maj3(lo.z, a.z, b.z), maj3(lo.w, a.w, b.w)};
  lo = W4{xor3(lo.x, a.x, b.x), xor3(lo.y, a.y, b.y), xor3(lo.z, a.z, b.z), xor3(lo.w, a.w, b.w)};
  return hi;
}

template <int NP>
struct Counter {
  W4 c[NP];
  // add a word of weight 2^K: ripple from plane K upwards
  template <int K>
  __device__ __forceinline__ void add(W4 v) {
#pragma unroll
    for (int p = K; p < NP; ++p) {
      const W4 carry{c[p].x & v.x, c[p].y & v.y, c[p].z & v.z, c[p].w & v.w};
      c[p] = W4{c[p].x ^ v.x, c[p].y ^ v.y, c[p].z ^ v.z, c[p].w ^ v.w};
      v = carry;
    }
  }
  __device__ __forceinline__ void add2(const W4& a, const W4& b) {
    if (NP >= 2) {
      const W4 h = csa(c[0], a, b);
      add<1>(h);
    }
  }
  __device__ __forceinline__ void add4(const W4* a) {
    if (NP >= 3) {
      const W4 hA = csa(c[0], a[0], a[1]);
      const W4 hB = csa(c[0], a[2], a[3]);
      const W4 q = csa(c[1], hA, hB);
      add<2>(q);
    }
  }
  __device__ __forceinline__ void add8(const W4* a) {
    if (NP >= 4) {
      const W4 hA = csa(c[0], a[0], a[1]);
      const W4 hB = csa(c[0], a[2], a[3]);
      const W4 qA = csa(c[1], hA, hB);
      const W4 hC = csa(c[0], a[4], a[5]);
      const W4 hD = csa(c[0], a[6], a[7]);
      const W4 qB = csa(c[1], hC, hD);
      const W4 e = csa(c[2], qA, qB);
      add<3>(e);
    }
  }
};

// The same counter on a single word per thread (used by the fused step kernel).
template <int NP>
struct Counter1 {
  unsigned c[NP];
  __device__ __forceinline__ void init(unsigned start_value) {
#pragma unroll
    for (int p = 0; p < NP; ++p) c[p] = ((start_value >> p) & 1u) ? 0xFFFFFFFFu : 0u;
  }
  template <int K>
  __device__ __forceinline__ void add(unsigned v) {
#pragma unroll
    for (int p = K; p < NP; ++p) {
      const unsigned carry = c[p] & v;
      c[p] ^= v;
      v = carry;
    }
  }
  __device__ __forceinline__ void add2(unsigned a, unsigned b) {
    if (NP >= 2) {
      const unsigned h = maj3(c[0], a, b);
      c[0] = xor3(c[0], a, b);
      add<1>(h);
    } else {
      add<0>(a);   // not reached: one plane means one row
    }
  }
  __device__ __forceinline__ unsigned top() const { return c[NP - 1]; }
};

// Four words of one output plane; bits at positions >= d are written as 0,
// whatever the rows held there, and words at or beyond ceil(d/32) are not written.
__device__ __forceinline__ void store_plane_words(uint32_t* __restrict__ out, unsigned long long q,
                                                  unsigned long long d, const W4& v) {
  const unsigned long long first = q * 128;  // first parameter of this chunk
  if (first + 128 <= d) {
    *reinterpret_cast<uint4*>(out + 4 * q) = make_uint4(v.x, v.y, v.z, v.w);
  } else {
    const unsigned w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const unsigned long long lo = first + 32ull * k;
      if (lo < d) {
        const unsigned long long left = d - lo;
        const unsigned mask = left >= 32 ? 0xFFFFFFFFu : ((1u << left) - 1u);
        out[4 * q + k] = w[k] & mask;
      }
    }
  }
}

// One thread owns four consecutive words (one 128-bit load per row) and walks
// down the M rows; one 256-thread CTA covers 1024 words.
//   COUNTS = false: out[W] receives the top plane, the voted bit (Algorithm 3).
//   COUNTS = true:  the counter starts at 0 and all NP planes are written,
//                   plane p at out + p * ldc: the number of +1 votes per parameter,
//                   bit-sliced, which is what the server sends back in the "(good)"
//                   scheme of Section 4.
template <int NP, bool COUNTS>
__global__ void __launch_bounds__(kThreads)
vote_kernel(const uint32_t* __restrict__ bits, unsigned M, unsigned long long d,
            unsigned long long W, unsigned long long ldw, uint32_t* __restrict__ out,
            unsigned long long ldc, unsigned start_value) {
  const unsigned long long chunks = (W + 3) / 4;
  const unsigned long long stride = (unsigned long long)gridDim.x * kThreads;
  for (unsigned long long q = (unsigned long long)blockIdx.x * kThreads + threadIdx.x;
       q < chunks; q += stride) {
    const uint32_t* col = bits + 4 * q;
    Counter<NP> cnt;
#pragma unroll
    for (int p = 0; p < NP; ++p) {
      const unsigned f = ((start_value >> p) & 1u) ? 0xFFFFFFFFu : 0u;
      cnt.c[p] = W4{f, f, f, f};
    }
    unsigned w = 0;
    if (NP >= 4) {
      for (; w + 8 <= M; w += 8) {
        W4 a[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) a[k] = ld_words(col + (unsigned long long)(w + k) * ldw);
        cnt.add8(a);
      }
    }
    if (NP >= 3 && w + 4 <= M) {
      W4 a[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) a[k] = ld_words(col + (unsigned long long)(w + k) * ldw);
      cnt.add4(a);
      w += 4;
    }
    if (NP >= 2 && w + 2 <= M) {
      const W4 a = ld_words(col + (unsigned long long)w * ldw);
      const W4 b = ld_words(col + (unsigned long long)(w + 1) * ldw);
      cnt.add2(a, b);
      w += 2;
    }
    if (w < M) {
      cnt.template add<0>(ld_words(col + (unsigned long long)w * ldw));
      w += 1;
    }
    if (COUNTS) {
#pragma unroll
      for (int p = 0; p < NP; ++p) store_plane_words(out + (unsigned long long)p * ldc, q, d, cnt.c[p]);
    } else {
      store_plane_words(out, q, d, cnt.c[NP - 1]);
    }
  }
}

// ---------------------------------------------------------------------------
// apply: x <- x -/+ delta by the voted bit.  Thread layout as in the worker
// kernel: lane l of a warp holds elements 4l..4l+3 of a 128-element step, whose
// four bits sit at position 4(l%8) of word l/8 of that step.

template <int UNROLL>
__global__ void __launch_bounds__(kThreads)
apply_kernel(float* __restrict__ x, const uint32_t* __restrict__ vote, unsigned long long d,
             unsigned long long total_tiles, float delta) {
  constexpr unsigned long long TILE = (unsigned long long)kThreads * 4 * UNROLL;
  constexpr unsigned SPAN = 128 * UNROLL;
  const unsigned lane = threadIdx.x & 31u;
  const unsigned warp = threadIdx.x >> 5;
  const float minus = -delta;
  for (unsigned long long t = blockIdx.x; t < total_tiles; t += gridDim.x) {
    const unsigned long long e0 = t * TILE + (unsigned long long)warp * SPAN;
    if (e0 >= d) continue;
    const uint32_t* vw = vote + (e0 >> 5);
    if (e0 + SPAN <= d) {
      float4 xv[UNROLL];
      unsigned wv[UNROLL];
#pragma unroll
      for (int u = 0; u < UNROLL; ++u) {
        xv[u] = ld128(x + e0 + u * 128 + lane * 4);
        wv[u] = __ldg(vw + u * 4 + (lane >> 3));
      }
#pragma unroll
      for (int u = 0; u < UNROLL; ++u)
        st128(x + e0 + u * 128 + lane * 4, apply4(xv[u], wv[u] >> (4u * (lane & 7u)), delta, minus));
    } else {
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
  }
}

// ---------------------------------------------------------------------------
// sum-apply: the "(good)" update of Section 4, x <- x - delta * sum_m sign(.),
// from the bit-sliced count P of +1 votes: the sum of signs is 2P - M.  One fused
// multiply-add per element, x <- fma(-delta, float(2P - M), x).  Lane layout as
// in the apply kernel; each lane reads its word of every count plane.

template <int NP>
__global__ void __launch_bounds__(kThreads)
sum_apply_kernel(float* __restrict__ x, const uint32_t* __restrict__ counts, unsigned M,
                 unsigned long long d, unsigned long long ldc, float delta) {
  const unsigned lane = threadIdx.x & 31u;
  const unsigned long long stride = (unsigned long long)gridDim.x * kThreads * 4;
  const float neg = -delta;
  for (unsigned long long e = ((unsigned long long)blockIdx.x * kThreads + threadIdx.x) * 4; e < d; e += stride) {
    const unsigned shift = 4u * (lane & 7u);        // e is a multiple of 4: (e % 32) = 4 (lane % 8)
    unsigned nib[NP];
#pragma unroll
    for (int p = 0; p < NP; ++p) nib[p] = __ldg(counts + (unsigned long long)p * ldc + (e >> 5)) >> shift;
    float s[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      int P = 0;
#pragma unroll
      for (int p = 0; p < NP; ++p) P |= (int)((nib[p] >> k) & 1u) << p;
      s[k] = (float)(2 * P - (int)M);
    }
    if (e + 4 <= d) {
      float4 v = ld128(x + e);
      v.x = __fmaf_rn(neg, s[0], v.x);
      v.y = __fmaf_rn(neg, s[1], v.y);
      v.z = __fmaf_rn(neg, s[2], v.z);
      v.w = __fmaf_rn(neg, s[3], v.w);
      st128(x + e, v);
    } else {
#pragma unroll
      for (int k = 0; k < 4; ++k)
        if (e + k < d) x[e + k] = __fmaf_rn(neg, s[k], x[e + k]);
    }
  }
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

constexpr int kFusedMaxWorkers = 8;   // rows walked by one CTA at most
constexpr int kFusedMaxPlanes = 4;    // planes needed for M <= 8

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

template <int MODE, int UNROLL, int NP>
__global__ void __launch_bounds__(kThreads, 5)
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

// ---------------------------------------------------------------------------
// host side

struct DeviceInfo {
  int sms;
};

bool device_info(DeviceInfo* out) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return false;
  static int cached_sms[64] = {0};
  if (dev < 0 || dev >= 64) return false;
  if (cached_sms[dev] == 0) {
    int sms = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
      return false;
    cached_sms[dev] = sms;
  }
  out->sms = cached_sms[dev];
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

// Elements per thread: 4 * unroll.  Large inputs take unroll 4 (eight 128-bit
// loads in flight per thread in the worker step); smaller ones shrink the tile so
// that the launch still fills the machine with a few CTAs per SM.
int pick_unroll(unsigned long long elements_per_row, unsigned long long rows, int sms) {
  const unsigned long long want = 8ull * sms;                  // CTAs
  for (int u = 4; u > 1; u /= 2) {
    const unsigned long long tile = (unsigned long long)kThreads * 4 * u;
    if (((elements_per_row + tile - 1) / tile) * rows >= want) return u;
  }
  return 1;
}

template <int MODE, int UNROLL>
void launch_worker_u(const float* g, float* m, size_t M, size_t d, size_t ld, float beta,
                     uint32_t* bits, size_t ldw, cudaStream_t s) {
  constexpr unsigned long long TILE = (unsigned long long)kThreads * 4 * UNROLL;
  const unsigned long long tiles_per_row = (d + TILE - 1) / TILE;
  const unsigned long long total = tiles_per_row * M;
  const float omb = 1.0f - beta;
  worker_pack_kernel<MODE, UNROLL><<<grid_for(total), kThreads, 0, s>>>(
      g, m, bits, d, ld, ldw, tiles_per_row, total, beta, omb);
}

template <int MODE>
ssgd_status launch_worker(const float* g, float* m, size_t M, size_t d, size_t ld, float beta,
                          uint32_t* bits, size_t ldw, cudaStream_t s) {
  DeviceInfo di;
  if (!device_info(&di)) return SSGD_ERR_CUDA;
  switch (pick_unroll(d, M, di.sms)) {
    case 4: launch_worker_u<MODE, 4>(g, m, M, d, ld, beta, bits, ldw, s); break;
    case 2: launch_worker_u<MODE, 2>(g, m, M, d, ld, beta, bits, ldw, s); break;
    default: launch_worker_u<MODE, 1>(g, m, M, d, ld, beta, bits, ldw, s); break;
  }
  return launch_status();
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

ssgd_status launch_vote(const uint32_t* bits, size_t M, size_t d, size_t ldw, uint32_t* vote,
                        cudaStream_t s) {
  return launch_vote_any<false>(bits, M, d, ldw, vote, 0, s);
}

template <int NP>
void launch_sum_apply_np(float* x, const uint32_t* counts, size_t M, size_t d, size_t ldc, float delta,
                         cudaStream_t s) {
  const unsigned long long ctas = ((d + 3) / 4 + kThreads - 1) / kThreads;
  sum_apply_kernel<NP><<<grid_for(ctas), kThreads, 0, s>>>(x, counts, (unsigned)M, d, ldc, delta);
}

ssgd_status launch_sum_apply(float* x, const uint32_t* counts, size_t M, size_t d, size_t ldc,
                             float delta, cudaStream_t s) {
  switch (count_planes(M)) {
    case 1: launch_sum_apply_np<1>(x, counts, M, d, ldc, delta, s); break;
    case 2: launch_sum_apply_np<2>(x, counts, M, d, ldc, delta, s); break;
    case 3: launch_sum_apply_np<3>(x, counts, M, d, ldc, delta, s); break;
    case 4: launch_sum_apply_np<4>(x, counts, M, d, ldc, delta, s); break;
    case 5: launch_sum_apply_np<5>(x, counts, M, d, ldc, delta, s); break;
    case 6: launch_sum_apply_np<6>(x, counts, M, d, ldc, delta, s); break;
    case 7: launch_sum_apply_np<7>(x, counts, M, d, ldc, delta, s); break;
    case 8: launch_sum_apply_np<8>(x, counts, M, d, ldc, delta, s); break;
    case 9: launch_sum_apply_np<9>(x, counts, M, d, ldc, delta, s); break;
    case 10: launch_sum_apply_np<10>(x, counts, M, d, ldc, delta, s); break;
    case 11: launch_sum_apply_np<11>(x, counts, M, d, ldc, delta, s); break;
    default: return SSGD_ERR_SIZE;
  }
  return launch_status();
}

template <int UNROLL>
void launch_apply_u(float* x, const uint32_t* vote, size_t d, float delta, cudaStream_t s) {
  constexpr unsigned long long TILE = (unsigned long long)kThreads * 4 * UNROLL;
  const unsigned long long total = (d + TILE - 1) / TILE;
  apply_kernel<UNROLL><<<grid_for(total), kThreads, 0, s>>>(x, vote, d, total, delta);
}

ssgd_status launch_apply(float* x, const uint32_t* vote, size_t d, float delta, cudaStream_t s) {
  DeviceInfo di;
  if (!device_info(&di)) return SSGD_ERR_CUDA;
  switch (pick_unroll(d, 1, di.sms)) {
    case 4: launch_apply_u<4>(x, vote, d, delta, s); break;
    case 2: launch_apply_u<2>(x, vote, d, delta, s); break;
    default: launch_apply_u<1>(x, vote, d, delta, s); break;
  }
  return launch_status();
}

struct StepArgs {
  const float* g;
  float* m;
  float* x;
  uint32_t* bits;
  uint32_t* vote;
  size_t M, d, ld, ldw;
  float beta, delta;
};

template <int MODE, int UNROLL, int NP>
void launch_fused_mun(const StepArgs& a, cudaStream_t s) {
  constexpr unsigned long long TILE = (unsigned long long)kThreads * 4 * UNROLL;
  const unsigned long long tiles = (a.d + TILE - 1) / TILE;
  fused_step_kernel<MODE, UNROLL, NP><<<(unsigned)tiles, kThreads, 0, s>>>(
      a.g, a.m, a.x, a.bits, a.vote, (unsigned)a.M, a.d, a.ld, a.ldw, a.beta, 1.0f - a.beta, a.delta,
      vote_start_value(a.M, NP));
}

template <int MODE, int UNROLL>
bool launch_fused_mu(const StepArgs& a, cudaStream_t s) {
  switch (vote_planes(a.M)) {
    case 1: launch_fused_mun<MODE, UNROLL, 1>(a, s); return true;
    case 2: launch_fused_mun<MODE, UNROLL, 2>(a, s); return true;
    case 3: launch_fused_mun<MODE, UNROLL, 3>(a, s); return true;
    case 4: launch_fused_mun<MODE, UNROLL, 4>(a, s); return true;
  }
  return false;
}

// Whether the step runs as the fused kernel: few workers, and a vector that fits
// one grid of tiles.  Everything else takes the three kernels.
template <int MODE>
ssgd_status launch_fused(const StepArgs& a, cudaStream_t s, bool* launched) {
  static_assert(kFusedMaxWorkers / 2 < (1 << (kFusedMaxPlanes - 1)), "planes cover the fused worker limit");
  *launched = false;
  if (a.M > (size_t)kFusedMaxWorkers) return SSGD_OK;
  DeviceInfo di;
  if (!device_info(&di)) return SSGD_ERR_CUDA;
  const int unroll = pick_unroll(a.d, 1, di.sms) >= 2 ? 2 : 1;
  const unsigned long long tile = (unsigned long long)kThreads * 4 * unroll;
  if ((a.d + tile - 1) / tile > kMaxGrid) return SSGD_OK;
  const bool ok = unroll == 2 ? launch_fused_mu<MODE, 2>(a, s) : launch_fused_mu<MODE, 1>(a, s);
  if (!ok) return SSGD_ERR_SIZE;
  *launched = true;
  return launch_status();
}

// One whole step in the given worker mode: the fused kernel where it applies,
// otherwise worker, vote and apply kernels on the same stream.
template <int MODE>
ssgd_status run_step(const StepArgs& a, cudaStream_t s) {
  bool launched = false;
  ssgd_status st = launch_fused<MODE>(a, s, &launched);
  if (st != SSGD_OK || launched) return st;
  st = launch_worker<MODE>(a.g, a.m, a.M, a.d, a.ld, a.beta, a.bits, a.ldw, s);
  if (st != SSGD_OK) return st;
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

size_t ssgd_count_planes(size_t M) { return (M >= 1 && M <= SSGD_MAX_WORKERS) ? count_planes(M) : 0; }

ssgd_status ssgd_vote_counts(const uint32_t* bits, size_t M, size_t d, size_t ldw, uint32_t* counts,
                             size_t ldc, void* stream) {
  if (!bits || !counts) return SSGD_ERR_NULL;
  if (!aligned16(bits) || !aligned16(counts)) return SSGD_ERR_ALIGN;
  ssgd_status st = check_rows(M, d, 0, ldw, false);
  if (st != SSGD_OK) return st;
  st = check_rows(count_planes(M), d, 0, ldc, false);   // the planes are rows of the same kind
  if (st != SSGD_OK || d == 0) return st;
  return launch_vote_any<true>(bits, M, d, ldw, counts, ldc, static_cast<cudaStream_t>(stream));
}

ssgd_status ssgd_sum_apply(float* x, const uint32_t* counts, size_t M, size_t d, size_t ldc,
                           float delta, void* stream) {
  if (!x || !counts) return SSGD_ERR_NULL;
  if (!aligned16(x) || !aligned16(counts)) return SSGD_ERR_ALIGN;
  if (M < 1 || M > SSGD_MAX_WORKERS) return SSGD_ERR_SIZE;
  const ssgd_status st = check_rows(count_planes(M), d, 0, ldc, false);
  if (st != SSGD_OK) return st;
  if (!isfinite(delta)) return SSGD_ERR_ARG;
  if (d == 0) return SSGD_OK;
  return launch_sum_apply(x, counts, M, d, ldc, delta, static_cast<cudaStream_t>(stream));
}

ssgd_status ssgd_signsgd_step_host(float* x, const float* g_host, float* m, size_t M, size_t d,
                                   size_t ld, float beta, float delta, float* g_stage,
                                   uint32_t* bits_ws, size_t ldw, uint32_t* vote_ws,
                                   uint32_t* vote_host, void* stream) {
  if (!g_host) return SSGD_ERR_NULL;
  ssgd_status st = check_step(x, g_stage, m, M, d, ld, beta, delta, bits_ws, ldw, vote_ws);
  if (st != SSGD_OK || d == 0) return st;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (cudaMemcpyAsync(g_stage, g_host, M * ld * sizeof(float), cudaMemcpyHostToDevice, s) != cudaSuccess)
    return SSGD_ERR_CUDA;
  st = ssgd_signsgd_step(x, g_stage, m, M, d, ld, beta, delta, bits_ws, ldw, vote_ws, stream);
  if (st != SSGD_OK) return st;
  if (vote_host &&
      cudaMemcpyAsync(vote_host, vote_ws, ssgd_words(d) * sizeof(uint32_t), cudaMemcpyDeviceToHost, s) !=
          cudaSuccess)
    return SSGD_ERR_CUDA;
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
