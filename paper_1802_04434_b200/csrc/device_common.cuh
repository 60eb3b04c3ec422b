// Device-side building blocks shared by the kernels of this library: 128-bit
// accesses, the sign rule, the momentum arithmetic, the warp-level word assembly
// and the bit-sliced vote counters.  Everything lives in an unnamed namespace, so
// each translation unit that includes this file gets its own copy.
#ifndef SSGD_DEVICE_COMMON_CUH_
#define SSGD_DEVICE_COMMON_CUH_

#include <cuda_runtime.h>
#include <stdint.h>

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

// Programmatic dependent launch.  A kernel launched with the programmatic-serialization attribute may
// be brought onto the SMs while the kernel before it on the stream is still draining; pdl_wait() then
// returns once that kernel has completed and its writes are visible (at once when there is no such
// kernel, or when the launch carried no such attribute).  pdl_launch_dependents() tells the scheduler
// that the next kernel on the stream, if it was launched with the attribute, may be brought in as soon as
// every CTA of this grid has started.  Every main kernel of this library begins with both, before it
// touches memory, and is launched with the attribute (launch_kernel in host_common.h): whatever kernel
// precedes it on the stream, this library's or not, it only overlaps its own launch and ramp-up with
// that kernel's tail, and completion still implies that everything before it on the stream completed.
// Measured on B200: about 0.5 us per launch in a sequence of launches (a 4.6 us vote at d = 2^26, M = 1
// becomes 4.0 us; a 1.9 us step at d = 2^10 becomes 1.5-1.7 us), 0.9-1.6 us per three-kernel step.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;"); }

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
//   kSignumWarmup  m updated as in kSignum, bit = sign(g): the warm-up iterations
//                  of Theorem 3 (the first C(beta) ones), whose momentum is
//                  already the running average while the vote is still on g
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
  // The same folds for any NP.  A carry that would leave the top plane is dropped: the callers size NP
  // so that the count stays below 2^NP, hence such a carry is always zero.
  __device__ __forceinline__ void fold4(const W4* a) {
    const W4 hA = csa(c[0], a[0], a[1]);
    const W4 hB = csa(c[0], a[2], a[3]);
    if constexpr (NP >= 2) {
      const W4 q = csa(c[1], hA, hB);
      if constexpr (NP >= 3) add<2>(q);
    }
  }
  __device__ __forceinline__ void fold8(const W4* a) {
    const W4 hA = csa(c[0], a[0], a[1]);
    const W4 hB = csa(c[0], a[2], a[3]);
    const W4 hC = csa(c[0], a[4], a[5]);
    const W4 hD = csa(c[0], a[6], a[7]);
    if constexpr (NP >= 2) {
      const W4 qA = csa(c[1], hA, hB);
      const W4 qB = csa(c[1], hC, hD);
      if constexpr (NP >= 3) {
        const W4 e = csa(c[2], qA, qB);
        if constexpr (NP >= 4) add<3>(e);
      }
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
//   GUARDED = false: after the batches of eight rows, the remaining rows come in
//                   batches of 4, 2 and 1, each loaded and folded in turn (fewest
//                   registers).
//   GUARDED = true: the remaining rows come as ONE batch of four or eight loads with
//                   the missing rows as words of zeros, so that a thread makes
//                   ceil(M / 8) round trips to memory instead of up to three more.
//                   Measured on B200: a round trip costs a short launch about 0.5 us,
//                   and this form is 5-20 % faster for M = 15 and 31 at every size;
//                   the host picks per launch (vote_guarded).
// Two to seven rows (two and three planes) go to vote_exact_kernel below instead.
template <int NP, bool COUNTS, bool GUARDED>
__global__ void __launch_bounds__(kThreads)
vote_kernel(const uint32_t* __restrict__ bits, unsigned M, unsigned long long d,
            unsigned long long W, unsigned long long ldw, uint32_t* __restrict__ out,
            unsigned long long ldc, unsigned start_value) {
  pdl_launch_dependents();
  pdl_wait();
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
    if constexpr (GUARDED) {
      const W4 zero{0u, 0u, 0u, 0u};
      unsigned w = 0;
      for (; w + 8 <= M; w += 8) {
        W4 a[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) a[k] = ld_words(col + (unsigned long long)(w + k) * ldw);
        cnt.fold8(a);
      }
      if (w < M) {
        const unsigned left = M - w;
        if (left <= 4) {
          W4 a[4];
#pragma unroll
          for (int k = 0; k < 4; ++k)
            a[k] = (unsigned)k < left ? ld_words(col + (unsigned long long)(w + k) * ldw) : zero;
          cnt.fold4(a);
        } else {
          W4 a[8];
#pragma unroll
          for (int k = 0; k < 8; ++k)
            a[k] = (unsigned)k < left ? ld_words(col + (unsigned long long)(w + k) * ldw) : zero;
          cnt.fold8(a);
        }
      }
    } else {
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
    }
    if (COUNTS) {
#pragma unroll
      for (int p = 0; p < NP; ++p) store_plane_words(out + (unsigned long long)p * ldc, q, d, cnt.c[p]);
    } else {
      store_plane_words(out, q, d, cnt.c[NP - 1]);
    }
  }
}


// The same vote for exactly MROWS = 2 .. 7 rows (two and three planes): all rows are loaded before the
// first use, without guards, and folded in one carry-save step, so that a thread makes ONE round trip to
// memory at 30-36 registers (vote_kernel needs up to three trips for these row counts, or 48-56 registers
// in its guarded form).  Measured on B200 against vote_kernel: M = 5: 2.66 -> 2.09 us at d = 2^22,
// 9.00 -> 8.64 at 2^26; M = 7: 20.9 -> 20.2 at 2^27; M = 2, 3: 1-5 % at every size.
template <int NP, bool COUNTS, int MROWS>
__global__ void __launch_bounds__(kThreads)
vote_exact_kernel(const uint32_t* __restrict__ bits, unsigned long long d, unsigned long long W,
                  unsigned long long ldw, uint32_t* __restrict__ out, unsigned long long ldc,
                  unsigned start_value) {
  static_assert(MROWS >= 2 && MROWS <= 7 && NP >= 2 && NP <= 3, "row counts with two or three planes");
  pdl_launch_dependents();
  pdl_wait();
  const unsigned long long chunks = (W + 3) / 4;
  const unsigned long long stride = (unsigned long long)gridDim.x * kThreads;
  for (unsigned long long q = (unsigned long long)blockIdx.x * kThreads + threadIdx.x; q < chunks; q += stride) {
    const uint32_t* col = bits + 4 * q;
    W4 a[8];
#pragma unroll
    for (int k = 0; k < MROWS; ++k) a[k] = ld_words(col + (unsigned long long)k * ldw);
#pragma unroll
    for (int k = MROWS; k < 8; ++k) a[k] = W4{0u, 0u, 0u, 0u};   // folded away at compile time
    Counter<NP> cnt;
#pragma unroll
    for (int p = 0; p < NP; ++p) {
      const unsigned f = ((start_value >> p) & 1u) ? 0xFFFFFFFFu : 0u;
      cnt.c[p] = W4{f, f, f, f};
    }
    if (MROWS <= 4) cnt.fold4(a);
    else cnt.fold8(a);
    if (COUNTS) {
#pragma unroll
      for (int p = 0; p < NP; ++p) store_plane_words(out + (unsigned long long)p * ldc, q, d, cnt.c[p]);
    } else {
      store_plane_words(out, q, d, cnt.c[NP - 1]);
    }
  }
}


// The vote of MANY rows on a SHORT vector.  vote_kernel's thread walks all M rows of its four words, eight
// at a time: ceil(M / 8) dependent round trips to memory, which a launch of less than a wave cannot hide.
// Here the rows are spread over the eight warps of a CTA (warp w takes rows w, w + 8, ..., four in flight
// per pass), a CTA covering 128 words (32 lanes x 4); each warp keeps the bit-sliced count of its rows,
// the partial counts meet in shared memory (NP x 4 KB) and the first warp adds them, plane by plane with
// a rippling carry, onto the start value.  Up to 32 rows are one round trip.  Measured on B200 against
// vote_kernel, us per launch: M = 31: 6.4 -> 3.2 at d = 2^20, 7.2 -> 6.3 at 2^22, 8.3 -> 11.1 at 2^23;
// M = 16: 3.8 -> 2.7 at 2^20, 4.4 -> 4.9 at 2^22; M = 100: 17.5 -> 7.1 at 2^20; M = 9 .. 12: no gain.
// With eight times the CTAs per word it loses once the launch exceeds a few waves; the host picks it by
// measured thresholds (vote_split).
template <int NP, bool COUNTS>
__global__ void __launch_bounds__(kThreads)
vote_split_kernel(const uint32_t* __restrict__ bits, unsigned M, unsigned long long d,
                  unsigned long long W, unsigned long long ldw, uint32_t* __restrict__ out,
                  unsigned long long ldc, unsigned start_value) {
  constexpr unsigned kWarps = kThreads / 32;
  __shared__ uint4 part[kWarps][NP][32];   // partial counts: [warp][plane][lane's four words]
  pdl_launch_dependents();
  pdl_wait();
  const unsigned lane = threadIdx.x & 31u;
  const unsigned warp = threadIdx.x >> 5;
  const unsigned long long chunks = (W + 3) / 4;
  const unsigned long long q = (unsigned long long)blockIdx.x * 32 + lane;   // this lane's chunk of four words
  const bool live = q < chunks;
  const uint32_t* col = bits + 4 * (live ? q : 0);
  const W4 zero{0u, 0u, 0u, 0u};
  Counter<NP> cnt;
#pragma unroll
  for (int p = 0; p < NP; ++p) cnt.c[p] = zero;
  for (unsigned r0 = warp; r0 < M; r0 += kWarps * 4) {
    W4 a[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const unsigned r = r0 + kWarps * k;
      a[k] = (live && r < M) ? ld_words(col + (unsigned long long)r * ldw) : zero;
    }
    cnt.fold4(a);
  }
#pragma unroll
  for (int p = 0; p < NP; ++p) part[warp][p][lane] = make_uint4(cnt.c[p].x, cnt.c[p].y, cnt.c[p].z, cnt.c[p].w);
  __syncthreads();
  if (warp != 0 || !live) return;
  W4 total[NP];   // the host sizes NP so that start value + M stays below 2^NP: no carry leaves the top plane
#pragma unroll
  for (int p = 0; p < NP; ++p) {
    const unsigned f = ((start_value >> p) & 1u) ? 0xFFFFFFFFu : 0u;
    total[p] = W4{f, f, f, f};
  }
#pragma unroll
  for (unsigned w = 0; w < kWarps; ++w) {
    W4 carry = zero;
#pragma unroll
    for (int p = 0; p < NP; ++p) {
      const uint4 v = part[w][p][lane];
      const W4 t = total[p];
      total[p] = W4{xor3(t.x, v.x, carry.x), xor3(t.y, v.y, carry.y), xor3(t.z, v.z, carry.z), xor3(t.w, v.w, carry.w)};
      carry = W4{maj3(t.x, v.x, carry.x), maj3(t.y, v.y, carry.y), maj3(t.z, v.z, carry.z), maj3(t.w, v.w, carry.w)};
    }
  }
  if (COUNTS) {
#pragma unroll
    for (int p = 0; p < NP; ++p) store_plane_words(out + (unsigned long long)p * ldc, q, d, total[p]);
  } else {
    store_plane_words(out, q, d, total[NP - 1]);
  }
}

}  // namespace

#endif  // SSGD_DEVICE_COMMON_CUH_
