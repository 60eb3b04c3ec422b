// Variants of the step that the paper discusses beside Algorithms 1-3:
//   * the "(good)" scheme of Section 4 (the server returns the vote count, not
//     its sign);
//   * "majority vote with abstention" of the Discussion: ternary {-1, 0, +1} in
//     both directions, a worker abstaining when unsure and the server answering 0
//     when no quorum is reached.
// See include/signsgd.h for the contract of each call.

#include "host_common.h"
#include "vote_launch.h"

namespace {

// ---------------------------------------------------------------------------
// sum-apply: the "(good)" update of Section 4, x <- x - delta * sum_m sign(.),
// from the bit-sliced count P of +1 votes: the sum of signs is 2P - M.  One fused
// multiply-add per element, x <- fma(-delta, float(2P - M), x).  Lane layout as
// in the apply kernel; each lane reads its word of every count plane.

constexpr int kApplyUnroll = 2;   // 128-bit loads of x in flight per thread, as in the apply kernel of the 1-bit path

// the sum of the M signs for the four elements of a lane, from its nibble of every count plane
template <int NP>
__device__ __forceinline__ void signed_sums(const unsigned (&nib)[NP], unsigned M, float (&s)[4]) {
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    int P = 0;
#pragma unroll
    for (int p = 0; p < NP; ++p) P |= (int)((nib[p] >> k) & 1u) << p;
    s[k] = (float)(2 * P - (int)M);
  }
}

// One tile of kThreads * 4 * kApplyUnroll elements per CTA; lane layout as in the apply kernel.
template <int NP>
__global__ void __launch_bounds__(kThreads)
sum_apply_kernel(float* __restrict__ x, const uint32_t* __restrict__ counts, unsigned M,
                 unsigned long long d, unsigned long long ldc, float delta) {
  constexpr int UNROLL = kApplyUnroll;
  constexpr unsigned long long TILE = (unsigned long long)kThreads * 4 * UNROLL;
  constexpr unsigned SPAN = 128 * UNROLL;
  const unsigned lane = threadIdx.x & 31u;
  const unsigned warp = threadIdx.x >> 5;
  const unsigned shift = 4u * (lane & 7u);
  const float neg = -delta;
  const unsigned long long e0 = (unsigned long long)blockIdx.x * TILE + (unsigned long long)warp * SPAN;
  if (e0 >= d) return;
  if (e0 + SPAN <= d) {
    float4 xv[UNROLL];
    unsigned nib[UNROLL][NP];
#pragma unroll
    for (int u = 0; u < UNROLL; ++u) {
      xv[u] = ld128(x + e0 + u * 128 + lane * 4);
#pragma unroll
      for (int p = 0; p < NP; ++p)
        nib[u][p] = __ldg(counts + (unsigned long long)p * ldc + (e0 >> 5) + u * 4 + (lane >> 3)) >> shift;
    }
#pragma unroll
    for (int u = 0; u < UNROLL; ++u) {
      float s[4];
      signed_sums<NP>(nib[u], M, s);
      float4 v = xv[u];
      v.x = __fmaf_rn(neg, s[0], v.x);
      v.y = __fmaf_rn(neg, s[1], v.y);
      v.z = __fmaf_rn(neg, s[2], v.z);
      v.w = __fmaf_rn(neg, s[3], v.w);
      st128(x + e0 + u * 128 + lane * 4, v);
    }
  } else {
#pragma unroll 1
    for (int u = 0; u < UNROLL; ++u) {
      const unsigned long long e = e0 + u * 128 + lane * 4;
      if (e >= d) break;
      unsigned nib[NP];
#pragma unroll
      for (int p = 0; p < NP; ++p) nib[p] = __ldg(counts + (unsigned long long)p * ldc + (e >> 5)) >> shift;
      float s[4];
      signed_sums<NP>(nib, M, s);
#pragma unroll
      for (int k = 0; k < 4; ++k)
        if (e + k < d) x[e + k] = __fmaf_rn(neg, s[k], x[e + k]);
    }
  }
}

template <int NP>
void launch_sum_apply_np(float* x, const uint32_t* counts, size_t M, size_t d, size_t ldc, float delta,
                         cudaStream_t s) {
  constexpr unsigned long long TILE = (unsigned long long)kThreads * 4 * kApplyUnroll;
  sum_apply_kernel<NP><<<grid_for((d + TILE - 1) / TILE), kThreads, 0, s>>>(x, counts, (unsigned)M, d, ldc, delta);
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

// ---------------------------------------------------------------------------
// majority vote with abstention (Discussion section).  The paper gives the scheme
// in words only; the thresholds are this library's:
//   worker   abstains on element i when |v_i| < tau (v = momentum or gradient);
//            it sends two planes, sign (bit = !(v < 0), the 1-bit words) and
//            active (bit = !(|v| < tau));
//   server   with P / N the numbers of active +1 / -1 votes, answers sign(P - N)
//            when |P - N| >= max(quorum, 1) and 0 otherwise, again as two planes,
//            vote_active and vote_sign (set only where active and positive);
//   worker   moves x by -/+ delta where the answer is active, else leaves it.

constexpr int kTernaryUnroll = 4;

__device__ __forceinline__ unsigned active_nibble(const float4& v, float tau) {
  return ((fabsf(v.x) < tau) ? 0u : 1u) | ((fabsf(v.y) < tau) ? 0u : 2u) | ((fabsf(v.z) < tau) ? 0u : 4u) |
         ((fabsf(v.w) < tau) ? 0u : 8u);
}

// One span that crosses the end of its row: element-wise guards; bits at
// positions >= d stay 0, nothing at or beyond d is written.
template <bool MOMENTUM>
__device__ __forceinline__ void ternary_ragged_span(const float* __restrict__ gr, float* __restrict__ mr,
                                                    uint32_t* __restrict__ sr, uint32_t* __restrict__ ar,
                                                    unsigned long long d, unsigned long long e0, float beta,
                                                    float omb, float tau) {
  const unsigned lane = threadIdx.x & 31u;
#pragma unroll 1
  for (int u = 0; u < kTernaryUnroll; ++u) {
    const unsigned long long e = e0 + u * 128 + lane * 4;
    unsigned snib = 0, anib = 0;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      if (e + k < d) {
        float v = gr[e + k];
        if (MOMENTUM) {
          v = momentum_update(beta, omb, mr[e + k], v);
          mr[e + k] = v;
        }
        snib |= sign_bit(v) << k;
        anib |= ((fabsf(v) < tau) ? 0u : 1u) << k;
      }
    }
    const unsigned sword = assemble_word(snib, lane);
    const unsigned aword = assemble_word(anib, lane);
    const unsigned long long first = e0 + u * 128 + (lane >> 3) * 32;  // first element of the word
    if ((lane & 7u) == 0 && first < d) {
      sr[u * 4 + (lane >> 3)] = sword;
      ar[u * 4 + (lane >> 3)] = aword;
    }
  }
}

// Same tiling and structure as the worker kernel of the 1-bit path (grid x = tile
// of kThreads * 16 elements within the row, y = row; all loads of a thread issued
// before their first use; RAGGED = false leaves the last partial span of a row to
// the tail kernel), with a second output plane.
template <bool MOMENTUM, bool RAGGED>
__global__ void __launch_bounds__(kThreads, 1)
ternary_pack_kernel(const float* __restrict__ g, float* __restrict__ m,
                    uint32_t* __restrict__ sign_bits, uint32_t* __restrict__ active_bits,
                    unsigned long long d, unsigned long long ld, unsigned long long ldw,
                    float beta, float omb, float tau) {
  constexpr int UNROLL = kTernaryUnroll;
  constexpr unsigned long long TILE = (unsigned long long)kThreads * 4 * UNROLL;
  constexpr unsigned SPAN = 128 * UNROLL;
  const unsigned lane = threadIdx.x & 31u;
  const unsigned warp = threadIdx.x >> 5;
  const unsigned long long row = blockIdx.y;
  const unsigned long long e0 = (unsigned long long)blockIdx.x * TILE + (unsigned long long)warp * SPAN;
  if (e0 + SPAN > d) {
    if (RAGGED && e0 < d)
      ternary_ragged_span<MOMENTUM>(g + row * ld, MOMENTUM ? m + row * ld : nullptr,
                                    sign_bits + row * ldw + (e0 >> 5), active_bits + row * ldw + (e0 >> 5), d, e0,
                                    beta, omb, tau);
    return;
  }
  const float* gr = g + row * ld + e0 + lane * 4;
  float* mr = MOMENTUM ? m + row * ld + e0 + lane * 4 : nullptr;
  float4 gv[UNROLL], mv[UNROLL];
#pragma unroll
  for (int u = 0; u < UNROLL; ++u) gv[u] = ld128(gr + u * 128);
  if (MOMENTUM) {
#pragma unroll
    for (int u = 0; u < UNROLL; ++u) mv[u] = ld128(mr + u * 128);
  }
  unsigned smine = 0, amine = 0;
#pragma unroll
  for (int u = 0; u < UNROLL; ++u) {
    float4 v = gv[u];
    if (MOMENTUM) {
      v = momentum_update4(beta, omb, mv[u], v);
      st128(mr + u * 128, v);
    }
    const unsigned sword = assemble_word(sign_nibble(v), lane);
    const unsigned aword = assemble_word(active_nibble(v, tau), lane);
    if ((lane & 7u) == (unsigned)u) {
      smine = sword;
      amine = aword;
    }
  }
  if ((lane & 7u) < (unsigned)UNROLL) {
    const unsigned long long w = row * ldw + (e0 >> 5) + own_word_index<UNROLL>(lane);
    sign_bits[w] = smine;
    active_bits[w] = amine;
  }
}

template <bool MOMENTUM>
__global__ void __launch_bounds__(32)
ternary_tail_kernel(const float* __restrict__ g, float* __restrict__ m, uint32_t* __restrict__ sign_bits,
                    uint32_t* __restrict__ active_bits, unsigned long long d, unsigned long long ld,
                    unsigned long long ldw, float beta, float omb, float tau) {
  constexpr unsigned SPAN = 128 * kTernaryUnroll;
  const unsigned long long row = blockIdx.x;
  const unsigned long long e0 = d / SPAN * SPAN;
  if (e0 < d)
    ternary_ragged_span<MOMENTUM>(g + row * ld, MOMENTUM ? m + row * ld : nullptr, sign_bits + row * ldw + (e0 >> 5),
                                  active_bits + row * ldw + (e0 >> 5), d, e0, beta, omb, tau);
}

// Large inputs (at least 8 CTAs per SM): interior-only main kernel, with the unused shared-memory request
// that the worker kernel of the 1-bit path uses as a carve-out hint, plus a one-warp-per-row tail launch
// when d is not a multiple of the span; smaller inputs: one launch with the guarded path inline.
template <bool MOMENTUM>
ssgd_status launch_ternary_pack(const float* g, float* m, size_t M, size_t d, size_t ld, float beta, float tau,
                                uint32_t* sign_bits, uint32_t* active_bits, size_t ldw, cudaStream_t s) {
  constexpr unsigned long long TILE = (unsigned long long)kThreads * 4 * kTernaryUnroll;
  DeviceInfo di;
  if (!device_info(&di)) return SSGD_ERR_CUDA;
  const unsigned long long tiles_per_row = (d + TILE - 1) / TILE;
  if (tiles_per_row > kMaxGrid) return SSGD_ERR_SIZE;
  const dim3 grid((unsigned)tiles_per_row, (unsigned)M);
  const float omb = 1.0f - beta;
  if (tiles_per_row * M >= 8ull * di.sms) {
    ternary_pack_kernel<MOMENTUM, false><<<grid, kThreads, 36 * 1024, s>>>(g, m, sign_bits, active_bits, d, ld, ldw,
                                                                             beta, omb, tau);
    if (d % (128 * kTernaryUnroll) != 0)
      ternary_tail_kernel<MOMENTUM><<<(unsigned)M, 32, 0, s>>>(g, m, sign_bits, active_bits, d, ld, ldw, beta, omb, tau);
  } else {
    ternary_pack_kernel<MOMENTUM, true><<<grid, kThreads, 0, s>>>(g, m, sign_bits, active_bits, d, ld, ldw, beta, omb,
                                                                  tau);
  }
  return launch_status();
}

// [D >= T] per bit position for a bit-sliced D held in NP planes (D < 2^NP):
// the carry out of D + (2^NP - T), rippled with one MAJ3 per plane.
template <int NP>
__device__ __forceinline__ W4 planes_ge(const Counter<NP>& c, unsigned T) {
  if (T == 0) return W4{0xFFFFFFFFu, 0xFFFFFFFFu, 0xFFFFFFFFu, 0xFFFFFFFFu};
  if (T >= (1u << NP)) return W4{0u, 0u, 0u, 0u};
  const unsigned K = (1u << NP) - T;
  W4 carry{0u, 0u, 0u, 0u};
#pragma unroll
  for (int p = 0; p < NP; ++p) {
    const unsigned k = ((K >> p) & 1u) ? 0xFFFFFFFFu : 0u;
    carry = W4{maj3(c.c[p].x, k, carry.x), maj3(c.c[p].y, k, carry.y), maj3(c.c[p].z, k, carry.z),
               maj3(c.c[p].w, k, carry.w)};
  }
  return carry;
}

// D = sum_w [active & sign] + sum_w [not (active & not sign)] = (P - N) + M, so
// both decisions are comparisons of one bit-sliced counter over 2M inputs:
// active-positive iff D >= M + Q', active-negative iff D <= M - Q'.
template <int NP>
__global__ void __launch_bounds__(kThreads)
quorum_vote_kernel(const uint32_t* __restrict__ sign_bits, const uint32_t* __restrict__ active_bits,
                   unsigned M, unsigned long long d, unsigned long long W, unsigned long long ldw,
                   uint32_t* __restrict__ vote_sign, uint32_t* __restrict__ vote_active,
                   unsigned t_hi, unsigned t_lo) {
  const unsigned long long chunks = (W + 3) / 4;
  const unsigned long long stride = (unsigned long long)gridDim.x * kThreads;
  for (unsigned long long q = (unsigned long long)blockIdx.x * kThreads + threadIdx.x; q < chunks; q += stride) {
    Counter<NP> cnt;
#pragma unroll
    for (int p = 0; p < NP; ++p) cnt.c[p] = W4{0u, 0u, 0u, 0u};
    for (unsigned w = 0; w < M; ++w) {
      const W4 s = ld_words(sign_bits + (unsigned long long)w * ldw + 4 * q);
      const W4 a = ld_words(active_bits + (unsigned long long)w * ldw + 4 * q);
      const W4 pos{a.x & s.x, a.y & s.y, a.z & s.z, a.w & s.w};
      const W4 notneg{~a.x | s.x, ~a.y | s.y, ~a.z | s.z, ~a.w | s.w};
      cnt.add2(pos, notneg);
    }
    const W4 hi = planes_ge<NP>(cnt, t_hi);         // P - N >= Q'
    const W4 lo = planes_ge<NP>(cnt, t_lo);         // P - N >= -Q' + 1, i.e. NOT decided negative
    store_plane_words(vote_sign, q, d, hi);
    store_plane_words(vote_active, q, d, W4{hi.x | ~lo.x, hi.y | ~lo.y, hi.z | ~lo.z, hi.w | ~lo.w});
  }
}

__device__ __forceinline__ float4 ternary_apply4(float4 v, unsigned snib, unsigned anib, float delta, float minus) {
  if (anib & 1u) v.x = __fadd_rn(v.x, (snib & 1u) ? minus : delta);
  if (anib & 2u) v.y = __fadd_rn(v.y, (snib & 2u) ? minus : delta);
  if (anib & 4u) v.z = __fadd_rn(v.z, (snib & 4u) ? minus : delta);
  if (anib & 8u) v.w = __fadd_rn(v.w, (snib & 8u) ? minus : delta);
  return v;
}

// One tile of kThreads * 4 * kApplyUnroll elements per CTA; lane layout as in the apply kernel.
__global__ void __launch_bounds__(kThreads)
ternary_apply_kernel(float* __restrict__ x, const uint32_t* __restrict__ vote_sign,
                     const uint32_t* __restrict__ vote_active, unsigned long long d, float delta) {
  constexpr int UNROLL = kApplyUnroll;
  constexpr unsigned long long TILE = (unsigned long long)kThreads * 4 * UNROLL;
  constexpr unsigned SPAN = 128 * UNROLL;
  const unsigned lane = threadIdx.x & 31u;
  const unsigned warp = threadIdx.x >> 5;
  const unsigned shift = 4u * (lane & 7u);
  const float minus = -delta;
  const unsigned long long e0 = (unsigned long long)blockIdx.x * TILE + (unsigned long long)warp * SPAN;
  if (e0 >= d) return;
  if (e0 + SPAN <= d) {
    float4 xv[UNROLL];
    unsigned sn[UNROLL], an[UNROLL];
#pragma unroll
    for (int u = 0; u < UNROLL; ++u) {
      xv[u] = ld128(x + e0 + u * 128 + lane * 4);
      sn[u] = __ldg(vote_sign + (e0 >> 5) + u * 4 + (lane >> 3)) >> shift;
      an[u] = __ldg(vote_active + (e0 >> 5) + u * 4 + (lane >> 3)) >> shift;
    }
#pragma unroll
    for (int u = 0; u < UNROLL; ++u)
      st128(x + e0 + u * 128 + lane * 4, ternary_apply4(xv[u], sn[u], an[u], delta, minus));
  } else {
#pragma unroll 1
    for (int u = 0; u < UNROLL; ++u) {
      const unsigned long long e = e0 + u * 128 + lane * 4;
      if (e >= d) break;
      const unsigned snib = __ldg(vote_sign + (e >> 5)) >> shift;
      const unsigned anib = __ldg(vote_active + (e >> 5)) >> shift;
#pragma unroll
      for (int k = 0; k < 4; ++k)
        if (e + k < d && ((anib >> k) & 1u)) x[e + k] = __fadd_rn(x[e + k], ((snib >> k) & 1u) ? minus : delta);
    }
  }
}

template <int NP>
void launch_quorum_np(const uint32_t* sb, const uint32_t* ab, size_t M, size_t d, size_t W, size_t ldw,
                      uint32_t* vs, uint32_t* va, unsigned t_hi, unsigned t_lo, cudaStream_t s) {
  const unsigned long long chunks = (W + 3) / 4;
  quorum_vote_kernel<NP><<<grid_for((chunks + kThreads - 1) / kThreads), kThreads, 0, s>>>(
      sb, ab, (unsigned)M, d, W, ldw, vs, va, t_hi, t_lo);
}

}  // namespace

extern "C" {

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
  if (d / ((size_t)kThreads * 4 * kApplyUnroll) >= kMaxGrid) return SSGD_ERR_SIZE;   // beyond any device's memory
  return launch_sum_apply(x, counts, M, d, ldc, delta, static_cast<cudaStream_t>(stream));
}

ssgd_status ssgd_ternary_pack(const float* g, float* m, size_t M, size_t d, size_t ld, float beta,
                              float tau, uint32_t* sign_bits, uint32_t* active_bits, size_t ldw,
                              void* stream) {
  if (!g || !sign_bits || !active_bits) return SSGD_ERR_NULL;
  if (!aligned16(g) || !aligned16(sign_bits) || !aligned16(active_bits) || (m && !aligned16(m)))
    return SSGD_ERR_ALIGN;
  const ssgd_status st = check_rows(M, d, ld, ldw, true);
  if (st != SSGD_OK) return st;
  if (!beta_ok(beta) || !(tau >= 0.0f) || !isfinite(tau)) return SSGD_ERR_ARG;
  if (!m && beta != 0.0f) return SSGD_ERR_NULL;
  if (d == 0) return SSGD_OK;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  return m ? launch_ternary_pack<true>(g, m, M, d, ld, beta, tau, sign_bits, active_bits, ldw, s)
           : launch_ternary_pack<false>(g, nullptr, M, d, ld, 0.0f, tau, sign_bits, active_bits, ldw, s);
}

ssgd_status ssgd_quorum_vote(const uint32_t* sign_bits, const uint32_t* active_bits, size_t M, size_t d,
                             size_t ldw, size_t quorum, uint32_t* vote_sign, uint32_t* vote_active,
                             void* stream) {
  if (!sign_bits || !active_bits || !vote_sign || !vote_active) return SSGD_ERR_NULL;
  if (!aligned16(sign_bits) || !aligned16(active_bits) || !aligned16(vote_sign) || !aligned16(vote_active))
    return SSGD_ERR_ALIGN;
  const ssgd_status st = check_rows(M, d, 0, ldw, false);
  if (st != SSGD_OK || d == 0) return st;
  const size_t Q = quorum < 1 ? 1 : quorum;            // a tie (P = N) never decides
  const unsigned planes = count_planes(2 * M);
  const unsigned t_hi = Q > M ? (1u << planes) : (unsigned)(M + Q);   // D >= M + Q
  const unsigned t_lo = Q > M ? 0u : (unsigned)(M - Q + 1);           // D >= M - Q + 1
  const size_t W = ssgd_words(d);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  switch (planes) {
    case 2: launch_quorum_np<2>(sign_bits, active_bits, M, d, W, ldw, vote_sign, vote_active, t_hi, t_lo, s); break;
    case 3: launch_quorum_np<3>(sign_bits, active_bits, M, d, W, ldw, vote_sign, vote_active, t_hi, t_lo, s); break;
    case 4: launch_quorum_np<4>(sign_bits, active_bits, M, d, W, ldw, vote_sign, vote_active, t_hi, t_lo, s); break;
    case 5: launch_quorum_np<5>(sign_bits, active_bits, M, d, W, ldw, vote_sign, vote_active, t_hi, t_lo, s); break;
    case 6: launch_quorum_np<6>(sign_bits, active_bits, M, d, W, ldw, vote_sign, vote_active, t_hi, t_lo, s); break;
    case 7: launch_quorum_np<7>(sign_bits, active_bits, M, d, W, ldw, vote_sign, vote_active, t_hi, t_lo, s); break;
    case 8: launch_quorum_np<8>(sign_bits, active_bits, M, d, W, ldw, vote_sign, vote_active, t_hi, t_lo, s); break;
    case 9: launch_quorum_np<9>(sign_bits, active_bits, M, d, W, ldw, vote_sign, vote_active, t_hi, t_lo, s); break;
    case 10: launch_quorum_np<10>(sign_bits, active_bits, M, d, W, ldw, vote_sign, vote_active, t_hi, t_lo, s); break;
    case 11: launch_quorum_np<11>(sign_bits, active_bits, M, d, W, ldw, vote_sign, vote_active, t_hi, t_lo, s); break;
    case 12: launch_quorum_np<12>(sign_bits, active_bits, M, d, W, ldw, vote_sign, vote_active, t_hi, t_lo, s); break;
    default: return SSGD_ERR_SIZE;
  }
  return launch_status();
}

ssgd_status ssgd_ternary_apply(float* x, const uint32_t* vote_sign, const uint32_t* vote_active, size_t d,
                               float delta, void* stream) {
  if (!x || !vote_sign || !vote_active) return SSGD_ERR_NULL;
  if (!aligned16(x) || !aligned16(vote_sign) || !aligned16(vote_active)) return SSGD_ERR_ALIGN;
  if (d > SIZE_MAX - 31) return SSGD_ERR_SIZE;
  if (!isfinite(delta)) return SSGD_ERR_ARG;
  if (d == 0) return SSGD_OK;
  constexpr unsigned long long TILE = (unsigned long long)kThreads * 4 * kApplyUnroll;
  if (d / TILE >= kMaxGrid) return SSGD_ERR_SIZE;   // beyond any device's memory
  ternary_apply_kernel<<<grid_for((d + TILE - 1) / TILE), kThreads, 0, static_cast<cudaStream_t>(stream)>>>(
      x, vote_sign, vote_active, d, delta);
  return launch_status();
}

}  // extern "C"
