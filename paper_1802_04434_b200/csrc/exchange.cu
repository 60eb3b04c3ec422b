// Algorithm 3 with one worker per GPU: the worker block fused with the exchange.
//
// In the paper the server pulls sign(g_m) from every worker.  With one worker per
// GPU and every GPU voting for itself, that pull is an all-gather of the packed
// sign rows.  Here the worker kernel does the gather's sending half itself: the
// lane that owns a sign word stores it straight into row `row` of the rows buffer
// of every rank (its own included) through peer pointers, while the same kernel
// streams g and m through HBM.  Per parameter a rank reads and writes 12 bytes of
// HBM and sends (P - 1) / 8 bytes over NVLink, so the transfer hides under the
// stream: there is no separate collective, only a barrier before the vote.
//
// Peer memory is only ever WRITTEN here, with plain 32-bit stores; the vote kernel
// later reads the rank's own copy of the rows from its own HBM.  No loads from
// peer memory, no cluster-wide copies, no waits inside the kernel: ordering between ranks
// (all rows have landed before a rank votes; a rank has finished voting before
// its rows are overwritten) is the caller's, on the host or by a barrier kernel
// between this launch and the vote.
// See include/signsgd.h for the contract.

#include "host_common.h"

namespace {

struct PeerRows {
  uint32_t* p[SSGD_MAX_PEERS];   // first word of the destination row on every rank
};

__device__ __forceinline__ void store_to_peers(const PeerRows& dst, unsigned P, unsigned long long word_index,
                                               unsigned word) {
  for (unsigned r = 0; r < P; ++r) dst.p[r][word_index] = word;
}

// One span that crosses the end of the vector: element-wise guards, padding bits
// stay 0, nothing at or beyond d is written.
template <bool MOMENTUM, int UNROLL>
__device__ __forceinline__ void scatter_ragged_span(const float* __restrict__ g, float* __restrict__ m,
                                                    const PeerRows& dst, unsigned P, unsigned long long d,
                                                    unsigned long long e0, float beta, float omb) {
  const unsigned lane = threadIdx.x & 31u;
#pragma unroll 1
  for (int u = 0; u < UNROLL; ++u) {
    const unsigned long long e = e0 + u * 128 + lane * 4;
    unsigned nib = 0;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      if (e + k < d) {
        float v = g[e + k];
        if (MOMENTUM) {
          v = momentum_update(beta, omb, m[e + k], v);
          m[e + k] = v;
        }
        nib |= sign_bit(v) << k;
      }
    }
    const unsigned word = assemble_word(nib, lane);
    const unsigned long long first = e0 + u * 128 + (lane >> 3) * 32;  // first element of the word
    if ((lane & 7u) == 0 && first < d) store_to_peers(dst, P, (e0 >> 5) + u * 4 + (lane >> 3), word);
  }
}

// Same tiling and lane layout as the worker kernel of the single-GPU step, one row.
template <bool MOMENTUM, int UNROLL, bool RAGGED>
__global__ void __launch_bounds__(kThreads, 1)
pack_scatter_kernel(const float* __restrict__ g, float* __restrict__ m, const PeerRows dst, unsigned P,
                    unsigned long long d, float beta, float omb) {
  constexpr unsigned long long TILE = (unsigned long long)kThreads * 4 * UNROLL;
  constexpr unsigned SPAN = 128 * UNROLL;
  const unsigned lane = threadIdx.x & 31u;
  const unsigned warp = threadIdx.x >> 5;
  const unsigned long long e0 = (unsigned long long)blockIdx.x * TILE + (unsigned long long)warp * SPAN;
  if (e0 + SPAN > d) {
    if (RAGGED && e0 < d) scatter_ragged_span<MOMENTUM, UNROLL>(g, m, dst, P, d, e0, beta, omb);
    return;
  }
  const float* gr = g + e0 + lane * 4;
  float* mr = MOMENTUM ? m + e0 + lane * 4 : nullptr;
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
    const unsigned word = assemble_word(sign_nibble(v), lane);
    if ((lane & 7u) == (unsigned)u) mine = word;
  }
  // the warp's 4 * UNROLL words sit in as many lanes: one 32-bit store per word and rank
  if ((lane & 7u) < (unsigned)UNROLL) store_to_peers(dst, P, (e0 >> 5) + own_word_index<UNROLL>(lane), mine);
}

template <bool MOMENTUM, int UNROLL>
__global__ void __launch_bounds__(32)
pack_scatter_tail_kernel(const float* __restrict__ g, float* __restrict__ m, const PeerRows dst, unsigned P,
                         unsigned long long d, float beta, float omb) {
  constexpr unsigned SPAN = 128 * UNROLL;
  const unsigned long long e0 = d / SPAN * SPAN;
  if (e0 < d) scatter_ragged_span<MOMENTUM, UNROLL>(g, m, dst, P, d, e0, beta, omb);
}

template <bool MOMENTUM, int UNROLL>
bool launch_scatter_u(const float* g, float* m, const PeerRows& dst, size_t P, size_t d, float beta,
                      cudaStream_t s) {
  constexpr unsigned long long TILE = (unsigned long long)kThreads * 4 * UNROLL;
  constexpr bool SPLIT = UNROLL >= 4;
  const unsigned long long tiles = (d + TILE - 1) / TILE;
  if (tiles > kMaxGrid) return false;
  const float omb = 1.0f - beta;
  // the same unused 36 KB shared-memory request as the worker kernel of the single-GPU step (carve-out hint)
  const size_t smem = SPLIT ? 36 * 1024 : 0;
  pack_scatter_kernel<MOMENTUM, UNROLL, !SPLIT><<<(unsigned)tiles, kThreads, smem, s>>>(g, m, dst, (unsigned)P, d, beta, omb);
  if constexpr (SPLIT) {
    if (d % (128 * UNROLL) != 0)
      pack_scatter_tail_kernel<MOMENTUM, UNROLL><<<1, 32, 0, s>>>(g, m, dst, (unsigned)P, d, beta, omb);
  }
  return true;
}

template <bool MOMENTUM>
ssgd_status launch_scatter(const float* g, float* m, const PeerRows& dst, size_t P, size_t d, float beta,
                           cudaStream_t s) {
  DeviceInfo di;
  if (!device_info(&di)) return SSGD_ERR_CUDA;
  // tile sizes as for the worker kernel with a momentum (one row)
  const bool ok = worker_unroll(d, 1, di.sms, true) == 4 ? launch_scatter_u<MOMENTUM, 4>(g, m, dst, P, d, beta, s)
                                                         : launch_scatter_u<MOMENTUM, 1>(g, m, dst, P, d, beta, s);
  return ok ? launch_status() : SSGD_ERR_SIZE;
}

}  // namespace

extern "C" ssgd_status ssgd_signum_momentum_pack_scatter(const float* g, float* m, size_t d, float beta,
                                                         uint32_t* const* rows, size_t P, size_t row,
                                                         size_t ldw, void* stream) {
  if (!g || !rows) return SSGD_ERR_NULL;
  if (!beta_ok(beta)) return SSGD_ERR_ARG;
  if (!m && beta != 0.0f) return SSGD_ERR_NULL;
  if (!aligned16(g) || (m && !aligned16(m))) return SSGD_ERR_ALIGN;
  if (P < 1 || P > SSGD_MAX_PEERS || row >= SSGD_MAX_WORKERS) return SSGD_ERR_SIZE;
  if (d > SIZE_MAX - 31) return SSGD_ERR_SIZE;
  if (ldw % 4 != 0) return SSGD_ERR_ALIGN;
  if (ldw < ssgd_words(d) || mul_overflows(row + 1, ldw) || mul_overflows((row + 1) * ldw, sizeof(uint32_t)))
    return SSGD_ERR_SIZE;
  PeerRows dst;
  for (size_t r = 0; r < P; ++r) {
    if (!rows[r]) return SSGD_ERR_NULL;
    if (!aligned16(rows[r])) return SSGD_ERR_ALIGN;
    dst.p[r] = rows[r] + row * ldw;
  }
  for (size_t r = P; r < SSGD_MAX_PEERS; ++r) dst.p[r] = nullptr;
  if (d == 0) return SSGD_OK;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  return m ? launch_scatter<true>(g, m, dst, P, d, beta, s) : launch_scatter<false>(g, nullptr, dst, P, d, beta, s);
}
