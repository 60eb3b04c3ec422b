/* signsgd.h -- C ABI of the B200 (sm_100a) signSGD / Signum / majority-vote library.
 *
 * The calls follow Algorithms 1-3 of Bernstein, Wang, Azizzadenesheli and
 * Anandkumar, "signSGD: Compressed Optimisation for Non-Convex Problems":
 * each of M workers turns its gradient (Algorithm 1) or its momentum
 * (Algorithm 2) into one sign bit per parameter, a server takes the majority
 * of the M bits per parameter, and every worker moves each parameter by
 * -delta or +delta according to the voted bit (Algorithm 3).  Here the M
 * workers are M rows of one buffer on one GPU.
 *
 * Notation: d parameters, M workers, W = ssgd_words(d) = ceil(d/32) words.
 *
 * Data layout (all fixed by this library; the paper only says "1-bit"):
 *   g, m   float [M][ld]   row w at g + w*ld; elements d..ld-1 of a row are
 *                          padding: they may be read, they are never written.
 *   x      float [d]
 *   bits   uint32 [M][ldw] row w at bits + w*ldw; word j of a row holds
 *                          elements 32j..32j+31, least significant bit first;
 *                          bit = 1 encodes sign +1, bit = 0 encodes sign -1;
 *                          bits at positions >= d are written as 0; words
 *                          W..ldw-1 of a row may be read, never written.
 *   vote   uint32 [W]      same bit layout as one row of bits.
 *
 * Sign and tie rules: sign(v) -> bit !(v < 0), so +0, -0 and NaN encode +1;
 * a vote with as many -1 as +1 (even M) resolves to +1, i.e. the voted bit is
 * [P >= ceil(M/2)] with P the number of set bits among the M workers.
 *
 * Unless a function says otherwise:
 *   - every pointer is a DEVICE pointer owned by the caller; the library does
 *     not allocate, free or retain memory, and keeps no state between calls;
 *   - float and word pointers must be 16-byte aligned; ld and ldw must be
 *     multiples of 4 with ld >= d and ldw >= W (so every row is 16-byte
 *     aligned); 1 <= M <= SSGD_MAX_WORKERS;
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream);
 *     work is enqueued on it and the call returns without waiting.  Stream
 *     order holds as for any kernel; the kernels of Algorithms 1-3 are
 *     launched as programmatic dependents of the kernel before them on the
 *     stream, i.e. they may be brought onto the GPU while that kernel drains,
 *     but touch no memory before it has completed;
 *   - d == 0 is valid: nothing is launched, SSGD_OK is returned;
 *   - buffers must not overlap except where "in place" is stated;
 *   - arguments are checked on the host before anything is launched; a failed
 *     check returns a status and touches no memory.  Nothing traps, aborts,
 *     throws or prints.  Input values are not scanned (NaN/Inf follow the bit
 *     rule above).
 */
#ifndef SIGNSGD_B200_H_
#define SIGNSGD_B200_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SSGD_MAX_WORKERS 1024

typedef enum {
  SSGD_OK = 0,
  SSGD_ERR_NULL = 1,  /* a required pointer is NULL                            */
  SSGD_ERR_ALIGN = 2, /* pointer not 16-byte aligned, or ld / ldw not 4-aligned */
  SSGD_ERR_SIZE = 3,  /* M out of range, ld < d, ldw < W, or a size overflows   */
  SSGD_ERR_ARG = 4,   /* beta outside [0,1) or NaN; delta not finite            */
  SSGD_ERR_CUDA = 5,  /* the CUDA runtime reported an error at launch / copy    */
  SSGD_ERR_SCRATCH = 6 /* problem needs more than the library's built-in scratch */
} ssgd_status;

/* ceil(d / 32): words per packed sign vector (d bits per vector, Table 1). */
size_t ssgd_words(size_t d);

/* Static, NUL-terminated description of a status code. */
const char* ssgd_status_str(ssgd_status s);

/* Algorithm 1, second line, and Algorithm 3 "pull sign(g_m)": each worker's
 * gradient becomes its 1-bit sign vector.
 *   g    in   [M][ld] gradients
 *   bits out  [M][ldw] packed signs, bit i of row w = !(g[w][i] < 0)          */
ssgd_status ssgd_sign_pack(const float* g, size_t M, size_t d, size_t ld,
                           uint32_t* bits, size_t ldw, void* stream);

/* Algorithm 2, lines 2-3, per worker, fused with the sign packing: in place
 *   m[w][i] <- fma(beta, m[w][i], fl((1 - beta) * g[w][i]))      (fp32, RN)
 * and bit i of row w = !(m_new[w][i] < 0): the sign of the NEW momentum is
 * what the worker sends.  beta in [0,1); beta == 0 gives m <- g and the bits
 * of ssgd_sign_pack.
 *   g    in      [M][ld]
 *   m    in/out  [M][ld], updated in place (elements >= d untouched)
 *   bits out     [M][ldw]                                                      */
ssgd_status ssgd_signum_momentum_pack(const float* g, float* m, size_t M,
                                      size_t d, size_t ld, float beta,
                                      uint32_t* bits, size_t ldw, void* stream);

/* Algorithm 3, server block: vote = sign[ sum_m sign(.) ] per parameter (the
 * "(best)" update of Section 4), from the M packed rows.
 *   bits in   [M][ldw]  (padding bits of each row must be 0, as written by the
 *                        two calls above)
 *   vote out  [W]       voted bit = [popcount over workers >= ceil(M/2)]       */
ssgd_status ssgd_majority_vote(const uint32_t* bits, size_t M, size_t d,
                               size_t ldw, uint32_t* vote, void* stream);

/* Algorithm 3, worker block (and the last line of Algorithms 1 and 2):
 *   x[i] <- x[i] - delta if voted bit i is 1, else x[i] + delta   (fp32, RN)
 *   x    in/out [d], in place;  vote in [W];  delta finite.                    */
ssgd_status ssgd_sign_apply(float* x, const uint32_t* vote, size_t d,
                            float delta, void* stream);

/* One whole step of Algorithm 3 with Signum workers: momentum + pack for all
 * M workers, majority vote, apply; same results as the three calls above in
 * sequence on `stream`.
 *   x        in/out [d]
 *   g        in     [M][ld]
 *   m        in/out [M][ld]; may be NULL only when beta == 0, which selects
 *                   Algorithm 3 as printed (workers send sign(g), no momentum)
 *   bits_ws  out    [M][ldw] workspace: holds the workers' wire words on return
 *   vote_ws  out    [W]      workspace: holds the server's wire words on return
 * Depending on M and d the step is issued as one kernel or as the worker, vote
 * and apply kernels, all on `stream` (ssgd_step_is_fused tells which).  The
 * results do not depend on the form.                                           */
ssgd_status ssgd_signsgd_step(float* x, const float* g, float* m, size_t M,
                              size_t d, size_t ld, float beta, float delta,
                              uint32_t* bits_ws, size_t ldw, uint32_t* vote_ws,
                              void* stream);

/* Launch shape of ssgd_signsgd_step on the current device (a query for
 * measurement tools; the result of the step does not depend on it): 1 when the
 * step for M workers and d parameters runs as ONE fused kernel (worker step of
 * every row, vote and apply on a tile of columns: Algorithm 3 as a whole in one
 * pass), 2 when it runs as the one-kernel form for short vectors (the rows of a
 * tile handled by different warps at the same time), 0 when it runs as the
 * worker, vote and apply kernels one after another.
 * momentum != 0 asks about the Signum step (m given), 0 about the sign-only step
 * (m == NULL).  Returns 0 for M or d out of range or when no device is current.  */
int ssgd_step_is_fused(size_t M, size_t d, int momentum);

/* Theorem 3 (Signum): the warm-up length C(beta), the least positive integer C
 * with (C/2) beta^C <= 1 / ((1 - beta^2)(C + 1)) and beta^(C+1) <= 1/2; the
 * paper notes C(0.9) = 54.  Pure host arithmetic, no GPU work.  Returns 0 when
 * beta is outside [0,1) or NaN.  The scan takes about 5/(1-beta) iterations. */
size_t ssgd_warmup_steps(float beta);

/* Theorem 3's warm-up iteration on the worker side: the momentum is updated as
 * in Algorithm 2, but the bit sent is the sign of the stochastic gradient.  Same
 * as ssgd_signum_momentum_pack (m updated in place, identical values) except that
 * bit i of row w = !(g[w][i] < 0), the words of ssgd_sign_pack.               */
ssgd_status ssgd_signum_warmup_pack(const float* g, float* m, size_t M, size_t d,
                                    size_t ld, float beta, uint32_t* bits,
                                    size_t ldw, void* stream);

/* One whole warm-up step: ssgd_signum_warmup_pack for all M workers, majority
 * vote, apply.  Arguments as ssgd_signsgd_step; m is required.  A training loop
 * calls this for iterations k < ssgd_warmup_steps(beta) and ssgd_signsgd_step
 * afterwards.                                                                  */
ssgd_status ssgd_signsgd_warmup_step(float* x, const float* g, float* m, size_t M,
                                     size_t d, size_t ld, float beta, float delta,
                                     uint32_t* bits_ws, size_t ldw,
                                     uint32_t* vote_ws, void* stream);

/* The "(good)" scheme of Section 4, x <- x - delta * sum_m sign(g_m): the server
 * sends back the vote COUNT instead of its sign, so the way down is no longer
 * 1-bit.  Here the count travels bit-sliced:
 *   counts uint32 [ssgd_count_planes(M)][ldc]: bit k of word j of plane p is bit
 *   p of P_(32j+k), the number of workers whose bit for parameter 32j+k is set
 *   (0 <= P <= M); ldc a multiple of 4, ldc >= W; bits at positions >= d are 0.
 * ssgd_count_planes(M) = bit length of M (planes needed for 0..M); 0 if M is
 * out of range.                                                               */
size_t ssgd_count_planes(size_t M);

/* Server side of the "(good)" scheme: count the +1 votes per parameter.
 *   bits in [M][ldw]; counts out [ssgd_count_planes(M)][ldc].                  */
ssgd_status ssgd_vote_counts(const uint32_t* bits, size_t M, size_t d, size_t ldw,
                             uint32_t* counts, size_t ldc, void* stream);

/* Worker side of the "(good)" scheme: with S = 2 P - M the sum of the M signs,
 *   x[i] <- fma(-delta, (float)S_i, x[i])       (one fp32 rounding), in place.
 * The sign of S is the majority vote (S = 0 being the tie).                    */
ssgd_status ssgd_sum_apply(float* x, const uint32_t* counts, size_t M, size_t d,
                           size_t ldc, float delta, void* stream);

/* "Majority vote with abstention" (Discussion section): ternary {-1, 0, +1}
 * messages in both directions.  The paper describes the scheme in words and gives
 * no thresholds; the two below (tau, quorum) are this library's definition.
 * A ternary vector travels as two bit planes with the layout of a sign row:
 * `sign` (bit = !(v < 0)) and `active` (bit set = a vote was cast).
 *
 * Worker side: v = g (m == NULL, beta == 0) or the updated momentum (as in
 * ssgd_signum_momentum_pack, m updated in place); the worker abstains on element
 * i when |v_i| < tau.  tau >= 0, finite; tau == 0 never abstains, and the sign
 * plane always equals the 1-bit words of ssgd_sign_pack / ssgd_signum_momentum_pack.
 *   sign_bits, active_bits out [M][ldw].                                       */
ssgd_status ssgd_ternary_pack(const float* g, float* m, size_t M, size_t d, size_t ld,
                              float beta, float tau, uint32_t* sign_bits,
                              uint32_t* active_bits, size_t ldw, void* stream);

/* Server side: with P / N the numbers of active +1 / -1 votes on a parameter, the
 * answer is sign(P - N) when |P - N| >= max(quorum, 1) ("quorum reached") and 0
 * otherwise (the margin among the cast votes is too small; a tie never decides).
 *   vote_active out [W]: bit set = a decision was taken;
 *   vote_sign   out [W]: bit set = decided +1 (0 where undecided).             */
ssgd_status ssgd_quorum_vote(const uint32_t* sign_bits, const uint32_t* active_bits,
                             size_t M, size_t d, size_t ldw, size_t quorum,
                             uint32_t* vote_sign, uint32_t* vote_active, void* stream);

/* Worker side: x[i] <- x[i] -/+ delta where vote_active is set (by vote_sign as
 * in ssgd_sign_apply); x[i] unchanged where the server answered 0.             */
ssgd_status ssgd_ternary_apply(float* x, const uint32_t* vote_sign,
                               const uint32_t* vote_active, size_t d, float delta,
                               void* stream);

/* Section 3, "density" of a vector: phi(v) = |v|_1^2 / (d |v|_2^2), 1 for a fully
 * dense vector and 1/d for a one-hot one.  ssgd_density_sums leaves
 *   sums[0] = sum_i |t_i|,  sums[1] = sum_i t_i^2      (DEVICE double[2], 16-byte
 * aligned, overwritten) with t = v when root == 0 and t = sqrt(v) when root != 0
 * (v >= 0 then; used for the noise vector, see below), accumulated in fp64; the
 * order of the additions is not fixed, so the last bits may vary from call to
 * call.  phi = ssgd_density_from_sums(sums[0], sums[1], d) on the host (0 when
 * d == 0 or the vector is all zero).                                           */
ssgd_status ssgd_density_sums(const float* v, size_t d, int root, double* sums, void* stream);
double ssgd_density_from_sums(double l1, double l2_squared, size_t d);

/* Section 3: Welford's single-pass algorithm for the mean gradient g and its
 * per-component variance.  Folds the n-th sample (n counts from 1, n <= 2^24)
 * into the running state, in place, per element, in fp32:
 *   d1 = g - mean;  mean <- mean + d1 / n;  d2 = g - mean;  m2 <- fma(d1, d2, m2).
 * After n samples mean is the sample mean and m2 / (n - 1) the sample variance;
 * the noise density phi(sigma) is ssgd_density_sums(m2, d, root = 1) since the
 * factor 1 / (n - 1) cancels in phi.  Start from mean = m2 = 0.
 *   g in [d];  mean, m2 in/out [d].                                            */
ssgd_status ssgd_welford_update(const float* g, size_t n, float* mean, float* m2,
                                size_t d, void* stream);

/* ssgd_signsgd_step for a caller whose gradients live in HOST memory
 * (Algorithm 3's "independent gradient estimate" arriving from outside the
 * device): copies g_host to the device staging buffer, runs the step, and
 * copies the voted words back to the host; everything is ordered after what
 * `stream` already holds, and complete once `stream` has been synchronised.
 * A large transfer (128 MB and more of gradients) is cut into up to 32 slabs of
 * columns, copied by a stream that the call creates and releases, while `stream`
 * runs the step on the slabs that have arrived (the step is elementwise in the
 * parameter index, so the results are those of one step on the whole vector);
 * smaller ones, and calls made while `stream` is being captured, are one copy
 * and one step on `stream`.
 *   g_host    in   HOST  [M][ld]; page-locked memory makes the copies
 *                  asynchronous and lets them overlap the kernels
 *   g_stage   out  DEVICE [M][ld] staging buffer for the gradients (elements
 *                  d..ld-1 of its rows may be left unwritten)
 *   vote_host out  HOST  [W] (may be NULL: no copy back); valid once `stream`
 *                  has been synchronised
 *   x, m, bits_ws, vote_ws: DEVICE, as in ssgd_signsgd_step.                   */
ssgd_status ssgd_signsgd_step_host(float* x, const float* g_host, float* m,
                                   size_t M, size_t d, size_t ld, float beta,
                                   float delta, float* g_stage,
                                   uint32_t* bits_ws, size_t ldw,
                                   uint32_t* vote_ws, uint32_t* vote_host,
                                   void* stream);

/* ssgd_majority_vote (Algorithm 3, server block) computed by a second kernel design: the M rows of a
 * 1024-word tile are staged through shared memory by bulk asynchronous copies (8 rows per mbarrier
 * phase, double-buffered) instead of being loaded into registers directly.  Same arguments, same
 * output words.  It is kept so that the two designs can be measured side by side (on B200 the direct
 * kernel is at least as fast; the step entry points use that one).
 *   status  in/out DEVICE unsigned (4-byte aligned), set it to 0 before the call: every wait in the
 *                  kernel has an iteration limit, and a CTA whose copies do not arrive within it
 *                  sets bit 0 here and writes no output instead of waiting forever.  Read it after
 *                  synchronising the stream; it stays 0 in normal operation. */
ssgd_status ssgd_majority_vote_staged(const uint32_t* bits, size_t M, size_t d,
                                      size_t ldw, uint32_t* vote, unsigned* status,
                                      void* stream);

/* Self-test of the bounded waits of ssgd_majority_vote_staged (no counterpart in the paper): the same
 * launch with every wait made to run out (each phase is armed for more bytes than its copies deliver;
 * all copies still complete).  The kernel must return within its iteration limits (about 0.2 s) with
 * bit 0 of *status set and `vote` untouched; the context stays usable.  d <= 32768 (one tile). */
ssgd_status ssgd_majority_vote_staged_wait_selftest(const uint32_t* bits, size_t M, size_t d,
                                                    size_t ldw, uint32_t* vote,
                                                    unsigned* status, void* stream);

/* Most ranks one ssgd_signum_momentum_pack_scatter call can send to. */
#define SSGD_MAX_PEERS 64

/* Algorithm 3 with one worker per GPU, the worker's half of a step in one kernel:
 * Algorithm 2's momentum update on THIS worker's g and m and the 1-bit packing of
 * its sign (exactly ssgd_signum_momentum_pack with M = 1; m == NULL with beta == 0
 * sends sign(g) as Algorithm 3 prints it), fused with the transport of Algorithm
 * 3's "pull sign(g_m)": every packed word is stored directly into row `row` of the
 * rows buffer of each of P ranks, so that afterwards every rank holds this
 * worker's d bits (Table 1: d bits up per worker) without a separate collective.
 *   g      in      DEVICE [d] (16-byte aligned), this worker's gradient
 *   m      in/out  DEVICE [d], updated in place; NULL allowed iff beta == 0
 *   rows   in      HOST array of P DEVICE pointers (read during the call only):
 *                  rows[r] is the [.][ldw] rows buffer of rank r, 16-byte aligned;
 *                  it may live in another GPU's memory that this GPU can write
 *                  (peer access enabled / symmetric memory), or in this GPU's own.
 *                  1 <= P <= SSGD_MAX_PEERS; list this rank's own buffer too.
 *   row            this worker's index: words go to rows[r] + row * ldw + j,
 *                  j < W; words W..ldw-1 of the row are not written; bits >= d are 0.
 *   ldw            row stride in words, a multiple of 4, >= W.
 * The kernel only WRITES the destination rows (plain 32-bit stores) and contains
 * no waits.  Ordering between ranks is the caller's: before a rank votes on its
 * rows buffer, every rank's call must have completed (e.g. a barrier across the
 * ranks enqueued after this call); before a rows buffer is written again, its
 * owner must have finished reading it.  Errors as for ssgd_signum_momentum_pack;
 * a NULL entry of rows gives SSGD_ERR_NULL, P or row out of range SSGD_ERR_SIZE. */
ssgd_status ssgd_signum_momentum_pack_scatter(const float* g, float* m, size_t d,
                                              float beta, uint32_t* const* rows,
                                              size_t P, size_t row, size_t ldw,
                                              void* stream);

/* Capacity, in 32-bit words, of the scratch area that ssgd_signsgd_step_noalloc
 * uses (16 MiB of device memory per GPU that loads the library, held until the
 * process exits). */
#define SSGD_NOALLOC_SCRATCH_WORDS ((size_t)4 << 20)

/* ssgd_signsgd_step for callers that cannot provide the two word workspaces.
 * (The paper has no counterpart to this call: it is a packaging variant of the
 * step above, with the same arithmetic and the same results for x and m.)
 *
 * Who needs it: code that runs where device memory can no longer be obtained --
 * for instance an optimiser hook inside a training process whose framework has
 * already reserved all device memory for its own pool, so that a raw cudaMalloc
 * would fail, or a latency-sensitive loop that must avoid cudaMalloc / cudaFree
 * because those calls may synchronise the whole device.  Such a caller owns x,
 * g and m anyway, but has nowhere to put the packed sign rows and the vote.
 *
 * This call takes no workspace arguments and allocates nothing (no cudaMalloc,
 * cudaFree, or allocating library routine): the M sign rows and the vote live in
 * a fixed array inside the library, SSGD_NOALLOC_SCRATCH_WORDS words long.  With
 * W = ssgd_words(d) and W4 = W rounded up to a multiple of 4, the call needs
 * (M + 1) * W4 words; a larger problem is rejected with SSGD_ERR_SCRATCH before
 * anything is launched (use ssgd_signsgd_step with your own buffers instead).
 *
 *   x in/out [d], g in [M][ld], m in/out [M][ld] (NULL allowed iff beta == 0):
 *   DEVICE pointers with the same rules as ssgd_signsgd_step.
 *
 * The first call on each device looks up the device address of the built-in
 * array (with that device current) and remembers it for as long as the device's
 * primary context lives (after cudaDeviceReset the remembered address is stale:
 * do not call this again in that process); make that first call before starting
 * any stream capture.  All calls on a device share the one array, and it keeps
 * whatever the previous call left there.  Nothing in it has to start at zero:
 * every sign word and vote word that can reach x is written by the call before
 * it is read; the only stale words a call may read are the up to three padding
 * words that round a row up to a multiple of 4, and the vote masks every bit at
 * a position >= d, so they cannot influence any output bit.  Two calls whose GPU
 * work can overlap (different streams, or different host threads on the same
 * device) race on that array: issue them on one stream, or order them yourself.
 * The wire words are not returned; callers who want them use ssgd_signsgd_step. */
ssgd_status ssgd_signsgd_step_noalloc(float* x, const float* g, float* m,
                                      size_t M, size_t d, size_t ld, float beta,
                                      float delta, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* SIGNSGD_B200_H_ */
