"""Thin Python binding of the C ABI in ``include/signsgd.h``.

Argument marshalling only: every function takes torch tensors (device memory
and streams are torch's), checks dtype / device / contiguity, and passes raw
pointers and sizes to the function of the same name in ``libsignsgd_b200.so``.
All arithmetic of Algorithms 1-3 runs inside that library's CUDA kernels.
There is no fallback: if the library is missing or a call fails, an exception
is raised.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libsignsgd_b200.so")
MAX_WORKERS = 1024

_lib = None


class SignSGDError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__("%s failed: status %d (%s)" % (where, status, status_str(status)))


def lib() -> ctypes.CDLL:
    """Load the CUDA library (built by ``_build.build()``); raises if it is absent."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            "%s not found: build it with `python -m paper_1802_04434_b200._build` "
            "(needs nvcc); there is no CPU fallback" % LIB_PATH)
    L = ctypes.CDLL(LIB_PATH)
    sz, f32, vp, ci = ctypes.c_size_t, ctypes.c_float, ctypes.c_void_p, ctypes.c_int
    L.ssgd_words.restype = sz
    L.ssgd_words.argtypes = [sz]
    L.ssgd_density_from_sums.restype = ctypes.c_double
    L.ssgd_density_from_sums.argtypes = [ctypes.c_double, ctypes.c_double, sz]
    L.ssgd_count_planes.restype = sz
    L.ssgd_count_planes.argtypes = [sz]
    L.ssgd_warmup_steps.restype = sz
    L.ssgd_warmup_steps.argtypes = [f32]
    L.ssgd_step_is_fused.restype = ci
    L.ssgd_step_is_fused.argtypes = [sz, sz, ci]
    L.ssgd_status_str.restype = ctypes.c_char_p
    L.ssgd_status_str.argtypes = [ci]
    sigs = {
        "ssgd_sign_pack": [vp, sz, sz, sz, vp, sz, vp],
        "ssgd_signum_momentum_pack": [vp, vp, sz, sz, sz, f32, vp, sz, vp],
        "ssgd_majority_vote": [vp, sz, sz, sz, vp, vp],
        "ssgd_sign_apply": [vp, vp, sz, f32, vp],
        "ssgd_signsgd_step": [vp, vp, vp, sz, sz, sz, f32, f32, vp, sz, vp, vp],
        "ssgd_signum_warmup_pack": [vp, vp, sz, sz, sz, f32, vp, sz, vp],
        "ssgd_signsgd_warmup_step": [vp, vp, vp, sz, sz, sz, f32, f32, vp, sz, vp, vp],
        "ssgd_vote_counts": [vp, sz, sz, sz, vp, sz, vp],
        "ssgd_sum_apply": [vp, vp, sz, sz, sz, f32, vp],
        "ssgd_ternary_pack": [vp, vp, sz, sz, sz, f32, f32, vp, vp, sz, vp],
        "ssgd_quorum_vote": [vp, vp, sz, sz, sz, sz, vp, vp, vp],
        "ssgd_ternary_apply": [vp, vp, vp, sz, f32, vp],
        "ssgd_welford_update": [vp, sz, vp, vp, sz, vp],
        "ssgd_density_sums": [vp, sz, ci, vp, vp],
        "ssgd_signsgd_step_host": [vp, vp, vp, sz, sz, sz, f32, f32, vp, vp, sz, vp, vp, vp],
        "ssgd_signsgd_step_noalloc": [vp, vp, vp, sz, sz, sz, f32, f32, vp],
        "ssgd_signum_momentum_pack_scatter": [vp, vp, sz, f32, vp, sz, sz, sz, vp],
        "ssgd_majority_vote_staged": [vp, sz, sz, sz, vp, vp, vp],
        "ssgd_majority_vote_staged_wait_selftest": [vp, sz, sz, sz, vp, vp, vp],
    }
    for name, args in sigs.items():
        fn = getattr(L, name)
        fn.restype = ci
        fn.argtypes = args
    _lib = L
    return L


def status_str(status: int) -> str:
    return lib().ssgd_status_str(int(status)).decode()


def words(d: int) -> int:
    """ceil(d / 32)."""
    return int(lib().ssgd_words(d))


def _ptr(t: Optional[torch.Tensor], dtype, name: str, cuda: bool = True) -> Optional[int]:
    if t is None:
        return None
    if not isinstance(t, torch.Tensor) or t.dtype != dtype:
        raise TypeError("%s must be a torch tensor of dtype %s" % (name, dtype))
    if t.is_cuda != cuda:
        raise ValueError("%s must live in %s memory" % (name, "device" if cuda else "host"))
    if not t.is_contiguous():
        raise ValueError("%s must be contiguous" % name)
    return t.data_ptr()


def _need(t: torch.Tensor, n: int, name: str) -> None:
    if t.numel() < n:
        raise ValueError("%s holds %d elements, the call needs %d" % (name, t.numel(), n))


def _stream(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def _check(status: int, where: str) -> None:
    if status != 0:
        raise SignSGDError(status, where)


# words are stored in int32 tensors on the torch side (torch has no full uint32 support);
# the library sees the same 32 bits.
WORD_DTYPE = torch.int32


def sign_pack(g: torch.Tensor, M: int, d: int, ld: int, bits: torch.Tensor, ldw: int,
              stream=None) -> None:
    """Algorithm 1 / 3 worker side: bits[w] <- packed sign(g[w])."""
    _need(g, M * ld, "g"); _need(bits, M * ldw, "bits")
    _check(lib().ssgd_sign_pack(_ptr(g, torch.float32, "g"), M, d, ld,
                                _ptr(bits, WORD_DTYPE, "bits"), ldw, _stream(stream)),
           "ssgd_sign_pack")


def signum_momentum_pack(g: torch.Tensor, m: torch.Tensor, M: int, d: int, ld: int, beta: float,
                         bits: torch.Tensor, ldw: int, stream=None) -> None:
    """Algorithm 2 per worker, fused with packing: m updated in place, bits <- sign(m_new)."""
    _need(g, M * ld, "g"); _need(m, M * ld, "m"); _need(bits, M * ldw, "bits")
    _check(lib().ssgd_signum_momentum_pack(
        _ptr(g, torch.float32, "g"), _ptr(m, torch.float32, "m"), M, d, ld, beta,
        _ptr(bits, WORD_DTYPE, "bits"), ldw, _stream(stream)), "ssgd_signum_momentum_pack")


def majority_vote(bits: torch.Tensor, M: int, d: int, ldw: int, vote: torch.Tensor,
                  stream=None) -> None:
    """Algorithm 3 server side: vote <- packed sign of the sum of the workers' signs."""
    _need(bits, M * ldw, "bits"); _need(vote, -(-d // 32), "vote")
    _check(lib().ssgd_majority_vote(_ptr(bits, WORD_DTYPE, "bits"), M, d, ldw,
                                    _ptr(vote, WORD_DTYPE, "vote"), _stream(stream)),
           "ssgd_majority_vote")


def majority_vote_staged(bits: torch.Tensor, M: int, d: int, ldw: int, vote: torch.Tensor, status: torch.Tensor,
                         stream=None) -> None:
    """The majority vote by the kernel that stages the rows through shared memory with bulk copies; same
    output as `majority_vote`.  `status` is a one-element int32 device tensor, zero before the call; it is
    non-zero afterwards only if a bounded wait in the kernel ran out."""
    _need(bits, M * ldw, "bits"); _need(vote, -(-d // 32), "vote"); _need(status, 1, "status")
    _check(lib().ssgd_majority_vote_staged(_ptr(bits, WORD_DTYPE, "bits"), M, d, ldw, _ptr(vote, WORD_DTYPE, "vote"),
                                           _ptr(status, torch.int32, "status"), _stream(stream)),
           "ssgd_majority_vote_staged")


def sign_apply(x: torch.Tensor, vote: torch.Tensor, d: int, delta: float, stream=None) -> None:
    """Algorithm 3 worker side: x <- x - delta * sign(vote), in place."""
    _need(x, d, "x"); _need(vote, -(-d // 32), "vote")
    _check(lib().ssgd_sign_apply(_ptr(x, torch.float32, "x"), _ptr(vote, WORD_DTYPE, "vote"), d,
                                 delta, _stream(stream)), "ssgd_sign_apply")


def signsgd_step(x: torch.Tensor, g: torch.Tensor, m: Optional[torch.Tensor], M: int, d: int,
                 ld: int, beta: float, delta: float, bits_ws: torch.Tensor, ldw: int,
                 vote_ws: torch.Tensor, stream=None) -> None:
    """One step of Algorithm 3 with Signum workers (m=None with beta=0: plain signSGD)."""
    _need(x, d, "x"); _need(g, M * ld, "g"); _need(bits_ws, M * ldw, "bits_ws")
    _need(vote_ws, -(-d // 32), "vote_ws")
    if m is not None:
        _need(m, M * ld, "m")
    _check(lib().ssgd_signsgd_step(
        _ptr(x, torch.float32, "x"), _ptr(g, torch.float32, "g"), _ptr(m, torch.float32, "m"),
        M, d, ld, beta, delta, _ptr(bits_ws, WORD_DTYPE, "bits_ws"), ldw,
        _ptr(vote_ws, WORD_DTYPE, "vote_ws"), _stream(stream)), "ssgd_signsgd_step")


def step_is_fused(M: int, d: int, momentum: bool) -> bool:
    """Whether signsgd_step runs as one kernel for this problem on the current device (else worker,
    vote and apply kernels); a query for measurement tools."""
    return lib().ssgd_step_is_fused(M, d, 1 if momentum else 0) != 0


def step_kernel_name(M: int, d: int, momentum: bool) -> str:
    """Name of the kernel that is the whole step, or '' when the step is three kernels."""
    return ("", "fused_step_kernel", "step_rows_kernel")[lib().ssgd_step_is_fused(M, d, 1 if momentum else 0)]


def warmup_steps(beta: float) -> int:
    """C(beta) of Theorem 3: how many warm-up iterations Signum's analysis asks for (54 at 0.9)."""
    return int(lib().ssgd_warmup_steps(beta))


def signum_warmup_pack(g: torch.Tensor, m: torch.Tensor, M: int, d: int, ld: int, beta: float,
                       bits: torch.Tensor, ldw: int, stream=None) -> None:
    """Warm-up worker step of Theorem 3: m updated as in Algorithm 2, bits <- sign(g)."""
    _need(g, M * ld, "g"); _need(m, M * ld, "m"); _need(bits, M * ldw, "bits")
    _check(lib().ssgd_signum_warmup_pack(
        _ptr(g, torch.float32, "g"), _ptr(m, torch.float32, "m"), M, d, ld, beta,
        _ptr(bits, WORD_DTYPE, "bits"), ldw, _stream(stream)), "ssgd_signum_warmup_pack")


def signsgd_warmup_step(x: torch.Tensor, g: torch.Tensor, m: torch.Tensor, M: int, d: int, ld: int,
                        beta: float, delta: float, bits_ws: torch.Tensor, ldw: int,
                        vote_ws: torch.Tensor, stream=None) -> None:
    """One whole warm-up step (momentum accumulates, the vote is over sign(g))."""
    _need(x, d, "x"); _need(g, M * ld, "g"); _need(m, M * ld, "m")
    _need(bits_ws, M * ldw, "bits_ws"); _need(vote_ws, -(-d // 32), "vote_ws")
    _check(lib().ssgd_signsgd_warmup_step(
        _ptr(x, torch.float32, "x"), _ptr(g, torch.float32, "g"), _ptr(m, torch.float32, "m"),
        M, d, ld, beta, delta, _ptr(bits_ws, WORD_DTYPE, "bits_ws"), ldw,
        _ptr(vote_ws, WORD_DTYPE, "vote_ws"), _stream(stream)), "ssgd_signsgd_warmup_step")


def count_planes(M: int) -> int:
    """Bit planes that hold a vote count 0..M (the bit length of M)."""
    return int(lib().ssgd_count_planes(M))


def vote_counts(bits: torch.Tensor, M: int, d: int, ldw: int, counts: torch.Tensor, ldc: int,
                stream=None) -> None:
    """Server side of the "(good)" scheme of Sec. 4: bit-sliced number of +1 votes per parameter."""
    _need(bits, M * ldw, "bits"); _need(counts, count_planes(M) * ldc, "counts")
    _check(lib().ssgd_vote_counts(_ptr(bits, WORD_DTYPE, "bits"), M, d, ldw,
                                  _ptr(counts, WORD_DTYPE, "counts"), ldc, _stream(stream)),
           "ssgd_vote_counts")


def sum_apply(x: torch.Tensor, counts: torch.Tensor, M: int, d: int, ldc: int, delta: float,
              stream=None) -> None:
    """Worker side of the "(good)" scheme: x <- x - delta * (sum of the M signs), in place."""
    _need(x, d, "x"); _need(counts, count_planes(M) * ldc, "counts")
    _check(lib().ssgd_sum_apply(_ptr(x, torch.float32, "x"), _ptr(counts, WORD_DTYPE, "counts"), M, d,
                                ldc, delta, _stream(stream)), "ssgd_sum_apply")


def ternary_pack(g: torch.Tensor, m: Optional[torch.Tensor], M: int, d: int, ld: int, beta: float,
                 tau: float, sign_bits: torch.Tensor, active_bits: torch.Tensor, ldw: int,
                 stream=None) -> None:
    """Abstaining worker (Discussion): sign plane as in the 1-bit path, active plane = !(|v| < tau)."""
    _need(g, M * ld, "g"); _need(sign_bits, M * ldw, "sign_bits"); _need(active_bits, M * ldw, "active_bits")
    if m is not None:
        _need(m, M * ld, "m")
    _check(lib().ssgd_ternary_pack(
        _ptr(g, torch.float32, "g"), _ptr(m, torch.float32, "m"), M, d, ld, beta, tau,
        _ptr(sign_bits, WORD_DTYPE, "sign_bits"), _ptr(active_bits, WORD_DTYPE, "active_bits"), ldw,
        _stream(stream)), "ssgd_ternary_pack")


def quorum_vote(sign_bits: torch.Tensor, active_bits: torch.Tensor, M: int, d: int, ldw: int, quorum: int,
                vote_sign: torch.Tensor, vote_active: torch.Tensor, stream=None) -> None:
    """Server with quorum: decided where |P - N| >= max(quorum, 1), sign of P - N there."""
    _need(sign_bits, M * ldw, "sign_bits"); _need(active_bits, M * ldw, "active_bits")
    _need(vote_sign, -(-d // 32), "vote_sign"); _need(vote_active, -(-d // 32), "vote_active")
    _check(lib().ssgd_quorum_vote(
        _ptr(sign_bits, WORD_DTYPE, "sign_bits"), _ptr(active_bits, WORD_DTYPE, "active_bits"), M, d, ldw,
        quorum, _ptr(vote_sign, WORD_DTYPE, "vote_sign"), _ptr(vote_active, WORD_DTYPE, "vote_active"),
        _stream(stream)), "ssgd_quorum_vote")


def ternary_apply(x: torch.Tensor, vote_sign: torch.Tensor, vote_active: torch.Tensor, d: int, delta: float,
                  stream=None) -> None:
    """x moves by -/+ delta where the server decided, stays where it answered 0."""
    _need(x, d, "x"); _need(vote_sign, -(-d // 32), "vote_sign"); _need(vote_active, -(-d // 32), "vote_active")
    _check(lib().ssgd_ternary_apply(
        _ptr(x, torch.float32, "x"), _ptr(vote_sign, WORD_DTYPE, "vote_sign"),
        _ptr(vote_active, WORD_DTYPE, "vote_active"), d, delta, _stream(stream)), "ssgd_ternary_apply")


def welford_update(g: torch.Tensor, n: int, mean: torch.Tensor, m2: torch.Tensor, d: int, stream=None) -> None:
    """Fold the n-th gradient sample (n from 1) into the running mean and sum of squared deviations."""
    _need(g, d, "g"); _need(mean, d, "mean"); _need(m2, d, "m2")
    _check(lib().ssgd_welford_update(_ptr(g, torch.float32, "g"), n, _ptr(mean, torch.float32, "mean"),
                                     _ptr(m2, torch.float32, "m2"), d, _stream(stream)), "ssgd_welford_update")


def density(v: torch.Tensor, d: int, root: bool = False, sums: Optional[torch.Tensor] = None, stream=None) -> float:
    """phi(v) = |v|_1^2 / (d |v|_2^2) (Sec. 3); with root=True the density of sqrt(v).

    `sums` is a float64 device tensor of 2 elements used for the two norms (allocated here if not
    given).  Waits for the result: this is a measurement call, not part of the step."""
    _need(v, d, "v")
    if sums is None:
        sums = torch.zeros(2, dtype=torch.float64, device=v.device)
    _check(lib().ssgd_density_sums(_ptr(v, torch.float32, "v"), d, 1 if root else 0,
                                   _ptr(sums, torch.float64, "sums"), _stream(stream)), "ssgd_density_sums")
    l1, l2 = sums.tolist()
    return float(lib().ssgd_density_from_sums(l1, l2, d))


def signsgd_step_host(x: torch.Tensor, g_host: torch.Tensor, m: Optional[torch.Tensor], M: int,
                      d: int, ld: int, beta: float, delta: float, g_stage: torch.Tensor,
                      bits_ws: torch.Tensor, ldw: int, vote_ws: torch.Tensor,
                      vote_host: Optional[torch.Tensor], stream=None) -> None:
    """The whole step with gradients in (pinned) host memory and the vote read back to the host."""
    _need(x, d, "x"); _need(g_host, M * ld, "g_host"); _need(g_stage, M * ld, "g_stage")
    _need(bits_ws, M * ldw, "bits_ws"); _need(vote_ws, -(-d // 32), "vote_ws")
    if m is not None:
        _need(m, M * ld, "m")
    if vote_host is not None:
        _need(vote_host, -(-d // 32), "vote_host")
    _check(lib().ssgd_signsgd_step_host(
        _ptr(x, torch.float32, "x"), _ptr(g_host, torch.float32, "g_host", cuda=False),
        _ptr(m, torch.float32, "m"), M, d, ld, beta, delta,
        _ptr(g_stage, torch.float32, "g_stage"), _ptr(bits_ws, WORD_DTYPE, "bits_ws"), ldw,
        _ptr(vote_ws, WORD_DTYPE, "vote_ws"), _ptr(vote_host, WORD_DTYPE, "vote_host", cuda=False),
        _stream(stream)), "ssgd_signsgd_step_host")


MAX_PEERS = 64


def signum_momentum_pack_scatter(g: torch.Tensor, m: Optional[torch.Tensor], d: int, beta: float, rows, row: int,
                                 ldw: int, stream=None) -> None:
    """One worker's momentum update + sign packing, with its words stored into row `row` of every rank's
    rows buffer.  `rows` is a sequence with one entry per rank: a device tensor of int32 words (this
    GPU's own memory) or a raw device address as int (another GPU's memory this GPU can write)."""
    _need(g, d, "g")
    if m is not None:
        _need(m, d, "m")
    addrs = []
    for i, r in enumerate(rows):
        if isinstance(r, torch.Tensor):
            _need(r, (row + 1) * ldw, "rows[%d]" % i)
            addrs.append(_ptr(r, WORD_DTYPE, "rows[%d]" % i))
        else:
            addrs.append(int(r))
    table = (ctypes.c_void_p * len(addrs))(*addrs)
    _check(lib().ssgd_signum_momentum_pack_scatter(
        _ptr(g, torch.float32, "g"), _ptr(m, torch.float32, "m"), d, beta, table, len(addrs), row, ldw,
        _stream(stream)), "ssgd_signum_momentum_pack_scatter")


NOALLOC_SCRATCH_WORDS = 4 << 20


def signsgd_step_noalloc(x: torch.Tensor, g: torch.Tensor, m: Optional[torch.Tensor], M: int, d: int,
                         ld: int, beta: float, delta: float, stream=None) -> None:
    """The whole step without workspace arguments, for callers that cannot allocate device memory.

    The packed sign rows and the vote go to a fixed 16 MiB array inside the library, so the problem
    must satisfy (M + 1) * round_up(ceil(d / 32), 4) <= NOALLOC_SCRATCH_WORDS; larger ones raise
    (status 6).  Calls on one device share that array: keep them on one stream.  The first call on a
    device does a one-time address look-up and should come before any stream capture.
    """
    _need(x, d, "x"); _need(g, M * ld, "g")
    if m is not None:
        _need(m, M * ld, "m")
    _check(lib().ssgd_signsgd_step_noalloc(
        _ptr(x, torch.float32, "x"), _ptr(g, torch.float32, "g"), _ptr(m, torch.float32, "m"),
        M, d, ld, beta, delta, _stream(stream)), "ssgd_signsgd_step_noalloc")
