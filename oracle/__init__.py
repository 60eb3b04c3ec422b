"""CPU oracle for signSGD / Signum / majority vote (Algorithms 1-3 of the paper).

TEST INFRASTRUCTURE ONLY: the slow, plain definition that the CUDA library is
checked against.  Only the tests, the smoke check and the benchmark's
cpu-baseline leg may import this package; the product never does, and this
package imports nothing from the product.

The arithmetic lives in ``signsgd_ref.cpp`` (plain scalar C++).  This module
compiles it with g++ on first use and wraps each function for numpy arrays.
All arrays are host arrays: float32 for g / m / x, uint32 for packed words.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "signsgd_ref.cpp")
_LIB = os.path.join(_HERE, "libsignsgd_ref.so")

# Plain optimisation level, no fast-math, no contraction: the fused
# multiply-add of the momentum step is the one written in the source.
_CXXFLAGS = ["-O2", "-std=c++17", "-ffp-contract=off", "-fPIC", "-shared"]

_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle into a shared library next to its source."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    tmp = _LIB + ".tmp.%d" % os.getpid()
    subprocess.run(["g++", *_CXXFLAGS, "-o", tmp, _SRC], check=True)
    os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is not None:
        return _lib
    L = ctypes.CDLL(build())
    sz, f32, vp = ctypes.c_size_t, ctypes.c_float, ctypes.c_void_p
    L.ssgd_words_ref.restype = sz
    L.ssgd_words_ref.argtypes = [sz]
    L.ssgd_density_ref.restype = ctypes.c_double
    L.ssgd_density_ref.argtypes = [vp, sz, vp, vp]
    L.ssgd_density_of_root_ref.restype = ctypes.c_double
    L.ssgd_density_of_root_ref.argtypes = [vp, sz, vp, vp]
    L.ssgd_count_planes_ref.restype = sz
    L.ssgd_count_planes_ref.argtypes = [sz]
    L.ssgd_warmup_steps_ref.restype = sz
    L.ssgd_warmup_steps_ref.argtypes = [f32]
    for name, args in {
        "ssgd_sign_unpacked_ref": [vp, sz, vp],
        "ssgd_pack_bits_ref": [vp, sz, vp],
        "ssgd_unpack_bits_ref": [vp, sz, vp],
        "ssgd_sign_pack_ref": [vp, sz, sz, sz, vp, sz],
        "ssgd_momentum_ref": [vp, vp, sz, f32],
        "ssgd_signum_momentum_pack_ref": [vp, vp, sz, sz, sz, f32, vp, sz],
        "ssgd_signum_warmup_pack_ref": [vp, vp, sz, sz, sz, f32, vp, sz],
        "ssgd_signsgd_warmup_step_ref": [vp, vp, vp, sz, sz, sz, f32, f32, vp, sz, vp],
        "ssgd_ternary_pack_ref": [vp, vp, sz, sz, sz, f32, f32, vp, vp, sz],
        "ssgd_quorum_vote_ref": [vp, vp, sz, sz, sz, sz, vp, vp],
        "ssgd_ternary_apply_ref": [vp, vp, vp, sz, f32],
        "ssgd_welford_update_ref": [vp, sz, vp, vp, sz],
        "ssgd_vote_counts_ref": [vp, sz, sz, sz, vp],
        "ssgd_vote_count_planes_ref": [vp, sz, sz, sz, vp, sz],
        "ssgd_sum_apply_ref": [vp, vp, sz, sz, sz, f32],
        "ssgd_majority_vote_ref": [vp, sz, sz, sz, vp],
        "ssgd_sign_apply_ref": [vp, vp, sz, f32],
        "ssgd_signsgd_step_ref": [vp, vp, vp, sz, sz, sz, f32, f32, vp, sz, vp],
    }.items():
        fn = getattr(L, name)
        fn.restype = None
        fn.argtypes = args
    _lib = L
    return L


def _chk(a, dtype, min_size, name, writable=False):
    if not isinstance(a, np.ndarray) or a.dtype != dtype:
        raise TypeError("%s must be a numpy %s array" % (name, np.dtype(dtype)))
    if not a.flags.c_contiguous:
        raise ValueError("%s must be C-contiguous" % name)
    if a.size < min_size:
        raise ValueError("%s holds %d elements, needs %d" % (name, a.size, min_size))
    if writable and not a.flags.writeable:
        raise ValueError("%s must be writable" % name)
    return a.ctypes.data


def words(d: int) -> int:
    """ceil(d / 32): words per packed sign vector (d bits, Table 1)."""
    return int(_load().ssgd_words_ref(d))


def sign_unpacked(v: np.ndarray) -> np.ndarray:
    """sign(.) of Algorithms 1-3, one byte per element: 1 for +1, 0 for -1."""
    d = v.size
    s = np.empty(d, dtype=np.uint8)
    _load().ssgd_sign_unpacked_ref(_chk(v, np.float32, d, "v"), d, s.ctypes.data)
    return s


def pack_bits(s: np.ndarray) -> np.ndarray:
    d = s.size
    out = np.empty(words(d), dtype=np.uint32)
    _load().ssgd_pack_bits_ref(_chk(s, np.uint8, d, "s"), d, out.ctypes.data)
    return out


def unpack_bits(w: np.ndarray, d: int) -> np.ndarray:
    s = np.empty(d, dtype=np.uint8)
    _load().ssgd_unpack_bits_ref(_chk(w, np.uint32, words(d), "w"), d, s.ctypes.data)
    return s


def _rows(M, d, ld, ldw):
    ld = d if ld is None else ld
    ldw = words(d) if ldw is None else ldw
    if ld < d or ldw < words(d):
        raise ValueError("row stride shorter than the row")
    return ld, ldw


def sign_pack(g: np.ndarray, M: int, d: int, ld: int | None = None,
              ldw: int | None = None) -> np.ndarray:
    """Algorithm 1 / 3 worker side: bits[w] = packed sign(g[w])."""
    ld, ldw = _rows(M, d, ld, ldw)
    bits = np.zeros(M * ldw, dtype=np.uint32)
    _load().ssgd_sign_pack_ref(_chk(g, np.float32, M * ld, "g"), M, d, ld,
                               bits.ctypes.data, ldw)
    return bits


def momentum(g: np.ndarray, m: np.ndarray, beta: float) -> None:
    """Algorithm 2, momentum update of one row, in place on m."""
    d = g.size
    _load().ssgd_momentum_ref(_chk(g, np.float32, d, "g"),
                              _chk(m, np.float32, d, "m", True), d, beta)


def signum_momentum_pack(g: np.ndarray, m: np.ndarray, M: int, d: int,
                         beta: float, ld: int | None = None,
                         ldw: int | None = None) -> np.ndarray:
    """Algorithm 2 per worker (m updated in place), returns packed sign(m_new)."""
    ld, ldw = _rows(M, d, ld, ldw)
    bits = np.zeros(M * ldw, dtype=np.uint32)
    _load().ssgd_signum_momentum_pack_ref(
        _chk(g, np.float32, M * ld, "g"), _chk(m, np.float32, M * ld, "m", True),
        M, d, ld, beta, bits.ctypes.data, ldw)
    return bits


def vote_counts(bits: np.ndarray, M: int, d: int, ldw: int | None = None) -> np.ndarray:
    """Number of +1 votes per element (the inner sum of Algorithm 3, shifted)."""
    _, ldw = _rows(M, d, None, ldw)
    P = np.empty(d, dtype=np.int32)
    _load().ssgd_vote_counts_ref(_chk(bits, np.uint32, M * ldw, "bits"), M, d, ldw,
                                 P.ctypes.data)
    return P


def majority_vote(bits: np.ndarray, M: int, d: int, ldw: int | None = None) -> np.ndarray:
    """Algorithm 3 server side: packed sign[sum_m sign(.)], tie -> +1."""
    _, ldw = _rows(M, d, None, ldw)
    vote = np.empty(words(d), dtype=np.uint32)
    _load().ssgd_majority_vote_ref(_chk(bits, np.uint32, M * ldw, "bits"), M, d, ldw,
                                   vote.ctypes.data)
    return vote


def sign_apply(x: np.ndarray, vote: np.ndarray, d: int, delta: float) -> None:
    """Algorithm 3 worker side: x <- x - delta * sign(vote), in place."""
    _load().ssgd_sign_apply_ref(_chk(x, np.float32, d, "x", True),
                                _chk(vote, np.uint32, words(d), "vote"), d, delta)


def signsgd_step(x: np.ndarray, g: np.ndarray, m: np.ndarray | None, M: int, d: int,
                 beta: float, delta: float, ld: int | None = None,
                 ldw: int | None = None):
    """One step of Algorithm 3 with Signum workers; returns (bits, vote)."""
    ld, ldw = _rows(M, d, ld, ldw)
    bits = np.zeros(M * ldw, dtype=np.uint32)
    vote = np.empty(words(d), dtype=np.uint32)
    mp = None if m is None else _chk(m, np.float32, M * ld, "m", True)
    if m is None and beta != 0.0:
        raise ValueError("m may only be omitted when beta == 0")
    _load().ssgd_signsgd_step_ref(
        _chk(x, np.float32, d, "x", True), _chk(g, np.float32, M * ld, "g"), mp,
        M, d, ld, beta, delta, bits.ctypes.data, ldw, vote.ctypes.data)
    return bits, vote


def warmup_steps(beta: float) -> int:
    """C(beta) of Theorem 3 (the paper notes C(0.9) = 54)."""
    return int(_load().ssgd_warmup_steps_ref(beta))


def signum_warmup_pack(g: np.ndarray, m: np.ndarray, M: int, d: int, beta: float,
                       ld: int | None = None, ldw: int | None = None) -> np.ndarray:
    """Theorem 3 warm-up on the worker: m updated as in Algorithm 2, returns packed sign(g)."""
    ld, ldw = _rows(M, d, ld, ldw)
    bits = np.zeros(M * ldw, dtype=np.uint32)
    _load().ssgd_signum_warmup_pack_ref(
        _chk(g, np.float32, M * ld, "g"), _chk(m, np.float32, M * ld, "m", True),
        M, d, ld, beta, bits.ctypes.data, ldw)
    return bits


def signsgd_warmup_step(x: np.ndarray, g: np.ndarray, m: np.ndarray, M: int, d: int,
                        beta: float, delta: float, ld: int | None = None,
                        ldw: int | None = None):
    """One whole warm-up step; returns (bits, vote)."""
    ld, ldw = _rows(M, d, ld, ldw)
    bits = np.zeros(M * ldw, dtype=np.uint32)
    vote = np.empty(words(d), dtype=np.uint32)
    _load().ssgd_signsgd_warmup_step_ref(
        _chk(x, np.float32, d, "x", True), _chk(g, np.float32, M * ld, "g"),
        _chk(m, np.float32, M * ld, "m", True), M, d, ld, beta, delta,
        bits.ctypes.data, ldw, vote.ctypes.data)
    return bits, vote


def count_planes(M: int) -> int:
    """Bit planes needed for a vote count in 0..M."""
    return int(_load().ssgd_count_planes_ref(M))


def vote_count_planes(bits: np.ndarray, M: int, d: int, ldw: int | None = None,
                      ldc: int | None = None) -> np.ndarray:
    """Server side of the "(good)" scheme (Sec. 4): bit-sliced counts of +1 votes, [planes][ldc]."""
    _, ldw = _rows(M, d, None, ldw)
    ldc = words(d) if ldc is None else ldc
    out = np.zeros(count_planes(M) * ldc, dtype=np.uint32)
    _load().ssgd_vote_count_planes_ref(_chk(bits, np.uint32, M * ldw, "bits"), M, d, ldw,
                                       out.ctypes.data, ldc)
    return out


def sum_apply(x: np.ndarray, counts: np.ndarray, M: int, d: int, delta: float,
              ldc: int | None = None) -> None:
    """Worker side of the "(good)" scheme: x <- x - delta * sum_m sign(.), in place."""
    ldc = words(d) if ldc is None else ldc
    _load().ssgd_sum_apply_ref(_chk(x, np.float32, d, "x", True),
                               _chk(counts, np.uint32, count_planes(M) * ldc, "counts"),
                               M, d, ldc, delta)


def ternary_pack(g: np.ndarray, m: np.ndarray | None, M: int, d: int, beta: float, tau: float,
                 ld: int | None = None, ldw: int | None = None):
    """Abstaining worker (Discussion; thresholds are this code base's): returns (sign, active) planes.
    Parity with the paper unpinned: the paper gives no threshold."""
    ld, ldw = _rows(M, d, ld, ldw)
    sb = np.zeros(M * ldw, dtype=np.uint32)
    ab = np.zeros(M * ldw, dtype=np.uint32)
    mp = None if m is None else _chk(m, np.float32, M * ld, "m", True)
    _load().ssgd_ternary_pack_ref(_chk(g, np.float32, M * ld, "g"), mp, M, d, ld, beta, tau,
                                  sb.ctypes.data, ab.ctypes.data, ldw)
    return sb, ab


def quorum_vote(sign_bits: np.ndarray, active_bits: np.ndarray, M: int, d: int, quorum: int,
                ldw: int | None = None):
    """Server with quorum: returns (vote_sign, vote_active).  Parity with the paper unpinned."""
    _, ldw = _rows(M, d, None, ldw)
    vs = np.empty(words(d), dtype=np.uint32)
    va = np.empty(words(d), dtype=np.uint32)
    _load().ssgd_quorum_vote_ref(_chk(sign_bits, np.uint32, M * ldw, "sign_bits"),
                                 _chk(active_bits, np.uint32, M * ldw, "active_bits"), M, d, ldw, quorum,
                                 vs.ctypes.data, va.ctypes.data)
    return vs, va


def ternary_apply(x: np.ndarray, vote_sign: np.ndarray, vote_active: np.ndarray, d: int,
                  delta: float) -> None:
    """x moves by -/+ delta where the server decided, stays elsewhere.  Parity with the paper unpinned."""
    _load().ssgd_ternary_apply_ref(_chk(x, np.float32, d, "x", True),
                                   _chk(vote_sign, np.uint32, words(d), "vote_sign"),
                                   _chk(vote_active, np.uint32, words(d), "vote_active"), d, delta)


def density(v: np.ndarray):
    """phi(v) = |v|_1^2 / (d |v|_2^2) of Sec. 3; returns (phi, |v|_1, |v|_2^2)."""
    l1, l2 = ctypes.c_double(), ctypes.c_double()
    phi = _load().ssgd_density_ref(_chk(v, np.float32, v.size, "v"), v.size, ctypes.addressof(l1),
                                   ctypes.addressof(l2))
    return float(phi), l1.value, l2.value


def density_of_root(v: np.ndarray):
    """phi(sqrt(v)) for a non-negative v (Sec. 3: the noise density from a vector of variances);
    returns (phi, sum sqrt(v_i), sum v_i)."""
    l1, l2 = ctypes.c_double(), ctypes.c_double()
    phi = _load().ssgd_density_of_root_ref(_chk(v, np.float32, v.size, "v"), v.size, ctypes.addressof(l1),
                                           ctypes.addressof(l2))
    return float(phi), l1.value, l2.value


def welford_update(g: np.ndarray, n: int, mean: np.ndarray, m2: np.ndarray) -> None:
    """Welford's update with the n-th sample (n from 1), in place on mean and m2 (Sec. 3)."""
    d = g.size
    _load().ssgd_welford_update_ref(_chk(g, np.float32, d, "g"), n, _chk(mean, np.float32, d, "mean", True),
                                    _chk(m2, np.float32, d, "m2", True), d)
