"""The four compute calls of the step, served by the CPU oracle on CPU torch tensors.

Used by CPU tests of the host-side logic that sits above the kernels (which rank's row goes where,
what is exchanged), where the CUDA library cannot run.  Same call signatures as the CUDA binding.
"""
import numpy as np
import torch

import oracle


def _u32(t: torch.Tensor) -> np.ndarray:
    return t.numpy().view(np.uint32)


def _put_rows(dst: torch.Tensor, src: np.ndarray, M: int, ldw: int, W: int) -> None:
    out = _u32(dst).reshape(-1)
    for w in range(M):                                   # words W..ldw-1 of a row are never written
        out[w * ldw:w * ldw + W] = src[w * ldw:w * ldw + W]


def sign_pack(g, M, d, ld, bits, ldw, stream=None):
    _put_rows(bits, oracle.sign_pack(g.numpy().reshape(-1), M, d, ld=ld, ldw=ldw), M, ldw, oracle.words(d))


def signum_momentum_pack(g, m, M, d, ld, beta, bits, ldw, stream=None):
    mf = m.numpy().reshape(-1)                           # shares memory: updated in place
    _put_rows(bits, oracle.signum_momentum_pack(g.numpy().reshape(-1), mf, M, d, beta, ld=ld, ldw=ldw),
              M, ldw, oracle.words(d))


def majority_vote(bits, M, d, ldw, vote, stream=None):
    _u32(vote)[:oracle.words(d)] = oracle.majority_vote(_u32(bits).reshape(-1), M, d, ldw=ldw)


def sign_apply(x, vote, d, delta, stream=None):
    oracle.sign_apply(x.numpy(), _u32(vote), d, delta)


def signum_momentum_pack_scatter(g, m, d, beta, rows, row, ldw, stream=None):
    """One worker's row computed by the oracle and copied into row `row` of every rows buffer given."""
    W = oracle.words(d)
    gf = g.numpy().reshape(-1)[:d]
    if m is None:
        words = oracle.sign_pack(np.ascontiguousarray(gf), 1, d)
    else:
        mf = m.numpy().reshape(-1)[:d]                   # a view: updated in place
        words = oracle.signum_momentum_pack(np.ascontiguousarray(gf), mf, 1, d, beta)
    for r in rows:
        _u32(r).reshape(-1)[row * ldw:row * ldw + W] = words[:W]
