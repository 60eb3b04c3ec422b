"""Seeded synthetic inputs for the signSGD / Signum / majority-vote step.

This module only draws random numbers and lays them out; it holds none of the
method's arithmetic (no momentum, no sign, no packing, no vote) and is the one
piece of code that both the CUDA path's callers and the CPU oracle's callers
use, so that both sides see the very same inputs.

The paper trains Resnet-20 / Resnet-50 and shows (Sec. 4, the noise histograms)
that per-parameter gradient noise is unimodal and roughly symmetric, Gaussian at
batch size 256.  Datasets and trained weights are not available here, so every
workload is a stand-in with the same vector sizes and with noise of that kind:
a per-element mean shared by all workers plus independent per-worker noise.

All tensors are float32.  Gradients are returned as a ``[M, ld]`` tensor (one
row per worker, row stride ``ld`` a multiple of 4 so that every row starts on a
16-byte boundary); elements ``d <= i < ld`` of a row are zero.  Draws come from
``torch.Generator`` objects seeded from (seed, workload, step, worker), on the
device asked for; CPU and CUDA generators give different streams, so a test
always hands the oracle a host copy of the very tensor the GPU consumed.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Callable, List, Optional

import torch

_CHUNK = 1 << 24  # elements drawn at a time, bounds temporary memory


def round_up(n: int, k: int) -> int:
    return (n + k - 1) // k * k


def _gen(device, *key: int) -> torch.Generator:
    """Generator on `device` seeded by mixing the integer key (splitmix-style)."""
    s = 0x9E3779B97F4A7C15
    for k in key:
        s = (s ^ (int(k) + 0x9E3779B97F4A7C15 + ((s << 6) & (2**64 - 1)) + (s >> 2))) & (2**64 - 1)
        s = (s * 0xBF58476D1CE4E5B9) & (2**64 - 1)
        s ^= s >> 31
    g = torch.Generator(device=device)
    g.manual_seed(s & (2**63 - 1))
    return g


def _randn(n: int, gen: torch.Generator, device) -> torch.Tensor:
    return torch.randn(n, generator=gen, device=device, dtype=torch.float32)


def _rand(n: int, gen: torch.Generator, device) -> torch.Tensor:
    return torch.rand(n, generator=gen, device=device, dtype=torch.float32)


def resnet50_tensor_sizes() -> List[int]:
    """Element counts of the 161 conv / batch-norm / fc tensors of a Resnet-50.

    Stem 7x7 conv 3->64; four bottleneck stages of [3, 4, 6, 3] blocks with
    widths 64/128/256/512 and 4x expansion, a 1x1 projection in the first block
    of each stage; one scale and one shift vector per conv; fc 2048->1000 with
    bias.
    """
    sizes: List[int] = []

    def conv_bn(cin: int, cout: int, k: int) -> None:
        sizes.extend([cout * cin * k * k, cout, cout])

    conv_bn(3, 64, 7)
    cin = 64
    for width, blocks in zip((64, 128, 256, 512), (3, 4, 6, 3)):
        for b in range(blocks):
            conv_bn(cin, width, 1)
            conv_bn(width, width, 3)
            conv_bn(width, 4 * width, 1)
            if b == 0:
                conv_bn(cin, 4 * width, 1)
            cin = 4 * width
    sizes.extend([2048 * 1000, 1000])
    assert len(sizes) == 161 and sum(sizes) == 25_557_032
    return sizes


@dataclasses.dataclass
class Workload:
    """One named configuration: sizes, hyper-parameters and input recipes."""
    name: str
    key: int                      # integer mixed into every seed
    d: int                        # parameters (after per-tensor padding, if any)
    M: int                        # workers
    beta: float                   # Signum momentum constant; 0 = signSGD
    delta: float                  # learning rate
    steps: int = 1
    seed: int = 0
    momentum_buffer: bool = True  # False: the beta = 0 path runs without m
    # fill(row_out[d], step, worker, gen, shared) -> None
    _fill: Optional[Callable] = None
    # shared(device) -> object drawn once per workload (e.g. the mean vector)
    _shared: Optional[Callable] = None
    segments: Optional[List[tuple]] = None  # (offset, size) of each tensor

    @property
    def ld(self) -> int:
        return round_up(self.d, 4)

    @property
    def words(self) -> int:
        return (self.d + 31) // 32

    @property
    def ldw(self) -> int:
        return round_up(self.words, 4)

    def x0(self, device="cpu") -> torch.Tensor:
        """Initial parameters x_0 ~ N(0, 0.05^2); padding elements are 0."""
        gen = _gen(device, self.seed, self.key, 101)
        x = torch.empty(self.d, dtype=torch.float32, device=device)
        for o in range(0, self.d, _CHUNK):
            n = min(_CHUNK, self.d - o)
            x[o:o + n] = _randn(n, gen, device) * 0.05
        if self.segments is not None:
            _zero_padding(x, self.segments, self.d)
        return x

    def m0(self, device="cpu") -> torch.Tensor:
        """Initial momentum m_0 = 0 for every worker."""
        return torch.zeros(self.M, self.ld, dtype=torch.float32, device=device)

    def shared(self, device="cpu"):
        return None if self._shared is None else self._shared(self, device)

    def prefix(self, n: int) -> "Workload":
        """The same recipe on a vector of the first min(n, d) parameters: same seeds, same per-tensor
        layout (tensors beyond n dropped, the one that straddles n cut short).  For callers that want a
        bounded sample of a large workload without drawing all of it."""
        n = min(int(n), self.d)
        segs = None
        if self.segments is not None:
            segs = [(off, min(size, n - off)) for off, size in self.segments if off < n]
        return dataclasses.replace(self, d=n, segments=segs)

    def g(self, step: int, device="cpu", shared=None, out: Optional[torch.Tensor] = None) -> torch.Tensor:
        """Gradients of all M workers at `step`, shape [M, ld]."""
        if shared is None:
            shared = self.shared(device)
        if out is None:
            out = torch.zeros(self.M, self.ld, dtype=torch.float32, device=device)
        self._fill(self, out, step, device, shared)
        return out


def _zero_padding(v: torch.Tensor, segments, d: int) -> None:
    end = 0
    for off, size in segments:
        if off > end:
            v[..., end:off] = 0
        end = off + size
    if end < d:
        v[..., end:d] = 0


# --------------------------------------------------------------------------
# recipes


def _shared_mean(scale: float):
    def make(wl: Workload, device):
        gen = _gen(device, wl.seed, wl.key, 202)
        mu = torch.empty(wl.d, dtype=torch.float32, device=device)
        for o in range(0, wl.d, _CHUNK):
            n = min(_CHUNK, wl.d - o)
            mu[o:o + n] = _randn(n, gen, device) * scale
        return mu
    return make


def _fill_mean_plus_gauss(sigma: float):
    def fill(wl: Workload, out, step, device, mu):
        for w in range(wl.M):
            gen = _gen(device, wl.seed, wl.key, 303, step, w)
            for o in range(0, wl.d, _CHUNK):
                n = min(_CHUNK, wl.d - o)
                z = _randn(n, gen, device)
                out[w, o:o + n] = z * sigma if mu is None else mu[o:o + n] + z * sigma
    return fill


def _shared_layerwise(wl: Workload, device):
    """Per-tensor noise scale sigma ~ logU[1e-4, 1e-1]; mean ~ N(0, (0.2 sigma)^2)."""
    gen_cpu = _gen("cpu", wl.seed, wl.key, 404)
    u = torch.rand(len(wl.segments), generator=gen_cpu, dtype=torch.float64)
    sig = torch.exp(math.log(1e-4) + u * (math.log(1e-1) - math.log(1e-4))).to(torch.float32)
    sigma = torch.zeros(wl.d, dtype=torch.float32, device=device)
    for (off, size), s in zip(wl.segments, sig.tolist()):
        sigma[off:off + size] = s
    gen = _gen(device, wl.seed, wl.key, 202)
    mu = _randn(wl.d, gen, device) * (0.2 * sigma)
    return mu, sigma


def _fill_layerwise(wl: Workload, out, step, device, shared):
    mu, sigma = shared
    for w in range(wl.M):
        gen = _gen(device, wl.seed, wl.key, 303, step, w)
        out[w, :wl.d] = mu + sigma * _randn(wl.d, gen, device)
        _zero_padding(out[w, :wl.d], wl.segments, wl.d)       # exact +0.0 between tensors


def _fill_tie_zero(wl: Workload, out, step, device, shared):
    """Even-M stress: 30 % of elements split exactly M/2 : M/2, 2 % exact zeros elsewhere."""
    M, half = wl.M, wl.M // 2
    gen = _gen(device, wl.seed, wl.key, 505, step)
    for o in range(0, wl.d, _CHUNK // 4):
        n = min(_CHUNK // 4, wl.d - o)
        mag = torch.randn(M, n, generator=gen, device=device, dtype=torch.float32).abs()
        mag = torch.where(mag == 0, torch.ones_like(mag), mag)
        is_tie = torch.rand(n, generator=gen, device=device) < 0.30
        keys = torch.rand(M, n, generator=gen, device=device)
        rank = keys.argsort(dim=0).argsort(dim=0)
        s_tie = torch.where(rank < half, 1.0, -1.0)
        u = torch.rand(M, n, generator=gen, device=device)
        pm = torch.where(torch.rand(M, n, generator=gen, device=device) < 0.5, 1.0, -1.0)
        s_free = torch.where(u < 0.02, torch.zeros_like(pm), pm)
        s = torch.where(is_tie.unsqueeze(0), s_tie, s_free).to(torch.float32)
        out[:, o:o + n] = (s * mag).abs() * s  # keeps exact +0.0 (never -0.0) where s == 0


def _fill_student_t(scale: float, nu: int = 3):
    def fill(wl: Workload, out, step, device, mu):
        for w in range(wl.M):
            gen = _gen(device, wl.seed, wl.key, 303, step, w)
            for o in range(0, wl.d, _CHUNK):
                n = min(_CHUNK, wl.d - o)
                z0 = _randn(n, gen, device)
                chi = torch.zeros(n, dtype=torch.float32, device=device)
                for _ in range(nu):
                    chi += _randn(n, gen, device).square_()
                t = z0 / (chi / nu).sqrt_()
                out[w, o:o + n] = mu[o:o + n] + scale * t
    return fill


# --------------------------------------------------------------------------
# the named workloads


def small_signum(d: int = 1_000_000, M: int = 3) -> Workload:
    """Small case: shared mean N(0, 0.1^2) plus unit Gaussian noise, 5 Signum steps."""
    return Workload("small_signum_d1e6_M3", 1, d, M, 0.9, 1e-4, steps=5,
                    _fill=_fill_mean_plus_gauss(1.0), _shared=_shared_mean(0.1))


def resnet50_signum(M: int = 7) -> Workload:
    """Resnet-50-sized vector: 161 tensors end to end, each start 32-aligned."""
    sizes = resnet50_tensor_sizes()
    segs, off = [], 0
    for s in sizes:
        segs.append((off, s))
        off += round_up(s, 32)
    assert off == 25_557_056
    return Workload("resnet50_d25557056_M7", 2, off, M, 0.9, 1e-4, steps=1,
                    _fill=_fill_layerwise, _shared=_shared_layerwise, segments=segs)


def tie_zero_stress(d: int = 1 << 24, M: int = 8) -> Workload:
    """Even M with exact ties and exact zeros; signSGD (beta = 0), no momentum buffer."""
    return Workload("tie_zero_d2p24_M8", 3, d, M, 0.0, 1e-3, steps=1,
                    momentum_buffer=False, _fill=_fill_tie_zero)


def bert_large_signum(d: int = 335_141_888, M: int = 16) -> Workload:
    """BERT-large-sized vector with heavy-tailed (Student-t, nu = 3) noise."""
    return Workload("bertlarge_d335141888_M16", 4, d, M, 0.9, 1e-4, steps=1,
                    _fill=_fill_student_t(1e-3), _shared=_shared_mean(2e-4))


def sweep_point(d: int, M: int) -> Workload:
    """One point of the bandwidth sweep: i.i.d. unit Gaussian gradients."""
    return Workload("sweep_d%d_M%d" % (d, M), 5, d, M, 0.9, 1e-4, steps=1,
                    _fill=_fill_mean_plus_gauss(1.0))


SWEEP_D = [1 << k for k in range(10, 29)]
SWEEP_M = [1, 3, 7, 15, 31]
