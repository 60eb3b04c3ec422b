"""The seeded input recipes: sizes, layout, determinism and the structure each
configuration promises (ties, zeros, per-tensor padding)."""
import numpy as np
import torch

from paper_1802_04434_b200 import workloads as wl


def test_resnet50_layout():
    sizes = wl.resnet50_tensor_sizes()
    assert len(sizes) == 161 and sum(sizes) == 25_557_032
    assert min(sizes) == 64 and max(sizes) == 2_359_296
    cfg = wl.resnet50_signum()
    assert cfg.d == 25_557_056 and cfg.M == 7
    assert all(off % 32 == 0 for off, _ in cfg.segments)
    assert sum(wl.round_up(s, 32) - s for s in sizes) == 24


def test_small_workload_is_deterministic_and_fresh_per_step():
    cfg = wl.small_signum(d=10_000)
    g0a, g0b, g1 = cfg.g(0), cfg.g(0), cfg.g(1)
    assert g0a.shape == (3, cfg.ld) and g0a.dtype == torch.float32
    assert torch.equal(g0a, g0b) and not torch.equal(g0a, g1)
    assert not torch.equal(g0a[0], g0a[1])
    x0 = cfg.x0()
    assert abs(float(x0.std()) - 0.05) < 0.005
    assert float(cfg.m0().abs().max()) == 0.0
    mu = cfg.shared()
    assert abs(float(mu.std()) - 0.1) < 0.01
    assert abs(float((g0a[0, :cfg.d] - mu).std()) - 1.0) < 0.05


def test_tie_zero_structure():
    cfg = wl.tie_zero_stress(d=1 << 16)
    g = cfg.g(0)[:, :cfg.d].numpy()
    pos = (g > 0).sum(axis=0)
    neg = (g < 0).sum(axis=0)
    zero = (g == 0)
    tie = (pos == 4) & (neg == 4)
    assert 0.30 <= tie.mean() <= 0.30 + 0.7 * 0.30   # planted ties plus chance ties
    assert abs(zero.mean() - 0.7 * 0.02) < 0.003
    assert not np.signbit(g[zero]).any()              # zeros are +0.0
    assert cfg.beta == 0.0 and not cfg.momentum_buffer


def test_padding_elements_are_zero():
    cfg = wl.small_signum(d=1001)
    assert cfg.ld == 1004
    g = cfg.g(0)
    assert float(g[:, 1001:].abs().max()) == 0.0


def test_student_t_is_heavy_tailed():
    cfg = wl.bert_large_signum(d=200_000, M=2)
    g = cfg.g(0)[:, :cfg.d] / 1e-3
    k = float(((g - g.mean()) ** 4).mean() / g.var() ** 2)
    assert k > 6.0        # Gaussian kurtosis is 3
