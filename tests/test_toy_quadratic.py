"""The toy problem of the paper's supplementary figure "A simple toy problem where signSGD converges
faster than SGD": f(x) = 1/2 |x|^2 on R^100, Gaussian noise N(0, 100^2) on the first gradient component
only, x_0 ~ N(0, I), constant learning rates 0.01 (signSGD) and 0.001 (SGD), 50 repeats.

The figure gives no numbers, so the check is qualitative: the mean objective under signSGD (Algorithm 1,
i.e. the step with M = 1 and beta = 0) falls well below SGD's.  The 50 repeats are laid side by side in
one vector of 50 x 100 parameters (the update is elementwise, so the repeats do not interact).  SGD is the
comparison system and is written inline with plain array arithmetic.
"""
import numpy as np
import pytest

R, D, K = 50, 100, 300
LR_SIGN, LR_SGD = 0.01, 0.001


def noise(r):
    n = np.zeros((R, D), dtype=np.float32)
    n[:, 0] = (100.0 * r.standard_normal(R)).astype(np.float32)
    return n


def objective(x):
    return 0.5 * (x.reshape(R, D).astype(np.float64) ** 2).sum(axis=1)


def run(step_fn):
    """step_fn(x_flat, g_flat) applies one signSGD step in place; returns (f_sign, f_sgd, x_sign)."""
    r = np.random.default_rng(1802)
    x0 = r.standard_normal((R, D)).astype(np.float32)
    xs, xg = x0.copy().reshape(-1), x0.copy()
    for _ in range(K):
        g = (xs.reshape(R, D) + noise(r)).reshape(-1)
        xs = step_fn(xs, g)
        xg = xg - np.float32(LR_SGD) * (xg + noise(r))
    return objective(xs), objective(xg), xs


def test_signsgd_beats_sgd_on_sparse_noise_oracle():
    import oracle

    def step(x, g):
        oracle.signsgd_step(x, g, None, 1, R * D, 0.0, LR_SIGN)
        return x

    f_sign, f_sgd, _ = run(step)
    assert f_sign.mean() < 0.1 * f_sgd.mean()
    assert f_sign.mean() + f_sign.std() < f_sgd.mean() - f_sgd.std()
    assert f_sign.mean() < 0.05 * objective(np.random.default_rng(1802).standard_normal((R, D))).mean()


@pytest.mark.gpu
def test_signsgd_beats_sgd_on_sparse_noise_gpu():
    import torch
    import oracle
    from paper_1802_04434_b200 import binding as B

    d = R * D
    W = (d + 31) // 32
    ldw = (W + 3) // 4 * 4
    bits = torch.zeros(ldw, dtype=torch.int32, device="cuda:0")
    vote = torch.zeros(W, dtype=torch.int32, device="cuda:0")

    def step(x, g):
        xd, gd = torch.from_numpy(x).to("cuda:0"), torch.from_numpy(g).to("cuda:0")
        B.signsgd_step(xd, gd, None, 1, d, d, 0.0, LR_SIGN, bits, ldw, vote)
        return xd.cpu().numpy()

    f_sign, f_sgd, x_gpu = run(step)
    assert f_sign.mean() < 0.1 * f_sgd.mean()

    def ostep(x, g):
        oracle.signsgd_step(x, g, None, 1, d, 0.0, LR_SIGN)
        return x

    _, _, x_cpu = run(ostep)
    assert np.array_equal(x_gpu.view(np.uint32), x_cpu.view(np.uint32))   # same trajectory, bit for bit
