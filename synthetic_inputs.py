"""Seeded synthetic inputs shared by the tests, the oracle legs and the benchmark.

This module only draws random numbers and lays them out; it contains none of the
method's arithmetic (no schedule, no weights, no update, no gradient).

All generators return fp32 ``torch`` tensors on the requested device.  On the CPU the
stream is torch's CPU generator, on a GPU it is torch's device generator; a test that
needs the same bytes on both sides generates once and copies.
"""
import torch


def _gen(seed, device):
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def padded_ld(d, multiple=32):
    """Smallest leading dimension >= d that keeps every row 128-byte aligned (32 floats)."""
    return (d + multiple - 1) // multiple * multiple


def empty_rows(n, d, device, ld=None):
    """An [n, d] fp32 view whose rows are ld >= d elements apart (ld = d when not given)."""
    ld = d if ld is None else ld
    return torch.empty((n, ld), dtype=torch.float32, device=device)[:, :d]


def _randn_rows(n, d, gen, device, mean=0.0, std=1.0, out=None, ld=None):
    """Row by row so that a 10 GB matrix never needs a second 10 GB temporary."""
    x = out if out is not None else empty_rows(n, d, device, ld)
    for i in range(n):
        x[i].normal_(mean=mean, std=std, generator=gen)
    return x


def consensus_inputs(n, d, seed=1, offset_rows=True, device="cpu"):
    """X[i, :] ~ N(0, 1) + i: the rows are offset by the agent index so that the average is
    far from zero and a relative consensus deviation means something."""
    gen = _gen(seed, device)
    x = _randn_rows(n, d, gen, device)
    if offset_rows:
        x += torch.arange(n, dtype=torch.float32, device=device).unsqueeze(1)
    return x


def step_inputs(n, d, seed=0, x_std=0.01, g_std=0.01, device="cpu", same_xy=True, ld=None):
    """Flat parameter vectors of a CNN's size: X0 iid N(0, x_std^2) per element, Y0 = X0
    (or an independent draw when ``same_xy`` is false), G iid N(0, g_std^2).  With ``ld`` the
    three matrices are [n, d] views of [n, ld] buffers (padded rows)."""
    gen = _gen(seed, device)
    x = _randn_rows(n, d, gen, device, std=x_std, ld=ld)
    if same_xy:
        y = empty_rows(n, d, device, ld)
        y.copy_(x)
    else:
        y = _randn_rows(n, d, gen, device, std=x_std, ld=ld)
    g = _randn_rows(n, d, gen, device, std=g_std, ld=ld)
    return x, y, g


def gradient_inputs(n, d, k, g_std=0.01, device="cpu", out=None):
    """The synthetic stochastic gradient of iteration k: iid N(0, g_std^2), seeded by k."""
    gen = _gen(1_000_003 + int(k), device)
    return _randn_rows(n, d, gen, device, std=g_std, out=out)


def logreg_problem(n, m, d, seed=0, flip=0.1, hetero_std=0.0, device="cpu"):
    """Per-agent binary classification data.

    x_star ~ N(0, 1)^d; agent i's features are N(mu_i, 1) with one shift vector
    mu_i ~ N(0, hetero_std^2)^d per agent (zero when hetero_std is 0); the label of a
    sample is the sign of <a, x_star>, flipped with probability ``flip``.
    Returns (A [n, m, d], labels [n, m] in {-1, +1}, x_star [d]).
    """
    gen = _gen(seed, device)
    x_star = torch.empty(d, dtype=torch.float32, device=device).normal_(generator=gen)
    a = torch.empty((n, m, d), dtype=torch.float32, device=device)
    labels = torch.empty((n, m), dtype=torch.float32, device=device)
    for i in range(n):
        a[i].normal_(generator=gen)
        if hetero_std > 0:
            mu = torch.empty(d, dtype=torch.float32, device=device).normal_(std=hetero_std, generator=gen)
            a[i] += mu
        clean = torch.where(a[i] @ x_star >= 0, 1.0, -1.0)
        flips = torch.rand(m, generator=gen, device=device) < flip
        labels[i] = torch.where(flips, -clean, clean)
    return a, labels, x_star


def lsq_problem(n, m, d, seed=0, sigma_s=0.1, device="cpu"):
    """Distributed least squares: A_i ~ N(0, I) (m x d per agent), x_star ~ N(0, 1)^d,
    b_i = A_i x_star + v_i with v_i ~ N(0, sigma_s^2 I).  Returns (A [n, m, d], B [n, m], x_star [d])."""
    gen = _gen(seed, device)
    x_star = torch.empty(d, dtype=torch.float32, device=device).normal_(generator=gen)
    a = torch.empty((n, m, d), dtype=torch.float32, device=device).normal_(generator=gen)
    v = torch.empty((n, m), dtype=torch.float32, device=device).normal_(std=sigma_s, generator=gen)
    b = torch.einsum("nmd,d->nm", a, x_star) + v
    return a, b, x_star


def gradient_noise(n, d, k, sigma_n, seed=0, device="cpu"):
    """The additive gradient noise eps_i ~ N(0, sigma_n^2 I) of iteration k (one draw per agent)."""
    gen = _gen(7_000_003 * (int(seed) + 1) + int(k), device)
    return torch.empty((n, d), dtype=torch.float32, device=device).normal_(std=sigma_n, generator=gen)
