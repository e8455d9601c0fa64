"""GPU parity: the CUDA library against the fp64 oracle, element by element, on the same seeded
fp32 inputs.  Every call goes through the C ABI (via the ctypes binding).

Tolerances (fp32 arithmetic against fp64):
  * one step / one round: max|delta| <= 2e-6 * scale, scale = max(|X|, |Y|, |gamma| |G|) of the inputs
    (the stated 2e-6 * max|X| bound, with the other operands included so that X0 = 0 is testable);
  * r rounds: r times that;
  * after tau aligned rounds the consensus deviation ||X - 1 xbar^T||_F / ||X||_F <= 1e-5;
  * logistic gradient: 8 sqrt(d) 2^-24 max|G| + 1e-7 (a length-d fp32 dot product feeding a
    1/4-Lipschitz sigmoid, then a length-m fp32 sum).
Schedules and peer indices are compared bit for bit in the CPU tests.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2306_00256_b200 as ceca
import synthetic_inputs as synth

pytestmark = pytest.mark.gpu

DEV = "cuda:0"
STEP_TOL = 2e-6


def _np(t):
    return t.detach().cpu().numpy()


def _scale(gamma, *tensors):
    vals = []
    for t, w in tensors:
        if t is not None:
            vals.append(float(t.abs().max()) * w)
    return max(vals + [1e-30])


def _padded(n, d, ld, offset=0):
    """A [n, d] view with row stride ld, starting `offset` floats into a fresh buffer."""
    buf = torch.full((n * ld + offset + 8,), float("nan"), dtype=torch.float32, device=DEV)
    return buf[offset:offset + n * ld].view(n, ld)[:, :d], buf


def _put(src, ld=None, offset=0):
    n, d = src.shape
    view, buf = _padded(n, d, ld or d, offset)
    view.copy_(src)
    return view, buf


def _variants(n):
    return [ceca.CECA_2P] if (n % 2 and n > 1) else [ceca.CECA_2P, ceca.CECA_1P]


def _tau(n):
    return max(oracle.round_info(n, 0).tau, 1)


# --------------------------------------------------------------------------------------------
# fused SGD step + gossip round
# --------------------------------------------------------------------------------------------

@pytest.mark.parametrize("n", [1, 2, 3, 5, 6, 24, 63, 64, 97, 100])
@pytest.mark.parametrize("d", [1, 3, 4, 5, 1023, 4100, 70001])
def test_step_matches_oracle_every_round(n, d):
    x, y, g = synth.step_inputs(n, d, seed=n * 1000 + d, x_std=1.0, g_std=1.0, same_xy=False)
    gamma = 0.1
    for variant in _variants(n):
        for k in list(range(_tau(n))) + [2**40 + 1]:
            X, Y, G = x.to(DEV), y.to(DEV), g.to(DEV)
            Xo, Yo = torch.empty_like(X), torch.empty_like(Y)
            ceca.ceca_gossip_sgd_step(X, Y, G, gamma, variant, k, X_out=Xo, Y_out=Yo)
            want_x, want_y = oracle.step(_np(x), _np(y), _np(g), np.float32(gamma), variant, k)
            tol = STEP_TOL * _scale(gamma, (x, 1), (y, 1), (g, gamma))
            assert np.abs(_np(Xo) - want_x).max() <= tol, (n, d, variant, k)
            assert np.abs(_np(Yo) - want_y).max() <= tol, (n, d, variant, k)
            # inputs untouched by the out-of-place call
            assert torch.equal(X.cpu(), x) and torch.equal(Y.cpu(), y) and torch.equal(G.cpu(), g)
            # in place gives the same bits
            ceca.ceca_gossip_sgd_step(X, Y, G, gamma, variant, k)
            assert torch.equal(X, Xo) and torch.equal(Y, Yo)


def test_step_every_n_from_2_to_130():
    """Every agent count of the n sweep (and the paper's n = 130), every round, both variants."""
    d, gamma = 260, 0.1
    for n in list(range(2, 131)):
        x, y, g = synth.step_inputs(n, d, seed=n, x_std=1.0, g_std=1.0, same_xy=False)
        X0, Y0, G = x.to(DEV), y.to(DEV), g.to(DEV)
        xn, yn, gn = _np(x), _np(y), _np(g)
        tol = STEP_TOL * _scale(gamma, (x, 1), (y, 1), (g, gamma))
        for variant in _variants(n):
            for k in range(_tau(n)):
                Xo, Yo = torch.empty_like(X0), torch.empty_like(Y0)
                ceca.ceca_gossip_sgd_step(X0, Y0, G, gamma, variant, k, X_out=Xo, Y_out=Yo)
                want_x, want_y = oracle.step(xn, yn, gn, np.float32(gamma), variant, k)
                assert np.abs(_np(Xo) - want_x).max() <= tol, (n, variant, k)
                assert np.abs(_np(Yo) - want_y).max() <= tol, (n, variant, k)


@pytest.mark.parametrize("n,variant", [(130, ceca.CECA_1P), (130, ceca.CECA_2P), (1026, ceca.CECA_1P), (1026, ceca.CECA_2P)])
def test_consensus_at_the_papers_network_sizes(n, variant):
    """n = 130 and n = 1026 (Sec. 5, "close to a power of two"): per-round kernel, tau rounds, random x and y;
    the residue sum_i ||x_i - mean|| drops to rounding level exactly at round tau, not before."""
    d = 515
    x = synth.consensus_inputs(n, d, seed=n, offset_rows=False)
    y = synth.consensus_inputs(n, d, seed=n + 1, offset_rows=False)
    tau = _tau(n)
    mean = x.double().mean(0)
    X, Y = x.to(DEV), y.to(DEV)
    for k in range(tau):
        ceca.ceca_consensus_rounds(X, Y, variant, k, 1, 0)
        residue = float((X.double().cpu() - mean).norm(dim=1).sum())
        if k < tau - 1:
            assert residue > 1e-2 * n
        else:
            assert residue < 1e-4 * n
    want_x, want_y = oracle.consensus(_np(x), _np(y), variant, 0, tau)
    tol = STEP_TOL * tau * _scale(0, (x, 1), (y, 1))
    assert np.abs(_np(X) - want_x).max() <= tol and np.abs(_np(Y) - want_y).max() <= tol


def test_step_with_more_cycles_than_one_grid_dimension_holds():
    """140,000 agents: the 1-port matching has 70,000 cycles (more than 65,535 grid rows), and the
    2-port shift n/2 as well."""
    n, d, gamma = 140_000, 5, 0.1
    x, y, g = synth.step_inputs(n, d, seed=1, x_std=1.0, g_std=1.0, same_xy=False)
    tau = _tau(n)
    tol = STEP_TOL * _scale(gamma, (x, 1), (y, 1), (g, gamma))
    for variant, k in [(ceca.CECA_1P, 0), (ceca.CECA_1P, tau - 1), (ceca.CECA_2P, 1), (ceca.CECA_2P, tau - 1)]:
        X, Y, G = x.to(DEV), y.to(DEV), g.to(DEV)
        ceca.ceca_gossip_sgd_step(X, Y, G, gamma, variant, k)
        want_x, want_y = oracle.step(_np(x), _np(y), _np(g), np.float32(gamma), variant, k)
        assert np.abs(_np(X) - want_x).max() <= tol and np.abs(_np(Y) - want_y).max() <= tol, (variant, k)


@pytest.mark.parametrize("n,d,ld,offset", [(6, 37, 40, 0), (6, 37, 41, 0), (24, 1000, 1024, 4), (24, 1000, 1024, 1),
                                           (24, 1000, 1024, 2), (24, 1003, 1024, 3), (5, 2, 8, 3), (5, 3, 8, 1), (5, 7, 8, 2),
                                           (97, 513, 517, 3), (100, 4096, 4100, 0)])
def test_step_padded_rows_and_unaligned_bases(n, d, ld, offset):
    x, y, g = synth.step_inputs(n, d, seed=7, x_std=1.0, g_std=0.5, same_xy=False)
    gamma = 0.25
    for variant in _variants(n):
        for k in range(_tau(n)):
            (X, xb), (Y, yb), (G, gb) = _put(x.to(DEV), ld, offset), _put(y.to(DEV), ld, offset), _put(g.to(DEV), ld, offset)
            (Xo, xob), (Yo, yob) = _padded(n, d, ld, offset), _padded(n, d, ld, offset)
            ceca.ceca_gossip_sgd_step(X, Y, G, gamma, variant, k, X_out=Xo, Y_out=Yo)
            want_x, want_y = oracle.step(_np(x), _np(y), _np(g), np.float32(gamma), variant, k)
            tol = STEP_TOL * _scale(gamma, (x, 1), (y, 1), (g, gamma))
            assert np.abs(_np(Xo) - want_x).max() <= tol
            assert np.abs(_np(Yo) - want_y).max() <= tol
            # the padding between rows (and around the buffer) is never written
            if ld > d:
                assert torch.isnan(xob[offset:offset + n * ld].view(n, ld)[:, d:]).all()
                assert torch.isnan(yob[offset:offset + n * ld].view(n, ld)[:, d:]).all()
            assert torch.isnan(xob[:offset]).all() and torch.isnan(xob[offset + n * ld:]).all()


def test_step_with_differently_misaligned_arrays():
    """X, Y, G and the outputs each start a different number of elements off a 16-byte boundary: no common
    scalar head exists, every column runs the scalar form, and the result is the same."""
    n, d, ld, gamma = 24, 1000, 1024, 0.25
    x, y, g = synth.step_inputs(n, d, seed=11, x_std=1.0, g_std=0.5, same_xy=False)
    for variant in _variants(n):
        for k in range(_tau(n)):
            (X, _), (Y, _), (G, _) = _put(x.to(DEV), ld, 1), _put(y.to(DEV), ld, 2), _put(g.to(DEV), ld, 3)
            (Xo, xob), (Yo, yob) = _padded(n, d, ld, 0), _padded(n, d, ld, 5)
            ceca.ceca_gossip_sgd_step(X, Y, G, gamma, variant, k, X_out=Xo, Y_out=Yo)
            want_x, want_y = oracle.step(_np(x), _np(y), _np(g), np.float32(gamma), variant, k)
            tol = STEP_TOL * _scale(gamma, (x, 1), (y, 1), (g, gamma))
            assert np.abs(_np(Xo) - want_x).max() <= tol
            assert np.abs(_np(Yo) - want_y).max() <= tol
            assert torch.isnan(yob[:5]).all() and torch.isnan(yob[5 + n * ld:]).all()
            assert torch.isnan(xob[n * ld:]).all()


def test_step_without_gradient_is_a_ceca_round_and_y_may_be_absent_in_round_zero():
    n, d = 24, 2051
    x, y, _ = synth.step_inputs(n, d, seed=3, x_std=1.0, same_xy=False)
    for variant in _variants(n):
        for k in range(_tau(n)):
            X, Y = x.to(DEV), y.to(DEV)
            Xo, Yo = torch.empty_like(X), torch.empty_like(Y)
            ceca.ceca_gossip_sgd_step(X, Y, None, 0.3, variant, k, X_out=Xo, Y_out=Yo)
            want_x, want_y = oracle.step(_np(x), _np(y), None, 0.0, variant, k)
            tol = STEP_TOL * _scale(0, (x, 1), (y, 1))
            assert np.abs(_np(Xo) - want_x).max() <= tol and np.abs(_np(Yo) - want_y).max() <= tol
        Xo2, Yo2 = torch.empty_like(X), torch.empty_like(Y)
        ceca.ceca_gossip_sgd_step(x.to(DEV), None, None, 0.0, variant, 0, X_out=Xo2, Y_out=Yo2)
        want_x, want_y = oracle.step(_np(x), np.zeros_like(_np(x)), None, 0.0, variant, 0)
        assert np.abs(_np(Xo2) - want_x).max() <= tol and np.abs(_np(Yo2) - want_y).max() <= tol
        with pytest.raises(ceca.CecaError):
            ceca.ceca_gossip_sgd_step(x.to(DEV), None, None, 0.0, variant, 1, X_out=Xo2, Y_out=Yo2)


@pytest.mark.parametrize("n", [1, 2, 4, 8, 64, 128])
@pytest.mark.parametrize("d", [5, 1023, 40004])
def test_x_only_step_for_power_of_two_agents(n, d):
    """n = 2^tau: every delta_r is 1, X never depends on Y, and the call without Y must give the oracle's X."""
    x, y, g = synth.step_inputs(n, d, seed=n + d, x_std=1.0, g_std=1.0, same_xy=False)
    gamma = 0.1
    tol = STEP_TOL * _scale(gamma, (x, 1), (g, gamma))
    for variant in _variants(n):
        for k in range(_tau(n) + 1):
            X, G = x.to(DEV), g.to(DEV)
            Xo = torch.full_like(X, float("nan"))
            ceca.ceca_gossip_sgd_step(X, None, G, gamma, variant, k, X_out=Xo)
            want_x, _ = oracle.step(_np(x), _np(y), _np(g), np.float32(gamma), variant, k)
            assert np.abs(_np(Xo) - want_x).max() <= tol, (n, d, variant, k)
            # the same bits as the full update's X, and in place
            Xf, Yf = torch.empty_like(X), torch.empty_like(X)
            ceca.ceca_gossip_sgd_step(X, y.to(DEV), G, gamma, variant, k, X_out=Xf, Y_out=Yf)
            assert torch.equal(Xo, Xf)
            ceca.ceca_gossip_sgd_step(X, None, G, gamma, variant, k)
            assert torch.equal(X, Xo)
    if n > 2:   # any other n needs Y
        bad = torch.zeros(n - 1, d, device=DEV)
        with pytest.raises(ceca.CecaError):
            ceca.ceca_gossip_sgd_step(bad, None, None, gamma, ceca.CECA_2P, 0, X_out=torch.empty_like(bad))


@pytest.mark.parametrize("n,variant", [(2, ceca.CECA_2P), (5, ceca.CECA_2P), (6, ceca.CECA_1P), (24, ceca.CECA_1P),
                                       (97, ceca.CECA_2P), (100, ceca.CECA_2P)])
def test_dead_y_may_be_dropped_in_the_last_round_of_a_cycle(n, variant):
    """Round tau-1 without storing y+, then round 0: the same X and Y bits as the full updates, because
    round 0 has b = 0 and builds its message from x."""
    d, gamma = 1029, 0.1
    tau = _tau(n)
    x, y, g = synth.step_inputs(n, d, seed=n, x_std=1.0, g_std=1.0, same_xy=False)
    g2 = synth.gradient_inputs(n, d, 1, g_std=1.0)
    k = 3 * tau + tau - 1
    Xf, Yf = x.to(DEV), y.to(DEV)                        # full path
    ceca.ceca_gossip_sgd_step(Xf, Yf, g.to(DEV), gamma, variant, k)
    Xl, Yl = x.to(DEV), y.to(DEV)                        # y+ dropped
    ceca.ceca_gossip_sgd_step(Xl, Yl, g.to(DEV), gamma, variant, k, drop_y=True)
    assert torch.equal(Xl, Xf) and torch.equal(Yl.cpu(), y)   # X as in the full update, Y untouched
    want_x, _ = oracle.step(_np(x), _np(y), _np(g), np.float32(gamma), variant, k)
    assert np.abs(_np(Xl) - want_x).max() <= STEP_TOL * _scale(gamma, (x, 1), (y, 1), (g, gamma))
    ceca.ceca_gossip_sgd_step(Xf, Yf, g2.to(DEV), gamma, variant, k + 1)
    ceca.ceca_gossip_sgd_step(Xl, Yl, g2.to(DEV), gamma, variant, k + 1)
    assert torch.equal(Xl, Xf) and torch.equal(Yl, Yf)
    if tau > 1:
        with pytest.raises(ceca.CecaError):
            ceca.ceca_gossip_sgd_step(Xl, Yl, g.to(DEV), gamma, variant, k + 1, drop_y=True)


@pytest.mark.parametrize("n,variant", [(5, ceca.CECA_2P), (6, ceca.CECA_1P), (63, ceca.CECA_2P), (64, ceca.CECA_1P)])
def test_mean_lemma_and_resume_on_gpu(n, variant):
    """Lemma "relation between averaged variables": with x0 = y0 the mean takes a plain SGD step.
    Also: stopping and restarting from (X, Y, k) gives the same bits as running straight through."""
    d = 3001
    x, y, _ = synth.step_inputs(n, d, seed=11, x_std=1.0)
    X, Y = x.to(DEV), y.to(DEV)
    gamma = 0.05
    tau = _tau(n)
    snap = None
    for k in range(2 * tau + 3):
        G = synth.gradient_inputs(n, d, k, g_std=1.0, device=DEV)
        mean_before = X.double().mean(0)
        ceca.ceca_gossip_sgd_step(X, Y, G, gamma, variant, k)
        want = mean_before - gamma * G.double().mean(0)
        assert (X.double().mean(0) - want).abs().max() <= 5e-6
        assert (Y.double().mean(0) - want).abs().max() <= 5e-6
        if k == tau:
            snap = (X.clone(), Y.clone())
    X2, Y2 = snap
    for k in range(tau + 1, 2 * tau + 3):
        G = synth.gradient_inputs(n, d, k, g_std=1.0, device=DEV)
        ceca.ceca_gossip_sgd_step(X2, Y2, G, gamma, variant, k)
    assert torch.equal(X, X2) and torch.equal(Y, Y2)


# --------------------------------------------------------------------------------------------
# consensus rounds: one launch per round, and the fused TMA kernel
# --------------------------------------------------------------------------------------------

BLOCK_MAX_N = 1152   # largest n the register-block kernel takes (16-column tiles of all rows on one SM)
BLOCK_MAX_N_1P = 416  # ... with the 1-port pairing (sixteen blocks of 26 agents)


def _fused_ws():
    return torch.zeros(64, dtype=torch.int32, device=DEV)


def _fused_kernels(n, variant=ceca.CECA_2P):
    """The fused kernels that take n agents and this variant: shared-memory exchange (n <= 2048),
    tensor-memory exchange (n <= 128), register blocks (CECA-2P: n <= 1152; CECA-1P: n <= 416)."""
    kernels = [ceca.FUSED_SMEM]
    if n <= 128:
        kernels.append(ceca.FUSED_TMEM)
    if n <= (BLOCK_MAX_N if variant == ceca.CECA_2P else BLOCK_MAX_N_1P):
        kernels.append(ceca.FUSED_BLOCK)
    return kernels


@pytest.mark.parametrize("fused", [ceca.UNFUSED, ceca.FUSED_SMEM, ceca.FUSED_TMEM, ceca.FUSED_BLOCK])
@pytest.mark.parametrize("n", [2, 3, 4, 5, 6, 7, 8, 9, 16, 17, 24, 31, 33, 63, 65, 97, 100, 127, 128, 129, 130, 150, 151, 161, 200, 201, 208, 209, 255, 256])
@pytest.mark.parametrize("d", [32, 1000, 4100])
def test_consensus_matches_oracle_and_reaches_the_mean(fused, n, d):
    if fused == ceca.FUSED_TMEM and n > 128:
        with pytest.raises(ceca.CecaError):   # outside that kernel's range: refused, nothing launched
            ceca.ceca_consensus_rounds(torch.zeros(n, d, device=DEV), None, ceca.CECA_2P, 0, 1, fused, workspace=_fused_ws(),
                                       want_y=False)
        return
    x = synth.consensus_inputs(n, d, seed=n + d)
    y0 = synth.consensus_inputs(n, d, seed=n + d + 1, offset_rows=False)
    tau = _tau(n)
    for variant in _variants(n):
        if fused == ceca.FUSED_BLOCK and fused not in _fused_kernels(n, variant):
            continue
        for k0, rounds in [(0, tau), (0, tau + 1), (0, 1), (1 % tau, 2 * tau + 3), (5 * tau, tau)]:
            X, Y = x.to(DEV), y0.to(DEV)
            Xo, Yo = torch.empty_like(X), torch.empty_like(Y)
            ws = _fused_ws()
            ceca.ceca_consensus_rounds(X, Y, variant, k0, rounds, fused, X_out=Xo, Y_out=Yo, workspace=ws)
            assert ceca.ceca_read_status(ws) == 0
            want_x, want_y = oracle.consensus(_np(x), _np(y0), variant, k0, rounds)
            tol = STEP_TOL * rounds * _scale(0, (x, 1), (y0, 1))
            assert np.abs(_np(Xo) - want_x).max() <= tol, (n, d, variant, k0, rounds)
            assert np.abs(_np(Yo) - want_y).max() <= tol, (n, d, variant, k0, rounds)
            assert torch.equal(X.cpu(), x) and torch.equal(Y.cpu(), y0)
            if k0 % tau == 0 and rounds >= tau:
                xd = Xo.double()
                mean = x.double().mean(0).to(DEV)
                dev = (xd - mean).norm() / xd.norm()
                assert float(dev) <= 1e-5
                if rounds == tau:  # Y holds the mean of the other agents
                    loo = (x.double().sum(0, keepdim=True) - x.double()) / (n - 1)
                    assert (Yo.double().cpu() - loo).abs().max() <= tol
            # in place gives the same bits
            ceca.ceca_consensus_rounds(X, Y, variant, k0, rounds, fused, workspace=ws)
            assert torch.equal(X, Xo) and torch.equal(Y, Yo)


@pytest.mark.parametrize("fused", [ceca.FUSED_AUTO, ceca.FUSED_SMEM, ceca.FUSED_BLOCK])
@pytest.mark.parametrize("n", [257, 258, 300, 367, 368, 369, 400, 401, 512, 513, 600, 800, 801, 1026, 1089, 1151, 1152, 1153, 1300, 2047, 2048])
@pytest.mark.parametrize("d", [8, 1000, 4100])
def test_fused_consensus_above_256_agents(fused, n, d):
    """Tiles taller than one TMA box (32-, 16- or 8-column tiles made of several boxes): tau rounds, extra rounds,
    unaligned starts; every fused kernel that takes this n, and the one the library picks by itself."""
    x = synth.consensus_inputs(n, d, seed=n + d)
    y0 = synth.consensus_inputs(n, d, seed=n + d + 1, offset_rows=False)
    tau = _tau(n)
    for variant in _variants(n):
        if fused == ceca.FUSED_BLOCK and fused not in _fused_kernels(n, variant):
            with pytest.raises(ceca.CecaError):   # outside that kernel's range: refused, nothing launched
                ceca.ceca_consensus_rounds(x.to(DEV), None, variant, 0, 1, fused, workspace=_fused_ws(), want_y=False)
            continue
        for k0, rounds in [(0, tau), (3, tau + 2), (tau, 1), (tau - 1, 2)]:
            X, Y = x.to(DEV), y0.to(DEV)
            Xo, Yo = torch.full_like(X, float("nan")), torch.full_like(Y, float("nan"))
            ws = _fused_ws()
            ceca.ceca_consensus_rounds(X, Y, variant, k0, rounds, fused, X_out=Xo, Y_out=Yo, workspace=ws)
            assert ceca.ceca_read_status(ws) == 0
            want_x, want_y = oracle.consensus(_np(x), _np(y0), variant, k0, rounds)
            tol = STEP_TOL * rounds * _scale(0, (x, 1), (y0, 1))
            assert np.abs(_np(Xo) - want_x).max() <= tol, (n, d, variant, k0, rounds)
            assert np.abs(_np(Yo) - want_y).max() <= tol, (n, d, variant, k0, rounds)
            if k0 == 0:
                xd = Xo.double()
                assert float((xd - x.double().mean(0).to(DEV)).norm() / xd.norm()) <= 1e-5
            ceca.ceca_consensus_rounds(X, Y, variant, k0, rounds, fused, workspace=ws)   # in place: same bits
            assert torch.equal(X, Xo) and torch.equal(Y, Yo)


@pytest.mark.parametrize("n", [2, 8, 64, 128])
def test_per_round_consensus_without_y_for_power_of_two_agents(n):
    """n = 2^tau and Y not wanted: no Y, no workspace, and the X of the full computation."""
    d = 1003
    x = synth.consensus_inputs(n, d, seed=n)
    y = synth.consensus_inputs(n, d, seed=n + 1, offset_rows=False)
    tau = _tau(n)
    for variant in _variants(n):
        for k0, rounds in [(0, tau), (2, tau + 3)]:
            Xo = torch.full((n, d), float("nan"), device=DEV)
            ceca.ceca_consensus_rounds(x.to(DEV), None, variant, k0, rounds, 0, X_out=Xo, want_y=False)
            want_x, _ = oracle.consensus(_np(x), _np(y), variant, k0, rounds)
            assert np.abs(_np(Xo) - want_x).max() <= STEP_TOL * rounds * float(x.abs().max()), (n, variant, k0)


def test_finite_time_consensus_for_every_network_size():
    """Sec. 5 "Finite-time exact consensus": for every n the residue sum_i ||x_i - mean|| is still large after
    tau - 1 rounds and at rounding level after tau = ceil(log2 n) rounds (fused kernel, random x and y)."""
    d = 96
    for n in range(2, 141):
        x = synth.consensus_inputs(n, d, seed=n, offset_rows=False)
        y = synth.consensus_inputs(n, d, seed=n + 7, offset_rows=False)
        mean = x.double().mean(0)
        tau = _tau(n)
        assert tau == int(np.ceil(np.log2(n)))
        for variant in _variants(n):
            ws = _fused_ws()
            for fused in _fused_kernels(n, variant):
                for rounds, reached in ((tau - 1, False), (tau, True)):
                    if rounds == 0:
                        continue
                    Xo, Yo = torch.empty(n, d, device=DEV), torch.empty(n, d, device=DEV)
                    ceca.ceca_consensus_rounds(x.to(DEV), y.to(DEV), variant, 0, rounds, fused, X_out=Xo, Y_out=Yo, workspace=ws)
                    residue = float((Xo.double().cpu() - mean).norm(dim=1).sum()) / n
                    assert (residue < 1e-5) == reached, (n, variant, fused, rounds, residue)
            assert ceca.ceca_read_status(ws) == 0


@pytest.mark.parametrize("fused", [0, 1, 2, 3, 4])
def test_consensus_optional_y(fused):
    n, d = 97, 1000
    x = synth.consensus_inputs(n, d, seed=5)
    tau = _tau(n)
    X = x.to(DEV)
    want_x, want_y = oracle.consensus(_np(x), np.zeros((n, d)), ceca.CECA_2P, 0, tau)
    tol = STEP_TOL * tau * float(x.abs().max())
    # no Y in (round 0 ignores it), Y out wanted
    Xo, Yo = torch.empty_like(X), torch.empty_like(X)
    ws = _fused_ws()
    ceca.ceca_consensus_rounds(X, None, ceca.CECA_2P, 0, tau, fused, X_out=Xo, Y_out=Yo, workspace=ws)
    assert np.abs(_np(Xo) - want_x).max() <= tol and np.abs(_np(Yo) - want_y).max() <= tol
    # no Y at all: fused needs only its status word, unfused keeps Y in the workspace
    Xo2 = torch.empty_like(X)
    if fused:
        ws2 = _fused_ws()
    else:
        ws2 = torch.empty(ceca.ceca_workspace_bytes(ceca.WS_CONSENSUS_UNFUSED, n, 0, d) // 4, dtype=torch.float32, device=DEV)
    ceca.ceca_consensus_rounds(X, None, ceca.CECA_2P, 0, tau, fused, X_out=Xo2, workspace=ws2, want_y=False)
    assert torch.equal(Xo2, Xo)
    # zero rounds and a single agent are copies
    Xc, Yc = torch.empty_like(X), torch.empty_like(X)
    ceca.ceca_consensus_rounds(X, X.clone(), ceca.CECA_2P, 3, 0, fused, X_out=Xc, Y_out=Yc, workspace=ws)
    assert torch.equal(Xc, X) and torch.equal(Yc, X)
    one = x[:1].to(DEV).contiguous()
    oc, yc = torch.empty_like(one), torch.empty_like(one)
    ceca.ceca_consensus_rounds(one, one.clone(), ceca.CECA_2P, 0, 4, fused, X_out=oc, Y_out=yc, workspace=ws)
    assert torch.equal(oc, one)


@pytest.mark.parametrize("fused", [ceca.FUSED_SMEM, ceca.FUSED_TMEM, ceca.FUSED_BLOCK])
def test_fused_consensus_many_rounds(fused):
    """More rounds than one launch takes: chunks of 64, continuing in place (the tensor-memory kernel
    also folds its running scales back every 16 rounds)."""
    n, d, rounds, k0 = 12, 200, 150, 5
    x = synth.consensus_inputs(n, d, seed=3)
    y = synth.consensus_inputs(n, d, seed=4, offset_rows=False)
    for variant in (ceca.CECA_2P, ceca.CECA_1P):
        if fused == ceca.FUSED_BLOCK and fused not in _fused_kernels(n, variant):
            continue
        Xo, Yo = torch.empty(n, d, device=DEV), torch.empty(n, d, device=DEV)
        ws = _fused_ws()
        ceca.ceca_consensus_rounds(x.to(DEV), y.to(DEV), variant, k0, rounds, fused, X_out=Xo, Y_out=Yo, workspace=ws)
        assert ceca.ceca_read_status(ws) == 0
        want_x, want_y = oracle.consensus(_np(x), _np(y), variant, k0, rounds)
        tol = STEP_TOL * rounds * _scale(0, (x, 1), (y, 1))
        assert np.abs(_np(Xo) - want_x).max() <= tol and np.abs(_np(Yo) - want_y).max() <= tol
        with pytest.raises(ceca.CecaError):   # nowhere to keep Y between the launches
            ceca.ceca_consensus_rounds(x.to(DEV), y.to(DEV), variant, k0, rounds, fused, X_out=Xo, workspace=ws, want_y=False)


@pytest.mark.parametrize("fused", [ceca.FUSED_SMEM, ceca.FUSED_TMEM, ceca.FUSED_BLOCK])
def test_fused_consensus_padded_rows(fused):
    n, d, ld = 100, 1000, 1024
    x = synth.consensus_inputs(n, d, seed=9)
    (X, xb), (Xo, xob), (Yo, yob) = _put(x.to(DEV), ld), _padded(n, d, ld), _padded(n, d, ld)
    ws = _fused_ws()
    for variant in (ceca.CECA_2P, ceca.CECA_1P):
        if fused == ceca.FUSED_BLOCK and fused not in _fused_kernels(n, variant):
            continue
        ceca.ceca_consensus_rounds(X, None, variant, 0, 7, fused, X_out=Xo, Y_out=Yo, workspace=ws)
        want_x, want_y = oracle.consensus(_np(x), np.zeros((n, d)), variant, 0, 7)
        tol = STEP_TOL * 7 * float(x.abs().max())
        assert np.abs(_np(Xo) - want_x).max() <= tol and np.abs(_np(Yo) - want_y).max() <= tol
        assert torch.isnan(xob[:n * ld].view(n, ld)[:, d:]).all()   # stores stop at column d
        assert torch.isnan(yob[:n * ld].view(n, ld)[:, d:]).all()
        assert ceca.ceca_read_status(ws) == 0


def test_step_and_consensus_on_random_shapes():
    """Seeded random draw of agent counts, widths, paddings, base offsets, iteration counters and call
    forms (in / out of place, with / without gradient, fused / per round)."""
    rng = np.random.default_rng(2024)
    for case in range(80):
        n = int(rng.choice([rng.integers(1, 9), rng.integers(9, 130), rng.integers(130, 700)]))
        d = int(rng.choice([rng.integers(1, 9), rng.integers(9, 300), rng.integers(300, 3000)]))
        ld = d + int(rng.choice([0, 0, 1, 3, 4, 28]))
        offset = int(rng.choice([0, 0, 4, 1]))
        variant = ceca.CECA_2P if (n % 2 and n > 1) else int(rng.choice([ceca.CECA_1P, ceca.CECA_2P]))
        k = int(rng.integers(0, 2**50))
        gamma = float(rng.choice([0.0, 0.05, 1.0]))
        with_g = bool(rng.integers(0, 2))
        x, y, g = synth.step_inputs(n, d, seed=case, x_std=1.0, g_std=1.0, same_xy=False)
        (X, _), (Y, _) = _put(x.to(DEV), ld, offset), _put(y.to(DEV), ld, offset)
        G = _put(g.to(DEV), ld, offset)[0] if with_g else None
        want_x, want_y = oracle.step(_np(x), _np(y), _np(g) if with_g else None, np.float32(gamma), variant, k)
        tol = STEP_TOL * _scale(gamma, (x, 1), (y, 1), (g if with_g else None, gamma))
        if rng.integers(0, 2):
            ceca.ceca_gossip_sgd_step(X, Y, G, gamma, variant, k)
            Xo, Yo = X, Y
        else:
            (Xo, _), (Yo, _) = _padded(n, d, ld, offset), _padded(n, d, ld, offset)
            ceca.ceca_gossip_sgd_step(X, Y, G, gamma, variant, k, X_out=Xo, Y_out=Yo)
        assert np.abs(_np(Xo) - want_x).max() <= tol, (case, n, d, ld, offset, variant, k)
        assert np.abs(_np(Yo) - want_y).max() <= tol, (case, n, d, ld, offset, variant, k)
        # consensus from the same data: a few rounds from a random start, fused where the layout allows
        rounds = int(rng.integers(1, 14))
        k0 = int(rng.integers(0, 40))
        ld4 = (d + 3) // 4 * 4 + 4 * int(rng.integers(0, 3))
        (Xc, _), (Yc, _) = _put(x.to(DEV), ld4, 0), _put(y.to(DEV), ld4, 0)
        fused = int(rng.choice([0, 1] + _fused_kernels(n, variant)))
        ws = _fused_ws()
        ceca.ceca_consensus_rounds(Xc, Yc, variant, k0, rounds, fused, workspace=ws)
        assert ceca.ceca_read_status(ws) == 0
        want_x, want_y = oracle.consensus(_np(x), _np(y), variant, k0, rounds)
        tol = STEP_TOL * rounds * _scale(0, (x, 1), (y, 1))
        assert np.abs(_np(Xc) - want_x).max() <= tol, (case, n, d, ld4, variant, k0, rounds, fused)
        assert np.abs(_np(Yc) - want_y).max() <= tol, (case, n, d, ld4, variant, k0, rounds, fused)


@pytest.mark.parametrize("fused", [ceca.FUSED_SMEM, ceca.FUSED_TMEM, ceca.FUSED_BLOCK])
def test_bounded_wait_of_the_fused_kernels_runs_out_and_reports(fused):
    """The only device-side wait in the library is the wait for the TMA landing.  The self-test entry arms
    that barrier for more bytes than arrive: every tile must give up after its poll budget, set the status
    word, store nothing, and leave the context usable for an ordinary call."""
    n, d = 6, 32
    x = synth.consensus_inputs(n, d, seed=11)
    X = x.to(DEV)
    Xo = torch.full_like(X, float("nan"))
    ws = _fused_ws()
    ceca.ceca_fused_wait_selftest(X, Xo, fused, ws)
    assert ceca.ceca_read_status(ws) == 1
    assert torch.isnan(Xo).all() and torch.equal(X.cpu(), x)
    ws.zero_()
    ceca.ceca_consensus_rounds(X, None, ceca.CECA_2P, 0, 3, fused, X_out=Xo, workspace=ws, want_y=False)
    assert ceca.ceca_read_status(ws) == 0
    want_x, _ = oracle.consensus(_np(x), np.zeros((n, d)), ceca.CECA_2P, 0, 3)
    assert np.abs(_np(Xo) - want_x).max() <= STEP_TOL * 3 * float(x.abs().max())
    # several tiles per group and a ragged last tile
    n, d = 97, 4100
    X = synth.consensus_inputs(n, d, seed=12).to(DEV)
    Xo = torch.full_like(X, float("nan"))
    ws.zero_()
    ceca.ceca_fused_wait_selftest(X, Xo, fused, ws)
    assert ceca.ceca_read_status(ws) == 1 and torch.isnan(Xo).all()


# --------------------------------------------------------------------------------------------
# logistic gradient
# --------------------------------------------------------------------------------------------

def _grad_tol(d, want):
    return 8 * np.sqrt(d) * 2.0 ** -24 * np.abs(want).max() + 1e-7


@pytest.mark.parametrize("n,m,d", [(5, 100, 32), (6, 100, 32), (3, 37, 4096), (2, 50, 8192), (2, 33, 1028),
                                   (4, 16, 2048), (3, 20, 30), (2, 9, 8200), (1, 5, 1), (7, 1, 64),
                                   # wider than one CTA's registers: clusters of 2 to 8 CTAs, one column chunk each
                                   (2, 21, 8196), (3, 37, 16384), (1, 18, 40000), (2, 33, 65536), (2, 5, 65540), (2, 4, 70000)])
def test_logreg_grad_matches_oracle(n, m, d):
    a, lab, x_star = synth.logreg_problem(n, m, d, seed=n + m + d, flip=0.1, hetero_std=0.5)
    gen = torch.Generator().manual_seed(1)
    x = 0.05 * torch.randn(n, d, generator=gen)
    y = 0.05 * torch.randn(n, d, generator=gen)
    A, L, X, Y = a.to(DEV), lab.to(DEV), x.to(DEV), y.to(DEV)
    ws = torch.empty(ceca.ceca_workspace_bytes(ceca.WS_LOGREG_GRAD, n, m, d) // 4 + 64, dtype=torch.float32, device=DEV)
    for variant in _variants(n):
        for k in range(_tau(n)):
            G = torch.full((n, d), float("nan"), device=DEV)
            ceca.dsgd_logreg_grad(A, L, X, Y, k, variant, G, ws)
            want = oracle.logreg_grad(_np(a), _np(lab), _np(x), _np(y), k)
            assert np.abs(_np(G) - want).max() <= _grad_tol(d, want), (n, m, d, k)
            G2 = torch.empty_like(G)
            ceca.dsgd_logreg_grad(A, L, X, Y, k, variant, G2, ws)
            assert torch.equal(G, G2)  # run-to-run identical


@pytest.mark.parametrize("n,m,d,ld", [(6, 40, 512, 516), (6, 40, 512, 513), (3, 33, 2052, 2080), (5, 50, 10, 12), (2, 9, 12288, 12292)])
def test_gradients_with_padded_rows_leave_padding_and_workspace_guard_alone(n, m, d, ld):
    """X, Y, G (and the least-squares noise) with ld > d; the columns between d and ld of G, and a guard
    area behind the stated workspace size, must keep their canary values."""
    a, lab, _ = synth.logreg_problem(n, m, d, seed=n + d, flip=0.1, hetero_std=0.3)
    a2, b2, _ = synth.lsq_problem(n, m, d, seed=n + d + 1)
    gen = torch.Generator().manual_seed(7)
    x = 0.1 * torch.randn(n, d, generator=gen); y = 0.1 * torch.randn(n, d, generator=gen)
    eps = synth.gradient_noise(n, d, 0, sigma_n=1.0)
    (X, _), (Y, _), (E, _) = _put(x.to(DEV), ld), _put(y.to(DEV), ld), _put(eps.to(DEV), ld)
    need = ceca.ceca_workspace_bytes(ceca.WS_LOGREG_GRAD, n, m, d)
    assert need % 4 == 0
    guard = 1024
    ws_all = torch.full((need // 4 + guard,), float("nan"), dtype=torch.float32, device=DEV)
    ws = ws_all[:need // 4]
    for k in range(_tau(n)):
        G, gbuf = _padded(n, d, ld)
        ceca.dsgd_logreg_grad(a.to(DEV), lab.to(DEV), X, Y, k, ceca.CECA_2P, G, ws)
        want = oracle.logreg_grad(_np(a), _np(lab), _np(x), _np(y), k)
        assert np.abs(_np(G) - want).max() <= _grad_tol(d, want)
        assert torch.isnan(gbuf[:n * ld].view(n, ld)[:, d:]).all() and torch.isnan(gbuf[n * ld:]).all()
        G2, gbuf2 = _padded(n, d, ld)
        ceca.dsgd_lsq_grad(a2.to(DEV), b2.to(DEV), X, Y, k, ceca.CECA_2P, G2, ws, noise=E)
        want = oracle.lsq_grad(_np(a2), _np(b2), _np(x), _np(y), k, noise=_np(eps))
        z = y if oracle.round_info(n, k).payload else x
        assert np.abs(_np(G2) - want).max() <= _lsq_tol(_np(a2), _np(b2), _np(z)) + 5e-6
        assert torch.isnan(gbuf2[:n * ld].view(n, ld)[:, d:]).all()
        assert torch.isnan(ws_all[need // 4:]).all()


@pytest.mark.parametrize("n,variant", [(5, ceca.CECA_2P), (6, ceca.CECA_1P)])
def test_small_logistic_regression_run(n, variant):
    """n agents, d = 32, 100 samples each, X0 = Y0 = 0, gamma = 0.05, 60 iterations: gradient kernel
    + fused step on the GPU against the same loop in the fp64 oracle."""
    m, d, gamma, iters = 100, 32, 0.05, 60
    a, lab, _ = synth.logreg_problem(n, m, d, seed=0, flip=0.1)
    A, L = a.to(DEV), lab.to(DEV)
    X = torch.zeros(n, d, device=DEV); Y = torch.zeros(n, d, device=DEV); G = torch.empty(n, d, device=DEV)
    ws = torch.empty(ceca.ceca_workspace_bytes(ceca.WS_LOGREG_GRAD, n, m, d) // 4, dtype=torch.float32, device=DEV)
    ox = np.zeros((n, d)); oy = np.zeros((n, d))
    an, ln = _np(a), _np(lab)
    for k in range(iters):
        ceca.dsgd_logreg_grad(A, L, X, Y, k, variant, G, ws)
        ceca.ceca_gossip_sgd_step(X, Y, G, gamma, variant, k)
        og = oracle.logreg_grad(an, ln, ox, oy, k)
        ox, oy = oracle.step(ox, oy, og, np.float32(gamma), variant, k)
        scale = max(np.abs(ox).max(), np.abs(oy).max(), 1e-3)
        tol = 4e-6 * (k + 1) * scale   # linear growth: each iteration adds a step's and a gradient's rounding
        assert np.abs(_np(X) - ox).max() <= tol, k
        assert np.abs(_np(Y) - oy).max() <= tol, k
    loss0 = oracle.logreg_loss(an, ln, np.zeros((n, d))).mean()
    loss1 = oracle.logreg_loss(an, ln, np.broadcast_to(_np(X).mean(0), (n, d))).mean()
    assert loss1 < loss0


# --------------------------------------------------------------------------------------------
# least-squares gradient and the paper's convex experiment (Sec. 5 "DSGD: least-squares problem")
# --------------------------------------------------------------------------------------------

@pytest.mark.parametrize("shards", [1, 2, 3])
@pytest.mark.parametrize("n,m,d,view", [(5, 100, 32, True), (6, 37, 1030, True), (3, 50, 4099, False), (63, 40, 512, False)])
def test_column_sharded_logistic_gradient(shards, n, m, d, view):
    """The gradient computed shard by shard (partial dot products per column block, their sum in shard order,
    coefficient + A^T pass per block) equals the oracle's and the unsharded kernel's; unequal block widths."""
    a, lab, _ = synth.logreg_problem(n, m, d, seed=n + d, flip=0.1, hetero_std=0.5)
    gen = torch.Generator().manual_seed(d)
    x, y = 0.1 * torch.randn(n, d, generator=gen), 0.1 * torch.randn(n, d, generator=gen)
    A, L, X, Y = a.to(DEV), lab.to(DEV), x.to(DEV), y.to(DEV)
    ws = torch.empty(ceca.ceca_workspace_bytes(ceca.WS_LOGREG_GRAD, n, m, d), dtype=torch.uint8, device=DEV)
    for k in (0, 1, 2):
        variant = ceca.CECA_2P
        Z = Y if ceca.ceca_schedule(n, variant, k, peers=False)[0].payload else X
        want = oracle.logreg_grad(_np(a), _np(lab), _np(x), _np(y), k)
        whole = torch.empty(n, d, device=DEV)
        ceca.dsgd_logreg_grad(A, L, X, Y, k, variant, whole, ws)
        G = torch.full((n, d), float("nan"), device=DEV)
        cuts = [ceca.shard_columns(d, shards, j) for j in range(shards)]
        assert cuts[0][0] == 0 and cuts[-1][1] == d and all(cuts[j][1] == cuts[j + 1][0] for j in range(shards - 1))
        total, part = torch.empty(n, m, device=DEV), torch.empty(n, m, device=DEV)
        blocks = []
        for j, (lo, hi) in enumerate(cuts):
            # a shard either views its columns of the full matrices or owns a dense copy of them
            As = A[:, :, lo:hi] if view else A[:, :, lo:hi].contiguous()
            Zs = Z[:, lo:hi] if view else Z[:, lo:hi].contiguous()
            blocks.append(As)
            ceca.dsgd_grad_shard_dots(As, Zs, part)
            ceca.dsgd_grad_shard_sum(total, part, first=(j == 0))
        for j, (lo, hi) in enumerate(cuts):
            dots = total.clone()          # every shard gets its own copy of the summed dots: apply overwrites it
            Gs = G[:, lo:hi] if view else torch.empty(n, hi - lo, device=DEV)
            ceca.dsgd_grad_shard_apply(blocks[j], L, dots, Gs)
            if not view:
                G[:, lo:hi] = Gs
        tol = _grad_tol(d, want)
        assert np.abs(_np(G) - want).max() <= tol, (k, shards)
        assert np.abs(_np(G) - _np(whole)).max() <= tol, (k, shards)


@pytest.mark.parametrize("shards", [1, 2, 3])
@pytest.mark.parametrize("n,m,d,view", [(6, 50, 10, True), (4, 64, 2048, False), (3, 37, 4100, True), (5, 33, 520, False)])
def test_column_sharded_least_squares_gradient(shards, n, m, d, view):
    """The least-squares form of the sharded gradient (residual as coefficient, the caller's noise added to each
    block): shard by shard against the oracle; widths that take the 128-bit A^T pass and widths that do not."""
    a, b, _ = synth.lsq_problem(n, m, d, seed=n + d, sigma_s=0.1)
    x = torch.randn(n, d, generator=torch.Generator().manual_seed(5))
    eps = synth.gradient_noise(n, d, 0, sigma_n=5.0)
    A, B, X, E = a.to(DEV), b.to(DEV), x.to(DEV), eps.to(DEV)
    k = 0                                                   # round 0 evaluates at x for every n
    want = oracle.lsq_grad(_np(a), _np(b), _np(x), _np(x), k, noise=_np(eps))
    tol = _lsq_tol(_np(a), _np(b), _np(x)) + 5e-6
    cuts = [ceca.shard_columns(d, shards, j) for j in range(shards)]
    total, part = torch.empty(n, m, device=DEV), torch.empty(n, m, device=DEV)
    blocks = []
    for j, (lo, hi) in enumerate(cuts):
        As = A[:, :, lo:hi] if view else A[:, :, lo:hi].contiguous()
        Zs = X[:, lo:hi] if view else X[:, lo:hi].contiguous()
        blocks.append(As)
        ceca.dsgd_grad_shard_dots(As, Zs, part)
        ceca.dsgd_grad_shard_sum(total, part, first=(j == 0))
    G = torch.full((n, d), float("nan"), device=DEV)
    for j, (lo, hi) in enumerate(cuts):
        Gs = G[:, lo:hi] if view else torch.empty(n, hi - lo, device=DEV)
        Es = E[:, lo:hi] if view else E[:, lo:hi].contiguous()
        ceca.dsgd_grad_shard_apply(blocks[j], B, total.clone(), Gs, loss=1, noise_shard=Es)
        if not view:
            G[:, lo:hi] = Gs
    assert np.abs(_np(G) - want).max() <= tol, (shards, n, m, d)


def _lsq_tol(a, b, z):
    """fp32 bound: a length-d dot product per residual, then a length-m sum of residual * feature."""
    n, m, d = a.shape
    u = 2.0 ** -24
    mag = np.einsum("nmd,nd->nm", np.abs(a), np.abs(z)) + np.abs(b)          # size of each residual's terms
    s = np.einsum("nmd,nm->nd", np.abs(a), mag).max()                         # size of each gradient entry's terms
    return 4 * u * (np.sqrt(d) + np.sqrt(m)) * s + 1e-7


@pytest.mark.parametrize("n,m,d", [(258, 50, 10), (6, 50, 10), (4, 64, 2048), (3, 37, 4096), (5, 20, 12), (2, 7, 1), (2, 30, 16384)])
def test_lsq_grad_matches_oracle(n, m, d):
    a, b, _ = synth.lsq_problem(n, m, d, seed=n + d, sigma_s=0.1)
    gen = torch.Generator().manual_seed(3)
    x = torch.randn(n, d, generator=gen); y = torch.randn(n, d, generator=gen)
    eps = synth.gradient_noise(n, d, 0, sigma_n=5.0)
    A, B, X, Y, E = a.to(DEV), b.to(DEV), x.to(DEV), y.to(DEV), eps.to(DEV)
    ws = torch.empty(ceca.ceca_workspace_bytes(ceca.WS_LOGREG_GRAD, n, m, d) // 4 + 64, dtype=torch.float32, device=DEV)
    for variant in _variants(n):
        for k in range(min(_tau(n), 4)):
            z = y if oracle.round_info(n, k).payload else x
            tol = _lsq_tol(_np(a), _np(b), _np(z))
            G = torch.full((n, d), float("nan"), device=DEV)
            ceca.dsgd_lsq_grad(A, B, X, Y, k, variant, G, ws)
            want = oracle.lsq_grad(_np(a), _np(b), _np(x), _np(y), k)
            assert np.abs(_np(G) - want).max() <= tol, (n, m, d, k)
            ceca.dsgd_lsq_grad(A, B, X, Y, k, variant, G, ws, noise=E)
            want = oracle.lsq_grad(_np(a), _np(b), _np(x), _np(y), k, noise=_np(eps))
            assert np.abs(_np(G) - want).max() <= tol + 5e-6, (n, m, d, k)


@pytest.mark.parametrize("variant", [ceca.CECA_1P, ceca.CECA_2P])
def test_least_squares_experiment(variant):
    """n = 258 agents, d = 10, 50 samples each, sigma_s = 0.1, gradient noise sigma_n = 5, step size 0.02
    divided by 1.5 every 20 iterations: gradient kernel + fused step on the GPU against the fp64 oracle
    on the same data and the same noise draws."""
    n, m, d, iters = 258, 50, 10, 120
    a, b, x_star = synth.lsq_problem(n, m, d, seed=0, sigma_s=0.1)
    x0 = torch.randn(n, d, generator=torch.Generator().manual_seed(5))
    A, B = a.to(DEV), b.to(DEV)
    X, Y, G = x0.to(DEV), x0.to(DEV), torch.empty(n, d, device=DEV)
    ws = torch.empty(ceca.ceca_workspace_bytes(ceca.WS_LOGREG_GRAD, n, m, d) // 4 + 64, dtype=torch.float32, device=DEV)
    ox, oy = _np(x0).astype(np.float64), _np(x0).astype(np.float64)
    an, bn = _np(a), _np(b)
    err0 = np.linalg.norm(ox.mean(0) - _np(x_star))
    gamma = 0.02
    for k in range(iters):
        if k and k % 20 == 0:
            gamma /= 1.5
        eps = synth.gradient_noise(n, d, k, sigma_n=5.0)
        ceca.dsgd_lsq_grad(A, B, X, Y, k, variant, G, ws, noise=eps.to(DEV))
        ceca.ceca_gossip_sgd_step(X, Y, G, gamma, variant, k)
        og = oracle.lsq_grad(an, bn, ox, oy, k, noise=_np(eps))
        ox, oy = oracle.step(ox, oy, og, np.float32(gamma), variant, k)
        # the local problems are contractive at this step size, so rounding does not accumulate
        # faster than linearly; the scale is what one step moves (gamma |G|) or the state itself
        scale = max(np.abs(ox).max(), np.abs(oy).max(), float(np.float32(gamma)) * np.abs(og).max())
        tol = 4e-6 * (k + 1) * scale
        assert np.abs(_np(X) - ox).max() <= tol, k
        assert np.abs(_np(Y) - oy).max() <= tol, k
    err1 = np.linalg.norm(_np(X).astype(np.float64).mean(0) - _np(x_star))
    assert err1 < 0.2 * err0      # the averaged model has moved most of the way to x*


# --------------------------------------------------------------------------------------------
# host-memory front end
# --------------------------------------------------------------------------------------------

@pytest.mark.parametrize("pinned", [True, False])
@pytest.mark.parametrize("n,d,ld,variant", [(6, 1000, 1000, ceca.CECA_1P), (24, 70001, 70004, ceca.CECA_2P),
                                             (100, 300000, 300000, ceca.CECA_2P)])
def test_host_step_matches_device_step(pinned, n, d, ld, variant):
    x, y, g = synth.step_inputs(n, ld, seed=2, x_std=1.0, g_std=1.0, same_xy=False)
    gamma = 0.1
    ws = torch.empty(32 << 20, dtype=torch.uint8, device=DEV)
    for k in range(_tau(n)):
        hx, hy, hg = x.clone(), y.clone(), g.clone()
        if pinned:
            hx, hy, hg = hx.pin_memory(), hy.pin_memory(), hg.pin_memory()
        ceca.ceca_gossip_sgd_step_host(hx[:, :d], hy[:, :d], hg[:, :d], gamma, variant, k, ws)
        X, Y, G = x[:, :d].to(DEV).contiguous(), y[:, :d].to(DEV).contiguous(), g[:, :d].to(DEV).contiguous()
        ceca.ceca_gossip_sgd_step(X, Y, G, gamma, variant, k)
        assert torch.equal(hx[:, :d], X.cpu()) and torch.equal(hy[:, :d], Y.cpu())
        assert torch.equal(hx[:, d:], x[:, d:]) and torch.equal(hg, g)   # padding and G untouched


# --------------------------------------------------------------------------------------------
# full-size workloads, checked on column windows (columns never interact in the update)
# --------------------------------------------------------------------------------------------

def _windows(d, width, count, seed):
    rng = np.random.default_rng(seed)
    starts = [0, max(d - width, 0)] + [int(s) for s in rng.integers(0, max(d - width, 1), size=count)]
    return [(s, min(s + width, d)) for s in starts]


def _need_free(bytes_needed):
    free, _ = torch.cuda.mem_get_info()
    if free < bytes_needed:
        pytest.skip("needs %.1f GB of free device memory" % (bytes_needed / 1e9))


@pytest.mark.parametrize("n,d,variant,iters", [(24, 11_689_512, ceca.CECA_1P, 5), (100, 25_557_032, ceca.CECA_2P, 7)])
def test_full_size_step_on_column_windows(n, d, variant, iters):
    """Flat CNN-sized parameter vectors (ResNet-18 / ResNet-50 sized), in place, the launch shape the
    benchmark times; windows include the first and the last (ragged) columns."""
    _need_free(int(3.3 * n * d * 4))
    ld = synth.padded_ld(d)   # the benchmark's layout: rows padded to a multiple of 128 bytes
    X, Y, G = synth.step_inputs(n, d, seed=4, x_std=0.01, g_std=0.01, device=DEV, ld=ld)
    assert X.stride(0) == ld and ld % 32 == 0 and d % 32 != 0
    gamma = 0.1
    wins = _windows(d, 4099, 4, seed=n)
    ref = [(_np(X[:, lo:hi]).astype(np.float64), _np(Y[:, lo:hi]).astype(np.float64)) for lo, hi in wins]
    for k in range(iters):
        synth.gradient_inputs(n, d, k, g_std=0.01, device=DEV, out=G)
        gw = [_np(G[:, lo:hi]) for lo, hi in wins]
        before = [( _np(X[:, lo:hi]), _np(Y[:, lo:hi])) for lo, hi in wins]
        ceca.ceca_gossip_sgd_step(X, Y, G, gamma, variant, k)
        for w, (lo, hi) in enumerate(wins):
            want_x, want_y = oracle.step(before[w][0], before[w][1], gw[w], np.float32(gamma), variant, k)
            tol = STEP_TOL * max(np.abs(before[w][0]).max(), np.abs(before[w][1]).max())
            assert np.abs(_np(X[:, lo:hi]) - want_x).max() <= tol, (k, lo)
            assert np.abs(_np(Y[:, lo:hi]) - want_y).max() <= tol, (k, lo)
            # and the whole trajectory against an fp64 run from the same start
            ref[w] = oracle.step(ref[w][0], ref[w][1], gw[w], np.float32(gamma), variant, k)
            assert np.abs(_np(X[:, lo:hi]) - ref[w][0]).max() <= tol * (k + 1)


def test_device_entry_points_reject_bad_arguments_and_launch_nothing():
    """The argument-error table of the C ABI with real device buffers: every call must come back with the
    stated status before anything is enqueued, so the NaN-filled outputs stay untouched."""
    import ctypes
    lib = ceca.library()
    big = 2050 * 8
    bufs = [torch.full((big + 4,), float("nan"), device=DEV) for _ in range(6)]
    x, y, g, xo, yo, ws = [ctypes.c_void_p(b.data_ptr()) for b in bufs]
    xo_off = ctypes.c_void_p(bufs[3].data_ptr() + 4)     # 4 bytes past a 16-byte boundary
    stream = ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
    step = lib.ceca_gossip_sgd_step
    assert step(None, y, g, xo, yo, 4, 8, 8, 0.1, 2, 0, stream) == 1
    assert step(x, y, g, xo, yo, 0, 8, 8, 0.1, 2, 0, stream) == 1
    assert step(x, y, g, xo, yo, 4, 8, 7, 0.1, 2, 0, stream) == 1        # ld < d
    assert step(x, y, g, xo, yo, 5, 8, 8, 0.1, 1, 0, stream) == 2        # odd n, 1-port
    assert step(x, None, g, xo, yo, 4, 8, 8, 0.1, 2, 1, stream) == 1     # round 1 needs Y
    assert step(x, y, g, xo, xo, 4, 8, 8, 0.1, 2, 1, stream) == 4        # X_out == Y_out
    assert step(x, y, g, y, yo, 4, 8, 8, 0.1, 2, 1, stream) == 4         # X_out == Y
    assert step(x, None, g, xo, None, 6, 8, 8, 0.1, 2, 0, stream) == 1   # X-only needs n = 2^tau
    assert step(x, y, g, xo, None, 8, 8, 8, 0.1, 2, 0, stream) == 1      # y+ may only be dropped at r = tau-1
    assert step(x, y, g, xo, yo, 4, 8, 8, 0.1, 3, 0, stream) == 1        # no such variant
    assert step(x, y, g, xo, yo, 4, 8, 8, 0.1, 2, -1, stream) == 1       # k < 0
    bf = lib.ceca_gossip_sgd_step_bf16
    assert bf(x, y, None, xo, yo, 4, 8, 8, 0, 0.1, 2, 0, stream) == 1    # the narrow gradient is required
    assert bf(x, y, g, xo, None, 4, 8, 8, 1, 0.1, 2, 0, stream) == 1     # so is Y_out
    assert bf(x, y, g, g, yo, 4, 8, 8, 1, 0.1, 2, 0, stream) == 4        # X_out == G
    cons = lib.ceca_consensus_rounds
    assert cons(x, y, xo, yo, 4, 8, 8, 2, 0, -1, 0, None, 0, stream) == 1
    assert cons(x, None, xo, None, 6, 8, 8, 2, 0, 2, 0, None, 0, stream) == 5      # no Y_out, no workspace (n not 2^tau)
    assert cons(x, None, xo, None, 2050, 8, 8, 2, 0, 2, 1, ws, 256, stream) == 4   # n > 2048 fused
    assert cons(x, None, xo, None, 200, 8, 8, 2, 0, 2, 3, ws, 256, stream) == 4    # tensor-memory kernel: n <= 128
    assert cons(x, None, xo, None, 418, 8, 8, 1, 0, 2, 4, ws, 256, stream) == 4    # register-block kernel: 1-port up to n = 416
    assert cons(x, None, xo, None, 1154, 8, 8, 2, 0, 2, 4, ws, 256, stream) == 4   # ... 2-port up to n = 1152
    assert cons(x, None, xo, None, 4, 8, 8, 2, 0, 2, 7, ws, 256, stream) == 1      # no such kernel
    assert cons(x, None, xo_off, None, 4, 8, 8, 2, 0, 2, 1, ws, 256, stream) == 3  # misaligned
    assert cons(x, None, xo, None, 4, 8, 6, 2, 0, 2, 1, ws, 256, stream) == 1      # ld < d
    assert cons(x, None, xo, None, 4, 6, 6, 2, 0, 2, 1, ws, 256, stream) == 3      # ld*4 % 16
    assert cons(x, None, xo, None, 4, 8, 8, 2, 1, 2, 1, ws, 256, stream) == 1      # starts at r=1, no Y
    assert cons(x, None, xo, None, 4, 8, 8, 2, 0, 2, 1, None, 0, stream) == 5      # fused needs the status word
    assert cons(x, None, xo, yo, 4, 8, 8, 2, 3, 0, 1, ws, 256, stream) == 1        # zero rounds, Y_out without Y
    self_test = lib.ceca_fused_wait_selftest
    assert self_test(x, x, 6, 32, 32, 2, ws, 256, stream) == 4                     # X_out must not alias X
    assert self_test(x, xo, 6, 32, 32, 1, ws, 256, stream) == 1                    # names a kernel, not "auto"
    grad = lib.dsgd_logreg_grad
    assert grad(x, y, g, g, 0, xo, 4, 0, 8, 8, 2, ws, 1 << 10, stream) == 1
    assert grad(x, y, g, g, 0, xo, 4, 5, 8, 8, 2, None, 0, stream) == 5
    assert grad(x, y, g, None, 1, xo, 6, 5, 8, 8, 2, ws, 1 << 10, stream) == 1     # n=6, k=1 evaluates at Y
    assert lib.dsgd_logreg_grad_static(x, y, g, None, 1, xo, 6, 5, 8, 8, 2, stream) == 1
    host = lib.ceca_gossip_sgd_step_host
    assert host(x, y, g, 4, 8, 8, 0.1, 2, 0, None, 0) == 5
    assert host(x, y, g, 5, 8, 8, 0.1, 1, 0, ws, 1 << 10) == 2
    torch.cuda.synchronize()
    for b in bufs:
        assert torch.isnan(b).all()


# --------------------------------------------------------------------------------------------
# bf16 storage (fp32 arithmetic): the gradient alone, or X, Y and the gradient
# --------------------------------------------------------------------------------------------

BF16_HALF_ULP = 2.0 ** -8    # round-to-nearest into 8 significant bits: at most 2^-8 relative


def _wide(t):
    """The exact fp64 values of a float32 / bfloat16 tensor."""
    return t.detach().float().cpu().numpy().astype(np.float64)


def _bf16_tol(want, scale, xy_bf16):
    """fp32 arithmetic on the stored values (2e-6 * scale, as for the fp32 step), plus one rounding of the
    result to bfloat16 when the models are stored narrow."""
    return STEP_TOL * scale + (BF16_HALF_ULP * np.abs(want) if xy_bf16 else 0.0)


@pytest.mark.parametrize("xy_bf16", [False, True])
@pytest.mark.parametrize("n,d,ld,offset", [(1, 9, 9, 0), (5, 37, 37, 0), (6, 64, 64, 0), (24, 1000, 1000, 0), (24, 1000, 1008, 8),
                                            (24, 1001, 1004, 4), (24, 1000, 1008, 3), (24, 1001, 1008, 5), (6, 5, 8, 6),
                                            (97, 4100, 4104, 0), (100, 70001, 70008, 0)])
def test_step_with_bf16_storage_matches_oracle(xy_bf16, n, d, ld, offset):
    gamma = 0.1
    x, y, g = synth.step_inputs(n, d, seed=n + d, x_std=1.0, g_std=1.0, same_xy=False)
    xy_t = torch.bfloat16 if xy_bf16 else torch.float32

    def put(src, dtype):
        buf = torch.full((n * ld + offset + 16,), float("nan"), dtype=dtype, device=DEV)
        view = buf[offset:offset + n * ld].view(n, ld)[:, :d]
        view.copy_(src.to(DEV))
        return view, buf

    for variant in _variants(n):
        for k in range(max(_tau(n), 1) + 1):
            (X, xb), (Y, yb), (G, gb) = put(x, xy_t), put(y, xy_t), put(g, torch.bfloat16)
            xs, ys, gs = _wide(X), _wide(Y), _wide(G)        # what the kernel reads, widened exactly
            want_x, want_y = oracle.step(xs, ys, gs, np.float32(gamma), variant, k)
            scale = max(np.abs(xs).max(), np.abs(ys).max(), gamma * np.abs(gs).max())
            (Xo, xob), (Yo, yob) = put(torch.zeros(n, d), xy_t), put(torch.zeros(n, d), xy_t)
            ceca.ceca_gossip_sgd_step_bf16(X, Y, G, gamma, variant, k, X_out=Xo, Y_out=Yo)
            assert (np.abs(_wide(Xo) - want_x) <= _bf16_tol(want_x, scale, xy_bf16)).all(), (variant, k)
            assert (np.abs(_wide(Yo) - want_y) <= _bf16_tol(want_y, scale, xy_bf16)).all(), (variant, k)
            assert torch.isnan(xob[:offset]).all() and torch.isnan(xob[offset + n * ld:]).all()
            if ld > d:
                assert torch.isnan(xob[offset:offset + n * ld].view(n, ld)[:, d:]).all()
                assert torch.isnan(yob[offset:offset + n * ld].view(n, ld)[:, d:]).all()
            ceca.ceca_gossip_sgd_step_bf16(X, Y, G, gamma, variant, k)     # in place: the same bits
            assert torch.equal(X, Xo) and torch.equal(Y, Yo)
    with pytest.raises(ceca.CecaError):   # the gradient is required in this form
        ceca.ceca_gossip_sgd_step_bf16(X, Y, None, gamma, ceca.CECA_2P, 0)


@pytest.mark.parametrize("xy_bf16", [False, True])
def test_full_size_step_with_bf16_storage_on_column_windows(xy_bf16):
    """n = 100, d = 25,557,032, CECA-2P, in place: the launch shape bench.py times for the narrow-storage
    workloads, checked on column windows that include the first and the last (ragged) columns."""
    n, d, variant, gamma = 100, 25_557_032, ceca.CECA_2P, 0.1
    _need_free(int(3.3 * n * d * 4))
    ld = synth.padded_ld(d)
    xy_t = torch.bfloat16 if xy_bf16 else torch.float32
    X32, Y32, G32 = synth.step_inputs(n, d, seed=4, x_std=0.01, g_std=0.01, device=DEV, ld=ld)
    if xy_bf16:
        X = torch.empty((n, ld), dtype=xy_t, device=DEV)[:, :d]; X.copy_(X32)
        Y = torch.empty((n, ld), dtype=xy_t, device=DEV)[:, :d]; Y.copy_(Y32)
        del X32, Y32
    else:
        X, Y = X32, Y32
    G = torch.empty((n, ld), dtype=torch.bfloat16, device=DEV)[:, :d]
    wins = _windows(d, 4099, 4, seed=n)
    for k in range(7):
        synth.gradient_inputs(n, d, k, g_std=0.01, device=DEV, out=G32)
        G.copy_(G32)
        before = [(_wide(X[:, lo:hi]), _wide(Y[:, lo:hi]), _wide(G[:, lo:hi])) for lo, hi in wins]
        ceca.ceca_gossip_sgd_step_bf16(X, Y, G, gamma, variant, k)
        for (xs, ys, gs), (lo, hi) in zip(before, wins):
            want_x, want_y = oracle.step(xs, ys, gs, np.float32(gamma), variant, k)
            scale = max(np.abs(xs).max(), np.abs(ys).max())
            assert (np.abs(_wide(X[:, lo:hi]) - want_x) <= _bf16_tol(want_x, scale, xy_bf16)).all(), (k, lo)
            assert (np.abs(_wide(Y[:, lo:hi]) - want_y) <= _bf16_tol(want_y, scale, xy_bf16)).all(), (k, lo)


@pytest.mark.parametrize("fused", [0, 1])
def test_full_size_consensus_on_column_windows(fused):
    """n = 97 (prime), d = 2^20, rows offset by the agent index, tau = 7 rounds, 2-port."""
    n, d, tau = 97, 1 << 20, 7
    x = synth.consensus_inputs(n, d, seed=1, device=DEV)
    Xo, Yo = torch.empty_like(x), torch.empty_like(x)
    ws = _fused_ws()
    ceca.ceca_consensus_rounds(x, None, ceca.CECA_2P, 0, tau, fused, X_out=Xo, Y_out=Yo, workspace=ws)
    assert ceca.ceca_read_status(ws) == 0
    xd = Xo.double()
    mean = x.double().mean(0)
    assert float((xd - mean).norm() / xd.norm()) <= 1e-5
    for lo, hi in _windows(d, 2048, 4, seed=97):
        want_x, want_y = oracle.consensus(_np(x[:, lo:hi]), np.zeros((n, hi - lo)), ceca.CECA_2P, 0, tau)
        tol = STEP_TOL * tau * float(x.abs().max())
        assert np.abs(_np(Xo[:, lo:hi]) - want_x).max() <= tol
        assert np.abs(_np(Yo[:, lo:hi]) - want_y).max() <= tol


@pytest.mark.parametrize("n,variant", [(63, ceca.CECA_2P), (62, ceca.CECA_1P), (64, ceca.CECA_1P)])
def test_heterogeneous_logreg_full_size_first_iterations(n, variant):
    """2000 samples per agent, d = 4096, per-agent feature shifts: gradient + fused step, checked against
    the oracle for the first iterations (a full CECA cycle and one more, so that rounds that evaluate the
    gradient at y are included).  The 1-port variant needs an even n: 62 and 64 stand beside n = 63."""
    m, d, gamma = 2000, 4096, 0.01
    _need_free(int(1.3 * n * m * d * 4))
    A, L, _ = synth.logreg_problem(n, m, d, seed=3, flip=0.05, hetero_std=0.5, device=DEV)
    X = torch.zeros(n, d, device=DEV); Y = torch.zeros(n, d, device=DEV); G = torch.empty(n, d, device=DEV)
    ws = torch.empty(ceca.ceca_workspace_bytes(ceca.WS_LOGREG_GRAD, n, m, d) // 4, dtype=torch.float32, device=DEV)
    agents = [0, n // 2, n - 1]
    an = {i: _np(A[i:i + 1]) for i in agents}
    ln = {i: _np(L[i:i + 1]) for i in agents}
    for k in range(_tau(n) + 1):
        ceca.dsgd_logreg_grad(A, L, X, Y, k, variant, G, ws)
        z = Y if oracle.round_info(n, k).payload else X
        for i in agents:   # the gradient of agent i depends on its own data and model only
            zi = _np(z[i:i + 1])
            want = oracle.logreg_grad(an[i], ln[i], zi, zi, 0)
            assert np.abs(_np(G[i:i + 1]) - want).max() <= _grad_tol(d, want), (k, i)
        bx, by, bg = _np(X), _np(Y), _np(G)
        ceca.ceca_gossip_sgd_step(X, Y, G, gamma, variant, k)
        want_x, want_y = oracle.step(bx, by, bg, np.float32(gamma), variant, k)
        tol = STEP_TOL * max(np.abs(bx).max(), np.abs(by).max(), gamma * np.abs(bg).max())
        assert np.abs(_np(X) - want_x).max() <= tol and np.abs(_np(Y) - want_y).max() <= tol


def test_register_block_consensus_over_the_whole_range_of_agent_counts():
    """The register-block kernel picks its tile width, block size and launch shape from n: every n up to its
    limit, with an odd width that ends in a lone column or a width of several tiles with a ragged last one, a
    start at the beginning of a cycle (Y ignored) and one in the middle of it (Y read)."""
    rng = np.random.default_rng(7)
    cases = [(n, ceca.CECA_2P) for n in range(2, BLOCK_MAX_N + 1)] + [(n, ceca.CECA_1P) for n in range(2, BLOCK_MAX_N_1P + 1, 2)]
    for n, variant in cases:
        d = 37 if (n // 2) % 2 else 130
        x = synth.consensus_inputs(n, d, seed=n, offset_rows=False)
        y = synth.consensus_inputs(n, d, seed=n + 1, offset_rows=False)
        tau = _tau(n)
        for k0, rounds in ((0, tau), (int(rng.integers(1, 3 * tau + 1)), int(rng.integers(1, tau + 3))),
                           (int(rng.integers(0, 3 * tau + 1)), 1)):
            ws = _fused_ws()
            ld = (d + 3) // 4 * 4 + 4     # padded rows, 16-byte aligned
            Xo, Yo = torch.full((n, ld), float("nan"), device=DEV)[:, :d], torch.full((n, ld), float("nan"), device=DEV)[:, :d]
            X = torch.empty((n, ld), device=DEV)[:, :d]; X.copy_(x)
            Y = torch.empty((n, ld), device=DEV)[:, :d]; Y.copy_(y)
            ceca.ceca_consensus_rounds(X, Y, variant, k0, rounds, ceca.FUSED_BLOCK, X_out=Xo, Y_out=Yo, workspace=ws)
            assert ceca.ceca_read_status(ws) == 0
            want_x, want_y = oracle.consensus(_np(x), _np(y), variant, k0, rounds)
            tol = STEP_TOL * rounds * _scale(0, (x, 1), (y, 1))
            assert np.abs(_np(Xo) - want_x).max() <= tol, (n, variant, k0, rounds)
            assert np.abs(_np(Yo) - want_y).max() <= tol, (n, variant, k0, rounds)
