"""Whole training loops on the GPU: warm-up averaging followed by DSGD-CECA iterations (the setting of
the convergence theorem), eagerly and replayed from a CUDA graph.  Every kernel call goes through the
C ABI; the loops only sequence them."""
import numpy as np
import pytest
import torch

import oracle
import paper_2306_00256_b200 as ceca
import synthetic_inputs as synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _np(t):
    return t.detach().cpu().numpy()


@pytest.mark.parametrize("n,variant", [(5, ceca.CECA_2P), (6, ceca.CECA_1P), (63, ceca.CECA_2P)])
def test_warm_up_averaging_then_training(n, variant):
    """Theorem "Convergence property": global averaging first (tau + 1 CECA rounds bring x and y to the
    mean), then the iterations of Algorithm 1; here with the logistic workload, against the oracle."""
    m, d, gamma, iters = 40, 64, 0.05, 25
    tau = oracle.round_info(n, 0).tau
    a, lab, _ = synth.logreg_problem(n, m, d, seed=1, flip=0.1, hetero_std=0.5)
    x0 = torch.randn(n, d, generator=torch.Generator().manual_seed(2))
    A, L = a.to(DEV), lab.to(DEV)
    X, Y, G = x0.to(DEV), torch.zeros(n, d, device=DEV), torch.empty(n, d, device=DEV)
    ws = torch.empty(ceca.ceca_workspace_bytes(ceca.WS_LOGREG_GRAD, n, m, d), dtype=torch.uint8, device=DEV)
    status = torch.zeros(64, dtype=torch.int32, device=DEV)
    ceca.ceca_consensus_rounds(X, Y, variant, 0, tau + 1, 1, workspace=status)
    assert ceca.ceca_read_status(status) == 0
    mean = x0.double().mean(0)
    assert (X.double().cpu() - mean).abs().max() <= 2e-6 * (tau + 1) * float(x0.abs().max())
    assert (Y.double().cpu() - mean).abs().max() <= 2e-6 * (tau + 1) * float(x0.abs().max())
    ox, oy = oracle.consensus(_np(x0), np.zeros((n, d)), variant, 0, tau + 1)
    an, ln = _np(a), _np(lab)
    for k in range(tau + 1, tau + 1 + iters):   # the iteration counter keeps running
        ceca.dsgd_logreg_grad(A, L, X, Y, k, variant, G, ws)
        ceca.ceca_gossip_sgd_step(X, Y, G, gamma, variant, k)
        og = oracle.logreg_grad(an, ln, ox, oy, k)
        ox, oy = oracle.step(ox, oy, og, np.float32(gamma), variant, k)
        tol = 4e-6 * (k + 1) * max(np.abs(ox).max(), np.abs(oy).max())
        assert np.abs(_np(X) - ox).max() <= tol and np.abs(_np(Y) - oy).max() <= tol, k


@pytest.mark.parametrize("n,variant,d", [(5, ceca.CECA_2P, 32), (6, ceca.CECA_1P, 32), (63, ceca.CECA_2P, 4096)])
def test_one_ceca_cycle_replayed_from_a_cuda_graph(n, variant, d):
    """tau iterations (gradient + fused step) captured once and replayed: the same bits as eager calls.
    The schedule depends on k only through k mod tau, so one captured cycle serves every cycle."""
    m, gamma, cycles = 100, 0.05, 4
    tau = oracle.round_info(n, 0).tau
    a, lab, _ = synth.logreg_problem(n, m, d, seed=0, flip=0.1)
    A, L = a.to(DEV), lab.to(DEV)
    ws = torch.empty(ceca.ceca_workspace_bytes(ceca.WS_LOGREG_GRAD, n, m, d), dtype=torch.uint8, device=DEV)

    def cycle(X, Y, G, k0):
        for k in range(k0, k0 + tau):
            ceca.dsgd_logreg_grad(A, L, X, Y, k, variant, G, ws)
            ceca.ceca_gossip_sgd_step(X, Y, G, gamma, variant, k)

    Xe, Ye, Ge = torch.zeros(n, d, device=DEV), torch.zeros(n, d, device=DEV), torch.empty(n, d, device=DEV)
    for c in range(cycles):
        cycle(Xe, Ye, Ge, c * tau)

    Xg, Yg, Gg = torch.zeros(n, d, device=DEV), torch.zeros(n, d, device=DEV), torch.empty(n, d, device=DEV)
    cycle(Xg, Yg, Gg, 0)            # eager first call on this device (one-time setup happens here)
    Xg.zero_(); Yg.zero_()
    graph = torch.cuda.CUDAGraph()
    torch.cuda.synchronize()
    with torch.cuda.graph(graph):
        cycle(Xg, Yg, Gg, 0)
    Xg.zero_(); Yg.zero_()
    for c in range(cycles):
        graph.replay()
    torch.cuda.synchronize()
    assert torch.equal(Xg, Xe) and torch.equal(Yg, Ye)
    assert float(Xg.abs().max()) > 0


@pytest.mark.parametrize("n,variant,d", [(5, ceca.CECA_2P, 32), (6, ceca.CECA_1P, 32), (63, ceca.CECA_2P, 4096), (97, ceca.CECA_2P, 256)])
def test_warm_up_and_a_ceca_cycle_in_one_cuda_graph(n, variant, d):
    """The theorem's setting as one captured graph: the warm-up averaging (tau + 1 fused consensus rounds,
    one launch) followed by a CECA cycle of gradient + step.  Replayed, it gives the bits of the eager calls.
    The fused consensus call encodes its tensor maps and sets its kernel attributes on the host, so the
    first (eager) call doubles as the one-time set-up that has to precede a capture."""
    m, gamma = 60, 0.05
    tau = oracle.round_info(n, 0).tau
    a, lab, _ = synth.logreg_problem(n, m, d, seed=5, flip=0.1, hetero_std=0.5)
    x0 = torch.randn(n, d, generator=torch.Generator().manual_seed(6))
    A, L = a.to(DEV), lab.to(DEV)
    ws = torch.empty(ceca.ceca_workspace_bytes(ceca.WS_LOGREG_GRAD, n, m, d), dtype=torch.uint8, device=DEV)
    status = torch.zeros(64, dtype=torch.int32, device=DEV)

    def warm_up_and_cycle(X, Y, G):
        ceca.ceca_consensus_rounds(X, Y, variant, 0, tau + 1, ceca.FUSED_AUTO, workspace=status)
        for k in range(tau + 1, 2 * tau + 1):
            ceca.dsgd_logreg_grad(A, L, X, Y, k, variant, G, ws)
            ceca.ceca_gossip_sgd_step(X, Y, G, gamma, variant, k)

    Xe, Ye, Ge = x0.to(DEV), torch.zeros(n, d, device=DEV), torch.empty(n, d, device=DEV)
    warm_up_and_cycle(Xe, Ye, Ge)
    torch.cuda.synchronize()
    # and against the oracle
    ox, oy = oracle.consensus(_np(x0), np.zeros((n, d)), variant, 0, tau + 1)
    for k in range(tau + 1, 2 * tau + 1):
        og = oracle.logreg_grad(_np(a), _np(lab), ox, oy, k)
        ox, oy = oracle.step(ox, oy, og, np.float32(gamma), variant, k)
    tol = 4e-6 * (2 * tau + 2) * float(x0.abs().max())
    assert np.abs(_np(Xe) - ox).max() <= tol and np.abs(_np(Ye) - oy).max() <= tol

    Xg, Yg, Gg = x0.to(DEV), torch.zeros(n, d, device=DEV), torch.empty(n, d, device=DEV)
    graph = torch.cuda.CUDAGraph()
    torch.cuda.synchronize()
    with torch.cuda.graph(graph):
        warm_up_and_cycle(Xg, Yg, Gg)
    for _ in range(3):   # every replay starts from the same inputs
        Xg.copy_(x0); Yg.zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert torch.equal(Xg, Xe) and torch.equal(Yg, Ye)
    assert ceca.ceca_read_status(status) == 0


@pytest.mark.parametrize("n,variant", [(5, ceca.CECA_2P), (6, ceca.CECA_1P), (24, ceca.CECA_2P)])
def test_periodic_global_averaging(n, variant):
    """DSGD-CECA with a global average every `period` CECA cycles (tau + 1 fused consensus rounds, which bring
    x and y to the mean, as in the theorem's warm-up), over four periods, against the oracle."""
    m, d, gamma, period = 40, 48, 0.05, 2
    tau = oracle.round_info(n, 0).tau
    a, lab, _ = synth.logreg_problem(n, m, d, seed=7, flip=0.1, hetero_std=0.5)
    x0 = torch.randn(n, d, generator=torch.Generator().manual_seed(8))
    A, L = a.to(DEV), lab.to(DEV)
    X, Y, G = x0.to(DEV), x0.to(DEV), torch.empty(n, d, device=DEV)
    ws = torch.empty(ceca.ceca_workspace_bytes(ceca.WS_LOGREG_GRAD, n, m, d), dtype=torch.uint8, device=DEV)
    status = torch.zeros(64, dtype=torch.int32, device=DEV)
    ox, oy = _np(x0).astype(np.float64), _np(x0).astype(np.float64)
    an, ln = _np(a), _np(lab)
    k, steps = 0, 0
    for p in range(4):
        for _ in range(period * tau):
            ceca.dsgd_logreg_grad(A, L, X, Y, k, variant, G, ws)
            ceca.ceca_gossip_sgd_step(X, Y, G, gamma, variant, k)
            og = oracle.logreg_grad(an, ln, ox, oy, k)
            ox, oy = oracle.step(ox, oy, og, np.float32(gamma), variant, k)
            k += 1
        # k is a multiple of tau here, so the averaging window is aligned
        ceca.ceca_consensus_rounds(X, Y, variant, k, tau + 1, ceca.FUSED_AUTO, workspace=status)
        ox, oy = oracle.consensus(ox, oy, variant, k, tau + 1)
        steps += period * tau + tau + 1
        tol = 4e-6 * steps * max(np.abs(ox).max(), np.abs(oy).max())
        assert np.abs(_np(X) - ox).max() <= tol and np.abs(_np(Y) - oy).max() <= tol, p
        # all agents agree after the averaging
        assert float((X - X.mean(0)).abs().max()) <= 1e-5 * float(X.abs().max())
        assert float((Y - X.mean(0)).abs().max()) <= 1e-5 * float(X.abs().max())
    assert ceca.ceca_read_status(status) == 0


def test_heterogeneous_logistic_regression_500_iterations():
    """Config 3's full length (500 iterations, gamma = 0.01, per-agent feature shifts, 5 % label flips) at
    reduced m and d, both variants, against the oracle with the linear-in-k tolerance of the short runs."""
    m, d, gamma, iters = 40, 64, 0.01, 500
    for n, variant in [(63, ceca.CECA_2P), (62, ceca.CECA_1P)]:
        a, lab, _ = synth.logreg_problem(n, m, d, seed=3, flip=0.05, hetero_std=0.5)
        A, L = a.to(DEV), lab.to(DEV)
        X, Y, G = torch.zeros(n, d, device=DEV), torch.zeros(n, d, device=DEV), torch.empty(n, d, device=DEV)
        ws = torch.empty(ceca.ceca_workspace_bytes(ceca.WS_LOGREG_GRAD, n, m, d), dtype=torch.uint8, device=DEV)
        ox, oy = np.zeros((n, d)), np.zeros((n, d))
        an, ln = _np(a), _np(lab)
        for k in range(iters):
            ceca.dsgd_logreg_grad(A, L, X, Y, k, variant, G, ws)
            ceca.ceca_gossip_sgd_step(X, Y, G, gamma, variant, k)
            og = oracle.logreg_grad(an, ln, ox, oy, k)
            ox, oy = oracle.step(ox, oy, og, np.float32(gamma), variant, k)
            if k % 50 == 49 or k < 8:
                scale = max(np.abs(ox).max(), np.abs(oy).max(), gamma * np.abs(og).max())
                tol = 4e-6 * (k + 1) * scale
                assert np.abs(_np(X) - ox).max() <= tol and np.abs(_np(Y) - oy).max() <= tol, (n, k)
        # the run has moved: the loss of the average model fell well below log 2
        loss = oracle.logreg_loss(an, ln, np.repeat(ox.mean(0, keepdims=True), n, 0)).mean()
        assert loss < 0.55
