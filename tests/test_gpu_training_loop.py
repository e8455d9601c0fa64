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
