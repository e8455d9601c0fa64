"""dsgd_logreg_grad_static: the logistic gradient for callers that cannot allocate device memory
(a plug-in whose host owns the device heap, code that must not re-enter an allocator, a loop that
has to stay clear of cudaMalloc).  Its scratch space is a fixed buffer inside the library, so the
call takes no workspace.  It must give what dsgd_logreg_grad gives, call after call, although all
calls share that one buffer and the buffer keeps whatever the previous call left in it.

This file sorts last on purpose: a run that stops at the first failure has then already run
every other test.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2306_00256_b200 as ceca
import synthetic_inputs as synth

DEV = "cuda:0"


def _tol(d, want):
    # the tolerance of the other logistic-gradient tests
    return 8 * np.sqrt(d) * 2.0 ** -24 * np.abs(want).max() + 1e-7


def _problem(n, m, d, seed):
    a, lab, _ = synth.logreg_problem(n, m, d, seed=seed, flip=0.1, hetero_std=0.5)
    gen = torch.Generator().manual_seed(seed + 1)
    x = 0.05 * torch.randn(n, d, generator=gen)
    y = 0.05 * torch.randn(n, d, generator=gen)
    return a, lab, x, y


@pytest.mark.gpu
def test_static_scratch_gradient_matches_workspace_gradient_on_consecutive_calls():
    # two calls in a row with different shapes: the second one finds the first one's partial sums
    # in the shared buffer and must not be disturbed by them (different block counts, a smaller
    # problem after a larger one, then the larger one again)
    cases = [(6, 300, 2048, 1, ceca.CECA_1P), (5, 37, 1028, 2, ceca.CECA_2P), (6, 300, 2048, 3, ceca.CECA_1P),
             (3, 20, 30, 1, ceca.CECA_2P)]   # the last one takes the unaligned fallback kernels
    for n, m, d, k, variant in cases:
        a, lab, x, y = _problem(n, m, d, seed=n + m + d)
        A, L, X, Y = a.to(DEV), lab.to(DEV), x.to(DEV), y.to(DEV)
        ws = torch.empty(ceca.ceca_workspace_bytes(ceca.WS_LOGREG_GRAD, n, m, d), dtype=torch.uint8, device=DEV)
        want_gpu = torch.full((n, d), float("nan"), device=DEV)
        ceca.dsgd_logreg_grad(A, L, X, Y, k, variant, want_gpu, ws)
        for call in range(2):   # twice in a row on the same inputs as well
            got = torch.full((n, d), float("nan"), device=DEV)
            torch.cuda.synchronize()
            free_before = torch.cuda.mem_get_info()[0]
            ceca.dsgd_logreg_grad_static(A, L, X, Y, k, variant, got)
            torch.cuda.synchronize()
            if call == 1 or (n, m, d) != cases[0][:3]:
                # the property in the name: the device has exactly as much free memory after the call as
                # before it (the very first call of a process may still load the kernels' module lazily)
                assert torch.cuda.mem_get_info()[0] == free_before
            want = oracle.logreg_grad(a.numpy(), lab.numpy(), x.numpy(), y.numpy(), k)
            assert np.abs(got.cpu().numpy() - want_gpu.cpu().numpy()).max() <= _tol(d, want)
            assert np.abs(got.cpu().numpy() - want).max() <= _tol(d, want)
            assert torch.equal(got, want_gpu)   # same kernels, same order of additions: same bits


@pytest.mark.gpu
def test_static_scratch_rejects_problems_that_do_not_fit():
    n, m, d = 20, 1000, 8192     # needs ~41 MB of partial sums: more than the built-in 32 MiB
    cap = ceca.dsgd_logreg_grad_static_capacity()
    assert ceca.ceca_workspace_bytes(ceca.WS_LOGREG_GRAD, n, m, d) > cap
    # real, full-size buffers: the call must return before touching them, but nothing is left to chance
    A = torch.zeros(n, m, d, device=DEV); L = torch.ones(n, m, device=DEV)
    X = torch.zeros(n, d, device=DEV); G = torch.full((n, d), 7.0, device=DEV)
    with pytest.raises(ceca.CecaError) as err:
        ceca.dsgd_logreg_grad_static(A, L, X, X, 0, ceca.CECA_2P, G)
    assert err.value.status == 7 and "scratch" in str(err.value)
    torch.cuda.synchronize()
    assert bool((G == 7.0).all())    # nothing was launched


def test_static_scratch_capacity_is_stated():
    assert ceca.dsgd_logreg_grad_static_capacity() == 32 << 20
    # the headline classification workload fits
    assert ceca.ceca_workspace_bytes(ceca.WS_LOGREG_GRAD, 63, 2000, 4096) <= 32 << 20
