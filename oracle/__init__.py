"""TEST INFRASTRUCTURE -- not part of the product.

ctypes front end of the plain-C fp64 oracle (``ceca_oracle.c``) plus the exact-rational
twin (``exact.py``).  Only tests, the smoke check and the benchmark's CPU-baseline leg may
import this package; the CUDA library never does.

Inputs are taken as whatever the caller holds (normally the fp32 bytes the GPU path also
reads) and widened to fp64 exactly; all arithmetic and all results are fp64.
"""
import ctypes
import os

import numpy as np

from . import build as _build
from . import exact  # noqa: F401  (re-exported)

VARIANT_1P = 1
VARIANT_2P = 2

OK, ERR_ARG, ERR_ODD_N_1P = 0, 1, 2


class OracleError(ValueError):
    def __init__(self, code):
        super().__init__({ERR_ARG: "invalid argument", ERR_ODD_N_1P: "CECA-1P needs even n"}.get(code, str(code)))
        self.code = code


class Round(ctypes.Structure):
    _fields_ = [("n", ctypes.c_int32), ("tau", ctypes.c_int32), ("r", ctypes.c_int32),
                ("delta", ctypes.c_int32), ("n_r", ctypes.c_int32), ("payload", ctypes.c_int32),
                ("a_num", ctypes.c_int32), ("a_den", ctypes.c_int32),
                ("b_num", ctypes.c_int32), ("b_den", ctypes.c_int32),
                ("a", ctypes.c_double), ("b", ctypes.c_double)]


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(_build.build())
        dp = ctypes.POINTER(ctypes.c_double)
        ip = ctypes.POINTER(ctypes.c_int32)
        _lib.ceca_oracle_round.argtypes = [ctypes.c_int32, ctypes.c_int64, ctypes.POINTER(Round)]
        _lib.ceca_oracle_peers.argtypes = [ctypes.c_int32, ctypes.c_int32, ctypes.c_int64, ip, ip]
        _lib.ceca_oracle_step.argtypes = [dp, dp, dp, ctypes.c_double, ctypes.c_int32, ctypes.c_int64,
                                          ctypes.c_int32, ctypes.c_int64, dp, dp]
        _lib.ceca_oracle_consensus.argtypes = [dp, dp, ctypes.c_int32, ctypes.c_int64, ctypes.c_int32,
                                               ctypes.c_int64, ctypes.c_int32]
        _lib.ceca_oracle_logreg_grad.argtypes = [dp, dp, dp, dp, ctypes.c_int64, dp, ctypes.c_int32,
                                                 ctypes.c_int32, ctypes.c_int64]
        _lib.ceca_oracle_lsq_grad.argtypes = [dp, dp, dp, dp, dp, ctypes.c_int64, dp, ctypes.c_int32,
                                              ctypes.c_int32, ctypes.c_int64]
        _lib.ceca_oracle_logreg_loss.argtypes = [dp, dp, dp, dp, ctypes.c_int32, ctypes.c_int32,
                                                 ctypes.c_int64]
    return _lib


def _check(code):
    if code != OK:
        raise OracleError(code)


def _f64(a):
    return np.ascontiguousarray(np.asarray(a), dtype=np.float64)


def _dp(a):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


def round_info(n, k):
    rd = Round()
    _check(lib().ceca_oracle_round(n, k, ctypes.byref(rd)))
    return rd


def peers(n, variant, k):
    """(recv_from, send_to) as int32 arrays: agent i receives from recv_from[i], sends to send_to[i]."""
    recv = np.empty(n, dtype=np.int32)
    send = np.empty(n, dtype=np.int32)
    ip = ctypes.POINTER(ctypes.c_int32)
    _check(lib().ceca_oracle_peers(n, variant, k, recv.ctypes.data_as(ip), send.ctypes.data_as(ip)))
    return recv, send


def step(X, Y, E, gamma, variant, k):
    """One DSGD-CECA iteration; E may be None (pure CECA round).  Returns fp64 (X+, Y+)."""
    X, Y = _f64(X), _f64(Y)
    n, d = X.shape
    E64 = None if E is None else _f64(E)
    Xo, Yo = np.empty_like(X), np.empty_like(Y)
    _check(lib().ceca_oracle_step(_dp(X), _dp(Y), None if E64 is None else _dp(E64), float(gamma),
                                  n, d, variant, k, _dp(Xo), _dp(Yo)))
    return Xo, Yo


def consensus(X, Y, variant, k0, rounds):
    """`rounds` CECA rounds starting at iteration index k0.  Returns fp64 (X, Y)."""
    X, Y = _f64(X).copy(), _f64(Y).copy()
    n, d = X.shape
    _check(lib().ceca_oracle_consensus(_dp(X), _dp(Y), n, d, variant, k0, rounds))
    return X, Y


def logreg_grad(A, labels, X, Y, k):
    """Per-agent logistic gradient at the model Algorithm 1 selects in iteration k."""
    A, labels, X, Y = _f64(A), _f64(labels), _f64(X), _f64(Y)
    n, m, d = A.shape
    G = np.empty((n, d), dtype=np.float64)
    _check(lib().ceca_oracle_logreg_grad(_dp(A), _dp(labels), _dp(X), _dp(Y), k, _dp(G), n, m, d))
    return G


def logreg_loss(A, labels, W):
    A, labels, W = _f64(A), _f64(labels), _f64(W)
    n, m, d = A.shape
    out = np.empty(n, dtype=np.float64)
    _check(lib().ceca_oracle_logreg_loss(_dp(A), _dp(labels), _dp(W), _dp(out), n, m, d))
    return out


def lsq_grad(A, B, X, Y, k, noise=None):
    """Per-agent least-squares gradient A_i^T (A_i z_i - b_i) (+ noise) at the model iteration k selects."""
    A, B, X, Y = _f64(A), _f64(B), _f64(X), _f64(Y)
    n, m, d = A.shape
    N = None if noise is None else _f64(noise)
    G = np.empty((n, d), dtype=np.float64)
    _check(lib().ceca_oracle_lsq_grad(_dp(A), _dp(B), _dp(X), _dp(Y), None if N is None else _dp(N), k, _dp(G),
                                      n, m, d))
    return G


def set_threads(t):
    """Number of OpenMP threads the C oracle uses (the loops over agents carry a pragma)."""
    os.environ["OMP_NUM_THREADS"] = str(t)
    try:
        omp = ctypes.CDLL("libgomp.so.1")
        omp.omp_set_num_threads(int(t))
    except OSError:
        pass
