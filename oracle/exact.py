"""TEST INFRASTRUCTURE -- not part of the product.

Exact-rational statement of CECA / DSGD-CECA (Python ``fractions``), written separately
from the fp64 C oracle so that the two can be checked against each other and against what
the paper fixes.  Nothing here is used by the CUDA library.

What follows which passage:
  * ``aux_sequence``   -- Sec. 3.1 "Auxiliary variables", Eq. (bin-n-1), Eq. (iter-nr)
  * ``comm_matrix``    -- Eq. (2p-gossip-matrix-d1/d0) and Eq. (1p-gossip-matrix); entry (i, j)
                          is 1 when agent j sends to agent i (Sec. 2.1)
  * ``weights``        -- Algorithm 1
  * ``ceca_round``     -- Sec. 3.1 / Sec. 3.2 "Main recursions", Algorithm 2
  * ``dsgd_step``      -- Eq. (x-iter-dsgd), Eq. (y-iter-dsgd)
  * ``mixing_matrices``-- Eq. (W-Wg-d1), Eq. (W-Wg-d0)

Indices are 0-based: paper agent p is index p-1.
"""
from fractions import Fraction
from functools import lru_cache

VARIANT_1P = 1
VARIANT_2P = 2


@lru_cache(maxsize=None)
def aux_sequence(n):
    """(tau, [delta_0..delta_{tau-1}], [n_0..n_tau]) with n-1 = (delta_0 ... delta_{tau-1})_2."""
    if n < 1:
        raise ValueError("n must be positive")
    digits = [int(ch) for ch in bin(n - 1)[2:]] if n > 1 else []
    tau = len(digits)
    n_seq = [0]
    for delta in digits:
        n_seq.append(2 * n_seq[-1] + delta)
    return tau, tuple(digits), tuple(n_seq)


@lru_cache(maxsize=64)
def comm_matrix(n, variant, r):
    """Dense 0/1 matrix Q^(r) as a list of rows."""
    tau, delta, n_seq = aux_sequence(n)
    if n == 1:
        return ((1,),)
    if variant == VARIANT_1P and n % 2:
        raise ValueError("CECA-1P needs an even number of agents")
    q = [[0] * n for _ in range(n)]
    for i in range(n):
        paper_i = i + 1
        if variant == VARIANT_2P:
            paper_j = paper_i - (n_seq[r] + delta[r])
        elif paper_i % 2 == 1:
            paper_j = paper_i + 2 * n_seq[r] + 1
        else:
            paper_j = paper_i - 2 * n_seq[r] - 1
        j = (paper_j - 1) % n
        q[i][j] = 1
    return tuple(tuple(row) for row in q)


def weights(n, r):
    """(a, b, payload) of Algorithm 1 for round r; payload 0 sends x (or I), 1 sends y (or J)."""
    tau, delta, n_seq = aux_sequence(n)
    if n == 1:
        return Fraction(1), Fraction(1), 0
    nr = n_seq[r]
    if delta[r] == 1:
        return Fraction(1, 2), Fraction(nr, 2 * nr + 1), 0
    return Fraction(nr + 1, 2 * nr + 1), Fraction(1, 2), 1


def _matvec(q, v):
    # q is sparse (one unit entry per row); skipping its zeros changes nothing
    return [sum(q[i][j] * v[j] for j in range(len(v)) if q[i][j]) for i in range(len(q))]


def dsgd_step(x, y, e, gamma, n, variant, k):
    """One iteration on scalar-per-agent lists x, y, e (Fractions).  Returns (x+, y+)."""
    tau, _, _ = aux_sequence(n)
    r = k % tau if tau else 0
    a, b, payload = weights(n, r)
    z = x if payload == 0 else y
    msg = [z[i] - gamma * e[i] for i in range(n)]
    recv = _matvec(comm_matrix(n, variant, r), msg)
    x_new = [a * (x[i] - gamma * e[i]) + (1 - a) * recv[i] for i in range(n)]
    y_new = [b * (y[i] - gamma * e[i]) + (1 - b) * recv[i] for i in range(n)]
    return x_new, y_new


def ceca_round(i_vals, j_vals, n, variant, r):
    """One CECA round written directly from the main recursions (not via dsgd_step)."""
    tau, delta, n_seq = aux_sequence(n)
    nr = n_seq[r]
    q = comm_matrix(n, variant, r)
    if delta[r] == 1:
        got = _matvec(q, i_vals)
        i_new = [Fraction(1, 2) * i_vals[i] + Fraction(1, 2) * got[i] for i in range(n)]
        j_new = [Fraction(nr, 2 * nr + 1) * j_vals[i] + Fraction(nr + 1, 2 * nr + 1) * got[i]
                 for i in range(n)]
    else:
        got = _matvec(q, j_vals)
        i_new = [Fraction(nr + 1, 2 * nr + 1) * i_vals[i] + Fraction(nr, 2 * nr + 1) * got[i]
                 for i in range(n)]
        j_new = [Fraction(1, 2) * j_vals[i] + Fraction(1, 2) * got[i] for i in range(n)]
    return i_new, j_new


def mixing_matrices(n, variant, k):
    """Dense 2n x 2n (W^(k), W_g^(k)) of Eq. (W-Wg-d1) / Eq. (W-Wg-d0) as lists of Fraction rows."""
    tau, delta, n_seq = aux_sequence(n)
    r = k % tau
    nr = n_seq[r]
    p = comm_matrix(n, variant, r)
    half = Fraction(1, 2)
    lo = Fraction(nr, 2 * nr + 1)
    hi = Fraction(nr + 1, 2 * nr + 1)
    eye = [[1 if i == j else 0 for j in range(n)] for i in range(n)]
    zero = [[0] * n for _ in range(n)]

    def comb(c1, m1, c2, m2):
        return [[c1 * m1[i][j] + c2 * m2[i][j] for j in range(n)] for i in range(n)]

    def blocks(b11, b12, b21, b22):
        top = [[Fraction(v) for v in b11[i] + b12[i]] for i in range(n)]
        bot = [[Fraction(v) for v in b21[i] + b22[i]] for i in range(n)]
        return top + bot

    if delta[r] == 1:
        w = blocks(comb(half, eye, half, p), zero, comb(hi, p, 0, eye), comb(lo, eye, 0, eye))
        wg = blocks(comb(half, eye, half, p), zero, comb(lo, eye, hi, p), zero)
    else:
        w = blocks(comb(hi, eye, 0, eye), comb(lo, p, 0, eye), zero, comb(half, eye, half, p))
        wg = blocks(zero, comb(hi, eye, lo, p), zero, comb(half, eye, half, p))
    return w, wg


def matmul(a, b):
    rows, inner, cols = len(a), len(b), len(b[0])
    return [[sum(a[i][t] * b[t][j] for t in range(inner)) for j in range(cols)] for i in range(rows)]
