"""Pins of the oracle against what the paper and the mathematics fix (CPU only).

Each test names the passage it takes its expected values from.  None of the expected
values comes from the oracle itself or from the CUDA library.
"""
import math
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle
from oracle import exact

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
V = {"1P": oracle.VARIANT_1P, "2P": oracle.VARIANT_2P}


def _load_example():
    table = {}
    for line in open(os.path.join(GOLDEN, "ceca_example_n6.txt")):
        if line.startswith("#") or not line.strip():
            continue
        parts = line.split()
        vals = [Fraction(p) for p in parts[2:]]
        table[(parts[0], int(parts[1]))] = (vals[0::2], vals[1::2])
    return table


def _load_aux():
    out = {}
    for line in open(os.path.join(GOLDEN, "aux_sequence.txt")):
        if line.startswith("#") or not line.strip():
            continue
        parts = line.split()
        out[parts[0]] = parts[1:]
    return out


# ---- Appendix B.1, Table "CECA_example": the printed worked example -----------------------

@pytest.mark.parametrize("name", ["2P", "1P"])
def test_worked_example_exact_recursions(name):
    table = _load_example()
    i_vals, j_vals = table[(name, 0)]
    for r in range(3):
        i_vals, j_vals = exact.ceca_round(i_vals, j_vals, 6, V[name], r)
        want_i, want_j = table[(name, r + 1)]
        assert i_vals == want_i, (name, r, i_vals)
        assert j_vals == want_j, (name, r, j_vals)


@pytest.mark.parametrize("name", ["2P", "1P"])
def test_worked_example_exact_dsgd_form_with_zero_step(name):
    table = _load_example()
    x, y = table[(name, 0)]
    zeros = [Fraction(0)] * 6
    for k in range(3):
        x, y = exact.dsgd_step(x, y, zeros, Fraction(1, 7), 6, V[name], k)
        assert (x, y) == table[(name, k + 1)]


@pytest.mark.parametrize("name", ["2P", "1P"])
def test_worked_example_fp64_oracle(name):
    table = _load_example()
    x = np.array([float(v) for v in table[(name, 0)][0]]).reshape(6, 1)
    y = np.array([float(v) for v in table[(name, 0)][1]]).reshape(6, 1)
    for k in range(3):
        x, y = oracle.step(x, y, None, 0.0, V[name], k)
        want_i, want_j = table[(name, k + 1)]
        np.testing.assert_allclose(x.ravel(), [float(v) for v in want_i], rtol=0, atol=1e-14)
        np.testing.assert_allclose(y.ravel(), [float(v) for v in want_j], rtol=0, atol=1e-14)
    # the whole run in one call
    x0 = np.arange(1.0, 7.0).reshape(6, 1)
    xc, yc = oracle.consensus(x0, np.zeros((6, 1)), V[name], 0, 3)
    np.testing.assert_allclose(xc, x, rtol=0, atol=0)
    np.testing.assert_allclose(yc, y, rtol=0, atol=0)


# ---- Sec. 3.1 "Auxiliary variables" and the 1-port example's matchings ----------------------

def test_aux_sequence_and_matchings_n6():
    g = _load_aux()
    n = int(g["n"][0])
    tau, delta, n_seq = exact.aux_sequence(n)
    assert tau == int(g["tau"][0])
    assert list(delta) == [int(v) for v in g["delta"]]
    assert list(n_seq) == [int(v) for v in g["n_seq"]]
    for r in range(tau):
        rd = oracle.round_info(n, r)
        assert (rd.tau, rd.r, rd.delta, rd.n_r) == (tau, r, delta[r], n_seq[r])
        want = set()
        for pair in g["pairs_round%d" % r]:
            p, q = (int(v) - 1 for v in pair.split("-"))
            want.add((p, q))
            want.add((q, p))
        recv, send = oracle.peers(n, oracle.VARIANT_1P, r)
        assert {(i, int(recv[i])) for i in range(n)} == want
        assert {(i, int(send[i])) for i in range(n)} == want
        q = exact.comm_matrix(n, exact.VARIANT_1P, r)
        assert {(i, j) for i in range(n) for j in range(n) if q[i][j]} == want


def test_two_port_direction_n6():
    # Appendix B.1: in round r agent i receives from agent i - n_r - delta_r (indices wrap).
    # Round 0 of the printed example: I_1 becomes (u_1 + u_6) / 2 = 3.5, so agent 1 hears agent 6.
    recv, send = oracle.peers(6, oracle.VARIANT_2P, 0)
    assert recv[0] == 5 and send[5] == 0
    shifts = [1, 1, 3]  # n_r + delta_r for (n_r, delta_r) = (0,1), (1,0), (2,1)
    for r, s in enumerate(shifts):
        recv, send = oracle.peers(6, oracle.VARIANT_2P, r)
        assert list(recv) == [(i - s) % 6 for i in range(6)]
        assert list(send) == [(i + s) % 6 for i in range(6)]


def test_n_tau_is_n_minus_one_and_tau_is_ceil_log2():
    # Sec. 3.1: "n_tau = n - 1"; tau = ceil(log2 n)
    for n in list(range(2, 3000)) + [2**20 - 1, 2**20, 2**20 + 1, 2**30 + 7]:
        tau, delta, n_seq = exact.aux_sequence(n)
        assert n_seq[-1] == n - 1
        assert delta[0] == 1
        assert 2 ** (tau - 1) < n <= 2 ** tau
        rd = oracle.round_info(n, tau - 1)
        assert rd.tau == tau and 2 * rd.n_r + rd.delta == n - 1


def test_round_index_wraps_with_period_tau():
    # Algorithm 1: r = k mod tau, also for very large k
    for n in (2, 3, 6, 97, 100, 1026):
        tau, delta, n_seq = exact.aux_sequence(n)
        for k in (0, 1, tau, tau + 1, 5 * tau + 2, 2**31 + 5, 2**40 + 3):
            rd = oracle.round_info(n, k)
            r = k % tau
            assert (rd.r, rd.delta, rd.n_r) == (r, delta[r], n_seq[r])


def test_weights_follow_algorithm_1():
    for n in range(2, 200):
        tau, delta, n_seq = exact.aux_sequence(n)
        for r in range(tau):
            rd = oracle.round_info(n, r)
            a, b, payload = exact.weights(n, r)
            assert Fraction(rd.a_num, rd.a_den) == a and Fraction(rd.b_num, rd.b_den) == b
            assert rd.payload == payload == 1 - delta[r]
            assert rd.a == float(a) and rd.b == float(b)
            if delta[r] == 1:
                assert a == Fraction(1, 2) and b == Fraction(n_seq[r], 2 * n_seq[r] + 1)
            else:
                assert a == Fraction(n_seq[r] + 1, 2 * n_seq[r] + 1) and b == Fraction(1, 2)
        assert exact.weights(n, 0)[1] == 0  # n_0 = 0: y carries no weight in round 0


# ---- Sec. 3.1 / 3.2 "Communication patterns": permutation, symmetry, one peer per agent ------

@pytest.mark.parametrize("n", list(range(2, 70)) + [97, 100, 130, 258, 1026])
def test_comm_matrix_is_a_permutation(n):
    tau, _, _ = exact.aux_sequence(n)
    for r in range(tau):
        for variant in (oracle.VARIANT_2P, oracle.VARIANT_1P):
            if variant == oracle.VARIANT_1P and n % 2:
                with pytest.raises(oracle.OracleError) as err:
                    oracle.peers(n, variant, r)
                assert err.value.code == oracle.ERR_ODD_N_1P
                continue
            recv, send = oracle.peers(n, variant, r)
            assert sorted(recv) == list(range(n)) and sorted(send) == list(range(n))
            assert all(send[recv[i]] == i for i in range(n))
            assert all(recv[i] != i for i in range(n))          # nobody talks to itself
            if variant == oracle.VARIANT_1P:
                assert all(recv[i] == send[i] for i in range(n))  # symmetric: a perfect matching
                assert all(recv[recv[i]] == i for i in range(n))
            if n <= 70:
                q = exact.comm_matrix(n, variant, r)
                assert [row.index(1) for row in q] == list(recv)
                assert all(sum(row) == 1 for row in q)
                if variant == oracle.VARIANT_1P:
                    assert all(q[i][j] == q[j][i] for i in range(n) for j in range(n))


# ---- Sec. 3.1 Eq. (z7u23bn) / Appendix B.1: window averages after every round ----------------

@pytest.mark.parametrize("n", list(range(2, 41)))
def test_window_average_closed_form(n):
    tau, delta, n_seq = exact.aux_sequence(n)
    u = [Fraction(3 * i * i - 7 * i + 2, 5) for i in range(n)]     # any distinct values
    for variant in (exact.VARIANT_2P, exact.VARIANT_1P):
        if variant == exact.VARIANT_1P and n % 2:
            continue
        i_vals, j_vals = list(u), [Fraction(0)] * n
        for r in range(tau):
            i_vals, j_vals = exact.ceca_round(i_vals, j_vals, n, variant, r)
            w = n_seq[r + 1]
            for i in range(n):
                # 2-port: every agent looks backwards; 1-port: paper-odd agents (even index)
                # look forwards, paper-even agents backwards (Appendix B.1, 1-port part)
                sign = 1 if (variant == exact.VARIANT_1P and i % 2 == 0) else -1
                win = [u[(i + sign * t) % n] for t in range(w + 1)]
                assert i_vals[i] == sum(win) / (w + 1)
                assert j_vals[i] == sum(win[1:]) / w
        assert all(v == sum(u) / n for v in i_vals)
        assert all(j_vals[i] == (sum(u) - u[i]) / (n - 1) for i in range(n))


# ---- Lemma "matrix consensus" (Appendix B.2): products of tau and of tau+1.. mixing matrices ---

def _apply_rounds_to_basis(n, variant, k_first, count, checkpoints=None):
    """Rows of the product of `count` mixing matrices, obtained by pushing every unit vector of
    R^{2n} through the exact DSGD step with a zero gradient.  With `checkpoints`, a dict
    {number of factors: product} is returned instead."""
    wanted = sorted(checkpoints) if checkpoints else [count]
    cols = {c: [] for c in wanted}
    zeros = [Fraction(0)] * n
    for basis in range(2 * n):
        x = [Fraction(int(basis == i)) for i in range(n)]
        y = [Fraction(int(basis == n + i)) for i in range(n)]
        for t in range(wanted[-1]):
            x, y = exact.dsgd_step(x, y, zeros, Fraction(0), n, variant, k_first + t)
            if t + 1 in cols:
                cols[t + 1].append(x + y)
    prods = {c: [[cols[c][col][row] for col in range(2 * n)] for row in range(2 * n)] for c in wanted}
    return prods if checkpoints else prods[count]


@pytest.mark.parametrize("n", list(range(2, 65)))
def test_product_lemma_exact(n):
    tau, _, _ = exact.aux_sequence(n)
    for variant in (exact.VARIANT_2P, exact.VARIANT_1P):
        if variant == exact.VARIANT_1P and n % 2:
            continue
        prods = _apply_rounds_to_basis(n, variant, 0, None, checkpoints={tau, tau + 1, tau + 2, 2 * tau})
        prod = prods[tau]
        for i in range(n):
            assert prod[i] == [Fraction(1, n)] * n + [0] * n
            assert prod[n + i] == [0 if j == i else Fraction(1, n - 1) for j in range(n)] + [0] * n
        for count in (tau + 1, tau + 2, 2 * tau):
            if count == tau:
                continue
            for i in range(2 * n):
                assert prods[count][i] == [Fraction(1, n)] * n + [0] * n


@pytest.mark.parametrize("n", [2, 3, 4, 5, 6, 7, 8, 11, 12])
def test_dense_mixing_matrices(n):
    """Eq. (W-Wg-d1/d0) multiplied out densely agree with the row-wise exact step (brute force),
    rows of W sum to one, and W commutes with block averaging (Lemma "matrix family")."""
    tau, _, _ = exact.aux_sequence(n)
    avg = [[Fraction(1, n) if (i < n) == (j < n) else 0 for j in range(2 * n)] for i in range(2 * n)]
    for variant in (exact.VARIANT_2P, exact.VARIANT_1P):
        if variant == exact.VARIANT_1P and n % 2:
            continue
        prod = None
        for k in range(tau + 1):
            w, wg = exact.mixing_matrices(n, variant, k)
            assert all(sum(row) == 1 for row in w)
            assert exact.matmul(w, avg) == exact.matmul(avg, w)
            prod = w if prod is None else exact.matmul(w, prod)
            assert prod == _apply_rounds_to_basis(n, variant, 0, k + 1)
            # one step with gradients: [x;y]+ = W [x;y] - gamma W_g [g;h]
            x = [Fraction(7 * i + 1, 3) for i in range(n)]
            y = [Fraction(2 - 5 * i, 7) for i in range(n)]
            g = [Fraction(i * i + 1, 11) for i in range(n)]
            h = [Fraction(3 - i, 13) for i in range(n)]
            gamma = Fraction(3, 10)
            a, b, payload = exact.weights(n, k % tau)
            e = g if payload == 0 else h
            x1, y1 = exact.dsgd_step(x, y, e, gamma, n, variant, k)
            col = [[v] for v in x + y]
            gcol = [[v] for v in g + h]
            lhs = exact.matmul(w, col)
            rhs = exact.matmul(wg, gcol)
            dense = [lhs[i][0] - gamma * rhs[i][0] for i in range(2 * n)]
            assert dense == x1 + y1


@pytest.mark.parametrize("n,variant", [(5, 2), (6, 1), (6, 2), (8, 2), (7, 2), (8, 1)])
def test_fp64_oracle_matches_dense_matrices(n, variant):
    """The C oracle's step equals the stacked dense form built from Eq. (W-Wg-d1/d0)."""
    rng = np.random.default_rng(11)
    d = 5
    x, y = rng.normal(size=(n, d)), rng.normal(size=(n, d))
    tau, _, _ = exact.aux_sequence(n)
    gamma = 0.3
    for k in range(2 * tau + 1):
        g, h = rng.normal(size=(n, d)), rng.normal(size=(n, d))
        w, wg = exact.mixing_matrices(n, variant, k)
        w = np.array([[float(v) for v in row] for row in w])
        wg = np.array([[float(v) for v in row] for row in wg])
        e = g if oracle.round_info(n, k).payload == 0 else h
        dense = w @ np.vstack([x, y]) - gamma * wg @ np.vstack([g, h])
        x1, y1 = oracle.step(x, y, e, gamma, variant, k)
        np.testing.assert_allclose(np.vstack([x1, y1]), dense, rtol=0, atol=1e-13)
        x, y = x1, y1


def test_fp64_oracle_matches_exact_twin_on_schedules():
    for n in range(1, 260):
        tau, delta, n_seq = exact.aux_sequence(n)
        for r in range(max(tau, 1)):
            for variant in (1, 2):
                if variant == 1 and n % 2 and n > 1:
                    continue
                recv, send = oracle.peers(n, variant, r)
                q = exact.comm_matrix(n, variant, r)
                assert [row.index(1) for row in q] == list(recv)


@pytest.mark.parametrize("n,variant", [(97, 2), (100, 1), (100, 2), (24, 1), (63, 2), (130, 1), (258, 2)])
def test_fp64_consensus_reaches_the_mean(n, variant):
    rng = np.random.default_rng(n)
    x0 = rng.normal(size=(n, 3)) + np.arange(n)[:, None]
    tau = exact.aux_sequence(n)[0]
    x, y = oracle.consensus(x0, np.zeros_like(x0), variant, 0, tau)
    mean = x0.mean(axis=0)
    np.testing.assert_allclose(x, np.broadcast_to(mean, x.shape), rtol=1e-14, atol=1e-13)
    loo = (x0.sum(axis=0)[None, :] - x0) / (n - 1)
    np.testing.assert_allclose(y, loo, rtol=1e-14, atol=1e-13)
    x2, y2 = oracle.consensus(x0, rng.normal(size=x0.shape), variant, 0, tau + 1)
    np.testing.assert_allclose(y2, np.broadcast_to(mean, x.shape), rtol=1e-14, atol=1e-13)
    np.testing.assert_allclose(x2, np.broadcast_to(mean, x.shape), rtol=1e-14, atol=1e-13)
    # a window of tau rounds that does not start at a multiple of tau is NOT an average of x
    x3, _ = oracle.consensus(x0, x0, variant, 1, tau)
    assert np.abs(x3 - mean).max() > 1e-3


# ---- Lemma "relation between averaged variables": the mean takes a plain SGD step -----------

@pytest.mark.parametrize("n,variant", [(5, 2), (6, 1), (24, 1), (63, 2), (100, 2), (100, 1)])
def test_mean_lemma(n, variant):
    rng = np.random.default_rng(5)
    d = 4
    x = rng.normal(size=(n, d))
    y = x.copy()
    gamma = 0.05
    for k in range(25):
        e = rng.normal(size=(n, d))
        x1, y1 = oracle.step(x, y, e, gamma, variant, k)
        np.testing.assert_allclose(x1.mean(0), x.mean(0) - gamma * e.mean(0), rtol=0, atol=1e-13)
        np.testing.assert_allclose(y1.mean(0), x1.mean(0), rtol=0, atol=1e-13)
        x, y = x1, y1


# ---- n = 2^tau: CECA-2P is the one-peer exponential graph (Sec. 1, contributions) -----------

@pytest.mark.parametrize("tau", [1, 2, 3, 5, 7])
def test_power_of_two_reduces_to_one_peer_exponential(tau):
    n = 2 ** tau
    rng = np.random.default_rng(tau)
    x = rng.normal(size=(n, 3))
    y = rng.normal(size=(n, 3))
    g = rng.normal(size=(n, 3))
    for k in range(2 * tau):
        rd = oracle.round_info(n, k)
        assert rd.delta == 1 and rd.a == 0.5 and rd.n_r == 2 ** (k % tau) - 1
        x1, y1 = oracle.step(x, y, g, 0.1, oracle.VARIANT_2P, k)
        u = x - 0.1 * g
        np.testing.assert_allclose(x1, 0.5 * (u + np.roll(u, 2 ** (k % tau), axis=0)), rtol=0, atol=1e-14)
        x, y = x1, y1


def test_single_agent_degenerates_to_plain_sgd():
    # reading for the case the paper leaves out (n = 1): no peer, both models take the step
    x = np.array([[1.0, 2.0]]); y = np.array([[3.0, -1.0]]); g = np.array([[0.5, 0.25]])
    x1, y1 = oracle.step(x, y, g, 0.1, oracle.VARIANT_2P, 4)
    np.testing.assert_allclose(x1, x - 0.1 * g)
    np.testing.assert_allclose(y1, y - 0.1 * g)
    assert oracle.round_info(1, 9).tau == 0


# ---- logistic gradient: not in the paper; pinned by calculus and hand cases --------------------

def test_logreg_hand_cases():
    # one agent, one sample, one feature: grad = -l * sigma(-l a w) * a
    a = np.array([[[2.0]]]); lab = np.array([[1.0]])
    g0 = oracle.logreg_grad(a, lab, np.array([[0.0]]), np.array([[9.0]]), 0)
    assert g0[0, 0] == pytest.approx(-1.0, abs=1e-15)
    g1 = oracle.logreg_grad(a, lab, np.array([[1.0]]), np.array([[9.0]]), 0)
    assert g1[0, 0] == pytest.approx(-2.0 / (1.0 + math.exp(2.0)), abs=1e-15)
    gneg = oracle.logreg_grad(a, -lab, np.array([[1.0]]), np.array([[9.0]]), 0)
    assert gneg[0, 0] == pytest.approx(2.0 / (1.0 + math.exp(-2.0)), abs=1e-15)
    # two samples average
    a2 = np.array([[[1.0], [3.0]]]); l2 = np.array([[1.0, -1.0]])
    g2 = oracle.logreg_grad(a2, l2, np.array([[0.0]]), np.array([[0.0]]), 0)
    assert g2[0, 0] == pytest.approx(0.5 * (-0.5 * 1.0 + 0.5 * 3.0), abs=1e-15)


def test_logreg_gradient_is_the_derivative_of_the_loss():
    rng = np.random.default_rng(3)
    n, m, d = 3, 17, 6
    a = rng.normal(size=(n, m, d)); lab = np.where(rng.random((n, m)) < 0.5, -1.0, 1.0)
    w = rng.normal(size=(n, d))
    grad = oracle.logreg_grad(a, lab, w, w, 0)

    def loss(wm):  # written with a library routine, independently of the oracle's own loss
        t = np.einsum("nmd,nd->nm", a, wm)
        return np.logaddexp(0.0, -lab * t).mean(axis=1)

    np.testing.assert_allclose(oracle.logreg_loss(a, lab, w), loss(w), rtol=1e-13)
    h = 1e-6
    for i in range(n):
        for c in range(d):
            wp, wm = w.copy(), w.copy()
            wp[i, c] += h; wm[i, c] -= h
            fd = (loss(wp)[i] - loss(wm)[i]) / (2 * h)
            assert grad[i, c] == pytest.approx(fd, abs=2e-9)


def test_logreg_uses_the_model_algorithm_1_selects():
    rng = np.random.default_rng(4)
    n, m, d = 6, 9, 4      # n = 6: delta = (1, 0, 1), so k = 1 evaluates at y
    a = rng.normal(size=(n, m, d)); lab = np.where(rng.random((n, m)) < 0.5, -1.0, 1.0)
    x = rng.normal(size=(n, d)); y = rng.normal(size=(n, d))
    np.testing.assert_array_equal(oracle.logreg_grad(a, lab, x, y, 0), oracle.logreg_grad(a, lab, x, x, 0))
    np.testing.assert_array_equal(oracle.logreg_grad(a, lab, x, y, 1), oracle.logreg_grad(a, lab, y, y, 0))
    np.testing.assert_array_equal(oracle.logreg_grad(a, lab, x, y, 2), oracle.logreg_grad(a, lab, x, x, 0))


# ---- least-squares gradient (Sec. 5 "DSGD: least-squares problem") ------------------------------

def test_lsq_gradient_vanishes_at_the_least_squares_solution_and_matches_differences():
    rng = np.random.default_rng(8)
    n, m, d = 4, 50, 10
    a = rng.normal(size=(n, m, d)); b = rng.normal(size=(n, m))
    # at the minimiser of each f_i (library routine) the gradient is zero
    w_ls = np.stack([np.linalg.lstsq(a[i], b[i], rcond=None)[0] for i in range(n)])
    g = oracle.lsq_grad(a, b, w_ls, w_ls, 0)
    assert np.abs(g).max() < 1e-10
    # elsewhere it is the derivative of (1/2)||A w - b||^2, and the noise is simply added
    w = rng.normal(size=(n, d)); eps = rng.normal(size=(n, d))
    g = oracle.lsq_grad(a, b, w, w, 0)
    loss = lambda wm: 0.5 * ((np.einsum("nmd,nd->nm", a, wm) - b) ** 2).sum(axis=1)
    h = 1e-5
    for i in range(n):
        for c in range(d):
            wp, wm = w.copy(), w.copy(); wp[i, c] += h; wm[i, c] -= h
            assert g[i, c] == pytest.approx((loss(wp)[i] - loss(wm)[i]) / (2 * h), rel=1e-7, abs=1e-7)
    np.testing.assert_allclose(oracle.lsq_grad(a, b, w, w, 0, noise=eps), g + eps, rtol=0, atol=1e-12)
    # hand case: one sample, one feature: a (a w - b)
    assert oracle.lsq_grad([[[3.0]]], [[2.0]], [[1.5]], [[0.0]], 0)[0, 0] == pytest.approx(3.0 * (4.5 - 2.0))
    # the model is the one Algorithm 1 selects (n = 6: round 1 evaluates at y)
    a6 = rng.normal(size=(6, 5, 3)); b6 = rng.normal(size=(6, 5)); x6 = rng.normal(size=(6, 3)); y6 = rng.normal(size=(6, 3))
    np.testing.assert_array_equal(oracle.lsq_grad(a6, b6, x6, y6, 1), oracle.lsq_grad(a6, b6, y6, y6, 0))
    np.testing.assert_array_equal(oracle.lsq_grad(a6, b6, x6, y6, 2), oracle.lsq_grad(a6, b6, x6, x6, 0))
