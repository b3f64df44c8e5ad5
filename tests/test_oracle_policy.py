"""Pins for the oracle's policy generator (Algorithm 3, Eq. 8-14, Eq. 22, Lemmas 1-2, Theorem 3)."""
import numpy as np
import pytest
from scipy.optimize import linprog

from oracle import policy
from paper_2009_05766_b200 import workloads


def _case(name):
    if name == "cfg1":
        w = workloads.config(1)
        return policy.iteration_times(w.link_speeds(0), w.d) + (w.lr, 20, 20)
    if name == "cfg2":
        w = workloads.config(2)
        return policy.iteration_times(w.link_speeds(0), w.d) + (w.lr, 10, 10)
    if name == "cfg3":
        w = workloads.config(3)
        return policy.iteration_times(w.link_speeds(0), w.d) + (w.lr, 6, 6)
    if name == "sparse7":
        rng = np.random.default_rng(5)
        M = 7
        s = np.exp(rng.uniform(np.log(1.0), np.log(50.0), (M, M)))
        s = np.triu(s, 1)
        s[0, 4] = s[1, 5] = s[2, 6] = 0.0      # missing links (d_im = 0)
        s = s + s.T
        return policy.iteration_times(s, 1_000_000) + (0.05, 8, 8)
    raise KeyError(name)


CASES = ["cfg1", "cfg2", "cfg3", "sparse7"]


@pytest.fixture(scope="module", params=CASES)
def solved(request):
    t, adj, alpha, K, R = _case(request.param)
    P, rho, info = policy.generate_policy(t, adj, alpha, K, R)
    return dict(t=t, adj=adj, alpha=alpha, P=P, rho=rho, info=info, M=t.shape[0])


def test_constraints_eq_10_to_13(solved):
    P, t, adj, a, rho, M = (solved[k] for k in ("P", "t", "adj", "alpha", "rho", "M"))
    off = ~np.eye(M, dtype=bool)
    np.testing.assert_allclose(P.sum(axis=1), 1.0, atol=1e-12)                       # Eq. 13
    assert (P >= 0).all() and (P[(adj == 0) & off] == 0).all()                       # Eq. 12
    floor = a * rho * (adj + adj.T)
    assert (P[(adj == 1)] >= floor[(adj == 1)] * (1 - 1e-9)).all()                   # Eq. 11 (closed)
    tbar_i = (t * P * (adj + np.eye(M))).sum(axis=1)                                 # Eq. 2 with d_ii = 1
    np.testing.assert_allclose(tbar_i, M * solved["info"]["tbar"], rtol=1e-8)        # Eq. 10
    np.testing.assert_allclose(policy.node_probabilities(P, t, adj), 1.0 / M, rtol=1e-8)   # Lemma 1


def test_y_matrix_lemmas_and_theorem_3(solved):
    P, t, adj, a, rho, M = (solved[k] for k in ("P", "t", "adj", "alpha", "rho", "M"))
    Y = policy.y_matrix(P, policy.node_probabilities(P, t, adj), adj, a, rho)
    np.testing.assert_allclose(Y, Y.T, atol=1e-12)                  # Lemma 1: symmetric
    np.testing.assert_allclose(Y.sum(axis=1), 1.0, atol=1e-9)       # Lemma 1: rows sum to 1
    assert (Y >= -1e-15).all()                                       # Lemma 2: non-negative
    lam = np.linalg.eigvalsh(Y)
    assert lam[-1] == pytest.approx(1.0, abs=1e-9)                   # Theorem 3
    assert lam[-2] < 1.0 - 1e-9
    assert lam[-2] == pytest.approx(solved["info"]["lam2"], abs=1e-10)
    if (adj + np.eye(M) == 1).all():                                 # fully connected: appendix bounds
        assert a * rho <= 1.0 / (2 * (M - 1))
        assert lam[-2] >= (M - 3) / (M - 1) - 1e-12


def test_y_matrix_equals_exact_expectation_of_DtD():
    """Enumerate the paper's one-worker-per-step process: worker i acts with probability p_i
    (Eq. 3), picks m with probability p_im, D = I + alpha*rho*gamma_im e_i (e_m - e_i)^T."""
    rng = np.random.default_rng(7)
    M, alpha, rho = 5, 0.1, 0.4
    P = rng.random((M, M)) + 0.1
    adj = (1 - np.eye(M)).astype(np.uint8)
    adj[1, 3] = adj[3, 1] = 0
    P[1, 3] = P[3, 1] = 0.0
    P /= P.sum(axis=1, keepdims=True)
    t = rng.uniform(1.0, 5.0, (M, M))
    p_node = policy.node_probabilities(P, t, adj)       # not uniform: P is not a feasible solution
    assert p_node.std() > 1e-3
    acc = np.zeros((M, M))
    for i in range(M):
        for m in range(M):
            D = np.eye(M)
            if m != i and P[i, m] > 0:
                g = (adj[i, m] + adj[m, i]) / (2 * P[i, m])
                e = np.zeros(M); e[m] = 1.0; e[i] -= 1.0
                D[i] += alpha * rho * g * e
            acc += p_node[i] * P[i, m] * (D.T @ D)
    np.testing.assert_allclose(policy.y_matrix(P, p_node, adj, alpha, rho), acc, atol=1e-13)


def test_lp_optimum_value_matches_an_independent_lp_solver(solved):
    """Eq. 14 at the selected (rho, t_bar): the row-wise solution reaches HiGHS's minimum of sum_i p_ii."""
    P, t, adj, a, rho, M = (solved[k] for k in ("P", "t", "adj", "alpha", "rho", "M"))
    T = M * solved["info"]["tbar"]
    n = M * M
    cost = np.eye(M).reshape(n)
    A_eq, b_eq = [], []
    for i in range(M):
        r1 = np.zeros((M, M)); r1[i] = 1.0
        r2 = np.zeros((M, M)); r2[i] = t[i] * (adj[i] + (np.arange(M) == i))
        A_eq += [r1.reshape(n), r2.reshape(n)]
        b_eq += [1.0, T]
    lo = (a * rho * (adj + adj.T) * adj).astype(np.float64)
    hi = np.where((adj == 1) | np.eye(M, dtype=bool), 1.0, 0.0)
    scale = 1.0 / t.max()
    A = np.array(A_eq); b = np.array(b_eq)
    A[1::2] *= scale; b[1::2] *= scale
    res = linprog(cost, A_eq=A, b_eq=b, bounds=list(zip(lo.reshape(n), hi.reshape(n))), method="highs")
    assert res.status == 0
    assert np.trace(P) == pytest.approx(res.fun, abs=1e-7)


def test_homogeneous_network_gives_uniform_neighbour_choice():
    M = 6
    t, adj = policy.iteration_times(np.full((M, M), 25.0) - 25.0 * np.eye(M), 1_000_000)
    P, rho, _ = policy.generate_policy(t, adj, 0.1, 8, 8)
    off = ~np.eye(M, dtype=bool)
    assert np.ptp(P[off]) < 1e-12
    assert np.ptp(np.diag(P)) < 1e-12


def test_faster_links_are_not_chosen_less_often(solved):
    P, t, adj, M = (solved[k] for k in ("P", "t", "adj", "M"))
    for i in range(M):
        nb = [m for m in range(M) if m != i and adj[i, m]]
        order = sorted(nb, key=lambda m: t[i, m])
        probs = P[i, order]
        assert (np.diff(probs) <= 1e-12).all() or solved["info"]["tbar"] * M > t[i, nb].mean()


def test_iteration_time_model():
    s = np.array([[0, 10.0, 1.0], [10.0, 0, 0.0], [1.0, 0.0, 0]])
    t, adj = policy.iteration_times(s, 1000)
    assert adj.tolist() == [[0, 1, 1], [1, 0, 0], [1, 0, 0]]
    assert t[0, 1] == pytest.approx(32e3 / 10e9) and t[0, 2] == pytest.approx(32e3 / 1e9)
    assert t[0, 0] == t[1, 1] == pytest.approx(0.25 * 32e3 / 10e9)
    assert t[1, 2] == 0.0


def test_tilt_hits_its_target_mean():
    times = np.array([1.0, 2.0, 4.0, 8.0])
    for target in (1.2, 3.75, 7.0):
        q = policy.tilt(times, target)
        assert q.sum() == pytest.approx(1.0) and (q > 0).all()
        assert (q * times).sum() == pytest.approx(target, rel=1e-9)
    np.testing.assert_allclose(policy.tilt(times, times.mean()), 0.25, atol=1e-9)   # eta = 0: maximum entropy
    assert (np.diff(policy.tilt(times, 2.0)) < 0).all()                             # fast peers preferred
