"""Pins for the oracle's policy generator under a constant pull weight (the paper's section
"Extension to existing decentralized PSGD approaches": Eq. 22 with alpha rho gamma_im replaced by w,
a positivity condition in place of Eq. 11, Eq. 8-13 solved again)."""
import itertools

import numpy as np
import pytest
from scipy.optimize import linprog

from oracle import policy
from paper_2009_05766_b200 import workloads


def _case(name):
    if name.startswith("cfg"):
        w = workloads.config(int(name[3]))
        return policy.iteration_times(w.link_speeds(0), w.d)
    rng = np.random.default_rng(5)
    M = 7
    s = np.triu(np.exp(rng.uniform(np.log(1.0), np.log(50.0), (M, M))), 1)
    s[0, 4] = s[1, 5] = s[2, 6] = 0.0            # missing links (d_im = 0)
    return policy.iteration_times(s + s.T, 1_000_000)


def test_y_matrix_equals_the_enumerated_expectation_of_DtD():
    """E[D^T D] over the M(M-1) possible (worker, peer) pairs, D = I + w e_i (e_m - e_i)^T, for a P and
    node probabilities that are NOT balanced: entries, and the row sums 1 + w (sum_m p_m p_mi - p_i sum_m p_im)
    that make the column constraint necessary."""
    rng = np.random.default_rng(1)
    M, w = 5, 0.37
    P = rng.random((M, M))
    P[1, 3] = P[4, 0] = 0.0
    P /= P.sum(axis=1, keepdims=True)              # rows sum to 1, self-draws included
    p_node = rng.random(M)
    p_node /= p_node.sum()
    want = np.zeros((M, M))
    for i, m in itertools.product(range(M), range(M)):
        D = np.eye(M)
        if m != i:
            D[i, i] -= w
            D[i, m] += w
        want += p_node[i] * P[i, m] * (D.T @ D)
    Y = policy.y_matrix_fixed_weight(P, p_node, w)
    np.testing.assert_allclose(Y, want, atol=1e-15)
    off = P * (1 - np.eye(M))
    pulls, pulled = p_node * off.sum(axis=1), (p_node[:, None] * off).sum(axis=0)
    np.testing.assert_allclose(Y.sum(axis=1), 1.0 + w * (pulled - pulls), atol=1e-15)
    assert np.abs(Y.sum(axis=1) - 1.0).max() > 1e-3          # unbalanced P: Y_P is not stochastic


def test_constant_weight_is_eq_22_with_the_weight_substituted():
    """With P from Algorithm 3 and w_im = alpha rho gamma_im the paper's Y_P (Eq. 22) is recovered entry by
    entry when each link's own weight is put into the constant-weight formula."""
    t, adj = _case("cfg1")
    alpha = 0.05
    P, rho, _ = policy.generate_policy(t, adj, alpha, 6, 6)
    M = P.shape[0]
    p_node = policy.node_probabilities(P, t, adj)
    Y = policy.y_matrix(P, p_node, adj, alpha, rho)
    W = np.zeros((M, M))
    pos = (P > 0) & ~np.eye(M, dtype=bool)
    W[pos] = alpha * rho * (adj + adj.T)[pos] / (2.0 * P[pos])
    a = p_node[:, None] * P
    off = ~np.eye(M, dtype=bool)
    want = a * (W - W ** 2) + (a * (W - W ** 2)).T
    np.testing.assert_allclose(Y[off], want[off], atol=1e-14)


@pytest.fixture(scope="module", params=[("cfg1", 0.0), ("cfg2", 0.3 / 7), ("cfg3", 0.0), ("sparse7", 0.05)],
                ids=lambda p: f"{p[0]}-{p[1]:.3f}")
def solved(request):
    name, floor_upper = request.param
    t, adj = _case(name)
    w = 0.5
    P, phi, info = policy.generate_policy_fixed_weight(t, adj, w, 3, 4, floor_upper=floor_upper)
    return dict(t=t, adj=adj, w=w, P=P, phi=phi, info=info, M=t.shape[0])


def test_constraints_of_the_extended_problem(solved):
    P, t, adj, phi, M = (solved[k] for k in ("P", "t", "adj", "phi", "M"))
    link = adj.astype(bool) & ~np.eye(M, dtype=bool)
    np.testing.assert_allclose(P.sum(axis=1), 1.0, atol=1e-9)                        # Eq. 13
    np.testing.assert_allclose(P.sum(axis=0), 1.0, atol=1e-9)                        # balance: pulled from as often as pulling
    assert (P[~link] == 0).all()                                                     # Eq. 12, and p_ii = 0
    assert (P[link] >= phi * (1 - 1e-9)).all()                                       # the floor that replaces Eq. 11
    np.testing.assert_allclose((t * P).sum(axis=1), M * solved["info"]["tbar"], rtol=1e-8)      # Eq. 10
    np.testing.assert_allclose(policy.node_probabilities(P, t, adj), 1.0 / M, rtol=1e-8)       # Lemma 1


def test_y_matrix_properties(solved):
    P, t, adj, w, M = (solved[k] for k in ("P", "t", "adj", "w", "M"))
    Y = policy.y_matrix_fixed_weight(P, np.full(M, 1.0 / M), w)
    link = adj.astype(bool) & ~np.eye(M, dtype=bool)
    np.testing.assert_allclose(Y, Y.T, atol=1e-14)
    np.testing.assert_allclose(Y.sum(axis=1), 1.0, atol=1e-9)
    assert (Y >= 0).all() and (Y[link] > 0).all()                                    # the positivity the section asks for
    lam = np.linalg.eigvalsh(Y)
    assert lam[-1] == pytest.approx(1.0, abs=1e-9) and lam[-2] < 1.0
    assert lam[-2] == pytest.approx(solved["info"]["lam2"], abs=1e-10)


def test_solution_is_the_entropy_maximum(solved):
    """The residual above the floor has the form exp(a_i + b_m - eta_i t_im) (the stationarity condition of
    the entropy maximum), and moving along any direction that keeps all constraints lowers the entropy."""
    P, t, adj, phi, M = (solved[k] for k in ("P", "t", "adj", "phi", "M"))
    link = adj.astype(bool) & ~np.eye(M, dtype=bool)
    r = (P - phi)[link]
    if r.max() < 1e-9:
        pytest.skip("the floors fill the rows at this grid point")
    assert (r >= 0).all()
    keep = r > 1e-9                                # (entries driven to the floor drop out of the stationarity fit)
    idx = np.argwhere(link)
    n = idx.shape[0]
    A = np.zeros((n, 3 * M))                       # log r = a_i + b_m - eta_i t_im
    A[np.arange(n), idx[:, 0]] = 1.0
    A[np.arange(n), M + idx[:, 1]] = 1.0
    A[np.arange(n), 2 * M + idx[:, 0]] = -t[link] / t[link].max()
    coef = np.linalg.lstsq(A[keep], np.log(r[keep]), rcond=None)[0]
    assert np.abs(A[keep] @ coef - np.log(r[keep])).max() < 1e-6
    # feasible directions: the null space of (row sums, column sums, row mean times) on the link entries
    C = np.zeros((3 * M, n))
    C[idx[:, 0], np.arange(n)] = 1.0
    C[M + idx[:, 1], np.arange(n)] = 1.0
    C[2 * M + idx[:, 0], np.arange(n)] = t[link] / t[link].max()
    _, sv, Vt = np.linalg.svd(C)
    null = Vt[(sv > 1e-10).sum():]
    entropy = lambda v: -(v * np.log(v)).sum()
    rng = np.random.default_rng(3)
    for _ in range(20):
        if null.shape[0] == 0:
            break
        step = null.T @ rng.standard_normal(null.shape[0])
        if (np.abs(step[~keep]) > 1e-12).any():
            continue                               # would leave the non-negative orthant
        step *= 0.2 * r[keep].min() / np.abs(step).max()
        assert entropy((r + step)[keep]) < entropy(r[keep]) + 1e-15


def test_p_ii_zero_is_lp_optimal_and_homogeneous_networks_get_uniform_policies(solved):
    P, t, adj, phi, M = (solved[k] for k in ("P", "t", "adj", "phi", "M"))
    # Eq. 14's objective sum_i p_ii over the same constraint set (self-draws allowed): its optimum is 0
    link = adj.astype(bool) & ~np.eye(M, dtype=bool)
    allowed = link | np.eye(M, dtype=bool)
    idx = np.argwhere(allowed)
    n = idx.shape[0]
    cost = (idx[:, 0] == idx[:, 1]).astype(float)
    Aeq = np.zeros((3 * M, n))
    Aeq[idx[:, 0], np.arange(n)] = 1.0
    Aeq[M + idx[:, 1], np.arange(n)] = 1.0
    Aeq[2 * M + idx[:, 0], np.arange(n)] = t[allowed] / t[link].max()
    beq = np.concatenate([np.ones(2 * M), np.full(M, M * solved["info"]["tbar"] / t[link].max())])
    bounds = [(phi if a != b else 0.0, None) for a, b in idx]
    res = linprog(cost, A_eq=Aeq, b_eq=beq, bounds=bounds, method="highs")
    assert res.status == 0 and res.fun == pytest.approx(0.0, abs=1e-9)
    # all links equally fast: the uniform policy
    Mh = 6
    th, adjh = policy.iteration_times((1 - np.eye(Mh)) * 25.0, 1_000_000)
    Ph, _, _ = policy.generate_policy_fixed_weight(th, adjh, 0.5, 3, 3)
    np.testing.assert_allclose(Ph[~np.eye(Mh, dtype=bool)], 1.0 / (Mh - 1), atol=1e-9)


def test_faster_links_are_not_chosen_less_often():
    t, adj = _case("cfg2")                         # two machines: intra-machine links are ten times faster
    M = t.shape[0]
    link = adj.astype(bool)
    uniform_T = float(t[0][link[0]].mean())        # the mean iteration time of a uniform row
    P = policy.solve_fixed_weight(t, adj, 0.2 / (M - 1), 0.8 * uniform_T)      # a faster network average than uniform
    assert P is not None
    assert P[0, 1] > 1.0 / (M - 1) > P[0, 5] > 0   # worker 0: peer 1 shares its machine, peer 5 does not
    for i in range(M):
        order = np.argsort(t[i][link[i]])
        assert (np.diff(P[i][link[i]][order]) <= 1e-12).all()      # within a row, a slower link never gets a larger probability
    rng = np.random.default_rng(10)                # and on a network without any symmetry
    s = np.triu(np.exp(rng.uniform(np.log(5.0), np.log(20.0), (6, 6))), 1)
    t, adj = policy.iteration_times(s + s.T, 2_000_000)
    link = adj.astype(bool)
    lo = max(float(t[i][link[i]].min()) for i in range(6))      # Eq. 10: every row has to reach the common mean time
    hi = min(float(t[i][link[i]].max()) for i in range(6))
    P = None
    for frac in np.linspace(0.05, 0.95, 19):       # the fastest network average that admits a balanced P
        P = policy.solve_fixed_weight(t, adj, 0.02, lo + frac * (hi - lo))
        if P is not None:
            break
    assert P is not None and frac < 0.3 and np.abs(P.sum(axis=0) - 1).max() < 1e-9
    slow_fast = [(P[i][link[i]][np.argmax(t[i][link[i]])], P[i][link[i]][np.argmin(t[i][link[i]])]) for i in range(6)]
    assert sum(a < b for a, b in slow_fast) >= 5    # the slowest link of a row gets less than its fastest (columns may bend one row)


def test_three_update_rules_on_a_two_machine_network():
    """The paper's comparison (section "Extension of AD-PSGD with Network Monitor"), on its own
    asynchronous process with quadratic objectives: NetMax, plain fixed-weight gossip (uniform peers,
    w = 1/2) and fixed-weight gossip with a monitor's policy (the constant-weight P for the average
    iteration time NetMax runs at).  The monitor variant needs MORE global steps than plain gossip to
    reach a given error (it pulls less often across the slow links at the same weight), LESS simulated
    time (its iterations are shorter), and more steps than NetMax, which weighs a rarely chosen peer
    more."""
    from oracle import oracle
    M, d, lr = 8, 1000, 0.1
    group = np.arange(M) // 4
    s = np.where(group[:, None] == group[None, :], 100.0, 1.0)
    np.fill_diagonal(s, 0.0)
    t, adj = policy.iteration_times(s, 11_173_962)
    c = workloads.clustered_centres(M, d, 4, spread=1.0, within=0.3, seed=1)
    cbar = c.astype(np.float64).mean(axis=0)
    P_nm, rho_nm, _ = policy.generate_policy(t, adj, lr, 10, 20, rho_upper=0.5 / lr)
    P_un = (1.0 - np.eye(M)) / (M - 1)
    P_fw = policy.solve_fixed_weight(t, adj, 0.3 / (M - 1), float((t * P_nm).sum(axis=1)[0]))
    assert P_fw is not None and P_fw[0, 1] > 1.3 * P_fw[0, 5]

    def to_level(P, rho, pull_weight, level, seed):
        sim = oracle.Sim(M, d, P, adj, alpha=lr, rho=rho, sigma=0.05, objective=1, seed=seed, pull_weight=pull_weight)
        sim.init(1.0, 0.0)
        sim.set_c(c)
        sim.async_begin(t, 0.9)
        for k in range(400):
            sim.async_steps(5)
            x = sim.x().astype(np.float64)
            if ((x - cbar) ** 2).sum(axis=1).mean() / d < level:
                return (k + 1) * 5, sim.async_now
        raise AssertionError("level not reached")

    def mean_to_level(P, rho, pull_weight, level):
        runs = np.array([to_level(P, rho, pull_weight, level, seed) for seed in range(5, 11)])
        return runs[:, 0].mean(), runs[:, 1].mean()

    for level in (0.2, 0.1):
        steps_nm, time_nm = mean_to_level(P_nm, rho_nm, 0.0, level)
        steps_un, time_un = mean_to_level(P_un, 0.0, 0.5, level)
        steps_fw, time_fw = mean_to_level(P_fw, 0.0, 0.5, level)
        assert steps_fw > 1.04 * steps_un, (level, steps_fw, steps_un)       # slower per step than plain gossip
        assert time_fw < 0.93 * time_un, (level, time_fw, time_un)           # but sooner on the clock
        assert steps_fw > 1.15 * steps_nm, (level, steps_fw, steps_nm)       # and slower per step than NetMax
        assert time_nm < time_fw                                             # NetMax is the soonest of the three
