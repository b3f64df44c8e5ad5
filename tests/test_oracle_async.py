"""Pins for the oracle's asynchronous timeline: the paper's own process, in which exactly one
worker updates at every global step (Section II-B, Eq. 2-3, Eq. 17-18, Eq. 22, Theorem 1)."""
import numpy as np
import pytest

from oracle import oracle
from oracle import policy as opolicy


def full_adj(M):
    return (1 - np.eye(M)).astype(np.uint8)


def random_policy(M, rng, self_prob=False):
    P = rng.random((M, M)) + 0.05
    if not self_prob:
        np.fill_diagonal(P, 0.0)
    return P / P.sum(axis=1, keepdims=True)


def random_times(M, rng):
    t = rng.uniform(1.0, 4.0, (M, M))
    t = 0.5 * (t + t.T)
    t[np.diag_indices(M)] = 0.2
    return t


def test_event_times_are_per_worker_cumulative_sums_and_globally_sorted():
    rng = np.random.default_rng(1)
    M = 5
    P, t = random_policy(M, rng, self_prob=True), random_times(M, rng)
    sim = oracle.Sim(M, 4, P, full_adj(M), alpha=0.1, rho=0.1, sigma=0.0, objective=0, seed=3)
    sim.async_begin(t, beta=0.5)
    sim.async_steps(400)
    worker, peer, local_iter, time = sim.async_trace()
    assert (np.diff(time) >= 0).all() and sim.async_now == time[-1]
    for i in range(M):
        mine = worker == i
        assert (local_iter[mine] == np.arange(mine.sum())).all()          # local steps count up
        np.testing.assert_allclose(time[mine], np.cumsum(t[i, peer[mine]]), rtol=1e-12)
        assert (P[i, peer[mine]] > 0).all()
    # the peers of worker i's local iterations are the PEER stream at counter (0, i, n): the same
    # draws the synchronous rounds use with n in place of the round number
    draws = oracle.peer_draws(P, 3, 0, int(local_iter.max()) + 1)
    assert (peer == draws[local_iter, worker]).all()


def test_global_steps_equal_products_of_D_k():
    """Zero gradient: x^{k+1} = D^k x^k with D^k = I + w_im e_i (e_m - e_i)^T (Eq. 18) and the
    peer's CURRENT replica; only worker i moves."""
    rng = np.random.default_rng(2)
    M, d, alpha = 4, 6, 0.1
    P, t = random_policy(M, rng, self_prob=True), random_times(M, rng)
    rho = 0.9 * P[~np.eye(M, dtype=bool)].min() / (2 * alpha)
    sim = oracle.Sim(M, d, P, full_adj(M), alpha=alpha, rho=rho, sigma=0.0, objective=0, seed=4)
    x0 = rng.standard_normal((M, d)).astype(np.float32)
    sim.set_x(x0)
    sim.async_begin(t, beta=0.0)
    x = x0.astype(np.float64)
    a32 = float(np.float32(alpha))
    for k in range(60):
        before = sim.x()
        sim.async_steps(1)
        worker, peer, _, _ = sim.async_trace(k, 1)
        i, m = int(worker[0]), int(peer[0])
        D = np.eye(M)
        if m != i:
            w = float(np.float32(a32 * rho * 2.0 / (2.0 * P[i, m])))
            D[i, i] -= w
            D[i, m] += w
        x = (D @ x).astype(np.float32).astype(np.float64)
        after = sim.x()
        assert (np.delete(after, i, axis=0) == np.delete(before, i, axis=0)).all()
    np.testing.assert_allclose(sim.x(), x, atol=1e-6)


def test_m2_alternating_closed_form():
    """M = 2, equal iteration times: the workers alternate (ties go to the lower index), each
    pull shrinks the difference by (1 - w): after 2r steps delta = (1 - w)^(2r) delta_0."""
    alpha, rho, d, r = 0.1, 2.0, 8, 10
    P = np.array([[0.0, 1.0], [1.0, 0.0]])
    t = np.array([[0.1, 1.0], [1.0, 0.1]])
    x0 = np.random.default_rng(3).standard_normal((2, d)).astype(np.float32)
    sim = oracle.Sim(2, d, P, full_adj(2), alpha=alpha, rho=rho, sigma=0.0, objective=0, seed=5)
    sim.set_x(x0)
    sim.async_begin(t, beta=0.0)
    sim.async_steps(2 * r)
    worker, _, _, time = sim.async_trace()
    assert (worker == np.tile([0, 1], r)).all()
    np.testing.assert_allclose(time, np.repeat(np.arange(1, r + 1), 2).astype(float))
    w = float(np.float32(np.float64(np.float32(alpha)) * rho))
    x = sim.x().astype(np.float64)
    np.testing.assert_allclose(x[0] - x[1], (1 - w) ** (2 * r) * (x0[0].astype(np.float64) - x0[1]), atol=2e-6)


def test_node_activation_frequencies_follow_eq_3():
    """p_i = (1/t_bar_i) / sum_m (1/t_bar_m) with t_bar_i = sum_m t_im p_im (Eq. 2-3)."""
    rng = np.random.default_rng(4)
    M, steps = 6, 120_000
    P, t = random_policy(M, rng, self_prob=True), random_times(M, rng)
    sim = oracle.Sim(M, 1, P, full_adj(M), alpha=0.1, rho=0.01, sigma=0.0, objective=0, seed=6)
    sim.async_begin(t, beta=0.9)
    sim.async_steps(steps)
    worker, peer, _, _ = sim.async_trace()
    freq = np.bincount(worker, minlength=M) / steps
    p_node = opolicy.node_probabilities(P, t, full_adj(M))
    np.testing.assert_allclose(freq, p_node, rtol=0.02)
    assert np.ptp(p_node) > 0.02          # a generic P makes the workers unequally active


def test_feasible_policy_equalises_the_workers_lemma_1():
    rng = np.random.default_rng(5)
    M = 6
    s = np.triu(np.exp(rng.uniform(np.log(1.0), np.log(30.0), (M, M))), 1)
    t, adj = opolicy.iteration_times(s + s.T, 1_000_000)
    P, rho, _ = opolicy.generate_policy(t, adj, 0.1, 6, 6)
    sim = oracle.Sim(M, 1, P, adj, alpha=0.1, rho=rho, sigma=0.0, objective=0, seed=7)
    sim.async_begin(t, beta=0.9)
    sim.async_steps(90_000)
    worker, _, _, _ = sim.async_trace()
    freq = np.bincount(worker, minlength=M) / worker.size
    np.testing.assert_allclose(freq, 1.0 / M, rtol=0.02)


def test_empirical_DtD_matches_eq_22():
    """Mean of (D^k)^T D^k over the simulated global steps against the closed form Y_P."""
    rng = np.random.default_rng(6)
    M, alpha, steps = 4, 0.1, 150_000
    P, t = random_policy(M, rng), random_times(M, rng)
    rho = 0.9 * P[~np.eye(M, dtype=bool)].min() / (2 * alpha)
    sim = oracle.Sim(M, 1, P, full_adj(M), alpha=alpha, rho=rho, sigma=0.0, objective=0, seed=8)
    sim.async_begin(t, beta=0.9)
    sim.async_steps(steps)
    worker, peer, _, _ = sim.async_trace()
    w = oracle.build_weights(P, full_adj(M), alpha, rho).astype(np.float64)
    counts = np.zeros((M, M))
    np.add.at(counts, (worker, peer), 1.0)
    acc = np.zeros((M, M))
    for i in range(M):
        for m in range(M):
            if counts[i, m] == 0:
                continue
            D = np.eye(M)
            if m != i:
                D[i, i] -= w[i, m]
                D[i, m] += w[i, m]
            acc += counts[i, m] * (D.T @ D)
    a32 = float(np.float32(alpha))
    Y = opolicy.y_matrix(P, opolicy.node_probabilities(P, t, full_adj(M)), full_adj(M), a32, rho)
    np.testing.assert_allclose(acc / steps, Y, atol=4e-3)


def test_ema_of_iteration_times():
    rng = np.random.default_rng(7)
    M, beta = 4, 0.8
    P, t = random_policy(M, rng), random_times(M, rng)
    sim = oracle.Sim(M, 1, P, full_adj(M), alpha=0.1, rho=0.01, sigma=0.0, objective=0, seed=9)
    sim.async_begin(t, beta=beta)
    sim.async_steps(300)
    ema, count = sim.async_ema()
    worker, peer, _, _ = sim.async_trace()
    want = np.zeros((M, M), dtype=np.int64)
    np.add.at(want, (worker, peer), 1)
    assert (count == want).all()
    np.testing.assert_allclose(ema, t * (1.0 - beta ** count), rtol=1e-12)     # EMA started from 0 (Algorithm 2)


def test_error_contracts_as_in_the_proof_of_theorem_1():
    """All workers share one optimum x* (c_i = c).  The proof of Theorem 1 gives, per global
    step, E||x - x*1 - alpha g||^2 <= (1 - 2 alpha mu L/(mu+L) p_min) ||x - x*1||^2 + alpha^2 sigma^2
    (its Eq. for the gradient step) and Y_P doubly stochastic makes the pull non-expansive in
    expectation.  For f = 1/2||x - c||^2 (mu = L = 1) and a feasible P (p_i = 1/M) the gradient
    step is exact: kappa = 1 - (2 alpha - alpha^2)/M, noise alpha^2 sigma^2 per step.
    (The theorem's headline rate lambda_2^k does not hold for the component along 1, whose
    eigenvalue in Y_P is 1; the consensus component does contract faster, checked below.)"""
    rng = np.random.default_rng(8)
    M, d, alpha, sigma = 5, 4000, 0.1, 0.05
    s = np.triu(np.exp(rng.uniform(np.log(1.0), np.log(20.0), (M, M))), 1)
    t, adj = opolicy.iteration_times(s + s.T, 1_000_000)
    P, rho, info = opolicy.generate_policy(t, adj, alpha, 6, 6)
    c = np.tile(rng.standard_normal(d).astype(np.float32), (M, 1))
    x0 = (c + 2.0 * rng.standard_normal((M, d))).astype(np.float32)
    sim = oracle.Sim(M, d, P, adj, alpha=alpha, rho=rho, sigma=sigma, objective=1, seed=10)
    sim.set_x(x0)
    sim.set_c(c)
    sim.async_begin(t, beta=0.9)
    e0 = ((x0.astype(np.float64) - c) ** 2).sum(axis=0).mean()      # per coordinate, averaged over coordinates
    kappa = 1.0 - (2 * alpha - alpha ** 2) / M
    floor = alpha ** 2 * sigma ** 2 / (1.0 - kappa)
    dev0 = ((x0.astype(np.float64) - x0.astype(np.float64).mean(axis=0)) ** 2).sum(axis=0).mean()
    for k in (50, 200, 600):
        sim.async_steps(k - sim.async_steps_done)
        x = sim.x().astype(np.float64)
        ek = ((x - c) ** 2).sum(axis=0).mean()
        assert ek <= (kappa ** k * e0 + floor) * 1.05, (k, ek)
        assert ek >= 0.2 * kappa ** k * e0                      # and it is not faster than the mean mode allows
    devk = ((x - x.mean(axis=0)) ** 2).sum(axis=0).mean()
    assert devk < 1e-3 * dev0                                   # the disagreement is gone long before


def test_policy_change_applies_to_iterations_started_afterwards():
    M = 3
    P1 = np.array([[0, 1.0, 0], [0, 0, 1.0], [1.0, 0, 0]])
    P2 = np.array([[0, 0, 1.0], [1.0, 0, 0], [0, 1.0, 0]])
    t = np.array([[0.1, 1.0, 1.0], [1.0, 0.1, 1.0], [1.0, 1.0, 0.1]])
    sim = oracle.Sim(M, 2, P1, full_adj(M), alpha=0.1, rho=0.1, sigma=0.0, objective=0, seed=11)
    sim.async_begin(t, beta=0.5)
    sim.async_steps(3)                      # all three pending iterations (drawn under P1) finish at t = 1
    sim.set_policy(P2, full_adj(M), 0.1)    # iterations already started (at t = 1) keep their P1 peers
    sim.async_steps(6)
    worker, peer, local_iter, _ = sim.async_trace()
    assert (peer[:6] == (worker[:6] + 1) % M).all()
    assert (peer[6:] == (worker[6:] + 2) % M).all()


def test_an_iteration_in_flight_keeps_the_weight_and_time_it_started_with():
    """Algorithm 2 reads P[i] and rho at the top of an iteration, before it draws the peer, and
    UpdateTimeVector folds in the time the iteration took.  An iteration that is in flight when
    the policy or the iteration times change therefore pulls with the OLD alpha rho / (2 p_im) and
    records the OLD t_im -- also when the new policy gives that peer probability zero."""
    M, d, alpha, beta = 3, 5, 0.1, 0.5
    P1 = np.array([[0, 1.0, 0], [0, 0, 1.0], [1.0, 0, 0]])          # i pulls from i + 1
    P2 = np.array([[0, 0, 1.0], [1.0, 0, 0], [0, 1.0, 0]])          # i pulls from i + 2: p_{i,i+1} becomes 0
    rho1, rho2 = 0.8, 2.4
    t1 = np.array([[0.1, 1.0, 1.0], [1.0, 0.1, 1.0], [1.0, 1.0, 0.1]])
    t2 = 3.0 * t1
    x0 = np.random.default_rng(12).standard_normal((M, d)).astype(np.float32)
    sim = oracle.Sim(M, d, P1, full_adj(M), alpha=alpha, rho=rho1, sigma=0.0, objective=0, seed=13)
    sim.set_x(x0)
    sim.async_begin(t1, beta=beta)
    # all three first iterations are in flight (peers drawn under P1, finishing at t = 1)
    sim.set_policy(P2, full_adj(M), rho2)
    sim.async_set_times(t2)
    a32 = float(np.float32(alpha))
    w_old = float(np.float32(a32 * rho1 * 2.0 / (2.0 * 1.0)))
    w_new = float(np.float32(a32 * rho2 * 2.0 / (2.0 * 1.0)))
    x = x0.astype(np.float64)
    for k in range(6):
        sim.async_steps(1)
        worker, peer, local_iter, time = sim.async_trace(k, 1)
        i, m, n = int(worker[0]), int(peer[0]), int(local_iter[0])
        w = w_old if n == 0 else w_new                             # iteration 0 started before the change
        assert m == ((i + 1) % M if n == 0 else (i + 2) % M)
        assert time[0] == pytest.approx(1.0 if n == 0 else 4.0)    # 1 s under t1, then 3 s under t2
        x[i] = np.float32(x[i] - w * (x[i] - x[m]))
        np.testing.assert_allclose(sim.x(), x, atol=1e-6)
        assert np.abs(sim.x()[i].astype(np.float64) - x0[i]).max() > 1e-3 or n > 0   # the old-policy pull happened
    ema, count = sim.async_ema()
    want = np.zeros((M, M))
    for i in range(M):
        want[i, (i + 1) % M] = (1 - beta) * 1.0                    # the iteration in flight took t1 = 1 s
        want[i, (i + 2) % M] = (1 - beta) * 3.0                    # the next one t2 = 3 s
    np.testing.assert_allclose(ema, want, rtol=1e-12)
    assert (count == (want > 0)).all()


def test_disagreement_contracts_by_lambda_max_when_the_policy_changes_theorem_2():
    """Theorem 2 (dynamic network): with the policy replaced every so often, the expected error
    contracts per global step by the largest lambda among the policies in force.  Zero gradients
    isolate the part Y_P governs: for x' = D x, ||x' - mean(x') 1||^2 <= ||D (x - mean(x) 1)||^2
    (D 1 = 1), whose expectation over the draw of D is (x - mean 1)^T Y_P (x - mean 1)
    <= lambda_2(Y_P) ||x - mean 1||^2.  Checked on links redrawn every 60 steps (the shape of the
    benchmark's third configuration); the expectation is a mean over 300 seeds (every column of a run
    sees the same D^k, so columns do not average the draws)."""
    M, d, alpha, period, epochs, runs = 6, 64, 0.1, 60, 4, 300
    rng = np.random.default_rng(11)
    policies = []
    for e in range(epochs):
        s = np.triu(np.exp(rng.uniform(np.log(1.0), np.log(100.0), (M, M))), 1)
        t, adj = opolicy.iteration_times(s + s.T, 1_000_000)
        P, rho, info = opolicy.generate_policy(t, adj, alpha, 6, 6)
        policies.append((t, adj, P, rho, info["lam2"]))
    lam = [p[4] for p in policies]
    lam_max = max(lam)
    assert max(lam) - min(lam) > 1e-3              # the epochs really differ
    x0 = rng.standard_normal((M, d)).astype(np.float32)
    checkpoints = list(range(20, epochs * period + 1, 20))
    total = np.zeros(len(checkpoints))

    def disagreement(sim):
        x = sim.x().astype(np.float64)
        return ((x - x.mean(axis=0)) ** 2).sum() / d

    for seed in range(runs):
        t, adj, P, rho, _ = policies[0]
        sim = oracle.Sim(M, d, P, adj, alpha=alpha, rho=rho, sigma=0.0, objective=0, seed=seed)
        sim.set_x(x0)
        sim.async_begin(t, 0.5)
        at = 0
        for e, (t, adj, P, rho, _) in enumerate(policies):
            if e > 0:
                sim.set_policy(P, adj, rho)
                sim.async_set_times(t)
            for _ in range(period // 20):
                sim.async_steps(20)
                total[at] += disagreement(sim)
                at += 1
        sim.close()
    mean = total / runs
    x064 = x0.astype(np.float64)
    e0 = ((x064 - x064.mean(axis=0)) ** 2).sum() / d
    # The theorem draws the acting worker independently at every step (probability p_i = 1/M); on the
    # timeline the workers' clocks make them take turns instead, which changes the constant but not the
    # picture: the measured decay stays between lambda_max^(3k/4) and (the smallest lambda)^(3k/2).
    for steps, now in zip(checkpoints, mean):
        assert now <= lam_max ** (0.75 * steps) * e0, (steps, now)
        assert now >= min(lam) ** (1.5 * steps) * e0, (steps, now)
    # Under the theorem's own sampling -- worker i uniform, peer m from P[i,:], D = I + w_im e_i (e_m - e_i)^T
    # with the simulator's fp32 weights -- the bound holds as stated, policy changes included.
    draws = np.random.default_rng(13)
    total = np.zeros(len(checkpoints))
    for run in range(runs):
        x = x064.copy()
        at = 0
        for t, adj, P, rho, _ in policies:
            w = oracle.build_weights(P, adj, alpha, rho).astype(np.float64)
            for step in range(period):
                i = int(draws.integers(M))
                m = int(draws.choice(M, p=P[i]))
                if m != i:
                    x[i] = x[i] - w[i, m] * (x[i] - x[m])
                if (step + 1) % 20 == 0:
                    total[at] += ((x - x.mean(axis=0)) ** 2).sum() / d
                    at += 1
    iid = total / runs
    bound = e0
    for e, lam2 in enumerate(lam):
        for k in range(period // 20):
            bound *= lam2 ** 20
            assert iid[e * (period // 20) + k] <= bound * 1.05                  # the sharper product of each epoch's own lambda_2
            assert iid[e * (period // 20) + k] <= lam_max ** (e * period + (k + 1) * 20) * e0 * 1.05      # Theorem 2
