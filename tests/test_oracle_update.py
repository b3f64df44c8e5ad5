"""Pins for the oracle's round update (Eq. 15-16 of arXiv 2009.05766) against what the
paper and the mathematics fix: fixed points, closed forms, the D^k matrix form, contraction."""
import math

import numpy as np
import pytest

from oracle import oracle


def full_adj(M):
    return (1 - np.eye(M)).astype(np.uint8)


def random_policy(M, rng, self_prob=False):
    P = rng.random((M, M)) + 0.05
    if not self_prob:
        np.fill_diagonal(P, 0.0)
    return P / P.sum(axis=1, keepdims=True)


def max_rho(P, alpha, margin=0.9):
    """Largest rho with alpha*rho*(d_im+d_mi) < p_im on every off-diagonal entry (Eq. 11), scaled."""
    M = P.shape[0]
    off = ~np.eye(M, dtype=bool)
    return margin * P[off].min() / (2.0 * alpha)


def test_zero_gradient_identical_replicas_do_not_move():
    rng = np.random.default_rng(0)
    M, d = 5, 37
    P = random_policy(M, rng, self_prob=True)
    sim = oracle.Sim(M, d, P, full_adj(M), alpha=0.1, rho=max_rho(P, 0.1), sigma=0.3, objective=0, seed=1)
    row = rng.standard_normal(d).astype(np.float32)
    x0 = np.tile(row, (M, 1))
    sim.set_x(x0)
    sim.set_c(rng.standard_normal((M, d)).astype(np.float32))   # centres are ignored when objective = 0
    sim.round(25)
    assert (sim.x() == x0).all()


def test_self_draw_is_a_plain_sgd_step():
    """p_ii = 1: the worker never communicates, so x' = x - alpha (x - c) exactly (sigma = 0)."""
    M, d, alpha = 3, 16, 0.25
    P = np.eye(M)
    rng = np.random.default_rng(1)
    x0 = rng.standard_normal((M, d)).astype(np.float32)
    c = rng.standard_normal((M, d)).astype(np.float32)
    sim = oracle.Sim(M, d, P, full_adj(M), alpha=alpha, rho=0.5, sigma=0.0, objective=1, seed=2)
    sim.set_x(x0)
    sim.set_c(c)
    sim.round(1)
    want = (x0.astype(np.float64) - np.float64(np.float32(alpha)) * (x0.astype(np.float64) - c)).astype(np.float32)
    assert (sim.x() == want).all()
    assert (sim.trace() == np.arange(M)).all()


@pytest.mark.parametrize("alpha,rho", [(0.05, 4.0), (0.1, 1.0), (0.3, 1.5)])
def test_m2_zero_gradient_closed_form(alpha, rho):
    """M = 2, P = [[0,1],[1,0]]: w = alpha*rho, the sum is conserved and the difference
    shrinks by (1 - 2w) per round."""
    d, rounds = 8, 12
    P = np.array([[0.0, 1.0], [1.0, 0.0]])
    rng = np.random.default_rng(2)
    x0 = rng.standard_normal((2, d)).astype(np.float32)
    sim = oracle.Sim(2, d, P, full_adj(2), alpha=alpha, rho=rho, sigma=0.0, objective=0, seed=3)
    sim.set_x(x0)
    sim.round(rounds)
    x = sim.x().astype(np.float64)
    w = float(np.float32(np.float64(np.float32(alpha)) * rho))
    s0, d0 = x0[0].astype(np.float64) + x0[1], x0[0].astype(np.float64) - x0[1]
    np.testing.assert_allclose(x[0] + x[1], s0, atol=2e-6)
    np.testing.assert_allclose(x[0] - x[1], (1 - 2 * w) ** rounds * d0, atol=2e-6)


@pytest.mark.parametrize("alpha,rho", [(0.05, 4.0), (0.2, 1.0)])
def test_m2_quadratic_closed_form(alpha, rho):
    """M = 2, quadratic objectives, no noise: with s = x1 + x2, delta = x1 - x2,
    s_r = C + (1 - a(1-w))^r (s_0 - C),  C = c1 + c2,
    delta_r = delta* + ((1-w)(1-a) - w)^r (delta_0 - delta*),  delta* = (1-w) a (c1-c2) / (a(1-w) + 2w)."""
    d, rounds = 8, 30
    P = np.array([[0.0, 1.0], [1.0, 0.0]])
    rng = np.random.default_rng(4)
    x0 = rng.standard_normal((2, d)).astype(np.float32)
    c = rng.standard_normal((2, d)).astype(np.float32)
    sim = oracle.Sim(2, d, P, full_adj(2), alpha=alpha, rho=rho, sigma=0.0, objective=1, seed=5)
    sim.set_x(x0)
    sim.set_c(c)
    sim.round(rounds)
    x = sim.x().astype(np.float64)
    a = float(np.float32(alpha))
    w = float(np.float32(a * rho))
    C, dc = c[0].astype(np.float64) + c[1], c[0].astype(np.float64) - c[1]
    s0, d0 = x0[0].astype(np.float64) + x0[1], x0[0].astype(np.float64) - x0[1]
    dstar = (1 - w) * a * dc / (a * (1 - w) + 2 * w)
    np.testing.assert_allclose(x[0] + x[1], C + (1 - a * (1 - w)) ** rounds * (s0 - C), atol=3e-6)
    np.testing.assert_allclose(x[0] - x[1], dstar + ((1 - w) * (1 - a) - w) ** rounds * (d0 - dstar), atol=3e-6)


def test_round_equals_product_with_row_stochastic_D():
    """Zero gradient: x^{r+1} = D^r x^r with D^r = I + sum_i w_{i,m_i} e_i (e_{m_i} - e_i)^T, all
    rows built from the round-start state; checked by explicit matrix products (M <= 8)."""
    rng = np.random.default_rng(6)
    M, d, alpha, rounds = 6, 24, 0.1, 15
    P = random_policy(M, rng, self_prob=True)
    rho = max_rho(P, alpha)
    sim = oracle.Sim(M, d, P, full_adj(M), alpha=alpha, rho=rho, sigma=0.0, objective=0, seed=7)
    x0 = rng.standard_normal((M, d)).astype(np.float32)
    sim.set_x(x0)
    sim.round(rounds)
    trace = sim.trace()
    a32 = np.float64(np.float32(alpha))
    x = x0.astype(np.float64)
    for r in range(rounds):
        D = np.eye(M)
        for i in range(M):
            m = trace[r, i]
            if m != i:
                w = np.float64(np.float32(a32 * rho * 2.0 / (2.0 * P[i, m])))
                D[i, i] -= w
                D[i, m] += w
        assert np.allclose(D.sum(axis=1), 1.0) and (D >= 0).all()
        x = (D @ x).astype(np.float32).astype(np.float64)
    np.testing.assert_allclose(sim.x(), x, atol=1e-6)


def test_zero_gradient_contracts_to_consensus_and_stays_in_the_hull():
    rng = np.random.default_rng(8)
    M, d, alpha = 8, 32, 0.1
    P = random_policy(M, rng)
    sim = oracle.Sim(M, d, P, full_adj(M), alpha=alpha, rho=max_rho(P, alpha), sigma=0.0, objective=0, seed=9)
    x0 = rng.standard_normal((M, d)).astype(np.float32)
    sim.set_x(x0)
    hi, lo = x0.max(axis=0), x0.min(axis=0)
    for _ in range(60):
        sim.round(5)
        x = sim.x()
        assert (x.max(axis=0) <= hi + 1e-6).all() and (x.min(axis=0) >= lo - 1e-6).all()
        hi, lo = np.minimum(hi, x.max(axis=0) + 1e-6), np.maximum(lo, x.min(axis=0) - 1e-6)
    cons, _ = sim.telemetry()
    assert cons[-1] < 1e-3 * cons[0]
    assert (np.diff(cons[::20]) < 0).all()


def test_expected_D_is_doubly_stochastic():
    """p_im * w_im = alpha*rho*(d_im+d_mi)/2 does not depend on P, so E[D] is symmetric: the
    replica mean is conserved in expectation (it is not conserved per realisation)."""
    rng = np.random.default_rng(10)
    M, alpha = 7, 0.1
    P = random_policy(M, rng, self_prob=True)
    adj = full_adj(M)
    adj[0, 3] = adj[3, 0] = 0
    P[0, 3] = P[3, 0] = 0.0
    P /= P.sum(axis=1, keepdims=True)
    off = (adj == 1)
    rho = 0.9 * P[off].min() / (2 * alpha)
    w = oracle.build_weights(P, adj, alpha, rho).astype(np.float64)
    ED = np.eye(M)
    for i in range(M):
        for m in range(M):
            if m != i:
                ED[i, i] -= P[i, m] * w[i, m]
                ED[i, m] += P[i, m] * w[i, m]
    np.testing.assert_allclose(ED.sum(axis=0), 1.0, atol=1e-6)
    np.testing.assert_allclose(ED, ED.T, atol=1e-6)
    a32 = float(np.float32(alpha))
    np.testing.assert_allclose(ED[off], a32 * rho, rtol=1e-6)      # (d_im + d_mi)/2 = 1 on every link
    assert w[0, 3] == 0 and w[3, 0] == 0 and (np.diag(w) == 0).all()
    assert (w[off] < 0.5).all()                                    # Eq. 11 => w < 1/2


def test_replica_mean_is_conserved_in_expectation_only():
    rng = np.random.default_rng(12)
    M, d, alpha = 4, 4, 0.1
    P = random_policy(M, rng)
    rho = max_rho(P, alpha)
    x0 = rng.standard_normal((M, d)).astype(np.float32)
    drift = []
    for seed in range(600):
        sim = oracle.Sim(M, d, P, full_adj(M), alpha=alpha, rho=rho, sigma=0.0, objective=0, seed=seed)
        sim.set_x(x0)
        sim.round(1)
        drift.append(sim.x().astype(np.float64).mean(axis=0) - x0.astype(np.float64).mean(axis=0))
        sim.close()
    drift = np.array(drift)
    assert np.abs(drift).max() > 1e-3                                  # a single realisation drifts
    sem = drift.std(axis=0) / math.sqrt(drift.shape[0])
    assert (np.abs(drift.mean(axis=0)) < 4.5 * sem).all()              # the expectation does not


def test_one_round_noise_scale():
    """Identical replicas sitting on identical centres: x' - x = -alpha*sigma*(1 - w_im) z."""
    M, d, alpha, sigma = 3, 40000, 0.05, 0.1
    P = np.array([[0, 0.5, 0.5], [0.25, 0, 0.75], [0.6, 0.4, 0]])
    rho = 1.5
    sim = oracle.Sim(M, d, P, full_adj(M), alpha=alpha, rho=rho, sigma=sigma, objective=1, seed=13)
    row = np.random.default_rng(13).standard_normal(d).astype(np.float32)
    sim.set_x(np.tile(row, (M, 1)))
    sim.set_c(np.tile(row, (M, 1)))
    sim.round(1)
    step = sim.x().astype(np.float64) - row
    peers = sim.trace()[0]
    w = oracle.build_weights(P, full_adj(M), alpha, rho)
    for i in range(M):
        want = alpha * sigma * (1.0 - w[i, peers[i]])
        assert step[i].std() == pytest.approx(want, rel=0.02)
        assert abs(step[i].mean()) < 5 * want / math.sqrt(d)
    z = -step[0] / (alpha * sigma * (1.0 - w[0, peers[0]]))
    np.testing.assert_allclose(z, oracle.noise(13, 0, 0, 0, d), atol=2e-4)  # fp32 storage of x limits this


def test_mean_replica_approaches_mean_centre_at_the_expected_rate():
    """Fully connected, p_ii = 0: E[xbar'] - cbar = (1 - a(1 - a rho (M-1))) (E[xbar] - cbar)."""
    rng = np.random.default_rng(14)
    M, d, alpha, rounds, seeds = 4, 6, 0.1, 12, 400
    P = random_policy(M, rng)
    rho = max_rho(P, alpha)
    x0 = (3.0 + rng.standard_normal((M, d))).astype(np.float32)
    c = rng.standard_normal((M, d)).astype(np.float32)
    acc = np.zeros((rounds + 1, d))
    for seed in range(seeds):
        sim = oracle.Sim(M, d, P, full_adj(M), alpha=alpha, rho=rho, sigma=0.05, objective=1, seed=1000 + seed)
        sim.set_x(x0)
        sim.set_c(c)
        acc[0] += x0.mean(axis=0)
        for r in range(rounds):
            sim.round(1)
            acc[r + 1] += sim.x().astype(np.float64).mean(axis=0)
        sim.close()
    gap = acc / seeds - c.astype(np.float64).mean(axis=0)
    a = float(np.float32(alpha))
    rate = 1 - a * (1 - a * rho * (M - 1))
    np.testing.assert_allclose(gap[rounds], rate ** rounds * gap[0], atol=0.02)
    assert np.abs(gap[rounds]).mean() < 0.5 * np.abs(gap[0]).mean()


def test_long_run_settles_near_the_mean_centre():
    rng = np.random.default_rng(15)
    M, d, alpha = 6, 64, 0.1
    P = random_policy(M, rng)
    c = rng.standard_normal((M, d)).astype(np.float32)
    sim = oracle.Sim(M, d, P, full_adj(M), alpha=alpha, rho=max_rho(P, alpha), sigma=0.0, objective=1, seed=16)
    sim.set_x(10.0 + rng.standard_normal((M, d)).astype(np.float32))
    sim.set_c(c)
    sim.round(400)
    x = sim.x().astype(np.float64)
    cbar = c.astype(np.float64).mean(axis=0)
    assert np.abs(x.mean(axis=0) - cbar).mean() < 0.35          # pulled from 10 to the centre of the c_i
    assert np.linalg.norm(x - cbar) < np.linalg.norm(c - cbar)  # closer to cbar than the c_i themselves


def test_split_calls_threads_and_column_samples_agree_bit_for_bit():
    rng = np.random.default_rng(17)
    M, d, alpha = 5, 5003, 0.05
    P = random_policy(M, rng, self_prob=True)
    rho = max_rho(P, alpha)
    kw = dict(alpha=alpha, rho=rho, sigma=0.1, objective=1, seed=18)
    a = oracle.Sim(M, d, P, full_adj(M), **kw)
    a.init(1.0, 1.0)
    a.round(9)
    b = oracle.Sim(M, d, P, full_adj(M), **kw)
    b.init(1.0, 1.0)
    b.round(4, threads=3)
    b.round(5, threads=2)
    assert (a.x() == b.x()).all() and (a.trace() == b.trace()).all()
    cols = np.array([0, 1, 2, 3, 4, 1000, 1001, 4097, 5000, 5001, 5002])
    s = oracle.Sim(M, d, P, full_adj(M), cols=cols, **kw)
    s.init(1.0, 1.0)
    s.round(9)
    assert (s.x() == a.x()[:, cols]).all() and (s.trace() == a.trace()).all()


def test_policy_refresh_between_rounds():
    rng = np.random.default_rng(19)
    M, d, alpha = 4, 16, 0.1
    P1, P2 = random_policy(M, rng), np.roll(np.eye(M), 1, axis=1)
    sim = oracle.Sim(M, d, P1, full_adj(M), alpha=alpha, rho=max_rho(P1, alpha), sigma=0.0, objective=0, seed=20)
    sim.set_x(rng.standard_normal((M, d)).astype(np.float32))
    sim.round(3)
    sim.set_policy(P2, full_adj(M), 2.0)
    sim.round(3)
    assert (sim.trace()[3:] == (np.arange(M) + 1) % M).all()


def test_telemetry_matches_its_definition():
    rng = np.random.default_rng(21)
    M, d = 5, 33
    P = random_policy(M, rng)
    sim = oracle.Sim(M, d, P, full_adj(M), alpha=0.1, rho=max_rho(P, 0.1), sigma=0.1, objective=1, seed=22)
    x0 = rng.standard_normal((M, d)).astype(np.float32)
    c = rng.standard_normal((M, d)).astype(np.float32)
    sim.set_x(x0)
    sim.set_c(c)
    sim.round(2)
    cons, loss = sim.telemetry()
    x64, c64 = x0.astype(np.float64), c.astype(np.float64)
    assert cons[0] == pytest.approx(((x64 - x64.mean(axis=0)) ** 2).sum() / M, rel=1e-12)
    assert loss[0] == pytest.approx(0.5 * ((x64 - c64) ** 2).sum() / M, rel=1e-12)


# ---------------------------------------------------------------- fixed pull weight (gossip / AD-PSGD style)
def test_fixed_weight_half_averages_two_workers_in_one_round():
    """w = 1/2, M = 2, both pull each other from the round-start snapshot: x1' = x2' = (x1+x2)/2."""
    d = 9
    P = np.array([[0.0, 1.0], [1.0, 0.0]])
    x0 = np.random.default_rng(30).standard_normal((2, d)).astype(np.float32)
    sim = oracle.Sim(2, d, P, full_adj(2), alpha=0.1, rho=123.0, sigma=0.0, objective=0, seed=1, pull_weight=0.5)
    sim.set_x(x0)
    sim.round(1)
    want = ((x0[0].astype(np.float64) + x0[1]) / 2).astype(np.float32)
    assert (sim.x()[0] == want).all() and (sim.x()[1] == want).all()
    assert (oracle.Sim(2, d, P, full_adj(2), 0.1, 123.0, 0.0, 0, 1, pull_weight=0.5).x() == 0).all()


def test_fixed_weight_ignores_rho_and_probabilities():
    rng = np.random.default_rng(31)
    M, d = 5, 16
    P = random_policy(M, rng)
    x0 = rng.standard_normal((M, d)).astype(np.float32)
    sims = []
    for rho in (0.01, 7.0):
        s = oracle.Sim(M, d, P, full_adj(M), alpha=0.1, rho=rho, sigma=0.0, objective=0, seed=2, pull_weight=0.25)
        s.set_x(x0)
        s.round(6)
        sims.append(s)
    assert (sims[0].x() == sims[1].x()).all()
    trace = sims[0].trace()
    x = x0.astype(np.float64)
    for r in range(6):                                   # D^r with the constant weight on every pull
        D = np.eye(M)
        for i in range(M):
            m = trace[r, i]
            if m != i:
                D[i, i] -= 0.25
                D[i, m] += 0.25
        x = (D @ x).astype(np.float32).astype(np.float64)
    np.testing.assert_allclose(sims[0].x(), x, atol=1e-6)


def test_rounds_numbered_from_a_later_start_use_that_rounds_counters():
    """A simulator that starts at round r0 draws the peers and the noise of rounds r0, r0 + 1, ...:
    checked against the two pinned stream functions across the 2^32 boundary of the round word,
    and against an uninterrupted run resumed half way."""
    M, d, alpha, sigma, seed = 4, 12, 0.1, 0.3, 77
    r0 = (1 << 32) - 3
    P = random_policy(M, np.random.default_rng(3), self_prob=True)
    rho = max_rho(P, alpha)
    sim = oracle.Sim(M, d, P, full_adj(M), alpha=alpha, rho=rho, sigma=sigma, objective=1, seed=seed, first_round=r0)
    sim.init(1.0, 1.0)
    x0, c = sim.x().astype(np.float64), sim.c().astype(np.float64)
    sim.round(6)
    assert sim.rounds_done == 6
    trace = sim.trace()
    assert (trace == oracle.peer_draws(P, seed, r0, 6)).all()
    assert not (trace == oracle.peer_draws(P, seed, 0, 6)).all()
    # first round by hand: Eq. 15 with the noise of round r0, then Eq. 16 against the snapshot
    a32, s32 = float(np.float32(alpha)), float(np.float32(sigma))
    w = oracle.build_weights(P, full_adj(M), a32, rho).astype(np.float64)
    one = oracle.Sim(M, d, P, full_adj(M), alpha=alpha, rho=rho, sigma=sigma, objective=1, seed=seed, first_round=r0)
    one.init(1.0, 1.0)
    one.round(1)
    want = np.empty_like(x0)
    for i in range(M):
        z = oracle.noise(seed, i, r0, 0, d)
        h = x0[i] - a32 * ((x0[i] - c[i]) + s32 * z)
        m = int(trace[0, i])
        want[i] = h if m == i else h - w[i, m] * (h - x0[m])
    np.testing.assert_array_equal(one.x(), want.astype(np.float32))
    # the initial state does not depend on where the rounds start
    base = oracle.Sim(M, d, P, full_adj(M), alpha=alpha, rho=rho, sigma=sigma, objective=1, seed=seed)
    base.init(1.0, 1.0)
    np.testing.assert_array_equal(base.x(), x0.astype(np.float32))
    # resume: 10 rounds from 0 == 4 rounds from 0, state handed over, 6 rounds numbered from 4
    base.round(4)
    rest = oracle.Sim(M, d, P, full_adj(M), alpha=alpha, rho=rho, sigma=sigma, objective=1, seed=seed, first_round=4)
    rest.set_x(base.x())
    rest.set_c(base.c())
    base.round(6)
    rest.round(6)
    np.testing.assert_array_equal(rest.x(), base.x())
    assert (rest.trace() == base.trace(4, 6)).all()
