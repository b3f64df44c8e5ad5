"""GPU tests of the constant-weight update rule with a policy from the extended Algorithm 3 (the
paper's sections "Extension to existing decentralized PSGD approaches" and "Extension of AD-PSGD
with Network Monitor"), on the asynchronous timeline."""
import numpy as np
import pytest

from oracle import oracle
from oracle import policy as opolicy
from paper_2009_05766_b200 import workloads

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def nm():
    import torch
    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device")
    from paper_2009_05766_b200 import binding
    binding.lib()
    return binding


def two_machines(M, inter_gbps):
    group = np.arange(M) // (M // 2)
    s = np.where(group[:, None] == group[None, :], 100.0, inter_gbps)
    np.fill_diagonal(s, 0.0)
    return s


def test_three_update_rules_on_a_two_machine_network(nm):
    """NetMax, plain fixed-weight gossip (uniform peers, w = 1/2) and fixed-weight gossip with a
    monitor's policy (the constant-weight P for the average iteration time NetMax runs at), from the
    same start on the same quadratic objectives.  As the paper reports for AD-PSGD with a Network
    Monitor: more global steps than plain gossip to a given error, less simulated time, and more
    steps than NetMax."""
    M, d, lr = 8, 2000, 0.1
    s = two_machines(M, 1.0)
    t, adj = nm.netmax_iteration_times(s, 11_173_962)
    c = workloads.clustered_centres(M, d, 4, spread=1.0, within=0.3, seed=1)
    cbar = c.astype(np.float64).mean(axis=0)
    P_nm, rho_nm, info = nm.netmax_policy_generate(t, adj, lr, 10, 20, rho_upper=0.5 / lr)
    P_un = (1.0 - np.eye(M)) / (M - 1)
    P_fw = nm.netmax_policy_fixed_weight_at(t, adj, 0.3 / (M - 1), info["tbar"])
    assert P_fw[0, 1] > 1.3 * P_fw[0, 5]
    np.testing.assert_allclose(P_fw.sum(axis=0), 1.0, atol=1e-9)

    def to_level(P, rho, pull_weight, level, seed):
        g = nm.Netmax(M=M, d=d, lr=lr, link_speed_gbps=s, prob=P, rho=rho, pull_weight=pull_weight, sigma=0.05, x0_std=1.0,
                      seed=seed)
        g.set_centres(c)
        g.async_begin(t, 0.9)
        try:
            for k in range(400):
                g.async_steps(5)
                x = g.read_replicas().astype(np.float64)
                if ((x - cbar) ** 2).sum(axis=1).mean() / d < level:
                    return (k + 1) * 5, g.async_time()[0]
            raise AssertionError("level not reached")
        finally:
            g.close()

    def mean_to_level(P, rho, pull_weight, level):
        runs = np.array([to_level(P, rho, pull_weight, level, seed) for seed in range(5, 11)])
        return runs[:, 0].mean(), runs[:, 1].mean()

    for level in (0.2, 0.1):
        steps_nm, time_nm = mean_to_level(P_nm, rho_nm, 0.0, level)
        steps_un, time_un = mean_to_level(P_un, 0.0, 0.5, level)
        steps_fw, time_fw = mean_to_level(P_fw, 0.0, 0.5, level)
        assert steps_fw > 1.04 * steps_un, (level, steps_fw, steps_un)
        assert time_fw < 0.93 * time_un, (level, time_fw, time_un)
        assert steps_fw > 1.15 * steps_nm, (level, steps_fw, steps_nm)
        assert time_nm < time_fw


def test_fixed_weight_context_gets_its_policy_from_the_extended_algorithm_3(nm):
    """A context with a constant pull weight and no P runs the extended generator at creation and at
    every refresh of the Network Monitor; the updates with that policy match the oracle."""
    M, d, lr = 8, 1500, 0.05
    s = two_machines(M, 10.0)
    t, adj = nm.netmax_iteration_times(s, d)                     # the context derives the same times from s and its d
    K = R = 4
    upper = 0.4 / (M - 1)
    g = nm.Netmax(M=M, d=d, lr=lr, link_speed_gbps=s, pull_weight=0.5, sigma=0.05, x0_std=1.0, c_std=1.0, seed=9,
                  policy_K=K, policy_R=R, policy_rho_upper=upper)
    P, _ = g.get_policy()
    P0, _, _ = opolicy.generate_policy_fixed_weight(t, adj, 0.5, K, R, floor_upper=upper)
    np.testing.assert_allclose(P, P0, atol=1e-8)
    o = oracle.Sim(M, d, P, adj, alpha=lr, rho=0.0, sigma=0.05, objective=1, seed=9, pull_weight=0.5)
    o.init(1.0, 1.0)
    t_async = t
    g.async_begin(None, 0.8)
    o.async_begin(t_async, 0.8)
    g.async_steps(6 * M)
    o.async_steps(6 * M)
    for a, b in zip(g.async_trace(), o.async_trace()):
        assert (a == b).all()
    got, want = g.read_replicas().astype(np.float64), o.x().astype(np.float64)
    assert (np.abs(got - want) <= 1e-5 * (1 + np.abs(want))).all()
    # the monitor: measured times equal the true ones here, so the refreshed policy is the generator's on t_async
    g.async_monitor(4 * float(t_async[adj == 1].mean()))
    g.async_steps(20 * M)
    assert g.async_monitor_refreshes >= 2
    P1, _ = g.get_policy()
    P2, _, _ = opolicy.generate_policy_fixed_weight(t_async, adj, 0.5, K, R, floor_upper=upper)
    np.testing.assert_allclose(P1, P2, atol=1e-7)
    np.testing.assert_allclose(P1.sum(axis=0), 1.0, atol=1e-8)
    g.close()


def test_disagreement_contracts_at_lambda_max_rate_under_redrawn_links(nm):
    """Theorem 2 on the GPU timeline: zero gradients, links redrawn and the policy replaced every 60
    global steps; the mean disagreement over many seeds decays between lambda_max^(3k/4) and (the
    smallest lambda)^(3k/2) (the workers' clocks make them take turns, so the theorem's constant, which
    assumes independent draws of the acting worker, is met up to that slack)."""
    M, d, alpha, period, epochs, runs = 6, 64, 0.1, 60, 4, 60
    rng = np.random.default_rng(11)
    policies = []
    for e in range(epochs):
        sp = np.triu(np.exp(rng.uniform(np.log(1.0), np.log(100.0), (M, M))), 1)
        t, adj = opolicy.iteration_times(sp + sp.T, 1_000_000)
        P, rho, info = opolicy.generate_policy(t, adj, alpha, 6, 6)
        policies.append((t, adj, P, rho, info["lam2"]))
    lam = [p[4] for p in policies]
    x0 = rng.standard_normal((M, d)).astype(np.float32)
    x064 = x0.astype(np.float64)
    e0 = ((x064 - x064.mean(axis=0)) ** 2).sum() / d
    total = np.zeros(epochs)
    for seed in range(runs):
        t, adj, P, rho, _ = policies[0]
        g = nm.Netmax(M=M, d=d, lr=alpha, prob=P, rho=rho, objective=0, seed=seed)
        g.set_replicas(x0)
        g.async_begin(t, 0.5)
        for e, (t, adj, P, rho, _) in enumerate(policies):
            if e > 0:
                g.set_policy(prob=P, rho=rho)
                g.async_set_times(t)
            g.async_steps(period)
            x = g.read_replicas().astype(np.float64)
            total[e] += ((x - x.mean(axis=0)) ** 2).sum() / d
        g.close()
    mean = total / runs
    for e in range(epochs):
        steps = (e + 1) * period
        assert mean[e] <= max(lam) ** (0.75 * steps) * e0 * 1.1, (steps, mean[e])
        assert mean[e] >= min(lam) ** (1.5 * steps) * e0 * 0.9, (steps, mean[e])
