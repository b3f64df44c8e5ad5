"""GPU parity at the benchmark's full sizes, in the launch configuration bench.py times.

The oracle cannot afford every element of 10^8-element replicas, but columns evolve
independently given the peer draws, so it simulates a sample of columns (always including
the first and last elements of the rows) for all workers and all rounds; peer traces are
compared in full.  Telemetry is checked against a direct fp64 evaluation of its definition."""
import os

import numpy as np
import pytest

from oracle import oracle
from oracle import policy as opolicy
from paper_2009_05766_b200 import workloads

pytestmark = pytest.mark.gpu
TOL = 1e-5


@pytest.fixture(scope="module")
def nm():
    import torch
    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device")
    from paper_2009_05766_b200 import binding
    binding.lib()
    return binding


def assert_replicas_close(got, want, tol=TOL):
    got64, want64 = got.astype(np.float64), want.astype(np.float64)
    excess = np.abs(got64 - want64) - tol * (1.0 + np.abs(want64))
    assert excess.max() <= 0.0, f"max excess {excess.max():.3e}"


def telemetry_from_device(g):
    """Consensus distance of the current replicas, computed by torch in fp64 from the device buffer."""
    ptr, ld = g.replicas_device()
    x = _as_tensor(ptr, g.M, ld)[:, :g.d].double()
    mean = x.mean(dim=0, keepdim=True)
    return float(((x - mean) ** 2).sum().item() / g.M)


def _as_tensor(ptr, rows, ld):
    """A torch view of a raw device pointer through the CUDA array interface."""
    import torch

    class _Holder:
        pass

    h = _Holder()
    h.__cuda_array_interface__ = {"shape": (rows, ld), "typestr": "<f4", "data": (ptr, False), "version": 3,
                                  "strides": None}
    return torch.as_tensor(h, device="cuda")


@pytest.mark.parametrize("idx", [2, 3, 4])
def test_full_size_configs_on_sampled_columns(nm, idx):
    import torch
    w = workloads.config(idx)
    cols = workloads.sample_columns(w.d, 2500, w.seed)
    period = w.policy_period or w.rounds
    g = o = None
    done = 0
    for epoch in range(w.n_epochs):
        s = w.link_speeds(epoch)
        t, adj = opolicy.iteration_times(s, w.d)
        P, rho, _ = opolicy.generate_policy(t, adj, w.lr, w.K if idx != 4 else 4, w.R if idx != 4 else 4)
        if g is None:
            g = nm.Netmax(M=w.M, d=w.d, lr=w.lr, link_speed_gbps=s, prob=P, rho=rho, sigma=w.sigma,
                          x0_std=w.x0_std, c_std=w.c_std, objective=1, seed=w.seed, trace_rounds=w.rounds + 1)
            o = oracle.Sim(w.M, w.d, P, adj, alpha=w.lr, rho=rho, sigma=w.sigma, objective=1, seed=w.seed, cols=cols)
            o.init(w.x0_std, w.c_std)
        else:
            g.set_policy(link_speed_gbps=s, prob=P, rho=rho)
            o.set_policy(P, adj, rho)
        n = min(period, w.rounds - done)
        g.round(n)
        o.round(n)
        done += n
    assert done == w.rounds
    assert (g.peer_trace() == o.trace()).all()
    assert_replicas_close(g.read_columns(cols), o.x())
    # telemetry of one more round is measured on the state just compared
    want_cons = telemetry_from_device(g)
    g.round(1)
    cons, loss = g.telemetry(w.rounds, 1)
    assert cons[0] == pytest.approx(want_cons, rel=1e-4)
    allcons, allloss = g.telemetry(0, w.rounds)
    assert np.isfinite(allcons).all() and np.isfinite(allloss).all() and (allloss > 0).all()
    assert allcons[-1] < allcons[0]          # replicas are pulled towards consensus
    g.close()
    torch.cuda.empty_cache()


def test_full_size_sampling_stress_config(nm):
    w = workloads.config(5)
    rounds = int(os.environ.get("NETMAX_CFG5_ROUNDS", "1000"))
    s = w.link_speeds(0)
    P = s / s.sum(axis=1, keepdims=True)      # dense heterogeneous rows: an input, not Algorithm 3
    cols = workloads.sample_columns(w.d, 40, w.seed)
    g = nm.Netmax(M=w.M, d=w.d, lr=w.lr, prob=P, sigma=w.sigma, x0_std=w.x0_std, c_std=w.c_std, objective=1,
                  seed=w.seed, trace_rounds=rounds + 1)
    _, rho = g.get_policy()
    o = oracle.Sim(w.M, w.d, P, (1 - np.eye(w.M)).astype(np.uint8), alpha=w.lr, rho=rho, sigma=w.sigma, objective=1,
                   seed=w.seed, cols=cols)
    o.init(w.x0_std, w.c_std)
    g.round(rounds)
    o.round(rounds)
    assert (g.peer_trace() == o.trace()).all()
    assert_replicas_close(g.read_columns(cols), o.x())
    want_cons = telemetry_from_device(g)
    g.round(1)
    assert g.telemetry(rounds, 1)[0][0] == pytest.approx(want_cons, rel=1e-4)
    g.close()
