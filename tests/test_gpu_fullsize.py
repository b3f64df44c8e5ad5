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
        P, rho, _ = opolicy.generate_policy(t, adj, w.lr, w.K, w.R)
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
    rounds = int(os.environ.get("NETMAX_CFG5_ROUNDS", str(w.rounds)))     # all 10,000 rounds (about 200 s of oracle time)
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


def test_maximum_vector_length(nm):
    """d just below the limit (a padded row of 2^32 - 128 bytes), odd so that the tail is ragged:
    every 64-bit offset, the ragged last group and the last elements of the rows are exercised.
    26 GB of device memory; the oracle follows a sample of columns."""
    import torch
    d, M = (1 << 30) - 33, 2
    free, _ = torch.cuda.mem_get_info()
    if free < 40 * (1 << 30):
        pytest.skip("needs 40 GB of free device memory")
    P = np.array([[0.1, 0.9], [0.7, 0.3]])
    adj = (1 - np.eye(M)).astype(np.uint8)
    cols = workloads.sample_columns(d, 3000, 77)
    assert cols[-1] == d - 1
    g = nm.Netmax(M=M, d=d, lr=0.1, prob=P, sigma=0.05, x0_std=1.0, c_std=1.0, objective=1, seed=77, trace_rounds=8)
    _, rho = g.get_policy()
    o = oracle.Sim(M, d, P, adj, alpha=0.1, rho=rho, sigma=0.05, objective=1, seed=77, cols=cols)
    o.init(1.0, 1.0)
    g.round(3)
    o.round(3)
    assert (g.peer_trace() == o.trace()).all()
    assert_replicas_close(g.read_columns(cols), o.x())
    ptr, ld = g.replicas_device()
    assert ld * 4 == (1 << 32) - 128
    pad = _as_tensor(ptr, M, ld)[:, d:]
    assert pad.numel() == M * (ld - d) and float(pad.abs().max().item()) == 0.0      # padding stays zero
    want_cons = telemetry_from_device(g)
    g.round(1)
    assert g.telemetry(3, 1)[0][0] == pytest.approx(want_cons, rel=1e-4)
    g.close()
    torch.cuda.empty_cache()
    with pytest.raises(nm.NetmaxError) as e:
        nm.Netmax(M=M, d=(1 << 30) - 32, lr=0.1, prob=P)
    assert e.value.code == -1


def test_maximum_worker_count(nm):
    """M at its limit (16384 workers, 1 GB threshold table, 1 GB weight table), short vectors."""
    M, d, rounds = 16384, 8, 3
    rng = np.random.default_rng(5)
    P = rng.random((M, M), dtype=np.float32).astype(np.float64)
    P[rng.random((M, M), dtype=np.float32) < 0.5] = 0.0
    P[np.arange(M), (np.arange(M) + 1) % M] = 1.0
    np.fill_diagonal(P, 0.0)
    P /= P.sum(axis=1, keepdims=True)
    adj = np.ones((M, M), dtype=np.uint8)
    np.fill_diagonal(adj, 0)
    g = nm.Netmax(M=M, d=d, lr=0.05, prob=P, sigma=0.1, x0_std=1.0, c_std=1.0, objective=1, seed=9, trace_rounds=4)
    _, rho = g.get_policy()
    o = oracle.Sim(M, d, P, adj, alpha=0.05, rho=rho, sigma=0.1, objective=1, seed=9)
    o.init(1.0, 1.0)
    g.round(rounds)
    o.round(rounds)
    assert (g.peer_trace() == o.trace()).all()
    assert_replicas_close(g.read_replicas(), o.x())
    gc, gl = g.telemetry()
    oc, ol = o.telemetry()
    np.testing.assert_allclose(gc, oc, rtol=1e-4)
    np.testing.assert_allclose(gl, ol, rtol=1e-4)
    g.close()
    with pytest.raises(nm.NetmaxError) as e:
        nm.Netmax(M=M + 1, d=d, lr=0.05)
    assert e.value.code == -1
