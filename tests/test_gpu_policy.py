"""GPU policy generator (Algorithm 3 on the device) against the oracle's numpy Algorithm 3 and
the library's host generator."""
import time

import numpy as np
import pytest

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


def _case(name):
    if name.startswith("cfg"):
        w = workloads.config(int(name[3]))
        K, R = {1: (20, 20), 2: (10, 10), 3: (6, 6), 4: (3, 3)}[w.index]
        return opolicy.iteration_times(w.link_speeds(1 if w.index == 3 else 0), w.d) + (w.lr, K, R)
    rng = np.random.default_rng(5)
    M = 7
    s = np.triu(np.exp(rng.uniform(np.log(1.0), np.log(50.0), (M, M))), 1)
    s[0, 4] = s[1, 5] = s[2, 6] = 0.0
    return opolicy.iteration_times(s + s.T, 1_000_000) + (0.05, 8, 8)


@pytest.mark.parametrize("name", ["cfg1", "cfg2", "cfg3", "cfg4", "sparse7"])
def test_device_policy_matches_oracle(nm, name):
    t, adj, lr, K, R = _case(name)
    P, rho, info = nm.netmax_policy_generate_device(t, adj, lr, K, R)
    P0, rho0, info0 = opolicy.generate_policy(t, adj, lr, K, R)
    assert (info["k"], info["r"]) == (info0["k"], info0["r"])
    assert rho == pytest.approx(rho0, rel=1e-14)
    np.testing.assert_allclose(P, P0, atol=1e-9)
    assert info["lam2"] == pytest.approx(info0["lam2"], abs=1e-9)
    assert info["t_conv"] == pytest.approx(info0["t_conv"], rel=1e-6)
    np.testing.assert_allclose(P.sum(axis=1), 1.0, atol=1e-12)


def test_device_policy_matches_host_generator_at_many_workers(nm):
    M = 512
    rng = np.random.default_rng(9)
    s = np.triu(np.exp(rng.uniform(np.log(0.1), np.log(100.0), (M, M))), 1)
    t, adj = nm.netmax_iteration_times(s + s.T, 1024)
    Pd, rhod, infod = nm.netmax_policy_generate_device(t, adj, 0.05, 4, 4)
    Ph, rhoh, infoh = nm.netmax_policy_generate(t, adj, 0.05, 4, 4)
    assert (infod["k"], infod["r"]) == (infoh["k"], infoh["r"]) and rhod == rhoh
    np.testing.assert_allclose(Pd, Ph, atol=1e-10)
    assert infod["lam2"] == pytest.approx(infoh["lam2"], abs=1e-10)
    Y = opolicy.y_matrix(Pd, opolicy.node_probabilities(Pd, t, adj), adj, 0.05, rhod)
    assert infod["lam2"] == pytest.approx(np.linalg.eigvalsh(Y)[-2], abs=1e-9)     # an independent dense solver


def test_device_policy_errors(nm):
    t, adj = opolicy.iteration_times(np.ones((3, 3)) - np.eye(3), 100)
    with pytest.raises(nm.NetmaxError) as e:
        nm.netmax_policy_generate_device(t, adj, -0.1, 4, 4)
    assert e.value.code == -1
    lone = adj.copy()
    lone[0, :] = lone[:, 0] = 0
    with pytest.raises(nm.NetmaxError) as e:
        nm.netmax_policy_generate_device(t, lone, 0.1, 4, 4)
    assert e.value.code == -6
    with pytest.raises(nm.NetmaxError) as e:
        nm.netmax_policy_generate_device(t, adj, 0.1, 4, 4, device=99)
    assert e.value.code == -4


def test_device_policy_on_the_sampling_stress_config(nm):
    """M = 4096: the device generator agrees with the host one and is much faster."""
    w = workloads.config(5)
    t, adj = nm.netmax_iteration_times(w.link_speeds(0), w.d)
    nm.netmax_policy_generate_device(*_case("cfg1")[:2], 0.05, 4, 4)              # warm-up (context, module load)
    t0 = time.perf_counter()
    Pd, rhod, infod = nm.netmax_policy_generate_device(t, adj, w.lr, w.K, w.R)
    dev_s = time.perf_counter() - t0
    t0 = time.perf_counter()
    Ph, rhoh, infoh = nm.netmax_policy_generate(t, adj, w.lr, w.K, w.R)
    host_s = time.perf_counter() - t0
    print(f"\nAlgorithm 3 at M={w.M}, K=R={w.K}: device {dev_s:.2f} s, host {host_s:.2f} s")
    assert (infod["k"], infod["r"]) == (infoh["k"], infoh["r"]) and rhod == rhoh
    np.testing.assert_allclose(Pd, Ph, atol=1e-10)
    assert infod["lam2"] == pytest.approx(infoh["lam2"], abs=1e-9)
    np.testing.assert_allclose(Pd.sum(axis=1), 1.0, atol=1e-12)
    off = ~np.eye(w.M, dtype=bool)
    assert (Pd[off] >= 2 * w.lr * rhod * (1 - 1e-9)).all()                     # Eq. 11 floors
    assert dev_s < host_s
