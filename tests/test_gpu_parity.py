"""GPU parity: the CUDA library (through its C ABI) against the CPU oracle, element by element,
on the same seeded inputs.  Peer traces must be bit-exact; fp32 replicas must agree within
|delta| <= 1e-5 (1 + |x|); telemetry within 1e-4 relative (its summation order differs)."""
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
    worst = np.unravel_index(np.argmax(excess), excess.shape)
    assert excess.max() <= 0.0, f"max excess {excess.max():.3e} at {worst}: {got[worst]} vs {want[worst]}"


def full_adj(M):
    return (1 - np.eye(M)).astype(np.uint8)


def random_policy(M, rng, self_prob=True, zeros=0.0):
    P = rng.random((M, M)) + 0.05
    if zeros > 0:
        mask = rng.random((M, M)) < zeros
        mask[np.arange(M), (np.arange(M) + 1) % M] = False
        P[mask] = 0.0
    if not self_prob:
        np.fill_diagonal(P, 0.0)
    return P / P.sum(axis=1, keepdims=True)


def pair(nm, M, d, P, lr, sigma, objective, seed, x0_std=1.0, c_std=1.0, rho=0.0, trace_rounds=1024):
    """The library context and the oracle simulator on the same inputs."""
    g = nm.Netmax(M=M, d=d, lr=lr, prob=P, rho=rho, sigma=sigma, x0_std=x0_std, c_std=c_std,
                  objective=objective, seed=seed, trace_rounds=trace_rounds)
    _, rho_used = g.get_policy()
    o = oracle.Sim(M, d, P, full_adj(M), alpha=lr, rho=rho_used, sigma=sigma, objective=objective, seed=seed)
    o.init(x0_std, c_std)
    return g, o


# ---------------------------------------------------------------- initial state and sampler
@pytest.mark.parametrize("M,d", [(2, 1), (3, 2), (4, 3), (3, 5), (5, 67), (4, 4096), (7, 4099), (2, 70001)])
def test_initial_state_matches_oracle(nm, M, d):
    rng = np.random.default_rng(M * 1000 + d)
    g, o = pair(nm, M, d, random_policy(M, rng), 0.05, 0.1, 1, seed=d, x0_std=1.5, c_std=0.5)
    np.testing.assert_allclose(g.read_replicas(), o.x(), atol=2e-6, rtol=2e-6)
    np.testing.assert_allclose(g.read_centres(), o.c(), atol=2e-6, rtol=2e-6)
    g.close()


@pytest.mark.parametrize("M", [2, 5, 64, 257, 1000])
def test_peer_sampler_is_bit_exact(nm, M):
    import torch
    rng = np.random.default_rng(M)
    P = random_policy(M, rng, zeros=0.4)
    g = nm.Netmax(M=M, d=8, lr=0.01, prob=P, seed=77 + M)
    rounds, first = 300, 12345678901
    out = torch.empty((rounds, M), dtype=torch.int32, device="cuda")
    g.sample_peers(first, rounds, out.data_ptr())
    torch.cuda.synchronize()
    want = oracle.peer_draws(P, 77 + M, first, rounds)
    assert (out.cpu().numpy() == want).all()
    assert (P[np.arange(M)[None, :].repeat(rounds, 0), want] > 0).all()
    g.close()


def test_peer_frequencies_chi_square_on_the_gpu(nm):
    import torch
    from scipy import stats
    w = workloads.config(1)
    t, adj = opolicy.iteration_times(w.link_speeds(0), w.d)
    P, rho, _ = opolicy.generate_policy(t, adj, w.lr, w.K, w.R)
    g = nm.Netmax(M=w.M, d=w.d, lr=w.lr, prob=P, rho=rho, seed=w.seed)
    rounds = 20000
    out = torch.empty((rounds, w.M), dtype=torch.int32, device="cuda")
    g.sample_peers(0, rounds, out.data_ptr())
    draws = out.cpu().numpy()
    for i in range(w.M):
        keep = P[i] > 0
        counts = np.bincount(draws[:, i], minlength=w.M)
        assert (counts[~keep] == 0).all()
        assert stats.chisquare(counts[keep], rounds * P[i][keep]).pvalue > 1e-3 / w.M
    g.close()


# ---------------------------------------------------------------- rounds, small shapes
SHAPES = [(2, 1), (2, 2), (3, 3), (4, 5), (5, 67), (8, 1000), (4, 4096), (6, 4099), (16, 3001), (3, 70001),
          (64, 515), (130, 37)]


@pytest.mark.parametrize("M,d", SHAPES)
def test_rounds_match_oracle_quadratic(nm, M, d):
    rng = np.random.default_rng(M * 7 + d)
    P = random_policy(M, rng, zeros=0.2)
    g, o = pair(nm, M, d, P, lr=0.05, sigma=0.1, objective=1, seed=1000 + d)
    x0 = rng.standard_normal((M, d)).astype(np.float32)
    c = rng.standard_normal((M, d)).astype(np.float32)
    g.set_replicas(x0)
    g.set_centres(c)
    o.set_x(x0)
    o.set_c(c)
    rounds = 40
    g.round(rounds)
    o.round(rounds)
    assert (g.peer_trace() == o.trace()).all()
    assert_replicas_close(g.read_replicas(), o.x())
    gc, gl = g.telemetry()
    oc, ol = o.telemetry()
    np.testing.assert_allclose(gc, oc, rtol=1e-4, atol=1e-9)
    np.testing.assert_allclose(gl, ol, rtol=1e-4, atol=1e-9)
    g.close()


@pytest.mark.parametrize("M,d", [(2, 5), (5, 67), (8, 4099), (64, 515)])
def test_rounds_match_oracle_zero_gradient(nm, M, d):
    rng = np.random.default_rng(M + d)
    P = random_policy(M, rng)
    g, o = pair(nm, M, d, P, lr=0.1, sigma=0.3, objective=0, seed=5)
    g.round(60)
    o.round(60)
    assert (g.peer_trace() == o.trace()).all()
    assert_replicas_close(g.read_replicas(), o.x())
    gc, _ = g.telemetry()
    oc, _ = o.telemetry()
    np.testing.assert_allclose(gc, oc, rtol=1e-4, atol=1e-9)
    assert gc[-1] < gc[0]
    g.close()


def test_zero_gradient_identical_replicas_do_not_move(nm):
    rng = np.random.default_rng(3)
    M, d = 6, 1003
    g = nm.Netmax(M=M, d=d, lr=0.1, prob=random_policy(M, rng), sigma=0.5, objective=0, seed=9)
    x0 = np.tile(rng.standard_normal(d).astype(np.float32), (M, 1))
    g.set_replicas(x0)
    g.round(25)
    assert (g.read_replicas() == x0).all()
    cons, _ = g.telemetry()
    assert (cons == 0.0).all()
    g.close()


def test_self_draw_rows_take_a_plain_sgd_step(nm):
    M, d, lr = 3, 130, 0.25
    rng = np.random.default_rng(4)
    x0 = rng.standard_normal((M, d)).astype(np.float32)
    c = rng.standard_normal((M, d)).astype(np.float32)
    g = nm.Netmax(M=M, d=d, lr=lr, prob=np.eye(M), rho=0.5, sigma=0.0, objective=1, seed=1)
    g.set_replicas(x0)
    g.set_centres(c)
    g.round(1)
    want = x0.astype(np.float64) - np.float64(np.float32(lr)) * (x0.astype(np.float64) - c)
    np.testing.assert_allclose(g.read_replicas(), want, rtol=3e-7, atol=1e-7)
    assert (g.peer_trace() == np.arange(M)).all()
    g.close()


def test_m2_closed_form_on_the_gpu(nm):
    lr, rho, d, rounds = 0.2, 1.0, 64, 30
    P = np.array([[0.0, 1.0], [1.0, 0.0]])
    rng = np.random.default_rng(6)
    x0 = rng.standard_normal((2, d)).astype(np.float32)
    c = rng.standard_normal((2, d)).astype(np.float32)
    g = nm.Netmax(M=2, d=d, lr=lr, prob=P, rho=rho, sigma=0.0, objective=1, seed=2)
    g.set_replicas(x0)
    g.set_centres(c)
    g.round(rounds)
    x = g.read_replicas().astype(np.float64)
    a = float(np.float32(lr))
    w = float(np.float32(a * rho))
    C, dc = c[0].astype(np.float64) + c[1], c[0].astype(np.float64) - c[1]
    s0, d0 = x0[0].astype(np.float64) + x0[1], x0[0].astype(np.float64) - x0[1]
    dstar = (1 - w) * a * dc / (a * (1 - w) + 2 * w)
    np.testing.assert_allclose(x[0] + x[1], C + (1 - a * (1 - w)) ** rounds * (s0 - C), atol=5e-6)
    np.testing.assert_allclose(x[0] - x[1], dstar + ((1 - w) * (1 - a) - w) ** rounds * (d0 - dstar), atol=5e-6)
    g.close()


def test_split_calls_change_no_bit_and_ring_wraps(nm):
    rng = np.random.default_rng(8)
    M, d = 5, 2051
    P = random_policy(M, rng)
    kw = dict(M=M, d=d, lr=0.05, prob=P, sigma=0.1, x0_std=1.0, c_std=1.0, objective=1, seed=11, trace_rounds=16)
    a, b = nm.Netmax(**kw), nm.Netmax(**kw)
    a.round(37)
    for n in (1, 0, 15, 16, 5):
        b.round(n)
    assert a.rounds_done == b.rounds_done == 37
    assert (a.read_replicas() == b.read_replicas()).all()
    assert (a.peer_trace(21, 16) == b.peer_trace(21, 16)).all()
    ta, tb = a.telemetry(21, 16), b.telemetry(21, 16)
    assert (ta[0] == tb[0]).all() and (ta[1] == tb[1]).all()
    o = oracle.Sim(M, d, P, full_adj(M), alpha=0.05, rho=a.get_policy()[1], sigma=0.1, objective=1, seed=11)
    o.init(1.0, 1.0)
    o.round(37)
    assert (a.peer_trace(21, 16) == o.trace(21, 16)).all()
    with pytest.raises(nm.NetmaxError) as e:
        a.peer_trace(20, 17)
    assert e.value.code == -5
    with pytest.raises(nm.NetmaxError):
        a.telemetry(30, 8)
    a.close()
    b.close()


def test_policy_refresh_between_rounds(nm):
    rng = np.random.default_rng(10)
    M, d = 6, 777
    P1, P2 = random_policy(M, rng), random_policy(M, rng, zeros=0.3)
    g, o = pair(nm, M, d, P1, lr=0.05, sigma=0.05, objective=1, seed=21)
    g.round(7)
    o.round(7)
    g.set_policy(prob=P2)
    o.set_policy(P2, full_adj(M), g.get_policy()[1])
    g.round(9)
    o.round(9)
    assert (g.peer_trace() == o.trace()).all()
    assert_replicas_close(g.read_replicas(), o.x())
    with pytest.raises(nm.NetmaxError):
        g.set_policy(prob=P2 * 1.1)
    g.round(1)
    o.round(1)
    assert (g.peer_trace(16, 1) == o.trace(16, 1)).all()
    g.close()


def test_caller_owned_workspace_and_stream(nm):
    import torch
    M, d = 4, 1234
    rng = np.random.default_rng(12)
    P = random_policy(M, rng)
    size = nm.Netmax.workspace_size(M, d, 64)
    ws = torch.empty(size + 256, dtype=torch.uint8, device="cuda")
    ptr = (ws.data_ptr() + 255) // 256 * 256
    stream = torch.cuda.Stream()
    g = nm.Netmax(M=M, d=d, lr=0.05, prob=P, sigma=0.1, x0_std=1.0, c_std=1.0, seed=3, trace_rounds=64,
                  stream=stream.cuda_stream, workspace=ptr, workspace_bytes=size)
    h = nm.Netmax(M=M, d=d, lr=0.05, prob=P, sigma=0.1, x0_std=1.0, c_std=1.0, seed=3, trace_rounds=64)
    g.round(10)
    h.round(10)
    assert (g.read_replicas() == h.read_replicas()).all()
    dev_ptr, ld = g.replicas_device()
    assert ld >= d and ptr <= dev_ptr < ptr + size
    with pytest.raises(nm.NetmaxError) as e:
        nm.Netmax(M=M, d=d, lr=0.05, prob=P, workspace=ptr, workspace_bytes=size // 2, trace_rounds=64)
    assert e.value.code == -3
    g.close()
    h.close()
    del ws


def test_read_columns_matches_full_read(nm):
    M, d = 5, 9001
    g = nm.Netmax(M=M, d=d, lr=0.05, prob=random_policy(M, np.random.default_rng(13)), sigma=0.1, x0_std=1.0,
                  c_std=1.0, seed=4)
    g.round(3)
    cols = workloads.sample_columns(d, 200, 5)
    assert (g.read_columns(cols) == g.read_replicas()[:, cols]).all()
    with pytest.raises(nm.NetmaxError):
        g.read_columns(np.array([d]))
    g.close()


@pytest.mark.parametrize("M,d", [(1024, 16_387), (2048, 8_195), (4096, 4_099)])
def test_many_workers_with_longer_vectors(nm, M, d):
    """So many rows that a tile of all of them would hold less than 128 bytes of each: the rows are split into
    groups instead (the short-vector launch shape), whatever the length of the vectors."""
    s = workloads.config(5).link_speeds(0)[:M, :M]
    P = s / s.sum(axis=1, keepdims=True)
    cols = np.unique(np.concatenate([np.arange(40), np.random.default_rng(d).integers(0, d, 600), np.arange(d - 40, d)])).astype(np.int64)
    g = nm.Netmax(M=M, d=d, lr=0.05, prob=P, sigma=0.1, x0_std=1.0, c_std=1.0, objective=1, seed=M + d, trace_rounds=16)
    o = oracle.Sim(M, d, P, full_adj(M), alpha=0.05, rho=g.get_policy()[1], sigma=0.1, objective=1, seed=M + d, cols=cols)
    o.init(1.0, 1.0)
    rounds = 6
    g.round(1)
    g.round(rounds - 1)
    o.round(rounds, threads=8)
    assert (g.peer_trace(0, rounds) == o.trace(0, rounds)).all()
    assert_replicas_close(g.read_columns(cols), o.x())
    # telemetry of the last round against its definition on the device buffer of the round before
    one = nm.Netmax(M=M, d=d, lr=0.05, prob=P, sigma=0.1, x0_std=1.0, c_std=1.0, objective=1, seed=M + d, trace_rounds=16, fuse_rounds=1)
    one.round(rounds)
    assert (one.read_replicas().view(np.uint32) == g.read_replicas().view(np.uint32)).all()
    np.testing.assert_allclose(g.telemetry(0, rounds)[0], one.telemetry(0, rounds)[0], rtol=2e-5)
    x = one.read_replicas().astype(np.float64)
    one.round(1)
    want = ((x - x.mean(axis=0)) ** 2).sum() / M
    assert one.telemetry(rounds, 1)[0][0] == pytest.approx(want, rel=1e-4)
    g.close()
    one.close()


def test_many_workers_small_vectors(nm):
    """The sampling-stress shape at reduced round count: M = 4096, d = 1024."""
    w = workloads.config(5)
    s = w.link_speeds(0)
    P = s / s.sum(axis=1, keepdims=True)          # a dense heterogeneous policy (an input, not Algorithm 3)
    g, o = pair(nm, w.M, w.d, P, lr=w.lr, sigma=w.sigma, objective=1, seed=w.seed, x0_std=w.x0_std, c_std=w.c_std)
    rounds = 20
    g.round(rounds)
    o.round(rounds, threads=8)
    assert (g.peer_trace() == o.trace()).all()
    assert_replicas_close(g.read_replicas(), o.x())
    gc, gl = g.telemetry()
    oc, ol = o.telemetry()
    np.testing.assert_allclose(gc, oc, rtol=1e-4)
    np.testing.assert_allclose(gl, ol, rtol=1e-4)
    g.close()


def test_column_shards_match_the_unsharded_problem(nm):
    """Two contexts holding disjoint column ranges (element_offset) of one problem reproduce the
    oracle's run of the whole problem: same peers, same noise streams, no exchange."""
    M, d, rounds = 5, 3001, 15
    d4 = (d + 3) // 4 * 4
    rng = np.random.default_rng(23)
    P = random_policy(M, rng)
    parts = []
    for rank in range(2):
        g = nm.Netmax(M=M, d=d, lr=0.05, prob=P, sigma=0.1, x0_std=1.0, c_std=1.0, seed=41,
                      element_offset=rank * d4)
        g.round(rounds)
        parts.append(g)
    rho = parts[0].get_policy()[1]
    cols = np.concatenate([rank * d4 + np.arange(d, dtype=np.int64) for rank in range(2)])
    o = oracle.Sim(M, 2 * d4, P, full_adj(M), alpha=0.05, rho=rho, sigma=0.1, objective=1, seed=41, cols=cols)
    o.init(1.0, 1.0)
    o.round(rounds)
    got = np.concatenate([g.read_replicas() for g in parts], axis=1)
    assert_replicas_close(got, o.x())
    assert (parts[0].peer_trace() == o.trace()).all() and (parts[1].peer_trace() == o.trace()).all()
    oc, ol = o.telemetry()
    gc = parts[0].telemetry()[0] + parts[1].telemetry()[0]
    gl = parts[0].telemetry()[1] + parts[1].telemetry()[1]
    np.testing.assert_allclose(gc, oc, rtol=1e-4)
    np.testing.assert_allclose(gl, ol, rtol=1e-4)
    with pytest.raises(nm.NetmaxError):
        nm.Netmax(M=M, d=d, lr=0.05, prob=P, element_offset=2)
    for g in parts:
        g.close()


@pytest.mark.parametrize("M,d", [(2, 9), (6, 4099), (64, 515)])
def test_fixed_pull_weight_matches_oracle(nm, M, d):
    """The gossip / AD-PSGD style rule: every pull averages with a constant weight."""
    rng = np.random.default_rng(M + 7 * d)
    P = random_policy(M, rng)
    g = nm.Netmax(M=M, d=d, lr=0.05, prob=P, sigma=0.1, x0_std=1.0, c_std=1.0, objective=1, seed=17, pull_weight=0.5)
    o = oracle.Sim(M, d, P, full_adj(M), alpha=0.05, rho=g.get_policy()[1], sigma=0.1, objective=1, seed=17,
                   pull_weight=0.5)
    o.init(1.0, 1.0)
    g.round(25)
    o.round(25)
    assert (g.peer_trace() == o.trace()).all()
    assert_replicas_close(g.read_replicas(), o.x())
    with pytest.raises(nm.NetmaxError):
        nm.Netmax(M=M, d=d, lr=0.05, prob=P, pull_weight=1.0)
    g.close()


def test_sparse_graph_with_clustered_centres(nm):
    """A ring of machines (most d_im = 0) and non-IID-like objectives: centres clustered by machine."""
    M, d, gsz = 12, 6007, 4
    s = workloads.sparse_ring_of_groups(M, gsz, 100.0, 5.0)
    t, adj = opolicy.iteration_times(s, 5_000_000)
    assert adj.sum() < M * (M - 1) / 2
    P, rho, _ = opolicy.generate_policy(t, adj, 0.05, 20, 20)   # slow ring links leave only small rho feasible
    assert (P[(adj == 0) & ~np.eye(M, dtype=bool)] == 0).all()
    c = workloads.clustered_centres(M, d, gsz, spread=1.0, within=0.05, seed=3)
    g = nm.Netmax(M=M, d=d, lr=0.05, link_speed_gbps=s, prob=P, rho=rho, sigma=0.05, x0_std=1.0, objective=1, seed=29)
    o = oracle.Sim(M, d, P, adj, alpha=0.05, rho=rho, sigma=0.05, objective=1, seed=29)
    o.init(1.0, 0.0)
    g.set_centres(c)
    o.set_c(c)
    g.round(200)
    o.round(200)
    assert (g.peer_trace(0, 200) == o.trace()).all()
    assert_replicas_close(g.read_replicas(), o.x())
    cons, loss = g.telemetry(0, 200)
    assert cons[-1] < 0.8 * cons[0]          # clustered optima and a weak coupling keep machines apart
    # the library's own Algorithm 3 on the same sparse graph gives the same policy
    h = nm.Netmax(M=M, d=5_000_000, lr=0.05, link_speed_gbps=s, policy_K=20, policy_R=20)
    np.testing.assert_allclose(h.get_policy()[0], P, atol=1e-9)
    with pytest.raises(nm.NetmaxError) as e:
        bad = P.copy()
        bad[0, 5] = 0.01
        bad[0] /= bad[0].sum()
        nm.Netmax(M=M, d=d, lr=0.05, link_speed_gbps=s, prob=bad)
    assert e.value.code == -2                              # Eq. 12: no probability on a missing link
    g.close()
    h.close()


def test_a_barrier_wait_that_runs_out_is_reported_and_the_context_survives(nm):
    """The multi-round launch polls its grid barrier a bounded number of times.  Made to wait for
    CTAs that do not exist, it gives up, the next synchronising call reports the error, and the
    same context then runs correctly again (no fault, no hang)."""
    import time
    M, d = 4, 4096
    rng = np.random.default_rng(33)
    P = random_policy(M, rng)
    x0 = rng.standard_normal((M, d)).astype(np.float32)
    # fuse_rounds = 1 keeps nothing resident on chip across rounds, which is what sends a short-vector
    # batch through the cooperative launch whose grid barrier is under test
    kw = dict(M=M, d=d, lr=0.05, prob=P, sigma=0.1, c_std=1.0, seed=3, fuse_rounds=1)
    g, ref = nm.Netmax(**kw), nm.Netmax(**kw)
    g.set_replicas(x0)
    g.debug_absent_ctas(1)
    t0 = time.perf_counter()
    g.round(5)
    with pytest.raises(nm.NetmaxError) as e:
        g.read_replicas()
    assert e.value.code == -4 and "barrier" in str(e.value)
    assert time.perf_counter() - t0 < 60.0
    # the context is still usable: rounds 5.. from a fresh state equal an undisturbed context's
    g.set_replicas(x0)
    ref.set_replicas(x0)
    ref.round(5)
    ref.set_replicas(x0)
    g.round(6)
    ref.round(6)
    assert (g.read_replicas() == ref.read_replicas()).all()
    assert (g.peer_trace(5, 6) == ref.peer_trace(5, 6)).all()
    g.close()
    ref.close()


def test_fast_gaussian_noise_stays_within_its_error_bound(nm):
    """The kernel's normals (hardware lg2 / sqrt / sin / cos approximations) against the oracle's
    fp64 Box-Muller on the same Philox words: with x = c = 0 and self-draws only, one round leaves
    x' = -alpha sigma z.  Typical error ~2e-7; the bound for radii below 1e-3 is 6e-4."""
    M, d, lr, sigma = 2, 2_000_003, 0.5, 0.5
    g = nm.Netmax(M=M, d=d, lr=lr, prob=np.eye(M), rho=0.1, sigma=sigma, objective=1, seed=123)
    g.round(1)
    z_gpu = -g.read_replicas().astype(np.float64) / (lr * sigma)
    err = np.concatenate([np.abs(z_gpu[i] - oracle.noise(123, i, 0, 0, d)) for i in range(M)])
    assert err.max() < 6e-4
    assert np.quantile(err, 0.9999) < 3e-6
    assert np.median(err) < 2e-7
    assert abs(z_gpu.mean()) < 4.0 / np.sqrt(z_gpu.size) and abs(z_gpu.var() - 1.0) < 4.0 * np.sqrt(2.0 / z_gpu.size)
    g.close()


def test_short_form_create(nm):
    """netmax_create(M, d, link_speed, prob, lr, seed): objective 1, sigma 0, unit-variance start."""
    import ctypes as C
    M, d = 4, 777
    P = random_policy(M, np.random.default_rng(44))
    L = nm.lib()
    h = C.c_void_p()
    assert L.netmax_create(M, d, None, P.ctypes.data_as(C.c_void_p), 0.05, 1234, C.byref(h)) == 0
    assert L.netmax_round(h, 9) == 0 and L.netmax_rounds_done(h) == 9
    out = np.empty((M, d), dtype=np.float32)
    assert L.netmax_read_replicas(h, out.ctypes.data_as(C.c_void_p)) == 0
    L.netmax_destroy(h)
    g = nm.Netmax(M=M, d=d, lr=0.05, prob=P, sigma=0.0, x0_std=1.0, c_std=1.0, objective=1, seed=1234)
    g.round(9)
    assert (g.read_replicas() == out).all()
    g.close()
    # prob = NULL: Algorithm 3 on equal link speeds gives uniform neighbour choice
    assert L.netmax_create(M, d, None, None, 0.05, 1, C.byref(h)) == 0
    Pu = np.empty((M, M))
    rho = C.c_double()
    assert L.netmax_get_policy(h, Pu.ctypes.data_as(C.c_void_p), C.byref(rho)) == 0
    off = ~np.eye(M, dtype=bool)
    assert np.ptp(Pu[off]) < 1e-12 and rho.value > 0
    L.netmax_destroy(h)
