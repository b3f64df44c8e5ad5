"""GPU parity of the bfloat16-storage option (NETMAX_STORAGE_BF16), through the C ABI.

A stored bfloat16 value is a quantised code, so the comparison is the one for codes: both sides
evaluate Eq. 15-16 in fp32 in the same stated order and round once, to nearest even.
  * Without gradient noise (zero gradients, or sigma = 0) every fp32 operation is the same on
    both sides: replicas must agree bit for bit, over many rounds, in every kernel shape.
  * With noise the kernel's normals come from hardware approximations and differ from the
    oracle's by about 2e-7; after scaling by alpha * sigma that can move a value across a
    rounding boundary only if it lies within a few fp32 units of the boundary.  From a common
    state, after one round, a stored code may therefore differ from the oracle's only by one
    step, and only where the oracle's unrounded value sits at the midpoint of the two codes.
  * Free-running noisy runs are compared statistically (a flipped code is a perturbation of
    one unit that the contraction damps).
Peer traces are bit-exact as always; telemetry within 1e-4 relative."""
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


def bf16_ulp(v):
    """Spacing of the bfloat16 grid at |v| (8 significant bits), for normal numbers."""
    v = np.abs(np.asarray(v, dtype=np.float64))
    e = np.floor(np.log2(np.maximum(v, 2.0 ** -126)))
    return 2.0 ** (e - 7)


def full_adj(M):
    return (1 - np.eye(M)).astype(np.uint8)


def random_policy(M, rng, zeros=0.0):
    P = rng.random((M, M)) + 0.05
    if zeros > 0:
        mask = rng.random((M, M)) < zeros
        mask[np.arange(M), (np.arange(M) + 1) % M] = False
        P[mask] = 0.0
    return P / P.sum(axis=1, keepdims=True)


def pair(nm, M, d, P, lr, sigma, objective, seed, x0_std=1.0, c_std=1.0, trace_rounds=1024, **kw):
    """A bfloat16 context and the oracle in its bfloat16 mode, started from the context's own
    initial state (already on the bfloat16 grid, so the hand-over is exact)."""
    g = nm.Netmax(M=M, d=d, lr=lr, prob=P, sigma=sigma, x0_std=x0_std, c_std=c_std, objective=objective, seed=seed,
                  trace_rounds=trace_rounds, storage="bf16", **kw)
    _, rho = g.get_policy()
    o = oracle.Sim(M, d, P, full_adj(M), alpha=lr, rho=rho, sigma=sigma, objective=objective, seed=seed, storage="bf16",
                   pull_weight=kw.get("pull_weight", 0.0))
    x0, c0 = g.read_replicas(), g.read_centres()
    assert (x0.view(np.uint32) & 0xFFFF == 0).all() and (c0.view(np.uint32) & 0xFFFF == 0).all()
    o.set_x(x0)
    o.set_c(c0)
    return g, o


def assert_codes_match_up_to_ties(gx, o, lr, sigma, x_prev, c):
    """After one round from a common state: see the module docstring."""
    ox, pre = o.x(), o.unrounded().astype(np.float64)
    gx64 = gx.astype(np.float64)
    scale = 1.0 + np.abs(x_prev).astype(np.float64) + np.abs(c) + 4.0 * sigma
    delta = lr * sigma * 2e-6 + 4 * 2.0 ** -24 * scale
    assert (np.abs(gx64 - pre) <= 0.5 * bf16_ulp(gx64) + delta).all()
    differ = gx != ox
    assert differ.mean() < 2e-3, f"{differ.mean():.2e} of the codes differ"
    if differ.any():
        a, b, p = gx64[differ], ox.astype(np.float64)[differ], pre[differ]
        assert (np.abs(a - b) <= 1.0001 * np.maximum(bf16_ulp(a), bf16_ulp(b))).all()   # neighbouring codes
        assert (np.abs(p - 0.5 * (a + b)) <= delta[differ]).all()                        # oracle value on the tie


# ---------------------------------------------------------------- host transfers and initial state
@pytest.mark.parametrize("M,d", [(2, 1), (3, 7), (2, 8), (3, 9), (5, 67), (4, 4096), (7, 4099), (3, 70001)])
def test_inputs_are_rounded_to_nearest_even_and_read_back_exactly(nm, M, d):
    rng = np.random.default_rng(M * 100 + d)
    x = (rng.standard_normal((M, d)) * 10.0 ** rng.integers(-4, 4, (M, d))).astype(np.float32)
    ties = ((rng.integers(0x3F00, 0x4100, (M, d)).astype(np.uint32) << 16) | 0x8000).view(np.float32)
    x = np.where(rng.random((M, d)) < 0.25, ties, x).astype(np.float32)
    c = -x[::-1].copy()
    g = nm.Netmax(M=M, d=d, lr=0.1, prob=random_policy(M, rng), storage="bf16")
    g.set_replicas(x)
    g.set_centres(c)
    assert (g.read_replicas().view(np.uint32) == oracle.bf16_round(x).view(np.uint32)).all()
    assert (g.read_centres().view(np.uint32) == oracle.bf16_round(c).view(np.uint32)).all()
    cols = np.unique(np.concatenate([[0, d - 1], rng.integers(0, d, 20)])).astype(np.int64)
    want = oracle.bf16_round(x)[:, cols]
    assert (g.read_columns(cols) == want).all() and (g.read_columns_static(cols) == want).all()
    # transfers stage through the idle half of the double buffer: the next round must not see leftovers
    g.round(1)
    g.close()


@pytest.mark.parametrize("M,d", [(3, 5), (4, 4096), (7, 4099)])
def test_initial_state_is_the_oracles_up_to_ties(nm, M, d):
    rng = np.random.default_rng(d)
    P = random_policy(M, rng)
    g = nm.Netmax(M=M, d=d, lr=0.05, prob=P, x0_std=1.5, c_std=0.5, seed=d, storage="bf16")
    o = oracle.Sim(M, d, P, full_adj(M), 0.05, 0.1, 0.0, 1, d, storage="bf16")
    o.init(1.5, 0.5)
    f = oracle.Sim(M, d, P, full_adj(M), 0.05, 0.1, 0.0, 1, d)   # fp32 state: the values before the bfloat16 rounding
    f.init(1.5, 0.5)
    for got, want, exact in ((g.read_replicas(), o.x(), f.x()), (g.read_centres(), o.c(), f.c())):
        assert (got.view(np.uint32) & 0xFFFF == 0).all()
        assert (got == want).mean() > 0.999
        assert (np.abs(got.astype(np.float64) - exact) <= 0.5 * bf16_ulp(got) + 4e-6).all()
    g.close()


def test_workspace_is_half_the_size_and_bad_arguments_are_refused(nm):
    M, d = 8, 1_000_000
    full, half = nm.Netmax.workspace_size(M, d), nm.Netmax.workspace_size(M, d, storage="bf16")
    assert 0.45 * full < half < 0.6 * full
    with pytest.raises(nm.NetmaxError) as e:
        nm.Netmax(M=2, d=64, lr=0.1, storage="bf16", element_offset=4)
    assert e.value.code == -1


# ---------------------------------------------------------------- rounds without noise: bit-exact
SHAPES = [(2, 1), (3, 9), (5, 67), (4, 4096), (7, 4099), (8, 70001), (64, 515), (300, 37), (512, 1024), (16, 300_000)]


@pytest.mark.parametrize("objective", [0, 1])
@pytest.mark.parametrize("M,d", SHAPES)
def test_noise_free_rounds_are_bit_exact(nm, M, d, objective):
    rng = np.random.default_rng(M * 7 + d)
    P = random_policy(M, rng, zeros=0.3 if M > 4 else 0.0)
    g, o = pair(nm, M, d, P, 0.07, 0.0, objective, seed=M + d)
    for n in (1, 9, 15):          # one launch per round, then batches (cooperative launches for short vectors)
        g.round(n)
        o.round(n)
    assert (g.peer_trace() == o.trace()).all()
    gx = g.read_replicas()
    assert (gx.view(np.uint32) == o.x().view(np.uint32)).all()
    gc, gl = g.telemetry()
    oc, ol = o.telemetry()
    np.testing.assert_allclose(gc, oc, rtol=1e-4, atol=1e-30)
    np.testing.assert_allclose(gl, ol, rtol=1e-4, atol=1e-30)
    cons, loss = g.measure()
    oc_now, ol_now = o.telemetry_now()
    assert cons == pytest.approx(oc_now, rel=1e-4, abs=1e-30) and loss == pytest.approx(ol_now, rel=1e-4, abs=1e-30)
    g.close()


def test_fixed_pull_weight_is_bit_exact(nm):
    M, d = 6, 1531
    P = random_policy(M, np.random.default_rng(3))
    g, o = pair(nm, M, d, P, 0.05, 0.0, 1, seed=5, pull_weight=0.5)
    g.round(20)
    o.round(20)
    assert (g.read_replicas().view(np.uint32) == o.x().view(np.uint32)).all()
    g.close()


def test_column_shards_reproduce_the_whole(nm):
    """Contexts that hold disjoint column ranges (element_offset, a multiple of 8 here) draw the
    noise the single context draws: GPU against GPU, bit for bit, noise included."""
    M, d, lr, sigma = 5, 4104, 0.05, 0.2
    P = random_policy(M, np.random.default_rng(8))
    whole = nm.Netmax(M=M, d=d, lr=lr, prob=P, rho=0.3, sigma=sigma, x0_std=1.0, c_std=1.0, seed=17, storage="bf16")
    x0, c0 = whole.read_replicas(), whole.read_centres()
    whole.round(12)
    want = whole.read_replicas()
    for lo, hi in ((0, 1000), (1000, 4104)):
        part = nm.Netmax(M=M, d=hi - lo, lr=lr, prob=P, rho=0.3, sigma=sigma, seed=17, storage="bf16", element_offset=lo)
        part.set_replicas(x0[:, lo:hi].copy())
        part.set_centres(c0[:, lo:hi].copy())
        part.round(12)
        assert (part.read_replicas() == want[:, lo:hi]).all()
        part.close()
    whole.close()


# ---------------------------------------------------------------- rounds with noise
@pytest.mark.parametrize("M,d", [(3, 9), (5, 67), (4, 4096), (7, 4099), (64, 515), (512, 1024), (8, 70001)])
def test_noisy_rounds_from_a_common_state_match_up_to_ties(nm, M, d):
    rng = np.random.default_rng(M * 3 + d)
    P = random_policy(M, rng)
    lr, sigma = 0.05, 0.1
    g, o = pair(nm, M, d, P, lr, sigma, 1, seed=d)
    c = o.c()
    for step in range(5):
        x_prev = o.x()
        g.set_replicas(x_prev)       # hand the oracle's state over (exact: it is on the bfloat16 grid)
        g.round(1)
        o.round(1)
        assert_codes_match_up_to_ties(g.read_replicas(), o, lr, sigma, x_prev, c)
    assert (g.peer_trace() == o.trace()).all()
    g.close()


@pytest.mark.parametrize("M,d", [(4, 4096), (64, 515), (8, 70001)])
def test_noisy_free_run_stays_within_a_few_units(nm, M, d):
    rng = np.random.default_rng(M + d)
    P = random_policy(M, rng)
    g, o = pair(nm, M, d, P, 0.05, 0.1, 1, seed=3 * d)
    g.round(60)
    o.round(60)
    assert (g.peer_trace() == o.trace()).all()
    gx, ox = g.read_replicas().astype(np.float64), o.x().astype(np.float64)
    units = np.abs(gx - ox) / bf16_ulp(np.maximum(np.abs(ox), 0.25))
    assert units.max() <= 2.0 and (units > 0).mean() < 2e-3, f"max {units.max():.2f} units, {(units > 0).mean():.2e} differ"
    gc, gl = g.telemetry()
    oc, ol = o.telemetry()
    np.testing.assert_allclose(gc, oc, rtol=1e-3)
    np.testing.assert_allclose(gl, ol, rtol=1e-3)
    g.close()


# ---------------------------------------------------------------- asynchronous timeline
@pytest.mark.parametrize("M,d", [(2, 5), (5, 67), (8, 4099), (64, 515)])
def test_async_steps_without_noise_are_bit_exact(nm, M, d):
    rng = np.random.default_rng(M * 13 + d)
    P = random_policy(M, rng)
    t = rng.uniform(1.0, 4.0, (M, M))
    g, o = pair(nm, M, d, P, 0.05, 0.0, 1, seed=d + 3)
    g.async_begin(t, beta=0.7)
    o.async_begin(t, beta=0.7)
    g.async_steps(12 * M)
    o.async_steps(12 * M)
    assert all((a == b).all() for a, b in zip(g.async_trace(), o.async_trace()))
    assert (g.read_replicas().view(np.uint32) == o.x().view(np.uint32)).all()
    g.close()


def test_async_steps_with_noise_stay_within_a_few_units(nm):
    M, d = 8, 4099
    rng = np.random.default_rng(4)
    P = random_policy(M, rng)
    t = rng.uniform(1.0, 4.0, (M, M))
    g, o = pair(nm, M, d, P, 0.05, 0.1, 1, seed=12)
    g.async_begin(t, beta=0.7)
    o.async_begin(t, beta=0.7)
    g.async_steps(40 * M)
    o.async_steps(40 * M)
    assert all((a == b).all() for a, b in zip(g.async_trace(), o.async_trace()))
    gx, ox = g.read_replicas().astype(np.float64), o.x().astype(np.float64)
    units = np.abs(gx - ox) / bf16_ulp(np.maximum(np.abs(ox), 0.25))
    assert units.max() <= 2.0 and (units > 0).mean() < 2e-3
    g.close()


# ---------------------------------------------------------------- full size, as the benchmark runs it
def _full_size_pair(nm, sigma):
    w = workloads.config(2)
    cols = workloads.sample_columns(w.d, 2500, w.seed)
    t, adj = opolicy.iteration_times(w.link_speeds(0), w.d)
    P, rho, _ = opolicy.generate_policy(t, adj, w.lr, w.K, w.R)
    g = nm.Netmax(M=w.M, d=w.d, lr=w.lr, link_speed_gbps=w.link_speeds(0), prob=P, rho=rho, sigma=sigma, x0_std=w.x0_std,
                  c_std=w.c_std, objective=1, seed=w.seed, trace_rounds=w.rounds + 1, storage="bf16")
    o = oracle.Sim(w.M, w.d, P, adj, alpha=w.lr, rho=rho, sigma=sigma, objective=1, seed=w.seed, cols=cols, storage="bf16")
    o.set_x(g.read_columns(cols))
    o.set_c(g.read_centres()[:, cols])
    return w, cols, g, o


def test_full_size_resnet18_config_without_noise_is_bit_exact_on_sampled_columns(nm):
    import torch
    w, cols, g, o = _full_size_pair(nm, 0.0)
    g.round(w.rounds)
    o.round(w.rounds)
    assert (g.peer_trace() == o.trace()).all()
    assert (g.read_columns(cols).view(np.uint32) == o.x().view(np.uint32)).all()
    g.close()
    torch.cuda.empty_cache()


def test_full_size_resnet18_config_with_noise_on_sampled_columns(nm):
    import torch
    w, cols, g, o = _full_size_pair(nm, workloads.config(2).sigma)
    g.round(w.rounds)
    o.round(w.rounds)
    assert (g.peer_trace() == o.trace()).all()
    gx, ox = g.read_columns(cols).astype(np.float64), o.x().astype(np.float64)
    units = np.abs(gx - ox) / bf16_ulp(np.maximum(np.abs(ox), 0.25 * w.x0_std))
    assert units.max() <= 2.0 and (units > 0).mean() < 2e-3, f"max {units.max():.2f} units, {(units > 0).mean():.2e} differ"
    # telemetry of one more round against a direct evaluation of its definition on the device buffer
    ptr, ld = g.replicas_device()

    class _Holder:
        pass

    h = _Holder()
    h.__cuda_array_interface__ = {"shape": (w.M, ld), "typestr": "<i2", "data": (ptr, False), "version": 3, "strides": None}
    x = torch.as_tensor(h, device="cuda").view(torch.bfloat16)[:, :w.d].double()
    want_cons = float(((x - x.mean(dim=0, keepdim=True)) ** 2).sum().item() / w.M)
    del x
    g.round(1)
    assert g.telemetry(w.rounds, 1)[0][0] == pytest.approx(want_cons, rel=1e-4)
    g.close()
    torch.cuda.empty_cache()
