"""GPU parity of the launch shape for short vectors that keeps whole columns (all M rows of a few
column groups) resident in shared memory for every round of a call.  Replicas and peer traces
must equal, bit for bit, those of the launch shapes that keep nothing on chip across rounds
(fuse_rounds = 1), and match the CPU oracle within the fp32 tolerance; telemetry sums are
accumulated in a different order and agree to fp32 rounding."""
import numpy as np
import pytest

from oracle import oracle

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


def full_adj(M):
    return (1 - np.eye(M)).astype(np.uint8)


def random_policy(M, rng, zeros=0.0):
    P = rng.random((M, M)) + 0.05
    if zeros > 0:
        mask = rng.random((M, M)) < zeros
        mask[np.arange(M), (np.arange(M) + 1) % M] = False
        P[mask] = 0.0
    return P / P.sum(axis=1, keepdims=True)


# a thread per column group (small M), rows split over threads (larger M), ragged tails, one column,
# more tiles than resident CTAs, the largest M that still fits (a 4-element column of 4700 rows)
SHAPES = [(2, 1), (3, 9), (4, 4096), (7, 4099), (5, 67), (2, 280_001), (66, 515), (67, 515), (130, 37), (300, 1030),
          (512, 1024), (1000, 131), (4096, 64), (4700, 7)]


@pytest.mark.parametrize("storage", ["f32", "bf16"])
@pytest.mark.parametrize("M,d", SHAPES)
def test_resident_columns_change_no_bit(nm, M, d, storage):
    rng = np.random.default_rng(M * 5 + d)
    P = random_policy(M, rng, zeros=0.3 if M > 4 else 0.0)
    kw = dict(M=M, d=d, lr=0.05, prob=P, sigma=0.1, x0_std=1.0, c_std=1.0, objective=1, seed=d + M, trace_rounds=16,
              storage=storage)
    plain = nm.Netmax(fuse_rounds=1, **kw)
    res = nm.Netmax(**kw)
    rounds = 0
    for n in (1, 7, 16, 2, 11):              # single rounds, batches, a full lap of the ring and a wrap
        launches = res.kernel_launches
        plain.round(n)
        res.round(n)
        rounds += n
        if n >= 2:                           # (a single round does not repay bringing the columns on chip)
            assert res.kernel_launches - launches == 3, "the rounds did not run on resident columns"
        else:
            assert res.kernel_launches - launches == 2, "a single round should take the per-round kernel"
    xa, xb = plain.read_replicas(), res.read_replicas()
    assert (xa.view(np.uint32) == xb.view(np.uint32)).all()
    assert (plain.peer_trace(rounds - 16, 16) == res.peer_trace(rounds - 16, 16)).all()
    (ca, la), (cb, lb) = plain.telemetry(rounds - 16, 16), res.telemetry(rounds - 16, 16)
    np.testing.assert_allclose(cb, ca, rtol=2e-5)
    np.testing.assert_allclose(lb, la, rtol=2e-5)
    plain.close()
    res.close()


def test_short_calls_do_not_pay_for_bringing_the_columns_on_chip(nm):
    """Resident columns are loaded and stored once per call; a call takes that shape only from the number of rounds at
    which it was measured to pay (2 up to a million elements, 6 up to four million, then 8 and 16)."""
    for M, d, short, long_ in ((4, 4096, 1, 2), (4096, 1024, 4, 6), (1024, 8192, 7, 8)):
        P = np.full((M, M), 1.0 / (M - 1))
        np.fill_diagonal(P, 0.0)
        kw = dict(M=M, d=d, lr=0.05, prob=P, sigma=0.1, x0_std=1.0, c_std=1.0, objective=1, seed=5, trace_rounds=32)
        a, b = nm.Netmax(**kw), nm.Netmax(fuse_rounds=1, **kw)
        for n, resident in ((short, False), (long_, True), (short, False)):
            before = a.kernel_launches
            a.round(n)
            b.round(n)
            launches = a.kernel_launches - before          # sampler + (resident kernel + tile sums | per-round kernels)
            assert (launches == 3) == resident, (M, d, n, launches)
        assert (a.read_replicas().view(np.uint32) == b.read_replicas().view(np.uint32)).all()
        assert (a.peer_trace() == b.peer_trace()).all()
        a.close()
        b.close()


@pytest.mark.parametrize("M,d", [(5048, 146), (5040, 9), (6000, 33)])
def test_more_workers_than_fit_on_chip(nm, M, d):
    """Beyond about 4700 workers the columns do not fit a CTA's shared memory and the per-round kernels run; around
    M = 5040 their table of draws needs just under 48 KB of dynamic shared memory, which with the kernels' static
    part is over the default limit (such a context once failed to plan its launch)."""
    rng = np.random.default_rng(M + d)
    P = random_policy(M, rng, zeros=0.5)
    kw = dict(M=M, d=d, lr=0.05, prob=P, sigma=0.1, x0_std=1.0, c_std=1.0, objective=1, seed=M, trace_rounds=8)
    one, many = nm.Netmax(fuse_rounds=1, **kw), nm.Netmax(**kw)
    o = oracle.Sim(M, d, P, full_adj(M), alpha=0.05, rho=one.get_policy()[1], sigma=0.1, objective=1, seed=M)
    o.init(1.0, 1.0)
    o.set_x(one.read_replicas())                       # (the two sides' initial normals differ in the last bit)
    o.set_c(one.read_centres())
    for n in (1, 5):
        one.round(n)
        many.round(n)
        o.round(n)
    xa, xb, xo = one.read_replicas(), many.read_replicas(), o.x().astype(np.float64)
    assert (xa.view(np.uint32) == xb.view(np.uint32)).all()
    assert (one.peer_trace(0, 6) == o.trace(0, 6)).all() and (many.peer_trace(0, 6) == o.trace(0, 6)).all()
    assert (np.abs(xa.astype(np.float64) - xo) <= TOL * (1.0 + np.abs(xo))).all()
    one.close()
    many.close()


@pytest.mark.parametrize("objective", [0, 1])
@pytest.mark.parametrize("M,d", [(4, 4096), (6, 4099), (64, 515), (130, 37), (1000, 131)])
def test_resident_columns_match_the_oracle(nm, M, d, objective):
    rng = np.random.default_rng(M + d)
    P = random_policy(M, rng, zeros=0.2)
    g = nm.Netmax(M=M, d=d, lr=0.05, prob=P, sigma=0.1, x0_std=1.0, c_std=1.0, objective=objective, seed=9, trace_rounds=64)
    o = oracle.Sim(M, d, P, full_adj(M), alpha=0.05, rho=g.get_policy()[1], sigma=0.1, objective=objective, seed=9)
    o.init(1.0, 1.0)
    x0, c0 = g.read_replicas(), g.read_centres()       # (the two sides' initial normals differ in the last bit)
    o.set_x(x0)
    o.set_c(c0)
    for n in (30, 1, 9):
        g.round(n)
        o.round(n)
    assert (g.peer_trace() == o.trace()).all()
    got, want = g.read_replicas().astype(np.float64), o.x().astype(np.float64)
    assert (np.abs(got - want) <= TOL * (1.0 + np.abs(want))).all()
    gc, gl = g.telemetry()
    oc, ol = o.telemetry()
    np.testing.assert_allclose(gc, oc, rtol=1e-4, atol=1e-9)
    np.testing.assert_allclose(gl, ol, rtol=1e-4, atol=1e-9)
    g.close()


def test_split_calls_change_no_bit_of_replicas_trace_or_telemetry(nm):
    """Every round runs on resident columns whatever the call pattern, so even telemetry is bit-identical."""
    rng = np.random.default_rng(8)
    M, d = 5, 2051
    kw = dict(M=M, d=d, lr=0.05, prob=random_policy(M, rng), sigma=0.1, x0_std=1.0, c_std=1.0, seed=11, trace_rounds=16)
    a, b = nm.Netmax(**kw), nm.Netmax(**kw)
    a.round(37)
    for n in (1, 0, 15, 16, 5):
        b.round(n)
    assert (a.read_replicas() == b.read_replicas()).all()
    ta, tb = a.telemetry(21, 16), b.telemetry(21, 16)
    assert (ta[0] == tb[0]).all() and (ta[1] == tb[1]).all()
    a.close()
    b.close()
