"""GPU parity across the 2^32 boundary of the round number.

The round number is a 64-bit quantity split over two words of every Philox counter (low word,
and high bits next to the stream tag).  A context that starts at netmax_config.first_round =
2^32 - 3 crosses the boundary after three rounds; every launch shape must then draw the peers and
the noise the oracle draws at those rounds, and a run resumed from saved replicas at a later
first_round must continue bit for bit."""
import numpy as np
import pytest

from oracle import oracle

pytestmark = pytest.mark.gpu
TOL = 1e-5
R0 = (1 << 32) - 3


@pytest.fixture(scope="module")
def nm():
    import torch
    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device")
    from paper_2009_05766_b200 import binding
    binding.lib()
    return binding


def bf16_ulp(v):
    """Spacing of bfloat16 (8 significant bits) at magnitude v."""
    return 2.0 ** (np.floor(np.log2(v)) - 7)


def full_adj(M):
    return (1 - np.eye(M)).astype(np.uint8)


def random_policy(M, rng):
    P = rng.random((M, M)) + 0.05
    return P / P.sum(axis=1, keepdims=True)


# (M, d, fuse_rounds, storage, what the shape exercises)
SHAPES = [
    (3, 303_200, 1, "f32", "one launch per round, long vectors"),
    (3, 303_200, 0, "f32", "four rounds per launch over resident tiles"),
    (4, 4_096, 0, "f32", "all rounds on shared-memory-resident columns"),
    (4, 4_096, 1, "f32", "cooperative multi-round launch"),
    (600, 520, 0, "f32", "resident columns, rows split over threads"),
    (3, 606_400, 0, "bf16", "fused, bfloat16 state"),
    (5, 2_051, 0, "bf16", "resident, bfloat16 state"),
]


@pytest.mark.parametrize("M,d,fuse,storage,what", SHAPES, ids=[s[4] for s in SHAPES])
def test_rounds_across_the_32_bit_boundary_match_the_oracle(nm, M, d, fuse, storage, what):
    rng = np.random.default_rng(M + d)
    P = random_policy(M, rng)
    rounds = 8
    g = nm.Netmax(M=M, d=d, lr=0.05, prob=P, sigma=0.1, x0_std=1.0, c_std=1.0, objective=1, seed=91, trace_rounds=32,
                  fuse_rounds=fuse, storage=storage, first_round=R0)
    assert g.rounds_done == R0
    cols = None if M * d < 2_000_000 else np.unique(np.concatenate([np.arange(0, 2048), np.arange(d - 2048, d),
                                                                     rng.integers(0, d, 20_000)])).astype(np.int64)
    o = oracle.Sim(M, d, P, full_adj(M), alpha=0.05, rho=g.get_policy()[1], sigma=0.1, objective=1, seed=91, cols=cols,
                   storage=storage, first_round=R0)
    if storage == "bf16":       # start both sides from the same stored codes
        x0, c0 = g.read_replicas(), g.read_centres()
        o.set_x(x0 if cols is None else x0[:, cols])
        o.set_c(c0 if cols is None else c0[:, cols])
    else:
        o.init(1.0, 1.0)
    g.round(rounds)
    o.round(rounds, threads=4)
    assert g.rounds_done == R0 + rounds
    assert (g.peer_trace() == o.trace()).all()                    # rounds R0 .. R0 + 7, absolute numbering
    assert (g.peer_trace(R0 + 2, 3) == o.trace(2, 3)).all()       # the three rounds around the boundary
    got = g.read_replicas() if cols is None else g.read_columns(cols)
    want = o.x()
    if storage == "bf16":
        # a code may differ by a bfloat16 step where the fast noise moves a value across a rounding
        # boundary, and such a step travels on with the pulls: a few steps of the state's scale at most
        units = np.abs(got.astype(np.float64) - want) / bf16_ulp(np.maximum(np.abs(want), 0.25))
        assert units.max() <= 2.0 and (units > 0).mean() < 2e-3, f"max {units.max():.2f} units, {(units > 0).mean():.2e} differ"
    else:
        assert (np.abs(got.astype(np.float64) - want) <= TOL * (1.0 + np.abs(want.astype(np.float64)))).all()
    gc, gl = g.telemetry()
    oc, ol = o.telemetry()
    if cols is None:
        np.testing.assert_allclose(gc, oc, rtol=1e-4)
        np.testing.assert_allclose(gl, ol, rtol=1e-4)
    # a context numbered from 0 draws other peers and other noise
    h = nm.Netmax(M=M, d=d, lr=0.05, prob=P, sigma=0.1, x0_std=1.0, c_std=1.0, objective=1, seed=91, trace_rounds=32,
                  fuse_rounds=fuse, storage=storage)
    h.round(rounds)
    assert not (h.peer_trace() == g.peer_trace()).all()
    with pytest.raises(nm.NetmaxError) as e:
        g.peer_trace(0, 1)                                        # before the context's first round
    assert e.value.code == -5
    g.close()
    h.close()


@pytest.mark.parametrize("M,d,fuse", [(3, 303_200, 0), (4, 4_096, 0), (64, 70_001, 0)])
def test_resumed_run_continues_bit_for_bit(nm, M, d, fuse):
    rng = np.random.default_rng(M * 3 + d)
    P = random_policy(M, rng)
    kw = dict(M=M, d=d, lr=0.05, prob=P, sigma=0.1, objective=1, seed=5, trace_rounds=16, fuse_rounds=fuse)
    whole = nm.Netmax(x0_std=1.0, c_std=1.0, **kw)
    whole.round(5)
    saved, centres = whole.read_replicas(), whole.read_centres()
    whole.round(7)
    rest = nm.Netmax(first_round=5, **kw)
    rest.set_replicas(saved)
    rest.set_centres(centres)
    rest.round(7)
    assert (rest.read_replicas().view(np.uint32) == whole.read_replicas().view(np.uint32)).all()
    assert (rest.peer_trace() == whole.peer_trace(5, 7)).all()
    np.testing.assert_allclose(rest.telemetry()[0], whole.telemetry(5, 7)[0], rtol=1e-6)
    whole.close()
    rest.close()


def test_first_round_is_validated(nm):
    P = random_policy(3, np.random.default_rng(0))
    for bad in (-1, 1 << 56):
        with pytest.raises(nm.NetmaxError) as e:
            nm.Netmax(M=3, d=8, lr=0.05, prob=P, first_round=bad)
        assert e.value.code == -1
