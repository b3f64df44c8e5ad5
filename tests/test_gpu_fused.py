"""GPU parity of the launch shape that advances a resident tile several rounds (long vectors,
few workers; netmax_config.fuse_rounds).  Columns evolve independently given the peer draws, so
fusing rounds must not change a bit of the replicas or of the peer trace: checked against one
launch per round on the same context inputs, and against the CPU oracle within the fp32
tolerance.  Telemetry sums are accumulated in a different order and agree to rounding."""
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


# long vectors: at least two 4 KB-wide tiles per SM, so that the streaming launch shapes are chosen
@pytest.mark.parametrize("M,d,fuse,storage", [(2, 400_003, 0, "f32"), (5, 320_001, 0, "f32"), (8, 400_002, 0, "f32"),
                                              (9, 310_000, 3, "f32"), (8, 400_001, 2, "f32"), (16, 320_001, 4, "f32"),
                                              (18, 310_003, 4, "f32"), (8, 700_003, 0, "bf16"), (3, 650_001, 4, "bf16"),
                                              (16, 620_006, 3, "bf16"), (24, 310_001, 0, "f32"), (36, 170_003, 0, "f32"),
                                              (22, 620_002, 0, "bf16"), (36, 330_001, 2, "bf16"), (8, 400_003, 8, "f32"),
                                              (5, 320_003, 6, "f32"), (16, 620_002, 8, "bf16")])
@pytest.mark.parametrize("objective", [0, 1])
def test_fused_rounds_change_no_bit(nm, M, d, fuse, storage, objective):
    rng = np.random.default_rng(M * 11 + d)
    P = random_policy(M, rng, zeros=0.2 if M > 4 else 0.0)
    kw = dict(M=M, d=d, lr=0.05, prob=P, sigma=0.1, x0_std=1.0, c_std=1.0, objective=objective, seed=d + M, trace_rounds=64,
              storage=storage)
    one = nm.Netmax(fuse_rounds=1, **kw)         # one launch per round
    many = nm.Netmax(fuse_rounds=fuse, **kw)
    rounds = 0
    for n in (11, 1, 2, 4, 3):                   # chunks of every length, a lone round in between, ring wrap-around
        launches = many.kernel_launches
        one.round(n)
        many.round(n)
        rounds += n
        if n >= 2:
            assert many.kernel_launches - launches < n + 1, "rounds were not fused"
    xa, xb = one.read_replicas(), many.read_replicas()
    assert (xa.view(np.uint32) == xb.view(np.uint32)).all()
    assert (one.peer_trace(0, rounds) == many.peer_trace(0, rounds)).all()
    (ca, la), (cb, lb) = one.telemetry(0, rounds), many.telemetry(0, rounds)
    # (with bfloat16 state the two launch shapes group a thread's fp32 partial sums by 8 and by 4 columns; beyond 24
    # workers the per-round kernel splits the rows of a column over two row lanes and adds their fp32 sums afterwards)
    rtol = 1e-12 if storage == "f32" and M <= 24 else 1e-6
    np.testing.assert_allclose(cb, ca, rtol=rtol)
    np.testing.assert_allclose(lb, la, rtol=rtol)
    # padding lanes of the rows stay zero
    import torch
    ptr, ld = many.replicas_device()

    class _Holder:
        pass

    h = _Holder()
    h.__cuda_array_interface__ = {"shape": (M, ld), "typestr": "<f4" if storage == "f32" else "<i2", "data": (ptr, False),
                                  "version": 3, "strides": None}
    assert int(torch.as_tensor(h, device="cuda")[:, d:].abs().max().item()) == 0
    one.close()
    many.close()


# more workers than the 128- and 256-thread CTAs hold: 64-thread CTAs of the same kernel up to M = 36 (19, 20, 24: three
# per SM; 25, 33, 35: two), beyond that the rows of a tile are split over the CTAs of a cluster (M = 44 -> 4 CTAs;
# 50 -> 5; 47, 57 -> 6; 56, 70 -> 7; 64, 100, 136 -> 8; ragged last CTAs, one with no row at all)
@pytest.mark.parametrize("M,d,fuse", [(64, 80_003, 0), (20, 303_201, 0), (33, 152_002, 3), (100, 38_001, 4), (136, 40_001, 2),
                                      (19, 310_000, 4), (24, 303_203, 0), (25, 160_001, 0), (44, 160_002, 0), (50, 80_001, 2),
                                      (57, 80_003, 0), (35, 160_003, 0), (47, 160_001, 0), (56, 80_001, 0), (70, 80_002, 0)])
@pytest.mark.parametrize("objective", [0, 1])
def test_cluster_resident_rounds_change_no_bit(nm, M, d, fuse, objective):
    rng = np.random.default_rng(M * 7 + d)
    P = random_policy(M, rng, zeros=0.3)
    kw = dict(M=M, d=d, lr=0.05, prob=P, sigma=0.1, x0_std=1.0, c_std=1.0, objective=objective, seed=d + M, trace_rounds=64)
    one = nm.Netmax(fuse_rounds=1, **kw)
    many = nm.Netmax(fuse_rounds=fuse, **kw)
    rounds = 0
    for n in (9, 1, 2, 4, 3):
        launches = many.kernel_launches
        one.round(n)
        many.round(n)
        rounds += n
        if n >= 2:
            assert many.kernel_launches - launches < n + 1, "rounds were not fused"
    assert (one.read_replicas().view(np.uint32) == many.read_replicas().view(np.uint32)).all()
    assert (one.peer_trace(0, rounds) == many.peer_trace(0, rounds)).all()
    (ca, la), (cb, lb) = one.telemetry(0, rounds), many.telemetry(0, rounds)
    np.testing.assert_allclose(cb, ca, rtol=2e-6)      # the column sums are added CTA by CTA here: fp32 rounding of partial sums
    np.testing.assert_allclose(lb, la, rtol=1e-6)
    one.close()
    many.close()


def test_cluster_shape_is_taken_only_where_it_pays(nm):
    """fuse_rounds = 0 fuses rounds for the worker counts where that was measured faster (in one CTA up to 36, over a
    cluster for 37 ... 66 and most of 68 ... 88) and runs one launch per round elsewhere; fuse_rounds >= 2 fuses
    wherever the rows fit (M <= 144)."""
    d = 400_001
    for M, fuse, fused in ((22, 0, True), (40, 0, True), (50, 0, True), (67, 0, False), (67, 4, True), (60, 0, True),
                           (81, 0, False), (81, 3, True), (100, 0, False), (150, 4, False)):
        P = np.full((M, M), 1.0 / (M - 1))
        np.fill_diagonal(P, 0.0)
        g = nm.Netmax(M=M, d=d, lr=0.05, prob=P, sigma=0.1, x0_std=1.0, c_std=1.0, seed=1, trace_rounds=16, fuse_rounds=fuse)
        g.round(1)
        before = g.kernel_launches
        g.round(8)
        launches = g.kernel_launches - before
        assert (launches < 8) == fused, (M, fuse, launches)
        g.close()


# 64-thread CTAs of the single-CTA kernel (M = 28), clusters of 6, 7 and 8 CTAs
@pytest.mark.parametrize("M,d", [(64, 80_003), (28, 160_003), (48, 80_001), (56, 80_002)])
def test_cluster_resident_rounds_match_the_oracle(nm, M, d):
    rng = np.random.default_rng(M + d)
    P = random_policy(M, rng, zeros=0.2)
    g = nm.Netmax(M=M, d=d, lr=0.05, prob=P, sigma=0.1, x0_std=1.0, c_std=1.0, objective=1, seed=7, trace_rounds=32)
    o = oracle.Sim(M, d, P, full_adj(M), alpha=0.05, rho=g.get_policy()[1], sigma=0.1, objective=1, seed=7)
    o.init(1.0, 1.0)
    rounds = 10
    launches = g.kernel_launches
    g.round(rounds)
    assert g.kernel_launches - launches <= 1 + (rounds + 3) // 4
    o.round(rounds, threads=8)
    assert (g.peer_trace() == o.trace()).all()
    got, want = g.read_replicas().astype(np.float64), o.x().astype(np.float64)
    assert (np.abs(got - want) <= TOL * (1.0 + np.abs(want))).all()
    gc, gl = g.telemetry()
    oc, ol = o.telemetry()
    np.testing.assert_allclose(gc, oc, rtol=1e-4)
    np.testing.assert_allclose(gl, ol, rtol=1e-4)
    g.close()


@pytest.mark.parametrize("M,d", [(3, 400_003), (8, 303_107)])
def test_fused_rounds_match_the_oracle(nm, M, d):
    rng = np.random.default_rng(M + d)
    P = random_policy(M, rng)
    g = nm.Netmax(M=M, d=d, lr=0.05, prob=P, sigma=0.1, x0_std=1.0, c_std=1.0, objective=1, seed=7, trace_rounds=32)
    o = oracle.Sim(M, d, P, full_adj(M), alpha=0.05, rho=g.get_policy()[1], sigma=0.1, objective=1, seed=7)
    o.init(1.0, 1.0)
    rounds = 14
    launches = g.kernel_launches
    g.round(rounds)
    assert g.kernel_launches - launches <= 1 + (rounds + 3) // 4     # the sampler and fused launches of four rounds
    o.round(rounds, threads=8)
    assert (g.peer_trace() == o.trace()).all()
    got, want = g.read_replicas().astype(np.float64), o.x().astype(np.float64)
    assert (np.abs(got - want) <= TOL * (1.0 + np.abs(want))).all()
    gc, gl = g.telemetry()
    oc, ol = o.telemetry()
    np.testing.assert_allclose(gc, oc, rtol=1e-4)
    np.testing.assert_allclose(gl, ol, rtol=1e-4)
    g.close()


def test_fuse_rounds_out_of_range_is_refused(nm):
    with pytest.raises(nm.NetmaxError) as e:
        nm.Netmax(M=2, d=64, lr=0.1, fuse_rounds=9)
    assert e.value.code == -1
