"""Pins for the oracle's initial state: x_i(0) = x0_std * z and c_i = c_std * z.

The fill is a composition of two primitives that are pinned on their own (Philox4x32-10
against cuRAND's host generator, the Box-Muller map against closed forms and the normal law),
so it is checked here (i) value by value against that composition written out in numpy,
(ii) against the normal law it must follow, and (iii) for the independence of the three
streams that share a counter (initial replicas, centres, round-0 gradient noise).
"""
import numpy as np
import pytest
from scipy import stats

from oracle import oracle
from oracle import policy as opolicy

SEED = 0x1234_5678_9ABC_DEF1


def _sim(M, d, cols=None, seed=SEED, storage="f32"):
    P = np.full((M, M), 1.0 / (M - 1))
    np.fill_diagonal(P, 0.0)
    adj = (1 - np.eye(M)).astype(np.uint8)
    return oracle.Sim(M, d, P, adj, alpha=0.05, rho=0.1, sigma=0.1, objective=1, seed=seed, cols=cols, storage=storage)


def _composed(seed, worker, e, tag, std):
    """float32(std * lane (e mod 4) of the normals of Philox block (e div 4, worker, 0, tag))."""
    key = [seed & 0xFFFFFFFF, seed >> 32]
    words = oracle.philox4x32_10([e >> 2, worker, 0, tag], key)
    return np.float32(std * oracle.normals_from_words(words)[e & 3])


def test_fill_is_the_composition_of_philox_and_box_muller():
    d = (1 << 30) - 33                                   # the longest vector the library accepts
    cols = np.array([0, 1, 2, 3, 4, 5, 6, 7, 1021, 1022, 1023, 65536 * 4 + 2,
                     d - 8, d - 7, d - 6, d - 5, d - 4, d - 3, d - 2, d - 1], dtype=np.int64)
    assert {int(e) & 3 for e in cols} == {0, 1, 2, 3}
    M, x0_std, c_std = 5, 0.37, 2.5
    s = _sim(M, d, cols)
    s.init(x0_std, c_std)
    x, c = s.x(), s.c()
    for i in range(M):
        for k, e in enumerate(cols):
            assert x[i, k] == _composed(SEED, i, int(e), oracle.TAG_X0, x0_std), (i, int(e))
            assert c[i, k] == _composed(SEED, i, int(e), oracle.TAG_C, c_std), (i, int(e))
    # the four lanes of one block are four different normals, in lane order
    words = oracle.philox4x32_10([0, 2, 0, oracle.TAG_X0], [SEED & 0xFFFFFFFF, SEED >> 32])
    z = oracle.normals_from_words(words)
    assert len(set(z.tolist())) == 4
    np.testing.assert_array_equal(x[2, :4], (x0_std * z).astype(np.float32))


def test_fill_scales_and_zero_std():
    cols = np.arange(64, dtype=np.int64)
    a, b = _sim(3, 64, cols), _sim(3, 64, cols)
    a.init(1.0, 1.0)
    b.init(0.25, 0.0)
    np.testing.assert_array_equal(b.x(), (a.x().astype(np.float64) * 0.25).astype(np.float32))   # power of two: exact
    assert (b.c() == 0.0).all()
    # the column sample does not change a value: column e of a sampled run is column e of the full run
    full = _sim(3, 64)
    full.init(1.0, 1.0)
    pick = np.array([5, 17, 18, 63], dtype=np.int64)
    part = _sim(3, 64, pick)
    part.init(1.0, 1.0)
    np.testing.assert_array_equal(part.x(), full.x()[:, pick])
    np.testing.assert_array_equal(part.c(), full.c()[:, pick])


def test_fill_follows_the_normal_law():
    M, d, std = 4, 100_000, 0.01
    s = _sim(M, d, seed=20090577)
    s.init(std, 3.0)
    for arr, scale in ((s.x(), std), (s.c(), 3.0)):
        z = arr.astype(np.float64).ravel() / scale
        assert abs(z.mean()) < 4.0 / np.sqrt(z.size)
        assert abs(z.var() - 1.0) < 4.0 * np.sqrt(2.0 / z.size)
        assert abs(stats.skew(z)) < 0.02 and abs(stats.kurtosis(z)) < 0.04
        assert stats.kstest(z, "norm").pvalue > 1e-3
        # workers are independent of each other, and so are neighbouring lanes
        rows = arr.astype(np.float64) / scale
        assert np.abs(np.corrcoef(rows) - np.eye(M)).max() < 0.02
        assert np.abs(np.corrcoef(rows[0].reshape(-1, 4).T) - np.eye(4)).max() < 0.02


def test_initial_replicas_centres_and_first_noise_are_independent_streams():
    M, d, seed = 3, 200_000, 99
    s = _sim(M, d, seed=seed)
    s.init(1.0, 1.0)
    x, c = s.x().astype(np.float64), s.c().astype(np.float64)
    for i in range(M):
        n0 = oracle.noise(seed, i, 0, 0, d)            # round-0 gradient noise of the same (i, e)
        for a, b in ((x[i], c[i]), (x[i], n0), (c[i], n0)):
            assert not np.allclose(a, b)
            assert abs(np.corrcoef(a, b)[0, 1]) < 5.0 / np.sqrt(d)
            assert (a == b).mean() < 1e-4
    # another seed gives another state
    t = _sim(M, d, seed=seed + 1)
    t.init(1.0, 1.0)
    assert abs(np.corrcoef(t.x()[0].astype(np.float64), x[0])[0, 1]) < 5.0 / np.sqrt(d)


def test_bfloat16_fill_is_one_fp32_product_rounded_once():
    cols = np.arange(4096, dtype=np.int64)
    M, std = 3, 0.0173
    a, b = _sim(M, 4096, cols), _sim(M, 4096, cols, storage="bf16")
    a.init(1.0, 1.0)
    b.init(std, std)
    z32 = a.x()                                           # fp32 roundings of the double normals (std 1)
    np.testing.assert_array_equal(b.x(), oracle.bf16_round(z32 * np.float32(std)))
    np.testing.assert_array_equal(b.c(), oracle.bf16_round(a.c() * np.float32(std)))


def test_second_eigenvalue_sparse_branch_matches_the_dense_one():
    # the branch taken above 512 workers (Lanczos through scipy) against eigvalsh on the same matrix
    M = 600
    rng = np.random.default_rng(8)
    s = np.exp(rng.uniform(np.log(1.0), np.log(100.0), (M, M)))
    s = np.triu(s, 1)
    s = s + s.T
    t, adj = opolicy.iteration_times(s, 1_000_000)
    alpha = 0.05
    P, rho, info = opolicy.generate_policy(t, adj, alpha, 2, 2)      # a coarse grid, every point through the sparse branch
    Y = opolicy.y_matrix(P, opolicy.node_probabilities(P, t, adj), adj, alpha, rho)
    dense = float(np.linalg.eigvalsh(0.5 * (Y + Y.T))[-2])
    assert opolicy.second_eigenvalue(Y) == pytest.approx(dense, abs=1e-10)
    assert info["lam2"] == pytest.approx(dense, abs=1e-10)
    assert 0.0 < dense < 1.0
