"""Pins for the oracle's Gaussian noise (Box-Muller on 24-bit uniforms) and peer sampler."""
import math

import numpy as np
import pytest
from scipy import stats

from oracle import oracle


# ------------------------------------------------------------------ normals
def test_box_muller_special_angles_and_radii():
    top = 0xFFFFFE00
    # angle 0: z0 = radius, z1 = 0; the radius for the largest u1 = 1 - 2^-24 is sqrt(-2 ln(1-2^-24))
    z = oracle.normals_from_words([top, 0, 0, 0])
    assert z[1] == 0.0
    assert z[0] == pytest.approx(math.sqrt(-2.0 * math.log1p(-2.0 ** -24)), rel=1e-9)
    # smallest u1 = 2^-24 gives the largest radius sqrt(48 ln 2)
    assert z[2] == pytest.approx(math.sqrt(48.0 * math.log(2.0)), rel=1e-12)
    # a quarter turn (u2 = 1/4): z0 ~ 0, z1 = radius; half a turn: z0 = -radius
    z = oracle.normals_from_words([0x80000000, 0x40000000, 0x80000000, 0x80000000])
    rad = math.sqrt(-2.0 * math.log((2 ** 22 + 0.5) / 2 ** 23))
    assert abs(z[0]) < 1e-15 and z[1] == pytest.approx(rad, rel=1e-12)
    assert z[2] == pytest.approx(-rad, rel=1e-12) and abs(z[3]) < 1e-15
    # the low 9 bits of the radius words and the low 8 bits of the angle words are not used
    assert (oracle.normals_from_words([0x800001FF, 0x400000FF, 0x800001FF, 0x800000FF]) == z).all()


def test_noise_is_standard_normal():
    z = oracle.noise(20090577, 3, 17, 0, 400_000)
    assert abs(z.mean()) < 4.0 / math.sqrt(z.size)
    assert abs(z.var() - 1.0) < 4.0 * math.sqrt(2.0 / z.size)
    assert abs(stats.skew(z)) < 0.02 and abs(stats.kurtosis(z)) < 0.04
    assert stats.kstest(z, "norm").pvalue > 1e-3
    # the four lanes of one Philox block are uncorrelated with each other
    lanes = z.reshape(-1, 4)
    corr = np.corrcoef(lanes.T)
    assert np.abs(corr - np.eye(4)).max() < 0.02


def test_noise_streams_depend_on_worker_round_and_element_only():
    a = oracle.noise(5, 2, 9, 0, 64)
    assert (oracle.noise(5, 2, 9, 13, 20) == a[13:33]).all()      # position-addressable
    assert not np.allclose(oracle.noise(5, 3, 9, 0, 64), a)       # another worker
    assert not np.allclose(oracle.noise(5, 2, 10, 0, 64), a)      # another round
    assert not np.allclose(oracle.noise(6, 2, 9, 0, 64), a)       # another seed
    assert not np.allclose(oracle.noise(5, 2, 9 + (1 << 32), 0, 64), a)  # the round's high word counts


# ------------------------------------------------------------------ sampler
def _rows():
    rng = np.random.default_rng(3)
    rows = [np.array([0.25, 0.25, 0.25, 0.25]),
            np.array([0.0, 0.5, 0.0, 0.5, 0.0]),
            np.array([0.0, 0.0, 1.0, 0.0]),
            np.array([1e-10, 0.3, 0.7 - 1e-10]),
            np.array([0.1] * 10)]
    for M in (7, 64, 257):
        p = rng.random(M) ** 3
        p[rng.random(M) < 0.3] = 0.0
        p[0] = max(p[0], 0.01)
        rows.append(p / p.sum())
    return rows


@pytest.mark.parametrize("p", _rows(), ids=lambda p: f"M{len(p)}")
def test_thresholds_partition_the_32_bit_range(p):
    M = len(p)
    P = np.tile(p, (M, 1))
    T, last = oracle.build_thresholds(P)
    T0, last0 = T[0].astype(np.int64), int(last[0])
    assert last0 == max(j for j in range(M) if p[j] > 0)
    assert (np.diff(T0) >= 0).all()
    # interval of index j is [T[j-1], T[j]) (the last positive index takes the rest)
    edges = np.concatenate([[0], T0[:last0], [1 << 32]])
    width = np.diff(edges)
    assert np.abs(width / 2.0 ** 32 - p[:last0 + 1]).max() <= 2.0 ** -32 * (M + 1)
    for j in range(last0 + 1):
        if p[j] == 0.0:
            assert width[j] == 0          # never drawn
    # exact sweeps of u across every boundary
    for j in range(last0 + 1):
        if width[j] == 0:
            continue
        lo, hi = int(edges[j]), int(edges[j + 1]) - 1
        for u in {lo, hi, (lo + hi) // 2}:
            assert oracle.sample(T[0], last0, u) == j, (j, u)
    assert oracle.sample(T[0], last0, 0xFFFFFFFF) == last0
    assert p[oracle.sample(T[0], last0, 0)] > 0


def test_peer_frequencies_match_probability_rows_chi_square():
    rng = np.random.default_rng(11)
    M, rounds = 12, 20000
    P = rng.random((M, M)) ** 2
    P[rng.random((M, M)) < 0.25] = 0.0
    P[np.arange(M), (np.arange(M) + 1) % M] += 0.05
    P /= P.sum(axis=1, keepdims=True)
    draws = oracle.peer_draws(P, seed=99, first_round=0, n_rounds=rounds)
    assert draws.shape == (rounds, M)
    for i in range(M):
        counts = np.bincount(draws[:, i], minlength=M)
        assert (counts[P[i] == 0] == 0).all()
        keep = P[i] > 0
        chi2, pval = stats.chisquare(counts[keep], rounds * P[i][keep])
        assert pval > 1e-3 / M, (i, pval)


def test_peer_draws_are_counter_based():
    P = np.full((5, 5), 0.2)
    a = oracle.peer_draws(P, 7, 0, 50)
    b = oracle.peer_draws(P, 7, 20, 30)
    assert (a[20:] == b).all()
    assert not (oracle.peer_draws(P, 8, 0, 50) == a).all()
    # different workers use different streams: columns are not identical
    assert not (a[:, 0] == a[:, 1]).all()
