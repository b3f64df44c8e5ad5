"""Pins of the oracle's bfloat16-storage mode (an option of the simulator, not of the paper).

The mode keeps the state on the bfloat16 grid, evaluates Eq. 15-16 in fp32 and rounds each new
parameter once, to nearest even.  Pinned against: a library bfloat16 conversion, hand-built
ties, the oracle's own double-precision mode (an independent code path: different arithmetic
type, no rounding step), and properties that round-to-nearest fixes (fixed points, stagnation
below half a unit in the last place).
"""
import numpy as np
import pytest
import torch

from oracle import oracle


def bf16_ulp(v):
    """Spacing of the bfloat16 grid at |v| (8 significant bits), for normal numbers."""
    v = np.abs(np.asarray(v, dtype=np.float64))
    e = np.floor(np.log2(np.maximum(v, 2.0 ** -126)))
    return 2.0 ** (e - 7)


def policy(M, rng):
    P = rng.random((M, M)) + 0.05
    P /= P.sum(axis=1, keepdims=True)
    return P


def test_rounding_matches_a_library_conversion():
    rng = np.random.default_rng(1)
    v = np.concatenate([rng.standard_normal(200_000) * s for s in (1e-6, 1e-2, 1.0, 1e4)]).astype(np.float32)
    ours = oracle.bf16_round(v)
    lib = torch.from_numpy(v).to(torch.bfloat16).to(torch.float32).numpy()
    assert (ours.view(np.uint32) == lib.view(np.uint32)).all()
    assert (ours.view(np.uint32) & 0xFFFF == 0).all()
    assert (np.abs(ours.astype(np.float64) - v) <= 0.5 * bf16_ulp(ours) * (1 + 1e-12)).all()


def test_ties_go_to_the_even_neighbour():
    # fp32 patterns whose low half is exactly 0x8000 lie midway between two bfloat16 values
    hi = np.arange(0x3F80, 0x3F80 + 64, dtype=np.uint32)  # 1.0 ... upward, consecutive bfloat16 codes
    ties = ((hi << 16) | 0x8000).view(np.float32)
    r = oracle.bf16_round(ties).view(np.uint32) >> 16
    want = np.where(hi % 2 == 0, hi, hi + 1)  # stay on an even code, move up from an odd one
    assert (r == want).all()
    # one fp32 step to either side of the tie goes to the nearer neighbour
    below = ((hi << 16) | 0x7FFF).view(np.float32)
    above = ((hi << 16) | 0x8001).view(np.float32)
    assert (oracle.bf16_round(below).view(np.uint32) >> 16 == hi).all()
    assert (oracle.bf16_round(above).view(np.uint32) >> 16 == hi + 1).all()
    neg = (-ties)
    assert (oracle.bf16_round(neg) == -oracle.bf16_round(ties)).all()
    # values already on the grid, and zero, are fixed points
    grid = (hi << 16).view(np.float32)
    assert (oracle.bf16_round(grid) == grid).all() and oracle.bf16_round([0.0])[0] == 0.0


@pytest.mark.parametrize("objective,sigma", [(1, 0.3), (1, 0.0), (0, 0.0)])
def test_one_round_is_the_double_precision_round_rounded_once(objective, sigma):
    """From one bfloat16 state, the bf16-mode round and the double-mode round (no storage
    rounding) must agree to half a bfloat16 unit plus fp32 rounding noise, and the value kept
    before the rounding must agree with the double result to a few fp32 units."""
    rng = np.random.default_rng(5)
    M, d, lr = 6, 1531, 0.07
    P = policy(M, rng)
    adj = np.ones((M, M), np.uint8)
    x0 = oracle.bf16_round(rng.standard_normal((M, d)).astype(np.float32))
    c0 = oracle.bf16_round(rng.standard_normal((M, d)).astype(np.float32))
    sims = {}
    for storage in ("bf16", "f32"):
        s = oracle.Sim(M, d, P, adj, lr, 0.1, sigma, objective, 99, storage=storage)
        s.set_x(x0)
        s.set_c(c0)
        s.round(1)
        sims[storage] = s
    xb, xd = sims["bf16"].x().astype(np.float64), sims["f32"].x().astype(np.float64)
    pre = sims["bf16"].unrounded()
    assert (sims["bf16"].trace() == sims["f32"].trace()).all()
    assert (oracle.bf16_round(pre) == sims["bf16"].x()).all()
    scale = 1.0 + np.abs(x0).astype(np.float64) + np.abs(c0) + 4.0 * sigma
    assert (np.abs(pre - xd) <= 6 * 2.0 ** -24 * scale).all()
    assert (np.abs(xb - xd) <= 0.5 * bf16_ulp(xb) + 6 * 2.0 ** -24 * scale).all()
    # away from ties the stored value is the double result rounded once
    same = oracle.bf16_round(sims["f32"].x()) == sims["bf16"].x()
    assert same.mean() > 0.999
    assert (xb.view(np.uint64) != xd.view(np.uint64)).mean() > 0.5  # the rounding really happened (self-draws without gradient move nothing)


def test_state_stays_on_the_bfloat16_grid_and_inputs_are_rounded():
    rng = np.random.default_rng(6)
    M, d = 4, 300
    P = policy(M, rng)
    s = oracle.Sim(M, d, P, np.ones((M, M), np.uint8), 0.05, 0.5, 0.1, 1, 3, storage="bf16")
    x0 = rng.standard_normal((M, d)).astype(np.float32)
    s.set_x(x0)
    s.set_c(-x0)
    assert (s.x() == oracle.bf16_round(x0)).all() and (s.c() == oracle.bf16_round(-x0)).all()
    s.round(5)
    assert (s.x().view(np.uint32) & 0xFFFF == 0).all()
    t = oracle.Sim(M, d, P, np.ones((M, M), np.uint8), 0.05, 0.5, 0.1, 1, 3, storage="bf16")
    t.init(1.0, 0.5)
    assert (t.x().view(np.uint32) & 0xFFFF == 0).all() and (t.c().view(np.uint32) & 0xFFFF == 0).all()
    u = oracle.Sim(M, d, P, np.ones((M, M), np.uint8), 0.05, 0.5, 0.1, 1, 3)
    u.init(1.0, 0.5)
    assert (np.abs(t.x().astype(np.float64) - u.x()) <= 0.5 * bf16_ulp(t.x()) + 1e-7).all()


def test_identical_replicas_without_gradient_do_not_move():
    rng = np.random.default_rng(7)
    M, d = 5, 257
    P = policy(M, rng)
    row = oracle.bf16_round(rng.standard_normal(d).astype(np.float32))
    s = oracle.Sim(M, d, P, np.ones((M, M), np.uint8), 0.05, 0.5, 0.0, 0, 11, storage="bf16")
    s.set_x(np.tile(row, (M, 1)))
    s.round(20)
    assert (s.x() == row).all()


def test_updates_below_half_a_unit_are_lost_and_larger_ones_are_kept():
    """Round-to-nearest at the store: a step smaller than half the grid spacing leaves the stored
    parameter where it was; a step of a few units moves it.  (The known price of narrow storage.)"""
    M, d, lr = 2, 64, 0.125
    P = np.eye(M)  # self-draws only: x' = x - lr (x - c)
    x0 = np.full((M, d), 1.0, np.float32)  # grid spacing at 1.0 is 2^-7
    for gap, moves in ((2.0 ** -7, False), (2.0 ** -3, True)):  # step = lr * gap: 2^-10 (lost), 2^-6 (two units)
        s = oracle.Sim(M, d, P, np.ones((M, M), np.uint8), lr, 0.1, 0.0, 1, 1, storage="bf16")
        s.set_x(x0)
        s.set_c(x0 + np.float32(gap))
        s.round(3)
        assert ((s.x() != x0).all()) == moves and ((s.x() == x0).all()) == (not moves)


def test_consensus_still_contracts_to_the_grid_floor():
    """Zero gradients: pulls are convex combinations, so the spread of every column shrinks until
    it reaches the rounding floor (a few grid units), and never grows beyond one unit per round."""
    rng = np.random.default_rng(8)
    M, d = 8, 400
    P = (1.0 - np.eye(M)) / (M - 1)
    s = oracle.Sim(M, d, P, np.ones((M, M), np.uint8), 0.1, 0.7, 0.0, 0, 5, storage="bf16")  # w = 0.49
    s.set_x(rng.standard_normal((M, d)).astype(np.float32))
    lo0, hi0 = s.x().min(axis=0), s.x().max(axis=0)
    spread0 = (hi0 - lo0).mean()
    s.round(400)
    x = s.x()
    assert ((x.max(axis=0) <= hi0 + bf16_ulp(hi0)) & (x.min(axis=0) >= lo0 - bf16_ulp(lo0))).all()
    assert (x.max(axis=0) - x.min(axis=0)).mean() < 0.05 * spread0


def test_asynchronous_step_is_the_double_precision_step_rounded_once():
    """One global step of the asynchronous timeline from a common bfloat16 state: the bf16-mode
    step and the double-mode step change the same single replica and agree to half a bfloat16
    unit plus fp32 rounding noise; every other replica is untouched, bit for bit."""
    rng = np.random.default_rng(9)
    M, d, lr, sigma = 5, 777, 0.06, 0.2
    P = policy(M, rng)
    t = rng.uniform(1.0, 3.0, (M, M))
    x0 = oracle.bf16_round(rng.standard_normal((M, d)).astype(np.float32))
    c0 = oracle.bf16_round(rng.standard_normal((M, d)).astype(np.float32))
    sims = {}
    for storage in ("bf16", "f32"):
        s = oracle.Sim(M, d, P, np.ones((M, M), np.uint8), lr, 0.3, sigma, 1, 21, storage=storage)
        s.set_x(x0)
        s.set_c(c0)
        s.async_begin(t, 0.5)
        s.async_steps(1)
        sims[storage] = s
    wb, wd = sims["bf16"].async_trace(), sims["f32"].async_trace()
    assert all((a == b).all() for a, b in zip(wb, wd))
    i = int(wb[0][0])
    xb, xd = sims["bf16"].x(), sims["f32"].x()
    others = np.arange(M) != i
    assert (xb[others] == x0[others]).all() and (xd[others] == x0[others]).all()
    assert (xb[i].view(np.uint32) & 0xFFFF == 0).all() and (xb[i] != x0[i]).mean() > 0.5
    scale = 1.0 + np.abs(x0[i]).astype(np.float64) + np.abs(c0[i]) + 4.0 * sigma
    assert (np.abs(xb[i].astype(np.float64) - xd[i]) <= 0.5 * bf16_ulp(xb[i]) + 6 * 2.0 ** -24 * scale).all()
    assert (oracle.bf16_round(sims["bf16"].unrounded()[i]) == xb[i]).all()
