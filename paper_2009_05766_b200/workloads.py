"""Seeded synthetic workloads shaped like the paper's experiments.

This module only describes inputs: sizes, hyper-parameters, seeds and link-speed matrices.
It holds none of the method's arithmetic (no policy, no sampling, no update), so both the
CUDA library and the CPU oracle can be driven from it without sharing any computation.

The paper trains ResNet18 / VGG19 replicas on 4-16 workers spread over machines joined by
fast intra-machine and slow, time-varying inter-machine links.  The stand-ins here are flat
fp32 vectors with those parameter counts, quadratic objectives f_i(x) = 1/2 ||x - c_i||^2,
and link-speed matrices with the same structure (machine groups; heterogeneous, periodically
redrawn inter-group speeds).
"""
from __future__ import annotations

import dataclasses
from typing import Optional

import numpy as np

BASE_SEED = 20090576


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    index: int
    M: int
    d: int
    x0_std: float
    c_std: float
    sigma: float
    lr: float
    rounds: int
    K: int                      # outer (rho) grid of the policy search
    R: int                      # inner (t_bar) grid of the policy search
    link_kind: str              # "groups", "groups_random_inter", "random"
    group_size: int = 1
    intra_gbps: float = 0.0
    inter_gbps: float = 0.0
    lo_gbps: float = 0.0
    hi_gbps: float = 0.0
    policy_period: Optional[int] = None   # rounds between link redraws / policy refreshes

    @property
    def seed(self) -> int:
        return BASE_SEED + self.index

    @property
    def n_epochs(self) -> int:
        if self.policy_period is None:
            return 1
        return (self.rounds + self.policy_period - 1) // self.policy_period

    def link_speeds(self, epoch: int = 0) -> np.ndarray:
        """Symmetric M x M link speeds in Gbps (diagonal 0) for one policy epoch."""
        M = self.M
        s = np.zeros((M, M), dtype=np.float64)
        group = np.arange(M) // self.group_size
        same = group[:, None] == group[None, :]
        iu = np.triu_indices(M, k=1)
        if self.link_kind == "groups":
            s[:] = np.where(same, self.intra_gbps, self.inter_gbps)
        else:
            rng = np.random.default_rng([self.seed, epoch])
            u = rng.random(iu[0].shape[0])
            draw = np.exp(np.log(self.lo_gbps) + u * (np.log(self.hi_gbps) - np.log(self.lo_gbps)))
            s[iu] = draw
            s = s + s.T
            if self.link_kind == "groups_random_inter":
                s = np.where(same, self.intra_gbps, s)
        np.fill_diagonal(s, 0.0)
        return s

    def scaled(self, **changes) -> "Workload":
        """A smaller (or otherwise altered) copy for tests; the name records the change."""
        tag = ",".join(f"{k}={v}" for k, v in sorted(changes.items()))
        return dataclasses.replace(self, name=f"{self.name}[{tag}]", **changes)


CONFIGS = (
    Workload(name="cfg1_M4_d4096", index=1, M=4, d=4096, x0_std=1.0, c_std=1.0, sigma=0.1, lr=0.05,
             rounds=500, K=20, R=20, link_kind="groups", group_size=2, intra_gbps=10.0, inter_gbps=1.0),
    Workload(name="cfg2_M8_resnet18", index=2, M=8, d=11_173_962, x0_std=0.01, c_std=0.01, sigma=0.01,
             lr=0.1, rounds=100, K=20, R=20, link_kind="groups", group_size=4, intra_gbps=100.0,
             inter_gbps=10.0),
    Workload(name="cfg3_M16_vgg19scale", index=3, M=16, d=20_000_000, x0_std=0.01, c_std=0.01, sigma=0.01,
             lr=0.1, rounds=100, K=20, R=20, link_kind="random", group_size=4, lo_gbps=1.0, hi_gbps=100.0,
             policy_period=20),
    Workload(name="cfg4_M64_resnet18", index=4, M=64, d=11_173_962, x0_std=0.01, c_std=0.01, sigma=0.01,
             lr=0.05, rounds=50, K=20, R=20, link_kind="groups_random_inter", group_size=8,
             intra_gbps=100.0, lo_gbps=1.0, hi_gbps=25.0),
    Workload(name="cfg5_M4096_sampling", index=5, M=4096, d=1024, x0_std=1.0, c_std=1.0, sigma=0.1, lr=0.05,
             rounds=10_000, K=8, R=8, link_kind="random", lo_gbps=0.1, hi_gbps=100.0),
)


def config(index: int) -> Workload:
    """Configs are numbered 1..5 as in the benchmark description."""
    return CONFIGS[index - 1]


def sample_columns(d: int, n: int, seed: int) -> np.ndarray:
    """A sorted sample of logical element indices that always holds the first and last
    few elements (row starts, the ragged tail) plus uniformly drawn ones."""
    rng = np.random.default_rng([seed, 7])
    edge = np.concatenate([np.arange(0, min(d, 9)), np.arange(max(0, d - 9), d)])
    body = rng.integers(0, d, size=max(0, n - edge.shape[0]))
    return np.unique(np.concatenate([edge, body])).astype(np.int64)


def clustered_centres(M: int, d: int, group_size: int, spread: float, within: float, seed: int) -> np.ndarray:
    """Non-IID-like objectives: the workers of one machine share a cluster centre (drawn with
    standard deviation `spread`), their own centres scatter around it with `within`."""
    rng = np.random.default_rng([seed, 11])
    groups = (M + group_size - 1) // group_size
    base = spread * rng.standard_normal((groups, d))
    c = base[np.arange(M) // group_size] + within * rng.standard_normal((M, d))
    return c.astype(np.float32)


def sparse_ring_of_groups(M: int, group_size: int, intra_gbps: float, inter_gbps: float) -> np.ndarray:
    """A sparse link graph: all-to-all inside a machine, and only the first worker of each
    machine linked to the first worker of the next machine (a ring of machines)."""
    s = np.zeros((M, M), dtype=np.float64)
    group = np.arange(M) // group_size
    s[group[:, None] == group[None, :]] = intra_gbps
    heads = np.arange(0, M, group_size)
    for a, b in zip(heads, np.roll(heads, -1)):
        if a != b:
            s[a, b] = s[b, a] = inter_gbps
    np.fill_diagonal(s, 0.0)
    return s
