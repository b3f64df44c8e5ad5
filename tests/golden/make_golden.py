"""Writes tests/golden/oracle_cfg1.txt from the CPU oracle alone (never from the CUDA path).

The paper prints no worked numeric example, so this fixture is not a pin of the oracle against
the paper; it freezes the oracle's own output on the small config (M = 4, d = 4096, 50 rounds),
so that an unintended change of its arithmetic, of the Philox counter layout or of the policy
generator shows up as a diff that has to be explained.  Run from the repository root:

    python tests/golden/make_golden.py
"""
import hashlib
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

from oracle import oracle, policy  # noqa: E402
from paper_2009_05766_b200 import workloads  # noqa: E402


def build():
    w = workloads.config(1)
    t, adj = policy.iteration_times(w.link_speeds(0), w.d)
    P, rho, info = policy.generate_policy(t, adj, w.lr, w.K, w.R)
    sim = oracle.Sim(w.M, w.d, P, adj, alpha=w.lr, rho=rho, sigma=w.sigma, objective=1, seed=w.seed)
    sim.init(w.x0_std, w.c_std)
    sim.round(50)
    x = sim.x()
    cons, loss = sim.telemetry()
    lines = [
        "# oracle output on cfg1 (M=4, d=4096, seed=%d), 50 synchronous rounds; written by make_golden.py" % w.seed,
        "policy_grid_point %d %d" % (info["k"], info["r"]),
        "rho %s" % float(rho).hex(),
        "P_row0 " + " ".join(float(v).hex() for v in P[0]),
        "trace_first_8_rounds " + " ".join(str(int(v)) for v in sim.trace(0, 8).reshape(-1)),
        "trace_sha256 " + hashlib.sha256(sim.trace().tobytes()).hexdigest(),
        "x_first_8_of_worker_2 " + " ".join(float(v).hex() for v in x[2, :8]),
        "x_sum_abs %s" % float(np.abs(x.astype(np.float64)).sum()).hex(),
        "consensus_round_0_and_49 %s %s" % (float(cons[0]).hex(), float(cons[49]).hex()),
        "loss_round_0_and_49 %s %s" % (float(loss[0]).hex(), float(loss[49]).hex()),
    ]
    return "\n".join(lines) + "\n"


if __name__ == "__main__":
    with open(os.path.join(os.path.dirname(os.path.abspath(__file__)), "oracle_cfg1.txt"), "w") as f:
        f.write(build())
    print("written")
