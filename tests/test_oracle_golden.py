"""The oracle still reproduces its frozen output on the small config (see tests/golden/make_golden.py).

Not a pin against the paper (it prints no numbers for this path): a tripwire for unintended
changes of the oracle's arithmetic, counter layout or policy generator.  Integers (grid point,
peer trace) must match exactly; floating-point values to a few ulps, since the host's libm may
round exp / log / sin / cos differently from the machine that wrote the file."""
import importlib.util
import os

import pytest


def _parse(text):
    out = {}
    for line in text.splitlines():
        if line.startswith("#") or not line.strip():
            continue
        key, *vals = line.split()
        out[key] = vals
    return out


def test_oracle_matches_its_frozen_output():
    here = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")
    spec = importlib.util.spec_from_file_location("make_golden", os.path.join(here, "make_golden.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    got = _parse(mod.build())
    want = _parse(open(os.path.join(here, "oracle_cfg1.txt")).read())
    assert got.keys() == want.keys()
    for key in ("policy_grid_point", "trace_first_8_rounds", "trace_sha256"):
        assert got[key] == want[key], key
    for key, rel, absolute in (("rho", 1e-12, 0.0), ("P_row0", 1e-10, 1e-14), ("x_first_8_of_worker_2", 0.0, 2e-6),
                               ("x_sum_abs", 1e-7, 0.0), ("consensus_round_0_and_49", 1e-7, 0.0),
                               ("loss_round_0_and_49", 1e-7, 0.0)):
        g = [float.fromhex(v) for v in got[key]]
        w = [float.fromhex(v) for v in want[key]]
        assert g == pytest.approx(w, rel=rel or None, abs=absolute or None), key
