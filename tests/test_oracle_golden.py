"""The oracle reproduces its stored config-1 results (guards against silent drift of the oracle
or of the seeded generator; the stored numbers were written from oracle/ only)."""
import importlib.util
import os

import pytest

HERE = os.path.dirname(os.path.abspath(__file__))


def test_cfg1_golden():
    spec = importlib.util.spec_from_file_location("make_cfg1_golden",
                                                  os.path.join(HERE, "golden", "make_cfg1_golden.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    got = mod.compute()
    want = {}
    for line in open(os.path.join(HERE, "golden", "cfg1_oracle.txt")):
        if line.startswith("#") or not line.strip():
            continue
        k, v = line.split()
        want[k] = float(v)
    assert got["n_policy"] == 170 and got["n_value"] == 42
    assert set(got) == set(want)
    for k in want:
        assert got[k] == pytest.approx(want[k], rel=1e-12, abs=1e-12), k
