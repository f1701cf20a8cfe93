"""The oracle still produces the values frozen in tests/golden/oracle_regression_c0.txt (its own
earlier output, not the paper's: the paper prints none).  A failure means the oracle's arithmetic
or the input generator changed; if that was intended, re-run the script beside the fixture."""
import importlib.util
import os

HERE = os.path.dirname(os.path.abspath(__file__))


def test_oracle_matches_its_frozen_values():
    spec = importlib.util.spec_from_file_location("make_oracle_regression",
                                                  os.path.join(HERE, "golden", "make_oracle_regression.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    want = {}
    with open(os.path.join(HERE, "golden", "oracle_regression_c0.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            name, val = line.rsplit(" ", 1)
            want[name] = float(val)
    got = dict(mod.values())
    assert set(got) == set(want)
    for k, v in want.items():
        assert abs(got[k] - v) <= 1e-12 * (1.0 + abs(v)), k
