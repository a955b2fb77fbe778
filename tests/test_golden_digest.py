"""The stored c1 digest (written by tests/golden/make_c1_digest.py from the oracle alone)
still matches what the oracle and the input recipe produce."""
import importlib.util
import json
import os


def test_c1_digest_matches(orc):
    here = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")
    spec = importlib.util.spec_from_file_location("make_c1_digest", os.path.join(here, "make_c1_digest.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    now = mod.digest()
    with open(os.path.join(here, "c1_oracle_digest.json")) as f:
        stored = json.load(f)

    def close(a, b):
        if isinstance(a, dict):
            return all(close(a[k], b[k]) for k in a)
        if isinstance(a, list):
            return all(close(x, y) for x, y in zip(a, b))
        if isinstance(a, float):
            return abs(a - b) <= 1e-10 * max(1.0, abs(a))
        return a == b
    assert close(stored, now)
