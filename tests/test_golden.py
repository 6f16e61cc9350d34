"""The stored oracle samples still come out of the oracle (guards against silent drift of
the oracle or of the seeded generators)."""
import importlib.util
import os

HERE = os.path.dirname(os.path.abspath(__file__))


def test_config1_golden_reproduces():
    spec = importlib.util.spec_from_file_location("make_golden", os.path.join(HERE, "golden", "make_golden.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    with open(os.path.join(HERE, "golden", "config1_oracle.txt")) as f:
        stored = [ln.strip() for ln in f if ln.strip() and not ln.startswith("#")]
    assert stored == mod.compute()
