"""The stored oracle results are reproduced by the oracle as it stands (CPU only)."""
import importlib.util
import json
import os

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def test_stored_oracle_results_reproduce():
    spec = importlib.util.spec_from_file_location("make_golden", os.path.join(GOLD, "make_golden.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    with open(os.path.join(GOLD, "oracle_small_cases.json")) as f:
        stored = json.load(f)
    assert mod.build() == stored
