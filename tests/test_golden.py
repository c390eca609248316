"""Regression pin: the oracle (and the seeded inputs) still produce the stored results of the tiny workload.
The stored file was written by tests/golden/make_golden.py, which calls only the input generator and the oracle."""
import importlib.util
import json
import os

HERE = os.path.dirname(os.path.abspath(__file__))


def test_oracle_reproduces_the_stored_results_of_config_1():
    spec = importlib.util.spec_from_file_location("make_golden", os.path.join(HERE, "golden", "make_golden.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    stored = json.load(open(os.path.join(HERE, "golden", "c1_tiny_oracle.json")))
    now = mod.compute()
    assert now.keys() == stored.keys()
    for k in stored:
        assert now[k] == stored[k], k
