"""The stored oracle/generator record still reproduces (see tests/golden/make_golden.py)."""
import importlib.util
import os


def test_golden_record_reproduces(oracle_lib):
    here = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")
    spec = importlib.util.spec_from_file_location("make_golden", os.path.join(here, "make_golden.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    stored = open(os.path.join(here, "oracle_regression.txt")).read().splitlines()
    assert stored == list(mod.lines())
