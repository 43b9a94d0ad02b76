"""Stored fixtures (written by tests/golden/make_golden.py from the generators and the oracle only)."""
import importlib.util
import os

HERE = os.path.dirname(os.path.abspath(__file__))
spec = importlib.util.spec_from_file_location("make_golden", os.path.join(HERE, "golden", "make_golden.py"))
make_golden = importlib.util.module_from_spec(spec)
spec.loader.exec_module(make_golden)


def _read(name):
    with open(os.path.join(HERE, "golden", name)) as f:
        return f.read().splitlines()


def test_seeded_generators_have_not_drifted():
    assert make_golden.inputs_lines() == _read("inputs_digest.txt")


def test_oracle_tiny_case_has_not_drifted():
    # bit-for-bit: the oracle is deterministic FP64 with a fixed summation order per row
    assert make_golden.oracle_lines() == _read("oracle_tiny.txt")
