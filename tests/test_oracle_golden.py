"""The oracle's frozen output on a tiny run (written by tests/golden/make_golden.py,
which calls only `oracle/`).  A regression guard: the pins live in the other
test_oracle_* files."""
import importlib.util
import os

HERE = os.path.dirname(os.path.abspath(__file__))


def test_oracle_output_unchanged_since_golden_was_written():
    spec = importlib.util.spec_from_file_location("make_golden", os.path.join(HERE, "golden", "make_golden.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    with open(os.path.join(HERE, "golden", "oracle_tiny_run.txt")) as f:
        assert mod.render() == f.read()
    with open(os.path.join(HERE, "golden", "oracle_widened_run.txt")) as f:      # warm-up, clipping, AdamW outer
        assert mod.render_widened() == f.read()
