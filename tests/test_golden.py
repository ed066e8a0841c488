"""The oracle still produces the stored summary of the tiny fp32 configuration (regression guard;
the fixture is written by tests/golden/make_golden.py from the oracle alone)."""
import importlib.util
import json
import os

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))


def test_oracle_matches_stored_summary():
    spec = importlib.util.spec_from_file_location("make_golden", os.path.join(HERE, "golden", "make_golden.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    got = mod.summary()
    want = json.load(open(os.path.join(HERE, "golden", "c0_oracle.json")))
    for k in ("workload", "parent_idx_sha", "child_idx_sha", "np", "selected"):
        assert got[k] == want[k], k
    np.testing.assert_allclose(got["importance_block0"], want["importance_block0"], rtol=0, atol=1e-8)
    np.testing.assert_allclose(got["Y_row0_first8"], want["Y_row0_first8"], rtol=0, atol=1e-11)
    assert abs(got["Y_abs_sum"] - want["Y_abs_sum"]) < 1e-6
