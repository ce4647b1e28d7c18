"""Drift guard: the oracle still gives the values stored by
tests/golden/make_golden.py (which calls only the oracle).  Not a pin of the
oracle -- those are the brute-force / closed-form / invariant tests."""
import importlib.util
import json
import os

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))


def _load_maker():
    spec = importlib.util.spec_from_file_location("make_golden", os.path.join(HERE, "golden", "make_golden.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    return mod


def test_oracle_matches_its_stored_outputs():
    mg = _load_maker()
    want = json.load(open(os.path.join(HERE, "golden", "oracle_tiny.json")))
    got = mg.oracle_outputs(mg.tiny_case())
    assert set(got) == set(want)
    for key in want:
        a, b = want[key], got[key]
        if key in ("argmax", "greedy", "sample"):
            assert a == b, key
        else:
            np.testing.assert_allclose(np.asarray(b, dtype=np.float64), np.asarray(a, dtype=np.float64), rtol=1e-12, atol=1e-13,
                                       err_msg=key)
