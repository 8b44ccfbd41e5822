"""The oracle against its stored outputs on one tiny block (tests/golden/tiny_block.json, written by
tests/golden/make_golden.py from the oracle alone): guards the oracle against accidental edits."""
import importlib.util
import json
import os

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))


def test_oracle_reproduces_its_stored_outputs():
    spec = importlib.util.spec_from_file_location("make_golden", os.path.join(HERE, "golden", "make_golden.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    now = mod.compute()
    with open(os.path.join(HERE, "golden", "tiny_block.json")) as f:
        ref = json.load(f)
    assert now["idx"] == ref["idx"]
    for key in ("gates", "F", "y2", "dy1"):
        assert np.allclose(np.array(now[key]), np.array(ref[key]), rtol=1e-12, atol=1e-14), key
    assert ref["max_abs_reconstruction_error"] <= 1e-12 and now["max_abs_reconstruction_error"] <= 1e-12
    for key in ("grad_sums", "grad_abs_sums"):
        for n, v in ref[key].items():
            assert np.isclose(now[key][n], v, rtol=1e-10, atol=1e-13), (key, n)
    assert np.abs(np.array(ref["F"])).max() > 1e-3          # the stored block is not degenerate
