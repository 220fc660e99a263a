"""The oracle still reproduces the values stored under tests/golden/ (written by
tests/golden/make_golden.py, which calls only the oracle)."""
import importlib.util
import json
import os

import numpy as np
import pytest

HERE = os.path.dirname(os.path.abspath(__file__))
spec = importlib.util.spec_from_file_location("make_golden", os.path.join(HERE, "golden", "make_golden.py"))
make_golden = importlib.util.module_from_spec(spec)
spec.loader.exec_module(make_golden)


@pytest.mark.parametrize("name", sorted(make_golden.CASES))
def test_oracle_reproduces_golden(name):
    with open(os.path.join(HERE, "golden", f"{name}.json")) as f:
        want = json.load(f)
    got = make_golden.compute(make_golden.CASES[name])
    for key in ("generator", "config", "draft_tok", "target_tok", "accept_len", "next_tok"):
        assert got[key] == want[key], key
    for key in ("top1", "gap"):
        np.testing.assert_allclose(np.array(got[key]), np.array(want[key]), rtol=0, atol=1e-10)
    gp = np.array([[np.nan if x is None else x for x in row] for row in got["judge_p"]])
    wp = np.array([[np.nan if x is None else x for x in row] for row in want["judge_p"]])
    np.testing.assert_allclose(gp, wp, rtol=0, atol=1e-10, equal_nan=True)


@pytest.mark.parametrize("name", sorted(make_golden.VARIANTS))
def test_oracle_reproduces_golden_variants(name):
    """Sampled target tokens (Appendix A) and a draft tree (Section 3.3, "Generality")."""
    with open(os.path.join(HERE, "golden", f"{name}.json")) as f:
        want = json.load(f)
    got = make_golden.compute_variant(**make_golden.VARIANTS[name])
    assert set(got) == set(want)
    for key in got:
        if key in ("top1", "noise"):
            np.testing.assert_allclose(np.array(got[key]), np.array(want[key]), rtol=0, atol=1e-10)
        elif key == "judge_p":
            gp = np.array([[np.nan if x is None else x for x in row] for row in got[key]])
            wp = np.array([[np.nan if x is None else x for x in row] for row in want[key]])
            np.testing.assert_allclose(gp, wp, rtol=0, atol=1e-10, equal_nan=True)
        else:
            assert got[key] == want[key], key
