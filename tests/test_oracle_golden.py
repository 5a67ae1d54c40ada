"""Regression anchor: the oracle still returns what the committed fixture froze.
(The fixture is written by tests/golden/make_golden.py, which calls only the oracle.)"""
import importlib.util
import json
import os

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))


def test_oracle_small_case_unchanged():
    spec = importlib.util.spec_from_file_location("make_golden", os.path.join(HERE, "golden", "make_golden.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    now = mod.compute()
    with open(os.path.join(HERE, "golden", "oracle_small_case.json")) as f:
        gold = json.load(f)
    for key in ("vl_idx", "k_scales_bits", "v_scales_bits", "q_codes_row200_head1", "v_codes_row5_head0"):
        assert now[key] == gold[key], key
    a = np.array([[[float.fromhex(x) for x in r] for r in h] for h in now["out_first8"]])
    b = np.array([[[float.fromhex(x) for x in r] for r in h] for h in gold["out_first8"]])
    np.testing.assert_allclose(a, b, rtol=0, atol=1e-13)
