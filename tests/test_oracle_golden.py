"""Regression anchor: the oracle still returns what the committed fixture froze.
(The fixture is written by tests/golden/make_golden.py, which calls only the oracle.)"""
import importlib.util
import json
import os

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))


def _make_golden():
    spec = importlib.util.spec_from_file_location("make_golden", os.path.join(HERE, "golden", "make_golden.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    return mod


def test_oracle_decode_case_unchanged():
    now = _make_golden().compute_decode()
    with open(os.path.join(HERE, "golden", "oracle_decode_case.json")) as f:
        gold = json.load(f)
    for key in ("mass_idx", "mass_scores_head2_first6", "quantized_positions_head1_first12", "kq_scales_bits", "vq_codes_row9_head0"):
        assert now[key] == gold[key], key
    for key in ("lse", "out_first8"):
        unhex = np.vectorize(float.fromhex)
        np.testing.assert_allclose(unhex(np.array(now[key])), unhex(np.array(gold[key])), rtol=0, atol=1e-13)


def test_oracle_small_case_unchanged():
    now = _make_golden().compute()
    with open(os.path.join(HERE, "golden", "oracle_small_case.json")) as f:
        gold = json.load(f)
    for key in ("vl_idx", "k_scales_bits", "v_scales_bits", "q_codes_row200_head1", "v_codes_row5_head0"):
        assert now[key] == gold[key], key
    a = np.array([[[float.fromhex(x) for x in r] for r in h] for h in now["out_first8"]])
    b = np.array([[[float.fromhex(x) for x in r] for r in h] for h in gold["out_first8"]])
    np.testing.assert_allclose(a, b, rtol=0, atol=1e-13)
