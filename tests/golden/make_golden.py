"""Writes tests/golden/oracle_small_case.json and tests/golden/oracle_decode_case.json from the CPU oracle alone.

The paper prints no worked numeric example for the prefill path, so this
fixture is a regression anchor, not an external pin: it freezes what the pinned
oracle returns on one small seeded case (vertical indices, a few codes and
scales, a few output values) so that any later change to the oracle's
arithmetic shows up as a diff.  Run:  python tests/golden/make_golden.py
"""
import json
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

import oracle  # noqa: E402
from paper_2608_27875_b200 import workloads as wl  # noqa: E402

CASE = dict(B=1, Hq=4, Hkv=2, L=320, window=48, k=12, n_plant=6, seed=4242)
ROWS = [0, 47, 48, 63, 64, 200, 319]


def compute():
    w = wl.CONFIGS["c0"].scaled(q_fmt=wl.FMT_INT4, k_fmt=wl.FMT_INT4, v_fmt=wl.FMT_FP8_E4M3, **CASE)
    Q, K, V = wl.make_inputs(w)
    r = oracle.hybrid_prefill(wl.bits(Q), wl.bits(K), wl.bits(V), w.window, w.k, w.fmts,
                              rows=np.array(ROWS, dtype=np.int32))
    return {
        "case": CASE, "rows": ROWS, "formats": "q,k int4; v fp8 e4m3; 64-token blocks",
        "vl_idx": r["idx"].tolist(),
        "k_scales_bits": r["k_scales"].view(np.uint32).tolist(),
        "v_scales_bits": r["v_scales"].view(np.uint32).tolist(),
        "q_codes_row200_head1": r["q_codes"][0, 1, 200].tolist(),
        "v_codes_row5_head0": r["v_codes"][0, 0, 5].tolist(),
        "out_first8": [[[float.hex(float(x)) for x in r["out"][0, h, n, :8]] for n in range(len(ROWS))]
                       for h in range(CASE["Hq"])],
    }


def compute_decode():
    """The decode side on the same tensors: Eq. 4-5 selection from 8 tail queries (first query head of every KV group),
    Freeze (Algorithm 4, K4V4, groups of 64), two staged rows, one token (Algorithm 3)."""
    from oracle import decode as od
    w = wl.CONFIGS["c0"].scaled(**CASE)
    Q, K, V = wl.make_inputs(w)
    g = CASE["Hq"] // CASE["Hkv"]
    idx_mass, scores = oracle.select_vertical_mass(wl.bits(Q), wl.bits(K), w.window, w.k, 8, return_scores=True)
    idx_kv = np.ascontiguousarray(idx_mass[:, ::g])
    cache = od.freeze(wl.bits(K), wl.bits(V), idx_kv, w.window)
    for i in (3, 17):
        od.append_staging(cache, wl.bits(K)[:, :, i], wl.bits(V)[:, :, i + 1])
    out, lse = od.decode_attention(wl.bits(Q[:, :, -1].contiguous()), cache)
    seg, _ = od.decode_attention_segmented(wl.bits(Q[:, :, -1].contiguous()), cache, splits=3, tile=16)
    assert np.allclose(seg, out, rtol=1e-11, atol=1e-13)
    return {
        "case": CASE, "n_queries": 8, "formats": "K4V4, groups of 64 compacted rows, staging rows 3 and 17/18",
        "mass_idx": idx_mass.tolist(),
        "mass_scores_head2_first6": [float.hex(float(x)) for x in scores[0, 2, :6]],
        "quantized_positions_head1_first12": cache["iq"][0, 1, :12].tolist(),
        "kq_scales_bits": cache["kq_scales"].view(np.uint32).tolist(),
        "vq_codes_row9_head0": cache["vq_codes"][0, 0, 9].tolist(),
        "lse": [float.hex(float(x)) for x in lse[0]],
        "out_first8": [[float.hex(float(x)) for x in out[0, h, :8]] for h in range(CASE["Hq"])],
    }


if __name__ == "__main__":
    here = os.path.dirname(os.path.abspath(__file__))
    for name, fn in (("oracle_small_case.json", compute), ("oracle_decode_case.json", compute_decode)):
        with open(os.path.join(here, name), "w") as f:
            json.dump(fn(), f, indent=1)
        print("wrote", os.path.join(here, name))
