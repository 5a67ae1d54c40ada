"""Writes tests/golden/oracle_small_case.json from the CPU oracle alone.

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


if __name__ == "__main__":
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "oracle_small_case.json")
    with open(path, "w") as f:
        json.dump(compute(), f, indent=1)
    print("wrote", path)
