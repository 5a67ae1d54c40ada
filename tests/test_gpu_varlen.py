"""Ragged prefill batches (the *_varlen calls): five prompts from shorter than the window to 10^4 tokens in one packed
batch.  Every sequence is its own problem, so each must come out exactly as the oracle computes it alone: index sets,
codes and scales bit for bit, the attention output within the parity tolerance - and identical, bit for bit, to what
the plain calls return for that sequence by itself."""
import numpy as np
import pytest
import torch

import oracle
from gpu_util import MAX_ABS_TOL, MEAN_REL_TOL, ensure_built, errors, rand_bf16
from paper_2608_27875_b200 import api, workloads as wl

pytestmark = pytest.mark.gpu
LENGTHS = [40, 333, 1000, 4097, 10000]


@pytest.mark.parametrize("fmts", [(0, 0, 0), (2, 2, 1)])
def test_every_sequence_of_a_ragged_batch_matches_the_oracle_and_the_plain_calls(fmts):
    ensure_built()
    Hq, Hkv, W = 4, 2, 128
    qs = [rand_bf16((Hq, L, 128), seed=10 + n) for n, L in enumerate(LENGTHS)]
    ks = [rand_bf16((Hkv, L, 128), seed=20 + n) for n, L in enumerate(LENGTHS)]
    vs = [rand_bf16((Hkv, L, 128), seed=30 + n) for n, L in enumerate(LENGTHS)]
    k_per = [max(1, (L - W) // 50) if L > W else 0 for L in LENGTHS]
    res = api.hybrid_prefill_varlen([t.cuda() for t in qs], [t.cuda() for t in ks], [t.cuda() for t in vs], W, k_per, fmts)
    assert len(res) == len(LENGTHS)
    for n, (L, r) in enumerate(zip(LENGTHS, res)):
        qb, kb, vb = wl.bits(qs[n][None]), wl.bits(ks[n][None]), wl.bits(vs[n][None])
        ref = oracle.hybrid_prefill(qb, kb, vb, W, k_per[n], fmts, rows=wl.sample_rows(L, W, n_random=8, edge=2) if L > 2000 else None)
        np.testing.assert_array_equal(r["idx"].cpu().numpy()[None], ref["idx"])
        for name in ("q_codes", "k_codes", "v_codes"):
            np.testing.assert_array_equal(r[name].cpu().numpy()[None], ref[name])
        for name in ("q_scales", "k_scales", "v_scales"):
            np.testing.assert_array_equal(r[name].cpu().numpy()[None].view(np.uint32), ref[name].view(np.uint32))
        got = r["out"].cpu().numpy()[None]
        assert np.isfinite(got).all()
        if L > 2000:
            got = got[:, :, wl.sample_rows(L, W, n_random=8, edge=2)]
        max_abs, mean_rel = errors(got, ref["out"])
        assert max_abs <= MAX_ABS_TOL and mean_rel <= MEAN_REL_TOL, (L, max_abs, mean_rel)
        # the plain calls on this sequence alone: the same bits
        alone = api.hybrid_prefill(qs[n][None].cuda(), ks[n][None].cuda(), vs[n][None].cuda(), W, k_per[n], fmts)
        assert torch.equal(alone["out"][0], r["out"])
        assert torch.equal(alone["idx"][0], r["idx"])


def test_argument_checks_of_the_ragged_calls():
    lib = ensure_built()
    import ctypes
    cu_bad = (ctypes.c_int32 * 3)(0, 5, 5)
    k0 = (ctypes.c_int32 * 2)(0, 0)
    assert lib.hyq_select_vertical_varlen(None, None, 2, cu_bad, 4, 2, 128, 16, 0, k0, None, None, 0, None) == 1
    assert lib.hyq_quantize_blocks_varlen(0x1000, 2, cu_bad, 4, 128, 64, 0, 0x2000, 0x3000, None) == 1
    cu = (ctypes.c_int32 * 3)(0, 100, 300)
    k_big = (ctypes.c_int32 * 2)(0, 300)
    assert lib.hyq_select_vertical_varlen(0x1000, 0x2000, 2, cu, 4, 2, 128, 16, 0, k_big, 0x3000, 0x4000, 1 << 20, None) == 1   # k > P
    assert lib.hyq_select_vertical_varlen(None, None, 2, cu, 4, 2, 128, 16, 0, k0, None, None, 0, None) == 0                      # nothing to select
