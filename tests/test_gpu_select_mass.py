"""GPU parity of the column-mass selector (Eq. 4-5) against the oracle.  Where scores nearly tie, several sets are
correct answers to the definition: every set the library returns is checked for VALIDITY against the
plain-definition oracle (nothing selected scores lower than anything left out, beyond fp64 rounding), and, as a
second and stricter assert, for bit-equality with the oracle's fixed-order recipe (the library's reproducibility
contract)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_27875_b200 import api, workloads as wl
from gpu_util import ensure_built, rand_bf16

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _lib():
    ensure_built()


SHAPES = [  # B, Hq, Hkv, Lq, Lk, W, n_queries, k
    (1, 4, 2, 200, 200, 40, 0, 7), (1, 2, 2, 70, 333, 64, 17, 5), (2, 8, 2, 130, 130, 5, 5, 9), (1, 1, 1, 64, 129, 64, 64, 3),
    (1, 8, 1, 300, 1000, 128, 70, 50), (1, 4, 4, 1, 65, 1, 1, 64), (1, 6, 2, 515, 515, 100, 9, 415), (1, 4, 2, 90, 90, 90, 0, 5),
]


def assert_valid_for_the_definition(got, q, kk, W, k, nT, alpha=None):
    """got [B,Hq,k]: size k, strictly ascending, inside [0, P), and no selected key scores lower under the plain
    definition than an unselected one (tolerance: 1e-12 of the largest score, the rounding of fp64 sums)."""
    P = max(0, kk.shape[2] - W)
    if P == 0:
        assert got.shape[2] == 0
        return
    _, sc = oracle.select_vertical_mass(wl.bits(q), wl.bits(kk), W, k, nT, alpha=alpha, return_scores=True, plain=True)
    assert got.shape == sc.shape[:2] + (k,)
    assert got.min() >= 0 and got.max() < P
    assert np.all(np.diff(got, axis=-1) > 0)
    for b in range(got.shape[0]):
        for h in range(got.shape[1]):
            chosen = np.zeros(P, dtype=bool)
            chosen[got[b, h]] = True
            if chosen.all():
                continue
            assert sc[b, h][chosen].min() >= sc[b, h][~chosen].max() - 1e-12 * sc[b, h].max(), (b, h)


@pytest.mark.parametrize("B,Hq,Hkv,Lq,Lk,W,nT,k", SHAPES)
def test_index_sets_are_valid_and_bit_exact(B, Hq, Hkv, Lq, Lk, W, nT, k):
    q, kk = rand_bf16((B, Hq, Lq, 128), 1, 1.2), rand_bf16((B, Hkv, Lk, 128), 2, 1.2)
    got = api.hyq_select_vertical_mass(q.cuda(), kk.cuda(), W, k, nT)
    torch.cuda.synchronize()
    got = got.cpu().numpy()
    assert_valid_for_the_definition(got, q, kk, W, k, nT)
    want = oracle.select_vertical_mass(wl.bits(q), wl.bits(kk), W, k, nT)
    assert got.shape == want.shape and np.array_equal(got, want)


def test_planted_keys_large_scores_and_a_custom_scale():
    w = wl.CONFIGS["c0"].scaled(L=1536, Hq=4, Hkv=2)
    Q, K, _ = wl.make_inputs(w)
    K[:, :, :500] = (K[:, :, :500].float() * 6).to(torch.bfloat16)          # scores in the hundreds
    for scale in (0.0, 0.05):
        want = oracle.select_vertical_mass(wl.bits(Q), wl.bits(K), w.window, w.k, 24, alpha=None if scale == 0 else np.float32(scale))
        got = api.hyq_select_vertical_mass(Q.cuda(), K.cuda(), w.window, w.k, 24, softmax_scale=scale).cpu().numpy()
        assert_valid_for_the_definition(got, Q, K, w.window, w.k, 24, alpha=None if scale == 0 else np.float32(scale))
        assert np.array_equal(got, want)


def test_benchmark_shape_heads_and_argument_checks():
    """c2's keys (32768 rows), two KV heads, 16 tail queries: all 8 query heads against the oracle."""
    w = wl.CONFIGS["c2"]
    Q, K, _ = wl.make_inputs(w, heads=[0, 5])
    Qt = Q[:, :, -64:].contiguous()
    want = oracle.select_vertical_mass(wl.bits(Qt), wl.bits(K), w.window, w.k, 16)
    got = api.hyq_select_vertical_mass(Qt.cuda(), K.cuda(), w.window, w.k, 16).cpu().numpy()
    assert_valid_for_the_definition(got, Qt, K, w.window, w.k, 16)
    assert np.array_equal(got, want)
    with pytest.raises(api.HyqError):
        api.hyq_select_vertical_mass(Qt.cuda(), K.cuda(), w.window, w.k, 65)       # more queries than rows given
    with pytest.raises(api.HyqError):
        api.hyq_select_vertical_mass(Q[:, :, -8:].contiguous().cuda(), K[:, :, :4].contiguous().cuda(), 2, 1, 2)   # Lq > Lk
