"""Pins for the oracle's column-mass selector (Eq. 4-5): vertical-line score = attention mass a key receives
from a set of tail queries, then top-k over the non-window prefix.  Two oracle functions are pinned: the plain
definition (two-pass softmax, libm exp, sequential sums) and the fixed-order recipe that the library reproduces
bit for bit; the recipe is additionally pinned to the plain definition."""
import math

import numpy as np
import pytest
import scipy.special
import torch

import oracle
from paper_2608_27875_b200 import workloads as wl


def _qk(B=1, Hq=4, Hkv=2, Lq=200, Lk=200, D=16, seed=0, scale=1.0):
    g = torch.Generator().manual_seed(seed)
    q = (torch.randn(B, Hq, Lq, D, generator=g) * scale).to(torch.bfloat16)
    k = (torch.randn(B, Hkv, Lk, D, generator=g) * scale).to(torch.bfloat16)
    return q, k


def _column_mass_lib(q, k, W, nT, alpha=None):
    """Column sums of library softmax rows (scipy), fp64."""
    B, Hq, Lq, D = q.shape
    _, Hkv, Lk, _ = k.shape
    g = Hq // Hkv
    P = Lk - W
    alpha = 1 / math.sqrt(D) if alpha is None else alpha
    out = np.zeros((B, Hq, P))
    for b in range(B):
        for h in range(Hq):
            kk = k[b, h // g].double().numpy()
            for i in range(Lq - nT, Lq):
                pos = Lk - Lq + i
                s = alpha * (kk[:pos + 1] @ q[b, h, i].double().numpy())
                out[b, h] += scipy.special.softmax(s)[:P]
    return out


def test_exp_det_is_exp_to_an_ulp():
    x = np.concatenate([np.linspace(-690, 0, 100001), -np.logspace(-300, 2.8, 2001), [0.0, -0.5 * math.log(2), -math.log(2)]])
    e = oracle.exp_det(x)
    ref = np.array([math.exp(v) for v in x])
    assert np.all(np.abs(e - ref) <= 2 * np.spacing(ref))
    assert oracle.exp_det(np.array([0.0]))[0] == 1.0
    assert np.all(oracle.exp_det(np.array([-690.0001, -1e4, -np.inf])) == 0.0)
    xs = np.sort(x)
    assert np.all(np.diff(oracle.exp_det(xs)) >= -np.spacing(oracle.exp_det(xs))[1:])        # monotone up to an ulp


PLAIN = [pytest.param(True, id="plain"), pytest.param(False, id="recipe")]


@pytest.mark.parametrize("plain", PLAIN)
@pytest.mark.parametrize("Lq,Lk,W,nT,Hq,Hkv", [(200, 200, 40, 0, 4, 2), (70, 333, 64, 17, 2, 2), (130, 130, 5, 5, 6, 2),
                                                (64, 129, 64, 64, 1, 1)])
def test_scores_are_the_column_sums_of_library_softmax(plain, Lq, Lk, W, nT, Hq, Hkv):
    q, k = _qk(1, Hq, Hkv, Lq, Lk, 16, seed=Lk, scale=1.5)
    n = nT or min(W, Lq)
    idx, sc = oracle.select_vertical_mass(wl.bits(q), wl.bits(k), W, 7, nT, return_scores=True, plain=plain)
    ref = _column_mass_lib(q, k, W, n)
    assert np.allclose(sc, ref, rtol=1e-12, atol=1e-300)
    for h in range(Hq):
        order = sorted(range(Lk - W), key=lambda p: (-sc[0, h, p], p))[:7]
        assert idx[0, h].tolist() == sorted(order)
        assert set(idx[0, h].tolist()) == set(np.argsort(-ref[0, h], kind="stable")[:7].tolist())


@pytest.mark.parametrize("plain", PLAIN)
def test_brute_force_on_a_tiny_case(plain):
    q, k = _qk(1, 2, 1, 6, 9, 4, seed=3)
    W, nT = 3, 2
    _, sc = oracle.select_vertical_mass(wl.bits(q), wl.bits(k), W, 2, nT, alpha=0.7, return_scores=True, plain=plain)
    qf, kf = q.double().numpy()[0], k.double().numpy()[0, 0]
    for h in range(2):
        want = [0.0] * 6
        for i in (4, 5):
            pos = 9 - 6 + i
            e = [math.exp(0.7 * sum(a * b for a, b in zip(qf[h, i].tolist(), kf[j].tolist()))) for j in range(pos + 1)]
            z = sum(e)
            for p in range(6):
                want[p] += e[p] / z
        assert np.allclose(sc[0, h], want, rtol=1e-12)


@pytest.mark.parametrize("plain", PLAIN)
def test_mass_is_conserved_and_a_planted_sink_is_found(plain):
    B, Hq, Hkv, L, D, W = 1, 4, 2, 300, 32, 32
    q, k = _qk(B, Hq, Hkv, L, L, D, seed=5)
    u = torch.nn.functional.normalize(torch.randn(D, generator=torch.Generator().manual_seed(6)), dim=0)
    k[:, :, 11] = (k[:, :, 11].float() + 6 * u).to(torch.bfloat16)
    q = (q.float() + 2 * u).to(torch.bfloat16)
    idx, sc = oracle.select_vertical_mass(wl.bits(q), wl.bits(k), W, 3, 0, return_scores=True, plain=plain)
    assert np.all(sc >= 0) and np.all(sc.sum(-1) <= W * (1 + 1e-12))       # each of the W query rows carries mass 1
    assert all(11 in idx[0, h] for h in range(Hq))
    assert np.all(np.argmax(sc, axis=-1) == 11)


@pytest.mark.parametrize("plain", PLAIN)
def test_gqa_equals_mha_on_repeated_kv_and_long_windows_select_nothing(plain):
    q, k = _qk(2, 4, 2, 90, 90, 16, seed=8)
    a = oracle.select_vertical_mass(wl.bits(q), wl.bits(k), 16, 5, plain=plain)
    b = oracle.select_vertical_mass(wl.bits(q), wl.bits(k.repeat_interleave(2, dim=1)), 16, 5, plain=plain)
    assert np.array_equal(a, b)
    assert oracle.select_vertical_mass(wl.bits(q), wl.bits(k), 90, 5, plain=plain).shape == (2, 4, 0)
    with pytest.raises(ValueError):
        oracle.select_vertical_mass(wl.bits(q), wl.bits(k), 16, 5, n_queries=17, plain=plain)     # more queries than window rows


@pytest.mark.parametrize("plain", PLAIN)
def test_large_scores_do_not_overflow(plain):
    q, k = _qk(1, 2, 2, 80, 80, 16, seed=9, scale=12.0)          # |s| in the hundreds
    _, sc = oracle.select_vertical_mass(wl.bits(q), wl.bits(k), 16, 4, return_scores=True, plain=plain)
    assert np.all(np.isfinite(sc))
    assert np.allclose(sc, _column_mass_lib(q, k, 16, 16), rtol=1e-11, atol=1e-300)


@pytest.mark.parametrize("Lq,Lk,W,nT,Hq,Hkv,scale", [(200, 200, 40, 0, 4, 2, 1.0), (70, 333, 64, 17, 2, 2, 1.5), (300, 1000, 128, 70, 4, 1, 1.2),
                                                      (80, 80, 16, 0, 2, 2, 12.0)])
def test_the_recipe_is_the_plain_definition_up_to_rounding(Lq, Lk, W, nT, Hq, Hkv, scale):
    """The fixed-order recipe (chunk maxima, pairwise trees, polynomial exp) against the definition itself: scores
    within 1e-12 of the largest score, and the recipe's set valid for the plain scores (nothing selected scores
    lower than anything left out, beyond that rounding)."""
    q, k = _qk(1, Hq, Hkv, Lq, Lk, 32, seed=Lk + Lq, scale=scale)
    kk = 9
    idx_r, sc_r = oracle.select_vertical_mass(wl.bits(q), wl.bits(k), W, kk, nT, return_scores=True)
    idx_p, sc_p = oracle.select_vertical_mass(wl.bits(q), wl.bits(k), W, kk, nT, return_scores=True, plain=True)
    tol = 1e-12 * sc_p.max()
    assert np.abs(sc_r - sc_p).max() <= tol
    for h in range(Hq):
        chosen = np.zeros(Lk - W, dtype=bool)
        chosen[idx_r[0, h]] = True
        assert sc_p[0, h][chosen].min() >= sc_p[0, h][~chosen].max() - tol
        if np.sort(sc_p[0, h])[-kk] - np.sort(sc_p[0, h])[-kk - 1] > 2 * tol:     # no near-tie at the boundary: one valid set
            assert np.array_equal(idx_r[0, h], idx_p[0, h])
