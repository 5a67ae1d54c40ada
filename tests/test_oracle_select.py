"""Pins for the oracle's vertical token identification (Algorithm 1)."""
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle
from paper_2608_27875_b200 import workloads as wl


def _qk(B=2, Hq=4, Hkv=2, L=96, D=16, seed=0):
    g = torch.Generator().manual_seed(seed)
    q = torch.randn(B, Hq, L, D, generator=g).to(torch.bfloat16)
    k = torch.randn(B, Hkv, L, D, generator=g).to(torch.bfloat16)
    return q, k


def _brute(q, k, W, kk, n_tail=0):
    """Exact rational dot products of the fp64 mean with the keys, sort with key
    (-score, position); random data has no near-ties, so the exact ranking and
    the fp64 ranking coincide."""
    B, Hq, L, D = q.shape
    Hkv = k.shape[1]
    g = Hq // Hkv
    P = max(0, L - W)
    t = n_tail or min(W, L)
    out = np.zeros((B, Hq, kk), dtype=np.int32)
    qd, kd = q.double().tolist(), k.double().tolist()
    for b in range(B):
        for h in range(Hq):
            qbar = [sum(qd[b][h][i][d] for i in range(L - t, L)) / t for d in range(D)]
            sc = []
            for p in range(P):
                s = sum(Fraction(qbar[d]) * Fraction(kd[b][h // g][p][d]) for d in range(D))
                sc.append((-s, p))
            sc.sort()
            out[b, h] = sorted(p for _, p in sc[:kk])
    return out


@pytest.mark.parametrize("W,kk,n_tail", [(16, 5, 0), (1, 1, 0), (40, 56, 0), (16, 7, 3)])
def test_against_brute_force(W, kk, n_tail):
    q, k = _qk(seed=W)
    got = oracle.select_vertical(wl.bits(q), wl.bits(k), W, kk, n_tail)
    np.testing.assert_array_equal(got, _brute(q, k, W, kk, n_tail))


def test_against_torch_einsum_topk():
    """Library route: fp64 einsum in the GQA-native form + torch.topk (sets equal when no tie)."""
    q, k = _qk(B=1, Hq=8, Hkv=2, L=512, D=128, seed=5)
    W, kk = 64, 20
    P = 512 - W
    qbar = q.double()[:, :, -W:].mean(2).reshape(1, 2, 4, 128)
    S = torch.einsum("bhrd,bhpd->bhrp", qbar, k.double()[:, :, :P]).reshape(1, 8, P)
    ref = torch.topk(S, kk, dim=-1, largest=True).indices.sort(-1).values.numpy()
    got, scores = oracle.select_vertical(wl.bits(q), wl.bits(k), W, kk, return_scores=True)
    np.testing.assert_array_equal(got, ref)
    np.testing.assert_allclose(scores, S.numpy(), rtol=0, atol=1e-12)


def test_mha_branch_equals_gqa_branch_on_repeated_kv():
    q, k = _qk(B=1, Hq=6, Hkv=2, L=128, D=32, seed=9)
    a = oracle.select_vertical(wl.bits(q), wl.bits(k), 32, 9)
    b = oracle.select_vertical(wl.bits(q), wl.bits(k.repeat_interleave(3, dim=1)), 32, 9)
    np.testing.assert_array_equal(a, b)


def test_set_follows_a_permutation_of_the_prefix_keys():
    q, k = _qk(B=1, Hq=2, Hkv=2, L=200, D=32, seed=11)
    W, kk = 40, 12
    P = 200 - W
    perm = torch.randperm(P, generator=torch.Generator().manual_seed(1))
    k2 = k.clone()
    k2[:, :, :P] = k[:, :, perm]              # new position n holds old key perm[n]
    a = oracle.select_vertical(wl.bits(q), wl.bits(k), W, kk)
    b = oracle.select_vertical(wl.bits(q), wl.bits(k2), W, kk)
    for h in range(2):
        assert set(perm[b[0, h]].tolist()) == set(a[0, h].tolist())


def test_invariance_to_query_scale_and_constant_key_shift():
    q, k = _qk(B=1, Hq=2, Hkv=1, L=160, D=16, seed=13)
    a = oracle.select_vertical(wl.bits(q), wl.bits(k), 32, 10)
    b = oracle.select_vertical(wl.bits(q * 4), wl.bits(k), 32, 10)          # exact power-of-two scaling
    np.testing.assert_array_equal(a, b)
    # adding one vector to every key adds the same constant to every score -> same ranking
    # (integers keep every bf16 sum exact)
    qi = (q * 8).round().clamp(-20, 20)
    ki = (k * 8).round().clamp(-20, 20)
    shift = torch.arange(16, dtype=torch.float32).to(torch.bfloat16) - 8
    c = oracle.select_vertical(wl.bits(qi), wl.bits(ki), 32, 10)
    d = oracle.select_vertical(wl.bits(qi), wl.bits((ki.float() + shift).to(torch.bfloat16)), 32, 10)
    np.testing.assert_array_equal(c, d)


def test_ties_go_to_the_lower_position_and_zero_signs_compare_equal():
    q = torch.ones(1, 1, 8, 4, dtype=torch.bfloat16)
    k = torch.zeros(1, 1, 8, 4, dtype=torch.bfloat16)
    k[0, 0, 1] = 1.0
    k[0, 0, 4] = 1.0            # duplicates of key 1
    k[0, 0, 5] = 1.0
    k[0, 0, 2, 0] = -0.0        # -0 scores tie with +0 scores
    got = oracle.select_vertical(wl.bits(q), wl.bits(k), 2, 2)     # P = 6
    np.testing.assert_array_equal(got[0, 0], [1, 4])
    got = oracle.select_vertical(wl.bits(q), wl.bits(k), 2, 5)
    np.testing.assert_array_equal(got[0, 0], [0, 1, 2, 4, 5])


def test_degenerate_sizes():
    q, k = _qk(B=1, Hq=2, Hkv=1, L=32, D=8, seed=2)
    assert oracle.select_vertical(wl.bits(q), wl.bits(k), 32, 4).shape == (1, 2, 0)     # P = 0
    assert oracle.select_vertical(wl.bits(q), wl.bits(k), 64, 4).shape == (1, 2, 0)     # W > L
    assert oracle.select_vertical(wl.bits(q), wl.bits(k), 8, 0).shape == (1, 2, 0)      # k = 0
    full = oracle.select_vertical(wl.bits(q), wl.bits(k), 8, 24)                        # k = P
    np.testing.assert_array_equal(full[0, 0], np.arange(24))
    with pytest.raises(ValueError):
        oracle.select_vertical(wl.bits(q), wl.bits(k), 8, 25)                           # k > P


def test_planted_vertical_keys_are_recovered():
    """The synthetic workloads plant strongly attended key columns; the tail-query
    proxy of Algorithm 1 must rank most of them on top."""
    w = wl.CONFIGS["c0"]
    Q, K, V = wl.make_inputs(w)
    idx = oracle.select_vertical(wl.bits(Q), wl.bits(K), w.window, w.k)
    for h in range(w.Hq):
        planted = set(wl.planted_positions(w, 0, h).tolist())
        assert len(planted & set(idx[0, h].tolist())) >= 0.7 * len(planted)
