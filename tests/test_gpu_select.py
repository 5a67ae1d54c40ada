"""GPU parity: hyq_select_vertical against the oracle - identical index sets, ascending."""
import numpy as np
import pytest
import torch

import oracle
from gpu_util import ensure_built, rand_bf16
from paper_2608_27875_b200 import api, workloads as wl

pytestmark = pytest.mark.gpu


def _check(Q, K, window, k, n_tail=0):
    ensure_built()
    got = api.hyq_select_vertical(Q.cuda(), K.cuda(), window, k, n_tail)
    torch.cuda.synchronize()
    ref = oracle.select_vertical(wl.bits(Q), wl.bits(K), window, k, n_tail)
    np.testing.assert_array_equal(got.cpu().numpy(), ref)


@pytest.mark.parametrize("B,Hq,Hkv,L,W,k,n_tail", [
    (1, 2, 2, 2048, 128, 32, 0), (2, 8, 2, 1000, 100, 17, 0), (1, 5, 1, 777, 64, 1, 0),
    (1, 4, 4, 300, 299, 1, 0), (1, 6, 2, 515, 3, 512, 0), (1, 4, 2, 4096, 512, 82, 64), (1, 3, 3, 129, 1, 128, 0),
])
def test_matches_oracle(B, Hq, Hkv, L, W, k, n_tail):
    _check(rand_bf16((B, Hq, L, 128), seed=L), rand_bf16((B, Hkv, L, 128), seed=L + 1), W, k, n_tail)


def test_ties_duplicates_and_signed_zeros():
    L, W = 600, 88
    Q = rand_bf16((1, 4, L, 128), seed=1)
    K = rand_bf16((1, 2, L, 128), seed=2)
    K[0, 0, 100:140] = K[0, 0, 50]          # 41 identical keys -> identical scores
    K[0, 1, 5:300] = 0.0                    # a run of exact-zero scores ...
    K[0, 1, 7] = -0.0                       # ... one of them from negative zeros
    K[0, 1, 300:] = -K[0, 1, 300:].abs() * torch.sign(Q[0, 2:, -W:].float().mean((0, 1))).to(torch.bfloat16)
    for k in (1, 20, 60, 300, L - W):
        _check(Q, K, W, k)


@pytest.mark.parametrize("seed", range(4))
def test_tail_queries_with_a_wide_exponent_spread(seed):
    """Tail rows mixing magnitudes from 1e-30 to 3e4 and large values of alternating sign: the fp64 partial sums of
    the tail mean are then inexact, so its value depends on the order of the additions - it has to be the row
    order of Algorithm 1 as the oracle takes it, or the index sets near ties come out different."""
    g = torch.Generator().manual_seed(700 + seed)
    B, Hq, Hkv, L, W, k = 1, 4, 2, 1200, 256, 40
    Q = torch.randn(B, Hq, L, 128, generator=g)
    mag = 10.0 ** (torch.rand(B, Hq, L, 128, generator=g) * 34.5 - 30.0)            # 1e-30 ... 3e4
    Q = Q.sign() * mag
    big = 3.0e4 * (1.0 + torch.rand(B, Hq, L, 1, generator=g))
    sign = torch.where(torch.arange(L) % 2 == 0, 1.0, -1.0).view(1, 1, L, 1)
    Q[..., ::3] = (sign * big).expand(B, Hq, L, 128)[..., ::3]                      # cancelling large terms in every third channel
    Q = Q.to(torch.bfloat16)
    K = rand_bf16((B, Hkv, L, 128), seed=800 + seed)
    K[0, :, 10:50] = K[0, :, 9:10]                                                  # equal keys: near-ties decided by the mean's last bits
    _check(Q, K, W, k)
    _check(Q, K, W, k, n_tail=77)


def test_empty_problems_touch_nothing():
    ensure_built()
    Q, K = rand_bf16((1, 2, 64, 128), 3).cuda(), rand_bf16((1, 2, 64, 128), 4).cuda()
    assert api.hyq_select_vertical(Q, K, 64, 4).shape == (1, 2, 0)        # P == 0
    assert api.hyq_select_vertical(Q, K, 16, 0).shape == (1, 2, 0)        # k == 0
    with pytest.raises(api.HyqError):
        api.hyq_select_vertical(Q, K, 16, 49)                             # k > P


@pytest.mark.parametrize("name", ["c0", "c1", "c2", "c4"])
def test_workload_configs(name):
    """Full-size selection of the benchmark configurations (the oracle does these in seconds)."""
    w = wl.CONFIGS[name]
    heads = None if name in ("c0", "c1") else [0, w.Hkv - 1]
    if w.B > 1:
        w = w.scaled(B=1)
    Q, K, _ = wl.make_inputs(w, heads=heads)
    _check(Q, K, w.window, w.k)


def test_longest_context_two_heads():
    w = wl.CONFIGS["c3"]
    Q, K, _ = wl.make_inputs(w, heads=[3])
    _check(Q, K, w.window, w.k)
