"""Pins for the oracle's hybrid-precision attention (Eq. 6-7; Algorithm 2, Stage 3)."""
import math

import numpy as np
import pytest
import torch
import torch.nn.functional as F

import oracle
from paper_2608_27875_b200 import workloads as wl

INT8, FP8, INT4 = oracle.FMT_INT8, oracle.FMT_FP8_E4M3, oracle.FMT_INT4


def _qkv(B=1, Hq=4, Hkv=2, L=40, D=16, seed=0):
    g = torch.Generator().manual_seed(seed)
    q = torch.randn(B, Hq, L, D, generator=g).to(torch.bfloat16)
    k = torch.randn(B, Hkv, L, D, generator=g).to(torch.bfloat16)
    v = torch.randn(B, Hkv, L, D, generator=g).to(torch.bfloat16)
    return q, k, v


def _quant(q, k, v, fmts, bt=64):
    out = []
    for t, f in zip((q, k, v), fmts):
        out.append(oracle.quantize(wl.bits(t), f, bt))
    return out


def _dequant_lib(codes, scales, fmt, bt):
    """Dequantized tensor through library casts only (torch float8 view, numpy int views)."""
    if fmt == INT8:
        val = torch.from_numpy(codes.view(np.int8).astype(np.float64))
    elif fmt == FP8:
        val = torch.from_numpy(codes.copy()).view(torch.float8_e4m3fn).double()
    else:
        lo = (codes & 0xF).astype(np.int16)
        hi = (codes >> 4).astype(np.int16)
        lo[lo >= 8] -= 16
        hi[hi >= 8] -= 16
        val = torch.from_numpy(np.stack([lo, hi], -1).reshape(codes.shape[:-1] + (-1,)).astype(np.float64))
    L = val.shape[2]
    sc = torch.from_numpy(scales.astype(np.float64)).repeat_interleave(bt, dim=2)[:, :, :L, None]
    return val * sc


def _call(q, k, v, qz, fmts, idx, W, rows=None, bt=64, **kw):
    (qc, qs), (kc, ks), (vc, vs) = qz
    return oracle.attention_rows(wl.bits(q), wl.bits(k), wl.bits(v), qc, kc, vc, qs, ks, vs, fmts, idx, W,
                                 rows, bt, **kw)


def _rand_idx(B, Hq, L, W, kk, seed=0):
    rng = np.random.default_rng(seed)
    P = L - W
    return np.stack([np.stack([np.sort(rng.choice(P, kk, replace=False)) for _ in range(Hq)])
                     for _ in range(B)]).astype(np.int32)


def test_full_window_equals_exact_causal_attention():
    """W >= L: every pair is full precision, so the result is plain softmax attention."""
    q, k, v = _qkv(Hq=4, Hkv=2, L=96, D=32, seed=1)
    qz = _quant(q, k, v, (INT8, INT8, INT8))
    got = _call(q, k, v, qz, (INT8, INT8, INT8), None, 96)
    kr, vr = (t.double().repeat_interleave(2, dim=1) for t in (k, v))
    ref = F.scaled_dot_product_attention(q.double(), kr, vr, is_causal=True)
    np.testing.assert_allclose(got, ref.numpy(), rtol=0, atol=1e-12)
    # the same through the vertical set: all prefix keys vertical, window covering the rest
    idx = np.broadcast_to(np.arange(64, dtype=np.int32), (1, 4, 64)).copy()
    got2 = _call(q, k, v, qz, (INT8, INT8, INT8), idx, 32)
    np.testing.assert_allclose(got2, ref.numpy(), rtol=0, atol=1e-12)


@pytest.mark.parametrize("fmts", [(INT8, INT8, INT8), (INT4, INT4, FP8), (FP8, FP8, FP8)])
def test_no_vertical_no_window_equals_fully_quantized_attention(fmts):
    q, k, v = _qkv(Hq=4, Hkv=2, L=150, D=32, seed=2)
    qz = _quant(q, k, v, fmts)
    got = _call(q, k, v, qz, fmts, None, 0)
    qh, kh, vh = (_dequant_lib(c, s, f, 64) for (c, s), f in zip(qz, fmts))
    ref = F.scaled_dot_product_attention(qh, kh.repeat_interleave(2, dim=1), vh.repeat_interleave(2, dim=1),
                                         is_causal=True)
    np.testing.assert_allclose(got, ref.numpy(), rtol=0, atol=1e-12)


def _brute(q, k, v, qh, kh, vh, idx, W, alpha):
    """Triple loop in Python floats over the definition of Eq. 7."""
    B, Hq, L, D = q.shape
    g = Hq // k.shape[1]
    ql, kl, vl_, qhl, khl, vhl = (t.double().tolist() for t in (q, k, v, qh, kh, vh))
    out = np.zeros((B, Hq, L, D))
    for b in range(B):
        for h in range(Hq):
            kv = h // g
            vset = set(idx[b, h].tolist()) if idx is not None else set()
            for i in range(L):
                s, vals = [], []
                for j in range(i + 1):
                    fp = (j in vset) or (i - j < W)
                    qq, kk, vv = (ql, kl, vl_) if fp else (qhl, khl, vhl)
                    s.append(alpha * sum(qq[b][h][i][d] * kk[b][kv][j][d] for d in range(D)))
                    vals.append(vv[b][kv][j])
                m = max(s)
                p = [math.exp(x - m) for x in s]
                z = sum(p)
                for d in range(D):
                    out[b, h, i, d] = sum(pj * vj[d] for pj, vj in zip(p, vals)) / z
    return out


@pytest.mark.parametrize("fmts,W,kk", [((INT8, INT8, INT8), 5, 4), ((INT4, INT4, FP8), 8, 3),
                                       ((FP8, FP8, FP8), 6, 5),
                                       ((INT8, INT8, INT8), 0, 6), ((INT8, INT8, INT8), 1, 0)])
def test_against_brute_force(fmts, W, kk):
    bt = 8
    q, k, v = _qkv(B=2, Hq=4, Hkv=2, L=27, D=8, seed=3 + W)
    qz = _quant(q, k, v, fmts, bt)
    idx = _rand_idx(2, 4, 27, W, kk, seed=W) if kk else None
    got = _call(q, k, v, qz, fmts, idx, W, bt=bt)
    qh, kh, vh = (_dequant_lib(c, s, f, bt) for (c, s), f in zip(qz, fmts))
    ref = _brute(q, k, v, qh, kh, vh, idx, W, 1 / math.sqrt(8))
    np.testing.assert_allclose(got, ref, rtol=0, atol=1e-12)


@pytest.mark.parametrize("tile_n", [1, 7, 64])
def test_segmented_walk_equals_single_softmax(tile_n):
    """Algorithm 2's three-segment online softmax is Eq. 7 in another order."""
    fmts = (INT4, INT4, FP8)
    q, k, v = _qkv(B=1, Hq=4, Hkv=2, L=130, D=16, seed=5)
    qz = _quant(q, k, v, fmts, 64)
    idx = _rand_idx(1, 4, 130, 20, 9, seed=2)
    (qc, qs), (kc, ks), (vc, vs) = qz
    a = _call(q, k, v, qz, fmts, idx, 20)
    b = oracle.attention_segmented_rows(wl.bits(q), wl.bits(k), wl.bits(v), qc, kc, vc, qs, ks, vs, fmts, idx, 20,
                                        None, tile_n)
    np.testing.assert_allclose(a, b, rtol=0, atol=1e-12)


def test_full_precision_pair_count_closed_form():
    """|FP pairs| = sum over heads of  W L - W(W-1)/2 + sum_{j in I} max(0, L - j - W)."""
    L, W, kk = 90, 17, 6
    q, k, v = _qkv(B=2, Hq=4, Hkv=2, L=L, D=8, seed=6)
    qz = _quant(q, k, v, (INT8,) * 3)
    idx = _rand_idx(2, 4, L, W, kk, seed=4)
    _, n_fp = _call(q, k, v, qz, (INT8,) * 3, idx, W, return_fp_pairs=True)
    closed = sum(W * L - W * (W - 1) // 2 + sum(max(0, L - int(j) - W) for j in idx[b, h])
                 for b in range(2) for h in range(4))
    assert n_fp == closed


def test_first_row_returns_first_value_and_rows_subset_matches_full():
    q, k, v = _qkv(B=1, Hq=4, Hkv=2, L=70, D=16, seed=7)
    qz = _quant(q, k, v, (INT8,) * 3)
    idx = _rand_idx(1, 4, 70, 8, 5, seed=1)
    full, lse = _call(q, k, v, qz, (INT8,) * 3, idx, 8, return_lse=True)
    np.testing.assert_array_equal(full[0, :, 0], v.double().numpy()[0].repeat(2, axis=0)[:, 0])   # W >= 1
    rows = np.array([0, 3, 69, 31], dtype=np.int32)
    sub = _call(q, k, v, qz, (INT8,) * 3, idx, 8, rows)
    np.testing.assert_array_equal(sub, full[:, :, rows])
    # with W = 0 the only key of row 0 is low-bit: the output is the dequantized V row
    w0 = _call(q, k, v, qz, (INT8,) * 3, None, 0, np.array([0], dtype=np.int32))
    vh = _dequant_lib(*qz[2], INT8, 64).numpy()[0].repeat(2, axis=0)[:, 0]
    np.testing.assert_allclose(w0[0, :, 0], vh, rtol=0, atol=1e-15)
    # log-sum-exp of row 0 is its single score
    assert np.isfinite(lse).all()


def test_hybrid_reduces_error_as_the_paper_reports():
    """Keeping vertical-line keys and the window in full precision lowers the error against
    exact attention; each alone helps, both together help most (Section 4.4, ablation)."""
    w = wl.CONFIGS["c0"].scaled(L=512, window=64, k=16, n_plant=8, Hq=2, Hkv=2)
    Q, K, V = wl.make_inputs(w)
    fmts = (INT4, INT4, INT4)
    qz = _quant(Q, K, V, fmts)
    idx = oracle.select_vertical(wl.bits(Q), wl.bits(K), w.window, w.k)
    exact = _call(Q, K, V, qz, fmts, None, w.L)
    err = {}
    err["uniform"] = np.abs(_call(Q, K, V, qz, fmts, None, 0) - exact).mean()
    err["window"] = np.abs(_call(Q, K, V, qz, fmts, None, w.window) - exact).mean()
    err["vl"] = np.abs(_call(Q, K, V, qz, fmts, idx, 0) - exact).mean()
    err["hybrid"] = np.abs(_call(Q, K, V, qz, fmts, idx, w.window) - exact).mean()
    assert err["hybrid"] < err["window"] < err["uniform"]
    assert err["hybrid"] < err["vl"] < err["uniform"]
    # and 8-bit is far more accurate than 4-bit (Fig. 2)
    qz8 = _quant(Q, K, V, (INT8,) * 3)
    e8 = np.abs(_call(Q, K, V, qz8, (INT8,) * 3, None, 0) - exact).mean()
    assert e8 < 0.25 * err["uniform"]


# ---- query block shorter than the keys (Algorithm 2: a query block against the full K, V; end-aligned) ----------
@pytest.mark.parametrize("fmts", [(INT8, INT8, INT8), (INT4, INT4, FP8)])
def test_block_aligned_query_block_reproduces_the_tail_rows_of_the_whole_prefill(fmts):
    """When the query block starts on a quantization-block boundary its codes and scales are slices of the
    whole prefill's, every (row, key) pair is classified and scored alike, and the rows must come out
    identical to the last rows of the whole prefill, bit for bit."""
    L, W, kk, bt, D = 200, 24, 7, 8, 16
    q, k, v = _qkv(B=2, Hq=4, Hkv=2, L=L, D=D, seed=3)
    qz = _quant(q, k, v, fmts, bt)
    idx = _rand_idx(2, 4, L, W, kk, seed=5)
    full = _call(q, k, v, qz, fmts, idx, W, bt=bt)
    for Lq in (bt, 5 * bt, L):                   # offsets L - Lq = 192, 160, 0: multiples of the block size
        off = L - Lq
        (qc, qs), kz, vz = qz
        qz_blk = ((qc[:, :, off:], qs[:, :, off // bt:]), kz, vz)
        got = _call(q[:, :, off:], k, v, qz_blk, fmts, idx, W, bt=bt)
        assert got.shape == (2, 4, Lq, D)
        assert np.array_equal(got, full[:, :, off:])


def test_single_query_row_with_a_covering_window_is_the_textbook_softmax():
    """L_Q = 1 and W >= L_K: every pair is full precision, the row is the last position."""
    L, D = 37, 16
    q, k, v = _qkv(B=1, Hq=2, Hkv=1, L=L, D=D, seed=8)
    q1 = q[:, :, -1:]
    fm = (INT8, INT8, INT8)
    qz = [oracle.quantize(wl.bits(q1), INT8, 64), oracle.quantize(wl.bits(k), INT8, 64), oracle.quantize(wl.bits(v), INT8, 64)]
    got, lse = _call(q1, k, v, qz, fm, None, L, return_lse=True)
    s = torch.einsum("bhqd,bkd->bhqk", q1.double(), k[:, 0].double()) / math.sqrt(D)
    ref = torch.einsum("bhqk,bkd->bhqd", torch.softmax(s, -1), v[:, 0].double())
    assert np.abs(got - ref.numpy()).max() < 1e-12
    assert np.abs(lse - torch.logsumexp(s, -1).numpy()).max() < 1e-12


@pytest.mark.parametrize("Lq", [1, 13, 70])
def test_query_block_off_the_block_grid_segmented_walk_and_pair_count(Lq):
    """A query block that does not start on a quantization-block boundary carries its own Q blocks.  The
    literal three-segment walk must agree with the single softmax, and the number of full-precision pairs
    has a closed form: row r sits at position p = L - Lq + r and has min(p + 1, W) window keys plus the
    vertical keys at positions <= p - W."""
    L, W, kk, bt, D = 150, 20, 9, 16, 16
    fmts = (INT8, INT8, INT8)
    q, k, v = _qkv(B=1, Hq=2, Hkv=2, L=L, D=D, seed=11)
    qb = q[:, :, L - Lq:]
    qz = _quant(qb, k, v, fmts, bt)
    idx = _rand_idx(1, 2, L, W, kk, seed=2)
    got, n_fp = _call(qb, k, v, qz, fmts, idx, W, bt=bt, return_fp_pairs=True)
    (qc, qs), (kc, ks), (vc, vs) = qz
    seg = oracle.attention_segmented_rows(wl.bits(qb), wl.bits(k), wl.bits(v), qc, kc, vc, qs, ks, vs, fmts, idx, W,
                                          None, 8, bt)
    assert np.abs(got - seg).max() < 1e-12
    expect = 0
    for h in range(2):
        for r in range(Lq):
            p = L - Lq + r
            expect += min(p + 1, W) + int((idx[0, h] <= p - W).sum())
    assert n_fp == expect


def test_query_block_longer_than_the_keys_is_rejected():
    q, k, v = _qkv(B=1, Hq=1, Hkv=1, L=20, D=16, seed=1)
    qz = _quant(q, k[:, :, :10], v[:, :, :10], (INT8, INT8, INT8), 64)
    with pytest.raises((ValueError, AssertionError)):
        _call(q, k[:, :, :10], v[:, :, :10], qz, (INT8, INT8, INT8), None, 4)


# ---- Algorithm 2's window taken literally: the last W keys for every row of the query block ------------------
def test_fixed_tail_window_agrees_with_the_sliding_window_on_the_last_row_only():
    """For the last row both window forms name the same keys, [L - W, L); for earlier rows the fixed window
    holds fewer causal keys, so the classes differ and (with quantization error) so do the outputs."""
    L, W, kk, bt = 120, 30, 6, 16
    fmts = (INT8, INT8, INT8)
    q, k, v = _qkv(B=1, Hq=2, Hkv=1, L=L, D=16, seed=21)
    qz = _quant(q, k, v, fmts, bt)
    idx = _rand_idx(1, 2, L, W, kk, seed=9)
    slide = _call(q, k, v, qz, fmts, idx, W, bt=bt)
    fixed = _call(q, k, v, qz, fmts, idx, W, bt=bt, fixed_window=True)
    assert np.array_equal(slide[:, :, -1], fixed[:, :, -1])
    assert not np.array_equal(slide[:, :, L // 2], fixed[:, :, L // 2])


@pytest.mark.parametrize("Lq", [1, 25, 64, 150])
def test_fixed_tail_window_pair_count_segments_and_full_precision_limit(Lq):
    """Row at position p has max(0, p - (L - W) + 1) window keys and the vertical keys at positions <= p
    (all of them lie below L - W); the literal three-segment walk agrees with the single softmax; and with
    W >= L the fixed window covers every key, i.e. exact causal attention."""
    L, W, kk, bt, D = 150, 40, 8, 16, 16
    fmts = (INT4, INT4, FP8)
    q, k, v = _qkv(B=1, Hq=2, Hkv=2, L=L, D=D, seed=31)
    qb = q[:, :, L - Lq:]
    qz = _quant(qb, k, v, fmts, bt)
    idx = _rand_idx(1, 2, L, W, kk, seed=4)
    got, n_fp = _call(qb, k, v, qz, fmts, idx, W, bt=bt, return_fp_pairs=True, fixed_window=True)
    (qc, qs), (kc, ks), (vc, vs) = qz
    seg = oracle.attention_segmented_rows(wl.bits(qb), wl.bits(k), wl.bits(v), qc, kc, vc, qs, ks, vs, fmts, idx, W,
                                          None, 8, bt, fixed_window=True)
    assert np.abs(got - seg).max() < 1e-12
    expect = 0
    for h in range(2):
        for r in range(Lq):
            p = L - Lq + r
            expect += max(0, p - (L - W) + 1) + int((idx[0, h] <= p).sum())
    assert n_fp == expect
    exact = _call(qb, k, v, qz, fmts, None, L, bt=bt, fixed_window=True)
    s = torch.einsum("bhqd,bhkd->bhqk", qb.double(), k.double()) / math.sqrt(D)
    pos = torch.arange(L - Lq, L)[:, None]
    s = s.masked_fill(torch.arange(L)[None, :] > pos, float("-inf"))
    ref = torch.einsum("bhqk,bhkd->bhqd", torch.softmax(s, -1), v.double())
    assert np.abs(exact - ref.numpy()).max() < 1e-12
