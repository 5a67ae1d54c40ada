"""Pins for the decode-side oracle: Freeze (Algorithm 4) and the hybrid KV-cache attention of one
token (Algorithm 3, Section 3.3)."""
import math

import numpy as np
import pytest
import scipy.special
import torch

import oracle
from oracle import decode as od
from paper_2608_27875_b200 import workloads as wl

INT8, FP8, INT4 = oracle.FMT_INT8, oracle.FMT_FP8_E4M3, oracle.FMT_INT4


def _kv(B=1, Hkv=2, N=300, D=16, seed=0):
    g = torch.Generator().manual_seed(seed)
    k = torch.randn(B, Hkv, N, D, generator=g).to(torch.bfloat16)
    v = torch.randn(B, Hkv, N, D, generator=g).to(torch.bfloat16)
    return k, v


def _q(B, Hq, D, seed=1):
    g = torch.Generator().manual_seed(seed)
    return torch.randn(B, Hq, D, generator=g).to(torch.bfloat16)


def _idx(B, H, P, kk, seed=0):
    rng = np.random.default_rng(seed)
    return np.stack([np.stack([np.sort(rng.choice(P, kk, replace=False)) for _ in range(H)])
                     for _ in range(B)]).astype(np.int32)


def _f64(t):
    return t.double().numpy()


def test_freeze_partitions_the_positions_and_keeps_rows_in_order():
    B, H, N, D, W, kk = 2, 3, 217, 16, 40, 9
    k, v = _kv(B, H, N, D)
    idx = _idx(B, H, N - W, kk)
    c = od.freeze(wl.bits(k), wl.bits(v), idx, W, group=32, fmts=(INT4, INT8))
    assert c["nQ"] == N - W - kk and c["kq_scales"].shape == (B, H, math.ceil(c["nQ"] / 32))
    for b in range(B):
        for h in range(H):
            allpos = np.concatenate([c["iq"][b, h], idx[b, h], np.arange(N - W, N)])
            assert sorted(allpos.tolist()) == list(range(N))            # each position exactly once
            assert np.all(np.diff(c["iq"][b, h]) > 0)
            assert np.array_equal(c["k_vl"][b, h], wl.bits(k)[b, h, idx[b, h]])
            assert np.array_equal(c["v_win"][b, h], wl.bits(v)[b, h, N - W:])
    assert c["n_s"] == 0 and c["k_s"].shape == (B, H, 128, D)


@pytest.mark.parametrize("fmt,c_b", [(INT4, 7.0), (INT8, 127.0)])
def test_freeze_codes_are_the_nearest_level_of_the_compacted_rows(fmt, c_b):
    """Independent of the quantizer's code: every group's scale is absmax / c_B of the GATHERED rows,
    the absmax element sits on +-c_B and every value is within half a step of its reconstruction."""
    B, H, N, D, W, kk, G = 1, 2, 200, 16, 30, 11, 32
    k, v = _kv(B, H, N, D, seed=3)
    idx = _idx(B, H, N - W, kk, seed=3)
    c = od.freeze(wl.bits(k), wl.bits(v), idx, W, group=G, fmts=(fmt, fmt))
    for name, src in (("kq", k), ("vq", v)):
        for h in range(H):
            rows = _f64(src)[0, h][c["iq"][0, h]]
            vals = od.code_values(c[name + "_codes"][0, h], fmt)
            for gi in range(math.ceil(rows.shape[0] / G)):
                blk, cv = rows[gi * G:(gi + 1) * G], vals[gi * G:(gi + 1) * G]
                amax = np.abs(blk).max()
                sc = float(c[name + "_scales"][0, h, gi])
                assert sc == np.float32(np.float32(amax) / np.float32(c_b))
                assert np.abs(cv).max() == c_b
                assert np.all(np.abs(blk - cv * sc) <= (0.5 + 1e-3) * sc)      # fp32 rounding of x * (c_B / absmax)


def test_memory_overhead_matches_the_papers_table():
    """Appendix memory table (W = 128, W_s = 128, 5 % vertical rows, K4V4, 16-bit full precision):
    +15.0 % for the vertical rows at any length; +4.7 % / +1.2 % for the window and for the staging
    buffer at 8K / 32K.  Overhead = bytes of the rows as stored minus bytes of the same rows at K4V4,
    over the strict K4V4 cache of the prefix."""
    for N, win_pct in ((8192, 4.7), (32768, 1.2)):
        kk = N * 5 // 100
        meta = dict(B=1, Hkv=8, D=128, nQ=N - 128 - kk, k=kk, window=128, fmts=(INT4, INT4),
                    k_s=np.zeros((1, 8, 128, 1), dtype=np.uint16))
        by = od.cache_code_bytes(meta)
        row_k4v4 = 8 * 128                                   # K and V at 4 bits: one byte per channel
        strict = N * row_k4v4
        assert by["quantized"] == meta["nQ"] * row_k4v4
        over = lambda name, rows: 100.0 * (by[name] - rows * row_k4v4) / strict   # noqa: E731
        assert round(over("vertical", kk), 1) == 15.0
        assert round(over("window", 128), 1) == win_pct
        assert round(over("staging", 128), 1) == win_pct


def test_definition_against_library_softmax():
    B, Hq, Hkv, N, D, W, kk = 1, 4, 2, 260, 16, 32, 12
    k, v = _kv(B, Hkv, N, D, seed=5)
    q = _q(B, Hq, D)
    idx = _idx(B, Hkv, N - W, kk, seed=5)
    c = od.freeze(wl.bits(k), wl.bits(v), idx, W, group=64, fmts=(INT4, INT4))
    od.append_staging(c, wl.bits(k)[:, :, 7], wl.bits(v)[:, :, 9])
    out, lse = od.decode_attention(wl.bits(q), c)
    for h in range(Hq):
        hk = h // 2
        # dequantized prefix through numpy integer views only
        def deq(codes, scales):
            lo = (codes & 0xF).astype(np.int8)
            hi = (codes >> 4).astype(np.int8)
            val = np.stack([np.where(lo > 7, lo - 16, lo), np.where(hi > 7, hi - 16, hi)], -1).reshape(len(codes), -1)
            return val * np.repeat(scales.astype(np.float64), 64)[:len(codes), None]
        K = np.concatenate([deq(c["kq_codes"][0, hk], c["kq_scales"][0, hk]), _f64(k)[0, hk][idx[0, hk]],
                            _f64(k)[0, hk, 7:8], _f64(k)[0, hk, N - W:]])
        V = np.concatenate([deq(c["vq_codes"][0, hk], c["vq_scales"][0, hk]), _f64(v)[0, hk][idx[0, hk]],
                            _f64(v)[0, hk, 9:10], _f64(v)[0, hk, N - W:]])
        s = (K @ _f64(q)[0, h]) / math.sqrt(D)
        assert np.allclose(out[0, h], scipy.special.softmax(s) @ V, rtol=1e-12, atol=1e-13)
        assert np.isclose(lse[0, h], scipy.special.logsumexp(s), rtol=1e-13)


@pytest.mark.parametrize("splits,tile", [(1, 64), (3, 16), (7, 5), (64, 64)])
def test_segmented_walk_equals_the_definition(splits, tile):
    B, Hq, Hkv, N, D, W, kk = 2, 6, 2, 333, 16, 48, 10
    k, v = _kv(B, Hkv, N, D, seed=8)
    q = _q(B, Hq, D, seed=9)
    idx = _idx(B, Hkv, N - W, kk, seed=8)
    c = od.freeze(wl.bits(k), wl.bits(v), idx, W, group=64, fmts=(INT4, INT8))
    for j in range(3):
        od.append_staging(c, wl.bits(k)[:, :, j], wl.bits(v)[:, :, j + 1])
    ref, lse_ref = od.decode_attention(wl.bits(q), c)
    out, lse = od.decode_attention_segmented(wl.bits(q), c, splits=splits, tile=tile)
    assert np.allclose(out, ref, rtol=1e-11, atol=1e-13) and np.allclose(lse, lse_ref, rtol=1e-12)


def test_brute_force_on_a_tiny_cache():
    B, Hq, Hkv, N, D, W, kk = 1, 2, 1, 12, 4, 3, 2
    k, v = _kv(B, Hkv, N, D, seed=11)
    q = _q(B, Hq, D, seed=12)
    idx = np.array([[[1, 6]]], dtype=np.int32)
    c = od.freeze(wl.bits(k), wl.bits(v), idx, W, group=4, fmts=(INT8, INT8))
    out, _ = od.decode_attention(wl.bits(q), c)
    kf, vf, qf = _f64(k)[0, 0], _f64(v)[0, 0], _f64(q)[0]
    quant_pos = [p for p in range(N - W) if p not in (1, 6)]
    def q8(rows):                                            # rows: list of lists; one group of <= 4 rows
        amax = max(abs(x) for r in rows for x in r)
        sc = float(np.float32(np.float32(amax) / np.float32(127.0)))
        inv = np.float32(127.0) / np.float32(amax)
        return [[float(np.rint(np.float32(x) * inv)) * sc for x in r] for r in rows]
    kd, vd = {}, {}
    for g0 in range(0, len(quant_pos), 4):
        pos = quant_pos[g0:g0 + 4]
        for p, rk, rv in zip(pos, q8([kf[p].tolist() for p in pos]), q8([vf[p].tolist() for p in pos])):
            kd[p], vd[p] = rk, rv
    for h in range(Hq):
        num, den = [0.0] * D, 0.0
        for p in range(N):
            kr = kd.get(p, kf[p].tolist())
            vr = vd.get(p, vf[p].tolist())
            w = math.exp(sum(a * b for a, b in zip(qf[h].tolist(), kr)) / math.sqrt(D))
            den += w
            num = [n + w * x for n, x in zip(num, vr)]
        assert np.allclose(out[0, h], [n / den for n in num], rtol=1e-12, atol=1e-14)


def test_everything_full_precision_equals_the_last_row_of_exact_attention():
    """W >= N (no prefix) and k = P (every prefix row vertical): nothing is quantized, so the token's
    output is the last row of exact causal attention - computed by the prefill oracle's C code."""
    B, Hq, Hkv, N, D = 1, 4, 2, 70, 16
    g = torch.Generator().manual_seed(21)
    Q = torch.randn(B, Hq, N, D, generator=g).to(torch.bfloat16)
    k, v = _kv(B, Hkv, N, D, seed=22)
    qz = [oracle.quantize(wl.bits(t), INT8, 64) for t in (Q, k, v)]
    (qc, qs), (kc, ks), (vc, vs) = qz
    exact = oracle.attention_rows(wl.bits(Q), wl.bits(k), wl.bits(v), qc, kc, vc, qs, ks, vs, (INT8,) * 3,
                                  np.zeros((B, Hq, 0), dtype=np.int32), N, np.array([N - 1]), 64)
    exact = np.asarray(exact[0] if isinstance(exact, tuple) else exact).reshape(B, Hq, D)
    qt = wl.bits(Q)[:, :, N - 1]
    for W, kk in ((N, 0), (N + 5, 0), (20, N - 20)):
        idx = None if kk == 0 else np.tile(np.arange(kk, dtype=np.int32), (B, Hkv, 1))
        c = od.freeze(wl.bits(k), wl.bits(v), idx, W)
        assert c["nQ"] == 0
        out, _ = od.decode_attention(qt, c)
        assert np.allclose(out, exact, rtol=1e-10, atol=1e-12)


def test_lossless_codes_make_the_partition_irrelevant():
    """Keys and values on an INT8 grid (multiples of 1/64 with +-127/64 present in every group) are
    reproduced exactly by the quantizer, so whatever is quantized, the output equals exact attention:
    this ties compaction order, group scales and the K/V pairing of the quantized segment to the
    full-precision result."""
    B, Hq, Hkv, N, D, W, kk, G = 1, 4, 2, 150, 8, 16, 7, 16
    rng = np.random.default_rng(31)
    def grid():
        a = rng.integers(-127, 128, size=(B, Hkv, N, D)).astype(np.float64)
        a[..., 0] = 127.0 * rng.choice([-1.0, 1.0], size=(B, Hkv, N))     # every row carries the absmax
        return torch.from_numpy(a / 64.0).to(torch.bfloat16)
    k, v = grid(), grid()
    assert np.array_equal(_f64(k) * 64, np.rint(_f64(k) * 64))
    q = _q(B, Hq, D, seed=32)
    idx = _idx(B, Hkv, N - W, kk, seed=33)
    c = od.freeze(wl.bits(k), wl.bits(v), idx, W, group=G, fmts=(INT8, INT8))
    assert np.array_equal(od.dequantize(c["kq_codes"], c["kq_scales"], INT8, G)[0, 1], _f64(k)[0, 1][c["iq"][0, 1]])
    out, _ = od.decode_attention_segmented(wl.bits(q), c, splits=3, tile=8)
    for h in range(Hq):
        s = (_f64(k)[0, h // 2] @ _f64(q)[0, h]) / math.sqrt(D)
        assert np.allclose(out[0, h], scipy.special.softmax(s) @ _f64(v)[0, h // 2], rtol=1e-11, atol=1e-13)


def test_full_precision_rows_may_sit_in_any_full_precision_segment():
    B, Hq, Hkv, N, D, W, kk = 1, 2, 1, 90, 8, 10, 5
    k, v = _kv(B, Hkv, N, D, seed=41)
    q = _q(B, Hq, D, seed=42)
    idx = _idx(B, Hkv, N - W, kk, seed=43)
    c = od.freeze(wl.bits(k), wl.bits(v), idx, W, group=16)
    ref, _ = od.decode_attention(wl.bits(q), c)
    c2 = dict(c)
    c2["k_s"], c2["v_s"] = c["k_s"].copy(), c["v_s"].copy()
    for j in range(3):                                       # three window rows move to the staging buffer
        od.append_staging(c2, c["k_win"][:, :, j], c["v_win"][:, :, j])
    c2["k_win"], c2["v_win"] = c["k_win"][:, :, 3:], c["v_win"][:, :, 3:]
    out, _ = od.decode_attention_segmented(wl.bits(q), c2, splits=2, tile=4)
    assert np.allclose(out, ref, rtol=1e-11, atol=1e-13)
