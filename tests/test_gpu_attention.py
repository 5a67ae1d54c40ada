"""GPU parity: hyq_hybrid_attention_prefill against the fp64 oracle (Eq. 6-7), element by element
at small sizes and on sampled rows at the benchmark sizes.  Tolerance: max-abs 1e-2 and
sum|err|/sum|ref| 2e-3 on the fp32 output."""
import numpy as np
import pytest
import torch

import oracle
from gpu_util import MAX_ABS_TOL, MEAN_REL_TOL, ensure_built, errors, gpu_attention, oracle_quant_all, rand_bf16
from paper_2608_27875_b200 import api, workloads as wl

pytestmark = pytest.mark.gpu
INT8 = (wl.FMT_INT8,) * 3
INT4FP8 = (wl.FMT_INT4, wl.FMT_INT4, wl.FMT_FP8_E4M3)
FP8ALL = (wl.FMT_FP8_E4M3,) * 3
IMPLS = [pytest.param(api.IMPL_SIMT, id="simt"), pytest.param(api.IMPL_TCGEN05, id="umma")]


def _rand_idx(B, Hq, P, k, seed):
    rng = np.random.default_rng(seed)
    return np.stack([np.stack([np.sort(rng.choice(P, k, replace=False)) for _ in range(Hq)])
                     for _ in range(B)]).astype(np.int32)


def _ref(Q, K, V, qz, fmts, idx, window, rows=None, **kw):
    (qc, qs), (kc, ks), (vc, vs) = qz
    return oracle.attention_rows(wl.bits(Q), wl.bits(K), wl.bits(V), qc, kc, vc, qs, ks, vs, fmts, idx, window, rows, **kw)


def _check(Q, K, V, fmts, idx, window, impl, rows=None):
    ensure_built()
    qz = oracle_quant_all(Q, K, V, fmts)
    got = gpu_attention(Q, K, V, qz, fmts, idx, window, impl).numpy()
    ref = _ref(Q, K, V, qz, fmts, idx, window, rows)
    if rows is not None:
        got = got[:, :, rows]
    assert np.isfinite(got).all()
    max_abs, mean_rel = errors(got, ref)
    assert max_abs <= MAX_ABS_TOL and mean_rel <= MEAN_REL_TOL, (max_abs, mean_rel)
    return max_abs, mean_rel


@pytest.mark.parametrize("impl", IMPLS)
@pytest.mark.parametrize("fmts", [INT8, INT4FP8, FP8ALL])
@pytest.mark.parametrize("B,Hq,Hkv,L,W,k", [
    (1, 2, 2, 512, 128, 16),      # several tiles
    (2, 4, 2, 333, 40, 9),        # ragged tail, window not a tile multiple
    (1, 4, 1, 130, 128, 2),       # window ~ L
    (1, 2, 2, 200, 0, 12),        # no window: the diagonal itself is low-bit
    (1, 2, 1, 257, 64, 0),        # no vertical keys
    (1, 1, 1, 1, 1, 0),           # a single token
    (1, 2, 2, 64, 200, 0),        # window >= L: exact attention
    (1, 2, 2, 640, 1, 639),       # every prefix key vertical
])
def test_small_shapes_match_oracle(impl, fmts, B, Hq, Hkv, L, W, k):
    Q, K, V = (rand_bf16((B, h, L, 128), seed=L + n) for n, h in enumerate((Hq, Hkv, Hkv)))
    P = max(0, L - W)
    idx = _rand_idx(B, Hq, P, k, seed=L) if k else None
    _check(Q, K, V, fmts, idx, W, impl)


@pytest.mark.parametrize("impl", IMPLS)
@pytest.mark.parametrize("bt", [32, 128])
@pytest.mark.parametrize("fmts", [INT8, INT4FP8, FP8ALL])
@pytest.mark.parametrize("B,Hq,Hkv,L,W,k", [(1, 2, 2, 512, 128, 16), (2, 4, 2, 333, 40, 9), (1, 2, 2, 200, 0, 12), (1, 4, 1, 1000, 64, 30)])
def test_other_quantization_block_sizes(impl, bt, fmts, B, Hq, Hkv, L, W, k):
    """32- and 128-token quantization blocks (scales per half tile / per two tiles); K rows of very different
    magnitude so that neighbouring blocks have very different scales."""
    Q, K, V = (rand_bf16((B, h, L, 128), seed=L + n + bt) for n, h in enumerate((Hq, Hkv, Hkv)))
    K = (K.float() * (1.0 + 3.0 * ((torch.arange(L) // 32) % 3).view(1, 1, L, 1))).to(torch.bfloat16)
    idx = _rand_idx(B, Hq, max(0, L - W), k, seed=L)
    ensure_built()
    qz = oracle_quant_all(Q, K, V, fmts, bt)
    got = gpu_attention(Q, K, V, qz, fmts, idx, W, impl, block_tokens=bt).numpy()
    ref = _ref(Q, K, V, qz, fmts, idx, W, None, block_tokens=bt)
    max_abs, mean_rel = errors(got, ref)
    assert np.isfinite(got).all() and max_abs <= MAX_ABS_TOL and mean_rel <= MEAN_REL_TOL, (max_abs, mean_rel)


@pytest.mark.parametrize("impl", IMPLS)
def test_vertical_keys_inside_the_window_and_beyond_the_diagonal(impl):
    """Index sets are free to name keys that a given row sees through its window or not at all."""
    L, W = 300, 50
    Q, K, V = (rand_bf16((1, 2, L, 128), seed=40 + n) for n in range(3))
    idx = np.array([[[0, 1, 2, 100, 101, 249], [5, 64, 127, 128, 200, 249]]], dtype=np.int32)
    _check(Q, K, V, INT8, idx, W, impl)


@pytest.mark.parametrize("impl", IMPLS)
def test_config0_full_output(impl):
    w = wl.CONFIGS["c0"]
    Q, K, V = wl.make_inputs(w)
    idx = oracle.select_vertical(wl.bits(Q), wl.bits(K), w.window, w.k)
    _check(Q, K, V, w.fmts, idx, w.window, impl)


@pytest.mark.parametrize("impl", IMPLS)
def test_bf16_output_is_the_rounded_fp32_output_and_lse(impl):
    ensure_built()
    w = wl.CONFIGS["c0"].scaled(L=700)
    Q, K, V = wl.make_inputs(w)
    qz = oracle_quant_all(Q, K, V, w.fmts)
    idx = oracle.select_vertical(wl.bits(Q), wl.bits(K), w.window, w.k)
    o32, lse = gpu_attention(Q, K, V, qz, w.fmts, idx, w.window, impl, lse=True)
    o16 = gpu_attention(Q, K, V, qz, w.fmts, idx, w.window, impl, out_dtype=torch.bfloat16)
    assert torch.equal(o16, o32.to(torch.bfloat16))
    _, ref_lse = _ref(Q, K, V, qz, w.fmts, idx, w.window, return_lse=True)
    np.testing.assert_allclose(lse.numpy(), ref_lse, rtol=0, atol=2e-3)


@pytest.mark.parametrize("name", ["c1", "c2", "c4"])
def test_benchmark_configs_on_sampled_rows(name):
    """Benchmark-size heads, tensor-core kernel, checked on rows the oracle can do one by one."""
    w = wl.CONFIGS[name]
    if w.B > 1:
        w = w.scaled(B=1)
    Q, K, V = wl.make_inputs(w, heads=[w.Hkv - 1])
    idx = oracle.select_vertical(wl.bits(Q), wl.bits(K), w.window, w.k)
    rows = wl.sample_rows(w.L, w.window, n_random=24)
    _check(Q, K, V, w.fmts, idx, w.window, api.IMPL_TCGEN05, rows)


def _run_whole_path(w):
    """The launch configuration bench.py times: every head of the workload, whole path on the device."""
    ensure_built()
    Q, K, V = wl.make_inputs(w)
    res = api.hybrid_prefill(Q.cuda(), K.cuda(), V.cuda(), w.window, w.k, w.fmts)
    torch.cuda.synchronize()
    return {n: t.cpu().numpy() for n, t in res.items()}


@pytest.mark.parametrize("name,kv_heads,n_random", [("c1", [0, 7], 24), ("c2", [2, 5], 16), ("c4", [2], 12), ("c3", [1, 6], 8)])
def test_full_size_workloads_in_the_benchmark_launch_configuration(name, kv_heads, n_random):
    """Full benchmark sizes, all heads launched at once; the oracle recomputes whole (batch, KV head)
    groups for selection and quantization (bit-exact) and sampled rows of the attention output."""
    w = wl.CONFIGS[name]
    got = _run_whole_path(w)
    g = w.Hq // w.Hkv
    b = w.B - 1
    rows = wl.sample_rows(w.L, w.window, n_random=n_random, edge=2)
    for kvh in kv_heads:
        Qh, Kh, Vh = wl.make_inputs(w.scaled(B=b + 1), heads=[kvh])
        Qh, Kh, Vh = Qh[b:b + 1], Kh[b:b + 1], Vh[b:b + 1]
        qs_ = slice(kvh * g, (kvh + 1) * g)
        ref_idx = oracle.select_vertical(wl.bits(Qh), wl.bits(Kh), w.window, w.k)
        np.testing.assert_array_equal(got["idx"][b:b + 1, qs_], ref_idx)
        qz = oracle_quant_all(Qh, Kh, Vh, w.fmts)
        for (codes, scales), cn, sn, hs in zip(qz, ("q_codes", "k_codes", "v_codes"), ("q_scales", "k_scales", "v_scales"),
                                               (qs_, slice(kvh, kvh + 1), slice(kvh, kvh + 1))):
            np.testing.assert_array_equal(got[cn][b:b + 1, hs], codes)
            np.testing.assert_array_equal(got[sn][b:b + 1, hs].view(np.uint32), scales.view(np.uint32))
        ref = _ref(Qh, Kh, Vh, qz, w.fmts, ref_idx, w.window, rows)
        out = got["out"][b:b + 1, qs_][:, :, rows]
        assert np.isfinite(got["out"]).all()
        max_abs, mean_rel = errors(out, ref)
        assert max_abs <= MAX_ABS_TOL and mean_rel <= MEAN_REL_TOL, (name, kvh, max_abs, mean_rel)


@pytest.mark.parametrize("name,Lq,mode", [("c1", 2048, 0), ("c2", 4096, 0), ("c2", 4096, 1)])
def test_benchmark_size_query_block_on_sampled_rows(name, Lq, mode):
    """The configuration `bench.py --lq` times: the last Lq rows of a benchmark-size context (one KV head's
    query heads), both window forms, checked against the oracle on sampled rows of the block."""
    ensure_built()
    w = wl.CONFIGS[name]
    Q, K, V = wl.make_inputs(w, heads=[w.Hkv - 1])
    Qb = Q[:, :, w.L - Lq:].contiguous()
    idx = oracle.select_vertical(wl.bits(Qb), wl.bits(K), w.window, w.k)
    rows = np.unique(np.concatenate([[0, 1, 63, 64, 255, 256, Lq - 2, Lq - 1],
                                     np.random.default_rng(7).integers(0, Lq, 12)])).astype(np.int32)
    qz = oracle_quant_all(Qb, K, V, w.fmts)
    got = gpu_attention(Qb, K, V, qz, w.fmts, idx, w.window, api.IMPL_TCGEN05, window_mode=mode).numpy()[:, :, rows]
    (qc, qs), (kc, ks), (vc, vs) = qz
    ref = oracle.attention_rows(wl.bits(Qb), wl.bits(K), wl.bits(V), qc, kc, vc, qs, ks, vs, w.fmts, idx, w.window,
                                rows, fixed_window=bool(mode))
    max_abs, mean_rel = errors(got, ref)
    assert max_abs <= MAX_ABS_TOL and mean_rel <= MEAN_REL_TOL, (name, Lq, mode, max_abs, mean_rel)


@pytest.mark.parametrize("fmts", [INT8, INT4FP8, FP8ALL])
@pytest.mark.parametrize("Lq,L,W,k,mode", [(1, 4096, 256, 40, 0), (100, 5000, 128, 64, 0), (256, 8192, 512, 80, 1),
                                           (300, 6000, 0, 30, 0), (512, 16384, 1024, 100, 0)])
def test_short_query_blocks_with_the_keys_split_over_ctas(fmts, Lq, L, W, k, mode):
    """Short query blocks against long contexts: the tensor-core path splits the keys over several CTAs per
    query tile and merges their partial results.  Outputs and the log-sum-exp must agree with the CUDA-core
    kernel (which never splits) everywhere, and with the oracle on sampled rows; the bf16 output must be the
    rounding of the fp32 one."""
    ensure_built()
    g = torch.Generator().manual_seed(Lq + L)
    Q = torch.randn(1, 2, Lq, 128, generator=g).to(torch.bfloat16).cuda()
    K = torch.randn(1, 1, L, 128, generator=g).to(torch.bfloat16).cuda()
    V = torch.randn(1, 1, L, 128, generator=g).to(torch.bfloat16).cuda()
    idx = torch.from_numpy(_rand_idx(1, 2, L - W, k, seed=L)).cuda()
    (qc, qs), (kc, ks), (vc, vs) = [api.hyq_quantize_blocks(t, f) for t, f in zip((Q, K, V), fmts)]
    lse = [torch.empty(1, 2, Lq, dtype=torch.float32, device="cuda") for _ in range(2)]
    tc, simt = [api.hyq_hybrid_attention_prefill(Q, K, V, qc, kc, vc, qs, ks, vs, fmts, idx, W, impl=impl, lse=l_,
                                                 window_mode=mode)
                for impl, l_ in zip((api.IMPL_TCGEN05, api.IMPL_SIMT), lse)]
    tc16 = api.hyq_hybrid_attention_prefill(Q, K, V, qc, kc, vc, qs, ks, vs, fmts, idx, W, impl=api.IMPL_TCGEN05,
                                            out_dtype=torch.bfloat16, window_mode=mode)
    torch.cuda.synchronize()
    assert torch.isfinite(tc).all()
    diff = (tc - simt).abs()
    assert float(diff.max()) <= MAX_ABS_TOL and float(diff.sum() / simt.abs().sum()) <= MEAN_REL_TOL
    assert float((lse[0] - lse[1]).abs().max()) <= 2e-3
    assert torch.equal(tc16, tc.to(torch.bfloat16))
    rows = np.unique(np.concatenate([[0, Lq - 1], np.random.default_rng(3).integers(0, Lq, 4)])).astype(np.int32)
    t = lambda x: x.cpu().numpy()   # noqa: E731
    ref = oracle.attention_rows(wl.bits(Q.cpu()), wl.bits(K.cpu()), wl.bits(V.cpu()), t(qc), t(kc), t(vc), t(qs), t(ks), t(vs),
                                fmts, t(idx), W, rows, fixed_window=bool(mode))
    max_abs, mean_rel = errors(t(tc)[:, :, rows], ref)
    assert max_abs <= MAX_ABS_TOL and mean_rel <= MEAN_REL_TOL, (max_abs, mean_rel)


def test_tensor_core_and_cuda_core_kernels_agree_on_every_output_of_config1():
    """Every row of every head at a benchmark size: two independent kernels, both within tolerance of the
    definition on the sampled rows, must agree with each other everywhere."""
    ensure_built()
    w = wl.CONFIGS["c1"]
    Q, K, V = (t.cuda() for t in wl.make_inputs(w))
    idx = api.hyq_select_vertical(Q, K, w.window, w.k)
    qz = [api.hyq_quantize_blocks(t, f) for t, f in zip((Q, K, V), w.fmts)]
    (qc, qs), (kc, ks), (vc, vs) = qz
    outs = [api.hyq_hybrid_attention_prefill(Q, K, V, qc, kc, vc, qs, ks, vs, w.fmts, idx, w.window, impl=impl)
            for impl in (api.IMPL_TCGEN05, api.IMPL_SIMT)]
    torch.cuda.synchronize()
    diff = (outs[0] - outs[1]).abs()
    assert torch.isfinite(outs[0]).all()
    assert float(diff.max()) <= MAX_ABS_TOL
    assert float(diff.sum() / outs[1].abs().sum()) <= MEAN_REL_TOL


# ---- query block shorter than the keys (Algorithm 2: a query block against the full K, V; end-aligned) ----------
@pytest.mark.parametrize("impl", IMPLS)
@pytest.mark.parametrize("fmts", [INT8, INT4FP8])
@pytest.mark.parametrize("Lq,L,W,k", [
    (64, 512, 128, 16),       # one block-aligned tile of queries at the end of eight key tiles
    (100, 333, 40, 9),        # ragged lengths, query block off the block grid (its own Q blocks)
    (1, 300, 64, 12),         # a single query row
    (300, 700, 0, 20),        # no window: every pair below the diagonal is low-bit or vertical
    (257, 1024, 300, 5),      # more than two query tiles, window longer than a query tile
    (130, 130, 16, 4),        # Lq == L given explicitly
])
def test_query_block_matches_oracle(impl, fmts, Lq, L, W, k):
    g = torch.Generator().manual_seed(Lq * 7 + L)
    Q = torch.randn(1, 4, Lq, 128, generator=g).to(torch.bfloat16)
    K = torch.randn(1, 2, L, 128, generator=g).to(torch.bfloat16)
    V = torch.randn(1, 2, L, 128, generator=g).to(torch.bfloat16)
    idx = _rand_idx(1, 4, max(1, L - W), k, seed=L) if k else None
    _check(Q, K, V, fmts, idx, W, impl)


@pytest.mark.parametrize("impl", IMPLS)
@pytest.mark.parametrize("fmts", [INT8, INT4FP8])
@pytest.mark.parametrize("Lq,L,W,k", [
    (64, 512, 128, 16),       # the block lies inside the fixed window
    (100, 333, 40, 9),        # rows before L - W have no window keys at all
    (1, 300, 64, 12),
    (600, 600, 100, 20),      # the whole prefill with the fixed tail window
    (257, 1024, 300, 5),
    (90, 400, 0, 7),          # no window
])
def test_fixed_tail_window_matches_oracle(impl, fmts, Lq, L, W, k):
    """Algorithm 2's K_Win taken literally: the last W keys are the window of every row of the query block."""
    ensure_built()
    g = torch.Generator().manual_seed(Lq * 11 + L)
    Q = torch.randn(1, 4, Lq, 128, generator=g).to(torch.bfloat16)
    K = torch.randn(1, 2, L, 128, generator=g).to(torch.bfloat16)
    V = torch.randn(1, 2, L, 128, generator=g).to(torch.bfloat16)
    idx = _rand_idx(1, 4, max(1, L - W), k, seed=L) if k else None
    qz = oracle_quant_all(Q, K, V, fmts)
    got = gpu_attention(Q, K, V, qz, fmts, idx, W, impl, window_mode=api.WINDOW_FIXED_TAIL).numpy()
    (qc, qs), (kc, ks), (vc, vs) = qz
    ref = oracle.attention_rows(wl.bits(Q), wl.bits(K), wl.bits(V), qc, kc, vc, qs, ks, vs, fmts, idx, W,
                                fixed_window=True)
    assert np.isfinite(got).all()
    max_abs, mean_rel = errors(got, ref)
    assert max_abs <= MAX_ABS_TOL and mean_rel <= MEAN_REL_TOL, (max_abs, mean_rel)


@pytest.mark.parametrize("fmts", [INT8, INT4FP8])
def test_query_block_on_the_cta_grid_repeats_the_tail_of_the_whole_prefill_bit_for_bit(fmts):
    """A query block that starts on a multiple of 256 rows is tiled by the tensor-core kernel exactly like the
    same rows of the whole prefill, and its codes and scales are slices of the whole prefill's: the outputs and
    the log-sum-exp must be identical."""
    ensure_built()
    L, Lq, W, k = 1280, 512, 128, 24
    g = torch.Generator().manual_seed(77)
    Q = torch.randn(1, 4, L, 128, generator=g).to(torch.bfloat16).cuda()
    K = torch.randn(1, 2, L, 128, generator=g).to(torch.bfloat16).cuda()
    V = torch.randn(1, 2, L, 128, generator=g).to(torch.bfloat16).cuda()
    idx = api.hyq_select_vertical(Q, K, W, k)
    (qc, qs), (kc, ks), (vc, vs) = [api.hyq_quantize_blocks(t, f) for t, f in zip((Q, K, V), fmts)]
    lse_full = torch.empty(1, 4, L, dtype=torch.float32, device="cuda")
    full = api.hyq_hybrid_attention_prefill(Q, K, V, qc, kc, vc, qs, ks, vs, fmts, idx, W, lse=lse_full)
    off = L - Lq
    Qb, qcb, qsb = Q[:, :, off:].contiguous(), qc[:, :, off:].contiguous(), qs[:, :, off // 64:].contiguous()
    lse_blk = torch.empty(1, 4, Lq, dtype=torch.float32, device="cuda")
    blk = api.hyq_hybrid_attention_prefill(Qb, K, V, qcb, kc, vc, qsb, ks, vs, fmts, idx, W, lse=lse_blk)
    torch.cuda.synchronize()
    assert blk.shape == (1, 4, Lq, 128)
    assert torch.equal(blk, full[:, :, off:])
    assert torch.equal(lse_blk, lse_full[:, :, off:])


def _two_kernels(Q, K, V, fmts, W, k):
    Qd, Kd, Vd = Q.cuda(), K.cuda(), V.cuda()
    if k == 0:
        idx = None
    elif W == 0:        # no observation window to select from: any ascending index set serves
        idx = torch.from_numpy(_rand_idx(Q.shape[0], Q.shape[1], Q.shape[2], k, seed=k)).cuda()
    else:
        idx = api.hyq_select_vertical(Qd, Kd, W, k)
    (qc, qs), (kc, ks), (vc, vs) = [api.hyq_quantize_blocks(t, f) for t, f in zip((Qd, Kd, Vd), fmts)]
    outs = [api.hyq_hybrid_attention_prefill(Qd, Kd, Vd, qc, kc, vc, qs, ks, vs, fmts, idx, W, impl=impl)
            for impl in (api.IMPL_TCGEN05, api.IMPL_SIMT, api.IMPL_TCGEN05)]
    torch.cuda.synchronize()
    return outs


@pytest.mark.parametrize("seed", range(32))
def test_random_shapes_tensor_core_matches_cuda_core_and_repeats_bit_for_bit(seed):
    """Seeded random shapes (ragged lengths, windows off the tile grid, GQA groups, both format sets, flat
    and steeply rising score profiles): the tensor-core kernel and the plain CUDA-core kernel are
    independent implementations of the same definition and must agree on every output; two runs of the
    tensor-core kernel on the same inputs must be identical bit for bit (no dependence on timing)."""
    ensure_built()
    rng = np.random.default_rng(1000 + seed)
    g = torch.Generator().manual_seed(2000 + seed)
    long_rows = seed >= 24                        # a few cases with dozens of key tiles per query tile
    B = 1 if long_rows else int(rng.integers(1, 3))
    Hkv = 1 if long_rows else int(rng.integers(1, 3))
    Hq = Hkv * int(rng.choice([1, 2, 4]))
    L = int(rng.integers(2000, 6000)) if long_rows else int(rng.integers(1, 1400))
    W = int(rng.choice([0, 1, 17, 64, 100, 128, 300, 1024]))
    k = int(rng.integers(0, max(1, min(L - W, 64)))) if L - W > 0 else 0
    fmts = (INT8, INT4FP8, FP8ALL)[seed % 3]
    u = torch.randn(128, generator=g)
    u = u / u.norm()
    slope = float(rng.choice([0.0, 0.0, 20.0, -20.0, 60.0]))
    ramp = torch.linspace(0.0, 1.0, L)[:, None]
    Q = (0.3 * torch.randn(B, Hq, L, 128, generator=g) + 6.0 * u).to(torch.bfloat16)
    K = (0.3 * torch.randn(B, Hkv, L, 128, generator=g) + (slope * ramp) * u).to(torch.bfloat16)
    V = torch.randn(B, Hkv, L, 128, generator=g).to(torch.bfloat16)
    tc, simt, tc_again = _two_kernels(Q, K, V, fmts, W, k)
    assert torch.isfinite(tc).all()
    assert torch.equal(tc, tc_again)
    diff = (tc - simt).abs()
    assert float(diff.max()) <= MAX_ABS_TOL, (B, Hq, Hkv, L, W, k, slope, float(diff.max()))
    assert float(diff.sum() / simt.abs().sum().clamp_min(1e-30)) <= MEAN_REL_TOL, (B, Hq, Hkv, L, W, k, slope)


@pytest.mark.parametrize("seed", range(16))
def test_random_query_blocks_and_window_forms_both_kernels_agree(seed):
    """Seeded random query blocks (any length up to the keys, on and off the tile grid) under both window
    forms: the tensor-core and the CUDA-core kernel must agree everywhere."""
    ensure_built()
    rng = np.random.default_rng(5000 + seed)
    g = torch.Generator().manual_seed(6000 + seed)
    L = int(rng.integers(2, 1500))
    Lq = int(rng.integers(1, L + 1))
    W = int(rng.choice([0, 1, 50, 64, 200, 700]))
    k = int(rng.integers(0, max(1, min(L - W, 48)))) if L - W > 0 else 0
    mode = int(rng.integers(0, 2))
    fmts = (INT8, INT4FP8, FP8ALL)[seed % 3]
    Hkv = int(rng.integers(1, 3))
    Hq = Hkv * int(rng.choice([1, 2]))
    Q = torch.randn(1, Hq, Lq, 128, generator=g).to(torch.bfloat16).cuda()
    K = torch.randn(1, Hkv, L, 128, generator=g).to(torch.bfloat16).cuda()
    V = torch.randn(1, Hkv, L, 128, generator=g).to(torch.bfloat16).cuda()
    idx = torch.from_numpy(_rand_idx(1, Hq, L - W, k, seed=seed)).cuda() if k else None
    (qc, qs), (kc, ks), (vc, vs) = [api.hyq_quantize_blocks(t, f) for t, f in zip((Q, K, V), fmts)]
    tc, simt = [api.hyq_hybrid_attention_prefill(Q, K, V, qc, kc, vc, qs, ks, vs, fmts, idx, W, impl=impl,
                                                 window_mode=mode) for impl in (api.IMPL_TCGEN05, api.IMPL_SIMT)]
    torch.cuda.synchronize()
    assert tc.shape == (1, Hq, Lq, 128) and torch.isfinite(tc).all()
    diff = (tc - simt).abs()
    assert float(diff.max()) <= MAX_ABS_TOL, (L, Lq, W, k, mode, float(diff.max()))
    assert float(diff.sum() / simt.abs().sum().clamp_min(1e-30)) <= MEAN_REL_TOL, (L, Lq, W, k, mode)


@pytest.mark.parametrize("impl", IMPLS)
@pytest.mark.parametrize("fmts", [INT8, INT4FP8])
def test_row_maximum_that_keeps_rising_along_the_keys(impl, fmts):
    """Scores that grow with the key position force the running maximum up tile after tile (every rescale
    path of the online softmax), with late keys dominating early ones by many orders of magnitude."""
    L, W, k = 900, 96, 10
    g = torch.Generator().manual_seed(5)
    u = torch.randn(128, generator=g)
    u = u / u.norm()
    ramp = torch.linspace(0.0, 1.0, L)[:, None]
    Q = (0.3 * torch.randn(1, 2, L, 128, generator=g) + 6.0 * u).to(torch.bfloat16)
    K = (0.3 * torch.randn(1, 2, L, 128, generator=g) + (40.0 * ramp) * u).to(torch.bfloat16)   # score ~ 21 * ramp (natural log units)
    V = torch.randn(1, 2, L, 128, generator=g).to(torch.bfloat16)
    idx = _rand_idx(1, 2, L - W, k, seed=3)
    _check(Q, K, V, fmts, idx, W, impl)


@pytest.mark.parametrize("impl", IMPLS)
def test_early_keys_dominate_and_all_zero_blocks(impl):
    """The opposite order (the first keys carry almost all the mass, later tiles underflow) plus all-zero
    K / V / Q blocks, whose scale is zero."""
    L, W, k = 700, 64, 6
    g = torch.Generator().manual_seed(9)
    u = torch.randn(128, generator=g)
    u = u / u.norm()
    ramp = torch.linspace(1.0, 0.0, L)[:, None]
    Q = (0.3 * torch.randn(1, 2, L, 128, generator=g) + 6.0 * u).to(torch.bfloat16)
    K = (0.3 * torch.randn(1, 1, L, 128, generator=g) + (40.0 * ramp) * u).to(torch.bfloat16)
    V = torch.randn(1, 1, L, 128, generator=g).to(torch.bfloat16)
    K[0, 0, 128:192] = 0
    V[0, 0, 256:320] = 0
    Q[0, 1, 320:384] = 0
    idx = _rand_idx(1, 2, L - W, k, seed=4)
    _check(Q, K, V, INT8, idx, W, impl)
