"""GPU parity of the decode side against the oracle: Freeze (Algorithm 4) bit-exact, the hybrid KV-cache
attention of one token (Algorithm 3) within the attention tolerances."""
import numpy as np
import pytest
import torch

import oracle
from oracle import decode as od
from paper_2608_27875_b200 import decode_api as dapi, workloads as wl
from gpu_util import MAX_ABS_TOL, MEAN_REL_TOL, ensure_built, errors, rand_bf16

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _lib():
    ensure_built()


def _idx(B, H, P, kk, seed):
    rng = np.random.default_rng(seed)
    return np.stack([np.stack([np.sort(rng.choice(P, kk, replace=False)) for _ in range(H)])
                     for _ in range(B)]).astype(np.int32)


def _v_tiles_to_rows(vq: np.ndarray) -> np.ndarray:
    """Undoes the fragment-major V layout as the header documents it, written out nibble by nibble:
    [.., tiles, 1024] bytes -> [.., tiles*16, 64] bytes in the row-major INT4 layout."""
    lead = vq.shape[:-2]
    tiles = vq.shape[-2]
    by = vq.reshape(lead + (tiles, 2, 32, 4, 4)).astype(np.uint32)                  # [.., tile, x >> 2, lane, x & 3, byte]
    words = by[..., 0] | (by[..., 1] << 8) | (by[..., 2] << 16) | (by[..., 3] << 24)
    words = np.moveaxis(words, -3, -2).reshape(lead + (tiles, 32, 8))               # [.., tile, lane, x]
    rows = np.zeros(lead + (tiles, 16, 128), dtype=np.uint8)
    for lane in range(32):
        r, j = lane >> 2, lane & 3
        for x in range(8):
            for n in range(8):
                ch = 64 * (x >> 2) + 8 * r + 2 * (x & 3) + (n & 1)
                key = 2 * j + (n >> 2) + 8 * ((n >> 1) & 1)
                rows[..., key, ch] = (words[..., lane, x] >> (4 * n)) & 0xF
    packed = rows[..., 0::2] | (rows[..., 1::2] << 4)
    return packed.reshape(lead + (tiles * 16, 64))


def _v8_tiles_to_rows(vq: np.ndarray) -> np.ndarray:
    """Undoes the INT8 fragment-major V layout as the header documents it: [.., tiles, 2048] -> [.., tiles*16, 128]."""
    lead, tiles = vq.shape[:-2], vq.shape[-2]
    rows = np.zeros(lead + (tiles, 16, 128), dtype=np.uint8)
    for key in range(16):
        for d in range(128):
            j, r, x = (key & 7) >> 1, (d >> 3) & 7, ((d >> 6) << 2) | ((d >> 1) & 3)
            w = 2 * x + (key >> 3)
            rows[..., key, d] = vq[..., (w >> 2) * 512 + (4 * r + j) * 16 + (w & 3) * 4 + (d & 1) * 2 + (key & 1)]
    return rows.reshape(lead + (tiles * 16, 128))


def _freeze_both(K, V, idx, W, Hq, staging_capacity=128, group=64, fmt=oracle.FMT_INT4):
    ref = od.freeze(wl.bits(K), wl.bits(V), idx, W, group=group, fmts=(fmt, fmt), staging_capacity=staging_capacity)
    idx_t = None if idx is None or idx.shape[2] == 0 else torch.from_numpy(idx).cuda()
    cache = dapi.hyq_freeze(K.cuda(), V.cuda(), idx_t, W, Hq, staging_capacity, group=group, fmt=fmt)
    torch.cuda.synchronize()
    return ref, cache


def _stage(ref, cache, n_s, seed):
    B, H, D = ref["B"], ref["Hkv"], ref["D"]
    for i in range(n_s):
        kn, vn = rand_bf16((B, H, D), seed + 2 * i), rand_bf16((B, H, D), seed + 2 * i + 1)
        od.append_staging(ref, wl.bits(kn), wl.bits(vn))
        cache.append(kn.cuda(), vn.cuda())


def _assert_cache_equal(ref, cache):
    nQ, kk, W = ref["nQ"], ref["k"], ref["window"]
    b = {n: t.cpu().numpy() if t.dtype != torch.bfloat16 else wl.bits(t.cpu()) for n, t in cache.buffers.items()}
    assert int(cache.sizes.quantized_rows) == nQ
    if nQ:
        ng = -(-nQ // ref["group"])
        assert np.array_equal(b["kq_codes"][:, :, :nQ], ref["kq_codes"])
        unpermute = _v_tiles_to_rows if ref["fmts"][1] == oracle.FMT_INT4 else _v8_tiles_to_rows
        assert np.array_equal(unpermute(b["vq_codes"])[:, :, :nQ], ref["vq_codes"])
        assert np.array_equal(b["kq_scales"][:, :, :ng].view(np.uint32), ref["kq_scales"].view(np.uint32))
        assert np.array_equal(b["vq_scales"][:, :, :ng].view(np.uint32), ref["vq_scales"].view(np.uint32))
    if kk:
        assert np.array_equal(b["k_vl"][:, :, :kk], ref["k_vl"]) and np.array_equal(b["v_vl"][:, :, :kk], ref["v_vl"])
    if W:
        assert np.array_equal(b["k_win"][:, :, :W], ref["k_win"]) and np.array_equal(b["v_win"][:, :, :W], ref["v_win"])


FREEZE_SHAPES = [  # B, Hkv, N, W, k
    (1, 2, 300, 40, 9), (2, 3, 1000, 128, 37), (1, 1, 64, 0, 0), (1, 2, 129, 1, 64), (1, 2, 50, 80, 0),
    (1, 2, 200, 20, 180), (2, 8, 4096, 512, 82), (1, 1, 65, 0, 1),
]


@pytest.mark.parametrize("B,Hkv,N,W,kk", FREEZE_SHAPES)
def test_freeze_is_bit_exact(B, Hkv, N, W, kk):
    K, V = rand_bf16((B, Hkv, N, 128), 1, 1.5), rand_bf16((B, Hkv, N, 128), 2)
    K[:, :, : N // 3] *= 0.01                               # groups with very different scales
    idx = _idx(B, Hkv, N - min(W, N), kk, 3) if kk else None
    ref, cache = _freeze_both(K, V, idx, W, Hq=Hkv)
    _assert_cache_equal(ref, cache)


def test_freeze_of_an_all_zero_group_and_clustered_vertical_rows():
    B, Hkv, N, W = 1, 2, 700, 60
    K, V = rand_bf16((B, Hkv, N, 128), 4), rand_bf16((B, Hkv, N, 128), 5)
    K[:, :, 100:300] = 0
    idx = np.tile(np.concatenate([np.arange(0, 40), np.arange(320, 330), np.arange(400, 600),     # a run longer than the
                                  np.arange(630, 640)]).astype(np.int32), (B, Hkv, 1))            # kernel's index window
    ref, cache = _freeze_both(K, V, idx, W, Hq=Hkv)
    assert (ref["kq_scales"] == 0).any()
    _assert_cache_equal(ref, cache)


def test_staging_rows_land_where_the_oracle_puts_them_and_a_full_buffer_is_refused():
    B, Hkv, N, W, cap = 3, 5, 200, 30, 6
    K, V = rand_bf16((B, Hkv, N, 128), 6), rand_bf16((B, Hkv, N, 128), 7)
    ref, cache = _freeze_both(K, V, _idx(B, Hkv, N - W, 4, 8), W, Hq=Hkv, staging_capacity=cap)
    cache.buffers["k_s"].fill_(-3.0), cache.buffers["v_s"].fill_(-3.0)          # untouched rows keep this marker
    marker = int(wl.bits(torch.tensor([-3.0], dtype=torch.bfloat16))[0])
    for n in range(1, cap + 1):
        _stage(ref, cache, 1, 10 * n)
        for name in ("k_s", "v_s"):
            got = wl.bits(cache.buffers[name].cpu())
            assert np.array_equal(got[:, :, :n], ref[name][:, :, :n]) and (got[:, :, n:] == marker).all()
    assert cache.n_staging == cap
    with pytest.raises(dapi.api.HyqError):
        cache.append(rand_bf16((B, Hkv, 128), 1).cuda(), rand_bf16((B, Hkv, 128), 2).cuda())
    assert cache.n_staging == cap


DECODE_SHAPES = [  # B, Hq, Hkv, N, W, k, n_s, splits
    (1, 4, 1, 300, 40, 9, 0, 1), (1, 4, 1, 300, 40, 9, 3, 0), (2, 8, 2, 1000, 128, 37, 5, 3), (1, 2, 2, 64, 0, 0, 1, 1),
    (1, 8, 1, 129, 1, 64, 0, 2), (1, 6, 2, 50, 80, 0, 0, 0), (1, 4, 2, 200, 20, 180, 17, 4), (1, 16, 2, 2000, 100, 50, 128, 0),
    (1, 5, 1, 777, 33, 21, 2, 7), (1, 4, 1, 40, 8, 3, 0, 50), (2, 32, 8, 4096, 512, 82, 16, 0), (1, 1, 1, 17, 16, 0, 0, 1),
]


@pytest.mark.parametrize("B,Hq,Hkv,N,W,kk,n_s,splits", DECODE_SHAPES)
def test_decode_attention_matches_oracle(B, Hq, Hkv, N, W, kk, n_s, splits):
    K, V = rand_bf16((B, Hkv, N, 128), 11, 1.3), rand_bf16((B, Hkv, N, 128), 12)
    q = rand_bf16((B, Hq, 128), 13, 1.5)
    idx = _idx(B, Hkv, N - min(W, N), kk, 14) if kk else None
    ref, cache = _freeze_both(K, V, idx, W, Hq)
    _stage(ref, cache, n_s, 100)
    want, lse_want = od.decode_attention(wl.bits(q), ref)
    lse = torch.empty(B, Hq, dtype=torch.float32, device="cuda")
    got = dapi.hyq_hybrid_attention_decode(q.cuda(), cache, splits=splits, out_dtype=torch.float32, lse=lse)
    torch.cuda.synchronize()
    mx, rel = errors(got.cpu().numpy(), want)
    assert mx <= MAX_ABS_TOL and rel <= MEAN_REL_TOL, (mx, rel)
    assert np.abs(lse.cpu().numpy() - lse_want).max() <= 2e-3
    got16 = dapi.hyq_hybrid_attention_decode(q.cuda(), cache, splits=splits, out_dtype=torch.bfloat16)
    assert torch.equal(got16.cpu(), got.cpu().to(torch.bfloat16))


@pytest.mark.parametrize("group", [32, 128])
@pytest.mark.parametrize("B,Hq,Hkv,N,W,kk,n_s", [(1, 4, 1, 300, 40, 9, 3), (2, 8, 2, 1000, 128, 37, 0), (1, 8, 2, 2117, 100, 50, 17),
                                                 (1, 2, 2, 64, 0, 0, 1)])
def test_other_group_sizes(group, B, Hq, Hkv, N, W, kk, n_s):
    """Algorithm 4's group size G = 32 and 128: cache bit-exact, attention within tolerance."""
    K, V = rand_bf16((B, Hkv, N, 128), 71, 1.3), rand_bf16((B, Hkv, N, 128), 72)
    K[:, :, : N // 2] *= 0.05
    q = rand_bf16((B, Hq, 128), 73, 1.5)
    idx = _idx(B, Hkv, N - min(W, N), kk, 74) if kk else None
    ref, cache = _freeze_both(K, V, idx, W, Hq, group=group)
    _assert_cache_equal(ref, cache)
    _stage(ref, cache, n_s, 500)
    want, _ = od.decode_attention(wl.bits(q), ref)
    for splits in (0, 3):
        got = dapi.hyq_hybrid_attention_decode(q.cuda(), cache, splits=splits, out_dtype=torch.float32)
        mx, rel = errors(got.cpu().numpy(), want)
        assert mx <= MAX_ABS_TOL and rel <= MEAN_REL_TOL, (splits, mx, rel)


@pytest.mark.parametrize("fmt", [oracle.FMT_INT8, oracle.FMT_FP8_E4M3])
@pytest.mark.parametrize("group", [32, 64, 128])
@pytest.mark.parametrize("B,Hq,Hkv,N,W,kk,n_s,splits", [(1, 4, 1, 300, 40, 9, 3, 0), (2, 8, 2, 1000, 128, 37, 0, 3), (1, 16, 2, 2117, 100, 50, 17, 0),
                                                        (1, 2, 2, 64, 0, 0, 1, 1), (1, 5, 1, 777, 33, 21, 2, 7), (1, 4, 2, 200, 20, 180, 5, 2)])
def test_byte_wide_caches(fmt, group, B, Hq, Hkv, N, W, kk, n_s, splits):
    """K8V8 with INT8 or FP8 e4m3 codes: codes, scales and layouts bit-exact; attention within tolerance."""
    K, V = rand_bf16((B, Hkv, N, 128), 81, 1.3), rand_bf16((B, Hkv, N, 128), 82)
    K[:, :, : N // 2] *= 0.05
    q = rand_bf16((B, Hq, 128), 83, 1.5)
    idx = _idx(B, Hkv, N - min(W, N), kk, 84) if kk else None
    ref, cache = _freeze_both(K, V, idx, W, Hq, group=group, fmt=fmt)
    _assert_cache_equal(ref, cache)
    _stage(ref, cache, n_s, 600)
    want, lse_want = od.decode_attention(wl.bits(q), ref)
    lse = torch.empty(B, Hq, dtype=torch.float32, device="cuda")
    got = dapi.hyq_hybrid_attention_decode(q.cuda(), cache, splits=splits, out_dtype=torch.float32, lse=lse)
    mx, rel = errors(got.cpu().numpy(), want)
    assert mx <= MAX_ABS_TOL and rel <= MEAN_REL_TOL, (mx, rel)
    assert np.abs(lse.cpu().numpy() - lse_want).max() <= 2e-3


@pytest.mark.parametrize("fmt", [oracle.FMT_INT4, oracle.FMT_INT8, oracle.FMT_FP8_E4M3])
@pytest.mark.parametrize("B,Hq,Hkv,N,W,kk,n_s,splits", [(1, 32, 2, 1500, 64, 30, 5, 0), (2, 12, 1, 700, 32, 11, 0, 3), (1, 18, 2, 333, 40, 9, 2, 1),
                                                        (1, 64, 1, 400, 16, 5, 1, 2)])
def test_more_than_eight_query_heads_per_kv_head(fmt, B, Hq, Hkv, N, W, kk, n_s, splits):
    """g = 16 (two KV heads for 32 query heads), 12, 9 and 64: eight heads per CTA, several CTAs per slice."""
    K, V = rand_bf16((B, Hkv, N, 128), 91, 1.3), rand_bf16((B, Hkv, N, 128), 92)
    q = rand_bf16((B, Hq, 128), 93, 1.5)
    idx = _idx(B, Hkv, N - W, kk, 94)
    ref, cache = _freeze_both(K, V, idx, W, Hq, fmt=fmt)
    _stage(ref, cache, n_s, 800)
    want, lse_want = od.decode_attention(wl.bits(q), ref)
    lse = torch.empty(B, Hq, dtype=torch.float32, device="cuda")
    got = dapi.hyq_hybrid_attention_decode(q.cuda(), cache, splits=splits, out_dtype=torch.float32, lse=lse)
    mx, rel = errors(got.cpu().numpy(), want)
    assert mx <= MAX_ABS_TOL and rel <= MEAN_REL_TOL, (mx, rel)
    assert np.abs(lse.cpu().numpy() - lse_want).max() <= 2e-3


def test_decode_with_peaked_scores_and_late_maxima():
    """A planted key that dominates (scores far above the rest) sits late in the quantized prefix, another
    in the window: the lazy reference maximum has to be raised mid-stream in several warps and slices."""
    B, Hq, Hkv, N, W, kk = 1, 8, 2, 3000, 64, 30
    K, V = rand_bf16((B, Hkv, N, 128), 21), rand_bf16((B, Hkv, N, 128), 22)
    q = rand_bf16((B, Hq, 128), 23)
    u = torch.nn.functional.normalize(torch.randn(128, generator=torch.Generator().manual_seed(24)), dim=0)
    qf = q.float() + 6.0 * u
    q = qf.to(torch.bfloat16)
    for pos, amp in ((2500, 8.0), (N - 5, 10.0), (17, 5.0)):
        K[:, :, pos] = (K[:, :, pos].float() + amp * u).to(torch.bfloat16)
    idx = _idx(B, Hkv, N - W, kk, 25)
    ref, cache = _freeze_both(K, V, idx, W, Hq)
    want, _ = od.decode_attention(wl.bits(q), ref)
    for splits in (1, 5, 0):
        got = dapi.hyq_hybrid_attention_decode(q.cuda(), cache, splits=splits, out_dtype=torch.float32)
        mx, rel = errors(got.cpu().numpy(), want)
        assert mx <= MAX_ABS_TOL and rel <= MEAN_REL_TOL, (splits, mx, rel)


def test_ragged_batch_whose_scale_slices_are_not_16_byte_aligned():
    """Short sequences: a sequence's slice of the batch's scale arrays starts at a multiple of 8 bytes only."""
    Hq, Hkv, W = 2, 1, 8
    seqs = [(100, 3), (70, 0), (90, 5)]
    rc = dapi.RaggedKvCache(len(seqs), Hq, Hkv, max_N=100, window=W, max_k=5)
    assert rc.batch.buffers["kq_scales"][1].data_ptr() % 16 == 8
    q = rand_bf16((len(seqs), Hq, 128), 120)
    refs = []
    for b, (N, kk) in enumerate(seqs):
        K, V = rand_bf16((1, Hkv, N, 128), 121 + b), rand_bf16((1, Hkv, N, 128), 131 + b)
        idx = _idx(1, Hkv, N - W, kk, 141 + b) if kk else None
        refs.append(od.freeze(wl.bits(K), wl.bits(V), idx, W))
        rc.freeze_sequence(b, K.cuda(), V.cuda(), None if idx is None else torch.from_numpy(idx).cuda())
    got = dapi.hyq_hybrid_attention_decode_ragged(q.cuda(), rc, out_dtype=torch.float32)
    for b, ref in enumerate(refs):
        want, _ = od.decode_attention(wl.bits(q[b:b + 1]), ref)
        mx, rel = errors(got[b:b + 1].cpu().numpy(), want)
        assert mx <= MAX_ABS_TOL and rel <= MEAN_REL_TOL, (b, mx, rel)


def test_a_dominant_full_precision_key_keeps_its_precision():
    """One window key takes almost all of the weight: the output is that key's value row, so any rounding of the
    weights in the full-precision product shows directly.  (A single bf16 weight would leave 1e-3 here.)"""
    B, Hq, Hkv, N, W = 1, 4, 2, 700, 64
    K, V = rand_bf16((B, Hkv, N, 128), 101, 0.3), rand_bf16((B, Hkv, N, 128), 102, 2.0)
    q = rand_bf16((B, Hq, 128), 103)
    u = torch.nn.functional.normalize(torch.randn(128, generator=torch.Generator().manual_seed(104)), dim=0)
    q = (q.float() + 8.0 * u).to(torch.bfloat16)
    for pos, amp in ((N - 7, 6.0), (N - 30, 5.5)):                      # two window keys of comparable, dominant weight
        K[:, :, pos] = (K[:, :, pos].float() + amp * u).to(torch.bfloat16)
    idx = _idx(B, Hkv, N - W, 20, 105)
    for fmt in (oracle.FMT_INT4, oracle.FMT_INT8, oracle.FMT_FP8_E4M3):
        ref, cache = _freeze_both(K, V, idx, W, Hq, fmt=fmt)
        want, _ = od.decode_attention(wl.bits(q), ref)
        got = dapi.hyq_hybrid_attention_decode(q.cuda(), cache, out_dtype=torch.float32)
        mx, rel = errors(got.cpu().numpy(), want)
        assert rel <= 4e-4, (fmt, mx, rel)


def test_decode_calls_can_be_captured_in_a_cuda_graph():
    """The call enqueues two kernels (the second as a programmatic dependent) and nothing else: it can be recorded in a
    CUDA graph and replayed, with the result of the eager call."""
    B, Hq, Hkv, N, W, kk = 2, 8, 2, 3000, 128, 40
    K, V = rand_bf16((B, Hkv, N, 128), 111), rand_bf16((B, Hkv, N, 128), 112)
    q = rand_bf16((B, Hq, 128), 113).cuda()
    _, cache = _freeze_both(K, V, _idx(B, Hkv, N - W, kk, 114), W, Hq)
    out = torch.empty(B, Hq, 128, dtype=torch.float32, device="cuda")
    ws = torch.empty(dapi.hyq_hybrid_attention_decode_workspace(cache) + 16, dtype=torch.uint8, device="cuda")
    eager = dapi.hyq_hybrid_attention_decode(q, cache, out_dtype=torch.float32).clone()      # also the first, uncaptured call
    graph, stream = torch.cuda.CUDAGraph(), torch.cuda.Stream()
    with torch.cuda.stream(stream):
        with torch.cuda.graph(graph, stream=stream):
            dapi.hyq_hybrid_attention_decode(q, cache, out=out, workspace=ws)
    out.zero_()
    graph.replay()
    torch.cuda.synchronize()
    assert torch.equal(out, eager)


def test_decode_at_benchmark_size_and_repeatable():
    """The benchmark's cache shape (32 / 8 heads, 32768 frozen rows, 2 % vertical, window 1024, a full staging
    buffer) at batch 2, every head against the oracle; two runs are bit-identical."""
    B, Hq, Hkv, N, W = 2, 32, 8, 32768, 1024
    kk = oracle_k = int(np.ceil((N - W) * 0.02))
    K, V = rand_bf16((B, Hkv, N, 128), 31), rand_bf16((B, Hkv, N, 128), 32)
    q = rand_bf16((B, Hq, 128), 33)
    idx = _idx(B, Hkv, N - W, kk, 34)
    ref, cache = _freeze_both(K, V, idx, W, Hq)
    _assert_cache_equal(ref, cache)
    _stage(ref, cache, 128, 300)
    want, _ = od.decode_attention(wl.bits(q), ref)
    got = dapi.hyq_hybrid_attention_decode(q.cuda(), cache, out_dtype=torch.float32)
    again = dapi.hyq_hybrid_attention_decode(q.cuda(), cache, out_dtype=torch.float32)
    mx, rel = errors(got.cpu().numpy(), want)
    assert mx <= MAX_ABS_TOL and rel <= MEAN_REL_TOL, (mx, rel)
    assert torch.equal(got, again)
    assert oracle_k == cache.desc.k


def test_ragged_batch_matches_the_oracle_sequence_by_sequence():
    """Sequences of different lengths, vertical counts and staging fills in one allocation (capacity strides) and
    one launch: every sequence against its own oracle cache; a sequence shorter than the window has no prefix."""
    Hq, Hkv, W = 8, 2, 64
    seqs = [(1000, 37, 5), (333, 0, 0), (40, 0, 3), (2000, 100, 128), (129, 1, 1)]          # N, k, staged rows
    rc = dapi.RaggedKvCache(len(seqs), Hq, Hkv, max_N=2000, window=W, max_k=100)
    refs, qs = [], []
    for b, (N, kk, n_s) in enumerate(seqs):
        K, V = rand_bf16((1, Hkv, N, 128), 40 + b, 1.3), rand_bf16((1, Hkv, N, 128), 50 + b)
        idx = _idx(1, Hkv, N - min(W, N), kk, 60 + b) if kk else None
        ref = od.freeze(wl.bits(K), wl.bits(V), idx, W)
        rc.freeze_sequence(b, K.cuda(), V.cuda(), None if idx is None else torch.from_numpy(idx).cuda())
        for i in range(n_s):
            kn, vn = rand_bf16((1, Hkv, 128), 700 + 10 * b + i), rand_bf16((1, Hkv, 128), 900 + 10 * b + i)
            od.append_staging(ref, wl.bits(kn), wl.bits(vn))
            rc.append(b, kn[0].cuda(), vn[0].cuda())
        refs.append(ref)
        qs.append(rand_bf16((1, Hq, 128), 80 + b, 1.5))
    q = torch.cat(qs)
    assert rc.lengths_host.tolist() == [[r["nQ"], r["k"], r["window"], r["n_s"]] for r in refs]
    for splits in (0, 1, 7):
        got = dapi.hyq_hybrid_attention_decode_ragged(q.cuda(), rc, splits=splits, out_dtype=torch.float32)
        torch.cuda.synchronize()
        for b, ref in enumerate(refs):
            want, _ = od.decode_attention(wl.bits(qs[b]), ref)
            mx, rel = errors(got[b:b + 1].cpu().numpy(), want)
            assert mx <= MAX_ABS_TOL and rel <= MEAN_REL_TOL, (splits, b, mx, rel)
    # the frozen codes of a sequence inside the batch allocation are those of a stand-alone Freeze
    b = 3
    nq = refs[b]["nQ"]
    assert np.array_equal(rc.batch.buffers["kq_codes"][b, :, :nq].cpu().numpy(), refs[b]["kq_codes"][0])
    assert np.array_equal(_v_tiles_to_rows(rc.batch.buffers["vq_codes"][b].cpu().numpy())[:, :nq], refs[b]["vq_codes"][0])
