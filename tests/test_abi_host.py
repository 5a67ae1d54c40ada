"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every symbol the
header declares, and rejects bad arguments before launching anything."""
import ctypes
import os
import re

import pytest

from paper_2608_27875_b200 import api, build, decode_api

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return api.lib()


def test_every_declared_symbol_is_exported(lib):
    for header_name, exports in (("hyq.h", api.EXPORTS), ("hyq_decode.h", decode_api.EXPORTS)):
        header = open(os.path.join(ROOT, "include", header_name)).read()
        header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)                 # declarations only, not prose
        declared = set(re.findall(r"\b(hyq_[a-z_0-9]+)\s*\(", header))
        assert declared == set(exports), header_name
        for name in declared:
            assert hasattr(lib, name), name


def test_status_strings_and_version(lib):
    assert lib.hyq_version() >= 1
    seen = {api.status_string(c) for c in range(7)}
    assert len(seen) == 7 and "ok" in seen
    assert api.status_string(99) == "unknown status"


def test_paper_k_formula(lib):
    # k = min(P, max(1, ceil(P r))), P = max(0, L - W)   (Algorithm 1)
    assert api.hyq_paper_k(8192, 512, 0.02) == 154
    assert api.hyq_paper_k(32768, 1024, 0.02) == 635
    assert api.hyq_paper_k(131072, 1024, 0.01) == 1301
    assert api.hyq_paper_k(16384, 512, 0.03) == 477
    assert api.hyq_paper_k(100, 100, 0.5) == 0          # P = 0
    assert api.hyq_paper_k(101, 100, 1e-9) == 1         # at least one
    assert api.hyq_paper_k(110, 100, 1.0) == 10         # at most P


def test_select_argument_checks(lib):
    n = ctypes.c_size_t(0)
    assert lib.hyq_select_vertical_workspace(1, 4, 2, 256, 256, 128, 64, 8, ctypes.byref(n)) == 0
    assert n.value >= 4 * 128 * 8 + 4 * 192 * 8
    assert lib.hyq_select_vertical_workspace(1, 4, 3, 256, 256, 128, 64, 8, ctypes.byref(n)) == 1   # Hq % Hkv
    assert lib.hyq_select_vertical_workspace(1, 4, 2, 256, 256, 64, 64, 8, ctypes.byref(n)) == 2    # D != 128
    assert lib.hyq_select_vertical_workspace(1, 4, 2, 256, 256, 128, 64, 193, ctypes.byref(n)) == 1  # k > P
    # k > P, bad tail, zero window with default tail: rejected before any pointer is touched
    assert lib.hyq_select_vertical(None, None, 1, 4, 2, 256, 256, 128, 64, 0, 193, None, None, 0, None) == 1
    assert lib.hyq_select_vertical(None, None, 1, 4, 2, 256, 256, 128, 64, 300, 8, None, None, 0, None) == 1
    assert lib.hyq_select_vertical(None, None, 1, 4, 2, 256, 256, 128, 0, 0, 8, None, None, 0, None) == 1
    # empty problems succeed without pointers
    assert lib.hyq_select_vertical(None, None, 1, 4, 2, 256, 256, 128, 256, 0, 8, None, None, 0, None) == 0
    assert lib.hyq_select_vertical(None, None, 1, 4, 2, 256, 256, 128, 64, 0, 0, None, None, 0, None) == 0
    # null pointers with real work
    assert lib.hyq_select_vertical(None, None, 1, 4, 2, 256, 256, 128, 64, 0, 8, None, None, 0, None) == 1
    # misaligned pointer / short workspace (fake addresses: checks come before any launch)
    assert lib.hyq_select_vertical(0x1008, 0x2000, 1, 4, 2, 256, 256, 128, 64, 0, 8, 0x3000, 0x4000, 1 << 30, None) == 4
    assert lib.hyq_select_vertical(0x1000, 0x2000, 1, 4, 2, 256, 256, 128, 64, 0, 8, 0x3000, 0x4000, 16, None) == 3


def test_quantize_argument_checks(lib):
    assert lib.hyq_quantize_blocks(None, 1, 1, 64, 128, 64, 0, None, None, None) == 1
    assert lib.hyq_quantize_blocks(0x1000, 1, 1, 64, 64, 64, 0, 0x2000, 0x3000, None) == 2      # D
    assert lib.hyq_quantize_blocks(0x1000, 1, 1, 64, 128, 48, 0, 0x2000, 0x3000, None) == 2     # block size (32, 64, 128 only)
    assert lib.hyq_quantize_blocks(0x1000, 1, 1, 64, 128, 64, 7, 0x2000, 0x3000, None) == 2     # format
    assert lib.hyq_quantize_blocks(0x1004, 1, 1, 64, 128, 64, 0, 0x2000, 0x3000, None) == 4
    assert lib.hyq_quantize_blocks(0x1000, 0, 1, 64, 128, 64, 0, 0x2000, 0x3000, None) == 1


def _args(**kw):
    a = api.AttnArgs()
    a.struct_size = ctypes.sizeof(api.AttnArgs)
    a.B, a.Hq, a.Hkv, a.L, a.D, a.window, a.k, a.block_tokens = 1, 4, 2, 256, 128, 64, 8, 64
    a.q_format = a.k_format = a.v_format = 0
    a.out_dtype, a.impl = 1, api.IMPL_SIMT
    for f in ("q", "k_", "v", "q_codes", "k_codes", "v_codes", "q_scales", "k_scales", "v_scales", "vl_idx", "out"):
        setattr(a, f, 0x10000)
    a.workspace, a.workspace_bytes = 0x20000, 1 << 30
    for key, val in kw.items():
        setattr(a, key, val)
    return a


def test_attention_argument_checks(lib):
    n = ctypes.c_size_t(0)
    for impl in (api.IMPL_SIMT, api.IMPL_AUTO):
        assert lib.hyq_hybrid_attention_prefill_workspace(ctypes.byref(_args(impl=impl)), ctypes.byref(n)) == 0
    call = lambda a: lib.hyq_hybrid_attention_prefill(ctypes.byref(a), None)   # noqa: E731
    assert call(_args(struct_size=8)) == 1
    assert call(_args(Hkv=3)) == 1
    assert call(_args(D=64)) == 2
    assert call(_args(block_tokens=48)) == 2
    assert call(_args(q_format=1, k_format=0, v_format=1)) == 2       # Q and K formats must match
    assert call(_args(q_format=2, k_format=2, v_format=0)) == 2       # INT4 with INT8 V not built
    assert call(_args(Lq=-1)) == 1
    assert call(_args(Lq=10 ** 6)) == 1                               # query block longer than the keys
    assert call(_args(window_mode=2)) == 1
    assert call(_args(out=None)) == 1
    assert call(_args(vl_idx=None)) == 1                              # k > 0 needs indices
    assert call(_args(q=0x10008)) == 4
    assert call(_args(workspace_bytes=0)) == 3
    assert call(_args(out_dtype=5)) == 1


def test_binding_fails_loudly_without_the_library(monkeypatch, tmp_path):
    monkeypatch.setattr(api, "_lib", None)
    monkeypatch.setattr(api, "LIB_PATH", str(tmp_path / "missing.so"))
    with pytest.raises(RuntimeError, match="missing"):
        api.lib()


def test_decode_side_argument_checks(lib):
    """Cache descriptions are checked on the host before anything is launched (no GPU needed: every call
    below must fail in the checks, or is a host-only size query)."""
    L = decode_api._lib()
    sizes = decode_api.KvCacheSizes()
    d = decode_api.make_desc(B=2, Hq=32, Hkv=8, N=1000, window=100, k=37)
    assert L.hyq_kv_cache_query_sizes(ctypes.byref(d), ctypes.byref(sizes)) == 0
    assert sizes.quantized_rows == 863 and sizes.padded_rows == 896
    assert sizes.kq_codes_bytes == sizes.vq_codes_bytes == 16 * 896 * 64 and sizes.scales_bytes == 16 * 14 * 4
    assert sizes.vertical_bytes == 16 * 37 * 256 and sizes.window_bytes == 16 * 100 * 256
    assert sizes.staging_bytes == 16 * 128 * 256
    n = ctypes.c_size_t(0)
    assert L.hyq_hybrid_attention_decode_workspace(ctypes.byref(d), 5, ctypes.byref(n)) == 0
    assert n.value == 16 * 5 * 8 * (128 + 2) * 4
    assert L.hyq_hybrid_attention_decode_workspace(ctypes.byref(d), 0, ctypes.byref(n)) == 0 and n.value > 0
    w_all = decode_api.make_desc(B=1, Hq=4, Hkv=4, N=50, window=80, k=0)          # window longer than the cache
    assert L.hyq_kv_cache_query_sizes(ctypes.byref(w_all), ctypes.byref(sizes)) == 0
    assert sizes.quantized_rows == 0 and sizes.window_bytes == 4 * 50 * 256
    bad = [dict(k=901), dict(Hq=30), dict(D=64), dict(group=48), dict(fmt=7), dict(Hq=1024),
           dict(n_staging=129), dict(N=0)]
    expect = [1, 1, 2, 2, 2, 2, 1, 1]
    for kw, code in zip(bad, expect):
        args = dict(B=2, Hq=32, Hkv=8, N=1000, window=100, k=37)
        args.update(kw)
        assert L.hyq_kv_cache_query_sizes(ctypes.byref(decode_api.make_desc(**args)), ctypes.byref(sizes)) == code, kw
    caps = decode_api.make_desc(B=2, Hq=32, Hkv=8, N=1000, window=100, k=37, cap_quantized_rows=1024, cap_vertical=64, cap_window=128)
    assert L.hyq_kv_cache_query_sizes(ctypes.byref(caps), ctypes.byref(sizes)) == 0
    assert sizes.kq_codes_bytes == 16 * 1024 * 64 and sizes.vertical_bytes == 16 * 64 * 256 and sizes.window_bytes == 16 * 128 * 256
    for kw in (dict(cap_quantized_rows=1000), dict(cap_quantized_rows=832), dict(cap_vertical=36), dict(cap_window=99)):
        args = dict(B=2, Hq=32, Hkv=8, N=1000, window=100, k=37)
        args.update(kw)
        assert L.hyq_kv_cache_query_sizes(ctypes.byref(decode_api.make_desc(**args)), ctypes.byref(sizes)) == 1, kw
    assert L.hyq_hybrid_attention_decode_ragged(None, ctypes.byref(d), None, 0.0, 0, 0, None, None, None, 0, None) == 1
    d.struct_size = 8
    assert L.hyq_kv_cache_query_sizes(ctypes.byref(d), ctypes.byref(sizes)) == 1
    d.struct_size = ctypes.sizeof(decode_api.KvCacheDesc)
    assert L.hyq_freeze(None, None, None, ctypes.byref(d), None) == 1            # null buffers
    assert L.hyq_kv_cache_append(None, None, ctypes.byref(d), None) == 1
    full = decode_api.make_desc(B=2, Hq=32, Hkv=8, N=1000, window=100, k=37)
    full.k_s, full.v_s, full.n_staging = 0x10000, 0x20000, full.staging_capacity
    assert L.hyq_kv_cache_append(0x30000, 0x40000, ctypes.byref(full), None) == 1          # staging buffer full
    full.n_staging = 3
    assert L.hyq_kv_cache_append(0x30008, 0x40000, ctypes.byref(full), None) == 4          # misaligned rows
    assert L.hyq_hybrid_attention_decode(None, ctypes.byref(d), 0.0, 0, 0, None, None, None, 0, None) == 1
