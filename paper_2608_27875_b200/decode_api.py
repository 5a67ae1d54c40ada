"""Thin Python binding of the decode side of the C ABI (``include/hyq_decode.h``): argument
marshalling only.  torch supplies device memory and the current stream; Freeze and the attention
run in the library's kernels.  No CPU fallback: the first call raises if ``libhyq.so`` is missing."""
from __future__ import annotations

import ctypes
from dataclasses import dataclass, field

import torch

from . import api
from .workloads import FMT_INT4, FMT_INT8

EXPORTS = ("hyq_kv_cache_query_sizes", "hyq_freeze", "hyq_kv_cache_append", "hyq_hybrid_attention_decode_workspace",
           "hyq_hybrid_attention_decode", "hyq_hybrid_attention_decode_ragged")


class KvCacheDesc(ctypes.Structure):
    """Mirror of ``hyq_kv_cache``."""
    _fields_ = ([("struct_size", ctypes.c_uint32)] +
                [(n, ctypes.c_int32) for n in ("B", "Hq", "Hkv", "D", "N", "window", "k", "group", "format",
                                               "staging_capacity", "n_staging")] +
                [(n, ctypes.c_void_p) for n in ("kq_codes", "vq_codes", "kq_scales", "vq_scales", "k_vl", "v_vl",
                                                "k_win", "v_win", "k_s", "v_s")] +
                [(n, ctypes.c_int32) for n in ("cap_quantized_rows", "cap_vertical", "cap_window")])


class KvCacheSizes(ctypes.Structure):
    """Mirror of ``hyq_kv_cache_sizes``."""
    _fields_ = ([("quantized_rows", ctypes.c_int64), ("padded_rows", ctypes.c_int64)] +
                [(n, ctypes.c_size_t) for n in ("kq_codes_bytes", "vq_codes_bytes", "scales_bytes", "vertical_bytes",
                                                "window_bytes", "staging_bytes")])


_bound = False


def _lib():
    global _bound
    L = api.lib()
    if not _bound:
        L.hyq_kv_cache_query_sizes.argtypes = [ctypes.POINTER(KvCacheDesc), ctypes.POINTER(KvCacheSizes)]
        L.hyq_freeze.argtypes = [ctypes.c_void_p] * 3 + [ctypes.POINTER(KvCacheDesc), ctypes.c_void_p]
        L.hyq_kv_cache_append.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.POINTER(KvCacheDesc), ctypes.c_void_p]
        L.hyq_hybrid_attention_decode_workspace.argtypes = [ctypes.POINTER(KvCacheDesc), ctypes.c_int,
                                                            ctypes.POINTER(ctypes.c_size_t)]
        L.hyq_hybrid_attention_decode.argtypes = [ctypes.c_void_p, ctypes.POINTER(KvCacheDesc), ctypes.c_float,
                                                  ctypes.c_int, ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p,
                                                  ctypes.c_void_p, ctypes.c_size_t, ctypes.c_void_p]
        L.hyq_hybrid_attention_decode_ragged.argtypes = [ctypes.c_void_p, ctypes.POINTER(KvCacheDesc), ctypes.c_void_p,
                                                         ctypes.c_float, ctypes.c_int, ctypes.c_int, ctypes.c_void_p,
                                                         ctypes.c_void_p, ctypes.c_void_p, ctypes.c_size_t, ctypes.c_void_p]
        _bound = True
    return L


def make_desc(B, Hq, Hkv, N, window, k, staging_capacity=128, n_staging=0, D=128, group=64, fmt=FMT_INT4,
              cap_quantized_rows=0, cap_vertical=0, cap_window=0) -> KvCacheDesc:
    d = KvCacheDesc()
    d.struct_size = ctypes.sizeof(KvCacheDesc)
    d.B, d.Hq, d.Hkv, d.D, d.N, d.window, d.k, d.group, d.format = B, Hq, Hkv, D, N, window, k, group, fmt
    d.staging_capacity, d.n_staging = staging_capacity, n_staging
    d.cap_quantized_rows, d.cap_vertical, d.cap_window = cap_quantized_rows, cap_vertical, cap_window
    return d


def hyq_kv_cache_query_sizes(desc: KvCacheDesc) -> KvCacheSizes:
    s = KvCacheSizes()
    api._check(_lib().hyq_kv_cache_query_sizes(ctypes.byref(desc), ctypes.byref(s)), "hyq_kv_cache_query_sizes")
    return s


@dataclass
class HybridKvCache:
    """The device buffers of one layer's hybrid cache plus the descriptor that points at them."""
    desc: KvCacheDesc
    sizes: KvCacheSizes
    buffers: dict = field(default_factory=dict)

    @property
    def n_staging(self) -> int:
        return int(self.desc.n_staging)

    def append(self, k_new: torch.Tensor, v_new: torch.Tensor) -> None:
        """Places one token's rows ([B,Hkv,D] bf16, contiguous) in the staging buffer (hyq_kv_cache_append)."""
        api._dev(k_new, torch.bfloat16, "k_new"), api._dev(v_new, torch.bfloat16, "v_new")
        api._check(_lib().hyq_kv_cache_append(k_new.data_ptr(), v_new.data_ptr(), ctypes.byref(self.desc), api._stream()),
                   "hyq_kv_cache_append")
        self.desc.n_staging = self.n_staging + 1

    def bytes_read_per_token(self) -> int:
        """Bytes of cache one attention call reads: codes, scales and the valid bf16 rows."""
        d, s = self.desc, self.sizes
        heads = d.B * d.Hkv
        nq = int(s.quantized_rows)
        w = min(d.window, d.N)
        code_bytes = d.D if d.format == FMT_INT4 else 2 * d.D    # K + V codes of one row
        return heads * (nq * code_bytes + 2 * (-(-nq // d.group)) * 4 + (d.k + w + d.n_staging) * d.D * 4)


def alloc_cache(desc: KvCacheDesc, device="cuda") -> HybridKvCache:
    s = hyq_kv_cache_query_sizes(desc)
    B, H, D = desc.B, desc.Hkv, desc.D
    w = desc.cap_window or min(desc.window, desc.N)
    nqp = desc.cap_quantized_rows or int(s.padded_rows)
    kcap = desc.cap_vertical or desc.k
    u8 = lambda *shape: torch.empty(*shape, dtype=torch.uint8, device=device)          # noqa: E731
    bf = lambda *shape: torch.empty(*shape, dtype=torch.bfloat16, device=device)       # noqa: E731
    rb = D // 2 if desc.format == FMT_INT4 else D               # code bytes per row
    buf = dict(kq_codes=u8(B, H, max(nqp, 1), rb), vq_codes=u8(B, H, max(nqp // 16, 1), 16 * rb),
               kq_scales=torch.empty(B, H, max(nqp // desc.group, 1), dtype=torch.float32, device=device),
               vq_scales=torch.empty(B, H, max(nqp // desc.group, 1), dtype=torch.float32, device=device),
               k_vl=bf(B, H, max(kcap, 1), D), v_vl=bf(B, H, max(kcap, 1), D),
               k_win=bf(B, H, max(w, 1), D), v_win=bf(B, H, max(w, 1), D),
               k_s=bf(B, H, max(desc.staging_capacity, 1), D), v_s=bf(B, H, max(desc.staging_capacity, 1), D))
    for name, t in buf.items():
        setattr(desc, name, t.data_ptr())
    return HybridKvCache(desc, s, buf)


def hyq_freeze(k: torch.Tensor, v: torch.Tensor, vl_idx: torch.Tensor | None, window: int, Hq: int,
               staging_capacity: int = 128, cache: HybridKvCache | None = None, group: int = 64,
               fmt: int = FMT_INT4) -> HybridKvCache:
    """Algorithm 4.  k, v [B,Hkv,N,D] bf16 CUDA; vl_idx int32 [B,Hkv,k] ascending (None: no vertical rows)."""
    api._dev(k, torch.bfloat16, "k"), api._dev(v, torch.bfloat16, "v")
    B, Hkv, N, D = k.shape
    kk = 0 if vl_idx is None else int(vl_idx.shape[2])
    if cache is None:
        cache = alloc_cache(make_desc(B, Hq, Hkv, N, window, kk, staging_capacity, D=D, group=group, fmt=fmt), k.device)
    if kk:
        api._dev(vl_idx, torch.int32, "vl_idx")
    api._check(_lib().hyq_freeze(k.data_ptr(), v.data_ptr(), vl_idx.data_ptr() if kk else None,
                                 ctypes.byref(cache.desc), api._stream()), "hyq_freeze")
    return cache


def hyq_hybrid_attention_decode_workspace(cache: HybridKvCache, splits: int = 0) -> int:
    n = ctypes.c_size_t(0)
    api._check(_lib().hyq_hybrid_attention_decode_workspace(ctypes.byref(cache.desc), splits, ctypes.byref(n)),
               "hyq_hybrid_attention_decode_workspace")
    return int(n.value)


def hyq_hybrid_attention_decode(q: torch.Tensor, cache: HybridKvCache, softmax_scale: float = 0.0, splits: int = 0,
                                out_dtype=torch.bfloat16, out: torch.Tensor | None = None,
                                lse: torch.Tensor | None = None, workspace: torch.Tensor | None = None) -> torch.Tensor:
    """Algorithm 3.  q [B,Hq,D] bf16 CUDA -> out [B,Hq,D]."""
    api._dev(q, torch.bfloat16, "q")
    B, Hq, D = q.shape
    if out is None:
        out = torch.empty(B, Hq, D, dtype=out_dtype, device=q.device)
    if workspace is None:
        workspace = torch.empty(max(hyq_hybrid_attention_decode_workspace(cache, splits), 16), dtype=torch.uint8,
                                device=q.device)
    api._check(_lib().hyq_hybrid_attention_decode(q.data_ptr(), ctypes.byref(cache.desc), softmax_scale, splits,
                                                  1 if out.dtype == torch.float32 else 0, out.data_ptr(),
                                                  lse.data_ptr() if lse is not None else None, workspace.data_ptr(),
                                                  workspace.numel(), api._stream()), "hyq_hybrid_attention_decode")
    return out


class RaggedKvCache:
    """A batch of sequences of different lengths in one allocation (capacity strides), for
    ``hyq_hybrid_attention_decode_ragged``.  Each sequence is frozen on its own (Algorithm 4 with B = 1 into its
    slice of the buffers); ``lengths`` [B,4] int32 holds the valid {quantized, vertical, window, staging} rows."""

    def __init__(self, B, Hq, Hkv, max_N, window, max_k, staging_capacity=128, D=128, device="cuda"):
        cap_q = -(-max_N // 64) * 64
        self.window = window
        self.batch = alloc_cache(make_desc(B, Hq, Hkv, max_N, window, 0, staging_capacity, D=D, cap_quantized_rows=cap_q,
                                           cap_vertical=max(max_k, 1), cap_window=max(min(window, max_N), 1)), device)
        self.lengths_host = torch.zeros(B, 4, dtype=torch.int32)
        self.lengths = torch.zeros(B, 4, dtype=torch.int32, device=device)

    def _sequence_view(self, b, N, k) -> HybridKvCache:
        bd = self.batch.desc
        d = make_desc(1, bd.Hq, bd.Hkv, N, self.window, k, bd.staging_capacity, D=bd.D, cap_quantized_rows=bd.cap_quantized_rows,
                      cap_vertical=bd.cap_vertical, cap_window=bd.cap_window)
        bufs = {n: t[b:b + 1] for n, t in self.batch.buffers.items()}
        for n, t in bufs.items():
            setattr(d, n, t.data_ptr())
        return HybridKvCache(d, hyq_kv_cache_query_sizes(d), bufs)

    def freeze_sequence(self, b: int, k: torch.Tensor, v: torch.Tensor, vl_idx: torch.Tensor | None) -> None:
        """k, v [1,Hkv,N_b,D] bf16; vl_idx [1,Hkv,k_b] int32 ascending or None."""
        N = k.shape[2]
        kk = 0 if vl_idx is None else int(vl_idx.shape[2])
        view = self._sequence_view(b, N, kk)
        hyq_freeze(k, v, vl_idx, self.window, self.batch.desc.Hq, cache=view)
        w = min(self.window, N)
        self.lengths_host[b] = torch.tensor([N - w - kk, kk, w, 0], dtype=torch.int32)
        self.lengths.copy_(self.lengths_host)

    def append(self, b: int, k_new: torch.Tensor, v_new: torch.Tensor) -> None:
        """One token's rows ([Hkv,D] bf16) of sequence b into its staging buffer."""
        n = int(self.lengths_host[b, 3])
        api._dev(k_new, torch.bfloat16, "k_new"), api._dev(v_new, torch.bfloat16, "v_new")
        one = KvCacheDesc()
        ctypes.memmove(ctypes.byref(one), ctypes.byref(self.batch.desc), ctypes.sizeof(KvCacheDesc))
        one.B, one.n_staging = 1, n                      # sequence b's staging buffers as a batch of one
        one.k_s, one.v_s = self.batch.buffers["k_s"][b].data_ptr(), self.batch.buffers["v_s"][b].data_ptr()
        api._check(_lib().hyq_kv_cache_append(k_new.data_ptr(), v_new.data_ptr(), ctypes.byref(one), api._stream()),
                   "hyq_kv_cache_append")
        self.lengths_host[b, 3] = n + 1
        self.lengths.copy_(self.lengths_host)


def hyq_hybrid_attention_decode_ragged(q: torch.Tensor, cache: RaggedKvCache, softmax_scale: float = 0.0, splits: int = 0,
                                       out_dtype=torch.bfloat16, out: torch.Tensor | None = None,
                                       lse: torch.Tensor | None = None, workspace: torch.Tensor | None = None) -> torch.Tensor:
    """Algorithm 3 for a batch of sequences of different lengths.  q [B,Hq,D] bf16 CUDA -> out [B,Hq,D]."""
    api._dev(q, torch.bfloat16, "q")
    B, Hq, D = q.shape
    if out is None:
        out = torch.empty(B, Hq, D, dtype=out_dtype, device=q.device)
    if workspace is None:
        workspace = torch.empty(max(hyq_hybrid_attention_decode_workspace(cache.batch, splits), 16), dtype=torch.uint8,
                                device=q.device)
    api._check(_lib().hyq_hybrid_attention_decode_ragged(q.data_ptr(), ctypes.byref(cache.batch.desc), cache.lengths.data_ptr(),
                                                         softmax_scale, splits, 1 if out.dtype == torch.float32 else 0,
                                                         out.data_ptr(), lse.data_ptr() if lse is not None else None,
                                                         workspace.data_ptr(), workspace.numel(), api._stream()),
               "hyq_hybrid_attention_decode_ragged")
    return out
