"""CPU oracle for the HyQuant prefill path (Algorithm 1, Algorithm 2, Eq. 6-7).

TEST INFRASTRUCTURE ONLY: imported by the test suite, the smoke check and the
CPU-baseline / reference legs of the benchmark.  The CUDA library never imports
it and it never imports the CUDA library.

The arithmetic lives in ``hyq_oracle.c`` (plain C, fp64, OpenMP over independent
rows); this module only compiles that file with gcc and marshals numpy arrays.
bf16 tensors are passed as ``uint16`` arrays holding the bit patterns.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "hyq_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")

FMT_INT8, FMT_FP8_E4M3, FMT_INT4 = 0, 1, 2


def build(force: bool = False) -> str:
    """Compile the oracle (gcc, no fast-math, no FMA contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-ffp-contract=off", "-std=c11", "-shared", "-fPIC",
             "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


class _AttnIn(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int) for n in
                ("B", "Hq", "Hkv", "L", "Lq", "fixed_window", "D", "W", "k", "block_tokens", "q_fmt", "k_fmt",
                 "v_fmt")] + [
        ("alpha", ctypes.c_double)] + [(n, ctypes.c_void_p) for n in
                                       ("q", "k_", "v", "q_codes", "k_codes", "v_codes",
                                        "q_scales", "k_scales", "v_scales", "vl_idx")]


_lib = None


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_num_threads.restype = ctypes.c_int
    return _lib


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def _u16(x, shape_len):
    x = np.ascontiguousarray(x)
    assert x.dtype == np.uint16 and x.ndim == shape_len, (x.dtype, x.shape)
    return x


def _ptr(a):
    return a.ctypes.data_as(ctypes.c_void_p)


def code_row_bytes(fmt: int, D: int) -> int:
    return D // 2 if fmt == FMT_INT4 else D


def e4m3_encode(y) -> np.ndarray:
    """fp32 -> e4m3 byte, round-to-nearest-even, saturating at +-448."""
    y = np.ascontiguousarray(y, dtype=np.float32)
    out = np.zeros(y.shape, dtype=np.uint8)
    _load().oracle_e4m3_encode(_ptr(y), ctypes.c_long(y.size), _ptr(out))
    return out


def e4m3_decode(c) -> np.ndarray:
    c = np.ascontiguousarray(c, dtype=np.uint8)
    out = np.zeros(c.shape, dtype=np.float64)
    _load().oracle_e4m3_decode(_ptr(c), ctypes.c_long(c.size), _ptr(out))
    return out


def quantize(x_bits, fmt: int, block_tokens: int = 64):
    """Algorithm 2 Stage 2.  x_bits: uint16 [B,H,L,D].  Returns (codes uint8
    [B,H,L,D or D/2], scales float32 [B,H,ceil(L/block_tokens)])."""
    x = _u16(x_bits, 4)
    B, H, L, D = x.shape
    nb = (L + block_tokens - 1) // block_tokens
    codes = np.zeros((B, H, L, code_row_bytes(fmt, D)), dtype=np.uint8)
    scales = np.zeros((B, H, nb), dtype=np.float32)
    rc = _load().oracle_quantize(_ptr(x), B, H, L, D, block_tokens, fmt, _ptr(codes), _ptr(scales))
    if rc:
        raise ValueError(f"oracle_quantize failed ({rc})")
    return codes, scales


def select_vertical(q_bits, k_bits, window: int, k: int, n_tail: int = 0, return_scores: bool = False):
    """Algorithm 1.  Returns int32 [B,Hq,k] ascending (and optionally the fp64
    scores [B,Hq,P])."""
    q = _u16(q_bits, 4)
    kk = _u16(k_bits, 4)
    B, Hq, Lq, D = q.shape
    Bk, Hkv, Lk, Dk = kk.shape
    assert B == Bk and D == Dk
    P = max(0, Lk - window)
    kk_eff = 0 if P == 0 else k
    idx = np.zeros((B, Hq, kk_eff), dtype=np.int32)
    scores = np.zeros((B, Hq, P), dtype=np.float64) if return_scores else None
    rc = _load().oracle_select(_ptr(q), _ptr(kk), B, Hq, Hkv, Lq, Lk, D, window, n_tail, kk_eff,
                               _ptr(idx), _ptr(scores) if return_scores else None)
    if rc:
        raise ValueError(f"oracle_select failed ({rc})")
    return (idx, scores) if return_scores else idx


def exp_det(x) -> np.ndarray:
    """The oracle's operation-by-operation exp for x <= 0 (Eq. 4 scores decide an index set)."""
    x = np.ascontiguousarray(x, dtype=np.float64)
    out = np.zeros(x.shape, dtype=np.float64)
    _load().oracle_exp_det(_ptr(x), ctypes.c_long(x.size), _ptr(out))
    return out


def select_vertical_mass(q_bits, k_bits, window: int, k: int, n_queries: int = 0, alpha: float | None = None,
                         return_scores: bool = False, plain: bool = False):
    """Eq. 4-5: column mass of the softmax rows of the last n_queries queries, top-k over the non-window
    prefix.  Returns int32 [B,Hq,k] ascending (and optionally the fp64 scores [B,Hq,P]).

    ``plain=True`` evaluates the definition itself (two-pass softmax per query with libm ``exp`` and
    sequential sums); the default is the library's fixed-order recipe, which is pinned to the plain form
    and which the GPU reproduces bit for bit."""
    q = _u16(q_bits, 4)
    kk = _u16(k_bits, 4)
    B, Hq, Lq, D = q.shape
    Bk, Hkv, Lk, Dk = kk.shape
    assert B == Bk and D == Dk
    P = max(0, Lk - window)
    kk_eff = 0 if P == 0 else k
    idx = np.zeros((B, Hq, kk_eff), dtype=np.int32)
    scores = np.zeros((B, Hq, P), dtype=np.float64) if return_scores else None
    a = 1.0 / np.sqrt(np.float64(D)) if alpha is None else float(alpha)
    fn = _load().oracle_select_mass_plain if plain else _load().oracle_select_mass
    rc = fn(_ptr(q), _ptr(kk), B, Hq, Hkv, Lq, Lk, D, window, n_queries, kk_eff,
            ctypes.c_double(a), _ptr(idx), _ptr(scores) if return_scores else None)
    if rc:
        raise ValueError(f"oracle_select_mass failed ({rc})")
    return (idx, scores) if return_scores else idx


def _attn_in(q_bits, k_bits, v_bits, qc, kc, vc, qs, ks, vs, fmts, vl_idx, window, block_tokens, alpha,
             fixed_window=False):
    q, kk, v = _u16(q_bits, 4), _u16(k_bits, 4), _u16(v_bits, 4)
    B, Hq, Lq, D = q.shape                      # Lq query rows, end-aligned with the L keys (Lq == L: whole prefill)
    Hkv, L = kk.shape[1], kk.shape[2]
    assert kk.shape == (B, Hkv, L, D) and v.shape == kk.shape and 0 < Lq <= L
    qc, kc, vc = (np.ascontiguousarray(c, dtype=np.uint8) for c in (qc, kc, vc))
    qs, ks, vs = (np.ascontiguousarray(s, dtype=np.float32) for s in (qs, ks, vs))
    nb = (L + block_tokens - 1) // block_tokens
    nbq = (Lq + block_tokens - 1) // block_tokens
    assert qc.shape == (B, Hq, Lq, code_row_bytes(fmts[0], D)), qc.shape
    assert kc.shape == (B, Hkv, L, code_row_bytes(fmts[1], D)), kc.shape
    assert vc.shape == (B, Hkv, L, code_row_bytes(fmts[2], D)), vc.shape
    assert qs.shape == (B, Hq, nbq) and ks.shape == (B, Hkv, nb) and vs.shape == (B, Hkv, nb)
    if vl_idx is None:
        vl_idx = np.zeros((B, Hq, 0), dtype=np.int32)
    vl = np.ascontiguousarray(vl_idx, dtype=np.int32)
    assert vl.shape[:2] == (B, Hq)
    a = _AttnIn(B=B, Hq=Hq, Hkv=Hkv, L=L, Lq=Lq, fixed_window=int(bool(fixed_window)), D=D, W=window, k=vl.shape[2], block_tokens=block_tokens,
                q_fmt=fmts[0], k_fmt=fmts[1], v_fmt=fmts[2],
                alpha=(1.0 / np.sqrt(D)) if alpha is None else float(alpha),
                q=q.ctypes.data, k_=kk.ctypes.data, v=v.ctypes.data,
                q_codes=qc.ctypes.data, k_codes=kc.ctypes.data, v_codes=vc.ctypes.data,
                q_scales=qs.ctypes.data, k_scales=ks.ctypes.data, v_scales=vs.ctypes.data,
                vl_idx=vl.ctypes.data)
    keep = (q, kk, v, qc, kc, vc, qs, ks, vs, vl)
    return a, keep, (B, Hq, Lq, D)


def attention_rows(q_bits, k_bits, v_bits, q_codes, k_codes, v_codes, q_scales, k_scales, v_scales,
                   fmts, vl_idx, window: int, rows=None, block_tokens: int = 64, alpha=None,
                   return_lse: bool = False, return_fp_pairs: bool = False, fixed_window: bool = False):
    """Eq. 6-7 by definition (two-pass fp64 softmax over every key j <= i).
    q holds Lq <= L query rows, end-aligned with the L keys (the query block of Algorithm 2; row r sits at
    position L - Lq + r); Lq == L is the whole prefill.
    fixed_window: the window keys are the last `window` keys for every row (Algorithm 2's K_Win taken literally)
    instead of each row's own last `window` positions.
    rows: rows of the query block to compute (default all).  Returns fp64 [B,Hq,n_rows,D]."""
    a, keep, (B, Hq, L, D) = _attn_in(q_bits, k_bits, v_bits, q_codes, k_codes, v_codes, q_scales,
                                      k_scales, v_scales, fmts, vl_idx, window, block_tokens, alpha, fixed_window)
    rows = np.arange(L, dtype=np.int32) if rows is None else np.ascontiguousarray(rows, dtype=np.int32)
    out = np.zeros((B, Hq, len(rows), D), dtype=np.float64)
    lse = np.zeros((B, Hq, len(rows)), dtype=np.float64)
    fp = ctypes.c_longlong(0)
    rc = _load().oracle_attention_rows(ctypes.byref(a), _ptr(rows), len(rows), _ptr(out), _ptr(lse),
                                       ctypes.byref(fp))
    if rc:
        raise ValueError(f"oracle_attention_rows failed ({rc})")
    res = (out,)
    if return_lse:
        res += (lse,)
    if return_fp_pairs:
        res += (int(fp.value),)
    return res[0] if len(res) == 1 else res


def attention_segmented_rows(q_bits, k_bits, v_bits, q_codes, k_codes, v_codes, q_scales, k_scales,
                             v_scales, fmts, vl_idx, window: int, rows=None, tile_n: int = 64,
                             block_tokens: int = 64, alpha=None, fixed_window: bool = False):
    """Algorithm 2 Stage 3 taken literally (segments A, B, C with the running
    (m, l, acc) update).  Returns fp64 [B,Hq,n_rows,D]."""
    a, keep, (B, Hq, L, D) = _attn_in(q_bits, k_bits, v_bits, q_codes, k_codes, v_codes, q_scales,
                                      k_scales, v_scales, fmts, vl_idx, window, block_tokens, alpha, fixed_window)
    rows = np.arange(L, dtype=np.int32) if rows is None else np.ascontiguousarray(rows, dtype=np.int32)
    out = np.zeros((B, Hq, len(rows), D), dtype=np.float64)
    rc = _load().oracle_attention_segmented_rows(ctypes.byref(a), _ptr(rows), len(rows), tile_n, _ptr(out))
    if rc:
        raise ValueError(f"oracle_attention_segmented_rows failed ({rc})")
    return out


def hybrid_prefill(q_bits, k_bits, v_bits, window: int, k: int, fmts=(FMT_INT8, FMT_INT8, FMT_INT8),
                   rows=None, block_tokens: int = 64, n_tail: int = 0):
    """The whole path in the paper's order: Algorithm 1, then Stage 2, then Eq. 7.
    Returns dict(idx, codes, scales, out)."""
    idx = select_vertical(q_bits, k_bits, window, k, n_tail)
    qc, qs = quantize(q_bits, fmts[0], block_tokens)
    kc, ks = quantize(k_bits, fmts[1], block_tokens)
    vc, vs = quantize(v_bits, fmts[2], block_tokens)
    out = attention_rows(q_bits, k_bits, v_bits, qc, kc, vc, qs, ks, vs, fmts, idx, window, rows, block_tokens)
    return dict(idx=idx, q_codes=qc, k_codes=kc, v_codes=vc, q_scales=qs, k_scales=ks, v_scales=vs, out=out)
