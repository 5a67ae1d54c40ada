"""CPU oracle for the decode side: Freeze (Algorithm 4) and the hybrid-precision KV-cache
attention of one new token (Algorithm 3).

TEST INFRASTRUCTURE ONLY, like the rest of this package: plain numpy in fp64, nothing here is
imported by the CUDA library and nothing here imports it.

Two forms of the attention are given and pinned against each other by the tests:
``decode_attention`` is the definition (one softmax over the concatenation of the dequantized
prefix, the vertical-line rows, the staging rows and the window rows, Section 3.3), and
``decode_attention_segmented`` walks Algorithm 3 in its own order (S chunks of the quantized
prefix from an empty state, ReduceSoftmax, then the three full-precision segments through the
same running state).

Readings taken where the paper leaves a choice (each is stated again where it is used):
  * Quant(.; G): the compacted non-window, non-vertical rows are cut into groups of G
    consecutive COMPACTED rows (all D channels) and each group is quantized as Algorithm 2
    Stage 2 quantizes a tile (one fp32 scale per group, c_B = 7 / 127 / 448).
  * Algorithm 1 returns one index set per query head while the cache has one row set per KV
    head; Freeze here takes one set per KV head as an input.
  * The new token's own key and value are in the cache (staging buffer, or the window when
    the staging buffer is empty) before its attention runs, as in any causal decoder.
"""
from __future__ import annotations

import numpy as np

from . import FMT_FP8_E4M3, FMT_INT4, FMT_INT8, e4m3_decode, quantize

_BITS = {FMT_INT4: 4, FMT_INT8: 8, FMT_FP8_E4M3: 8}


def bf16_to_f64(bits) -> np.ndarray:
    b = np.ascontiguousarray(bits, dtype=np.uint16)
    return (b.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def code_values(codes: np.ndarray, fmt: int) -> np.ndarray:
    """Numeric value of every code (fp64); INT4 rows unpack to D values, low nibble first."""
    if fmt == FMT_INT8:
        return codes.view(np.int8).astype(np.float64)
    if fmt == FMT_FP8_E4M3:
        return e4m3_decode(codes)
    lo = (codes & 0xF).astype(np.int16)
    hi = (codes >> 4).astype(np.int16)
    lo[lo >= 8] -= 16
    hi[hi >= 8] -= 16
    return np.stack([lo, hi], axis=-1).reshape(codes.shape[:-1] + (2 * codes.shape[-1],)).astype(np.float64)


def dequantize(codes: np.ndarray, scales: np.ndarray, fmt: int, group: int) -> np.ndarray:
    """DeQuant of Section 3.3: code value times the scale of the row's group."""
    val = code_values(codes, fmt)
    n = val.shape[-2]
    sc = np.repeat(scales.astype(np.float64), group, axis=-1)[..., :n]
    return val * sc[..., None]


def quantized_positions(N: int, window: int, vl_idx_row) -> np.ndarray:
    """Algorithm 4: I_Q = [0, N - W) minus I_VL, ascending."""
    P = max(0, N - window)
    keep = np.ones(P, dtype=bool)
    keep[np.asarray(vl_idx_row, dtype=np.int64)] = False
    return np.nonzero(keep)[0].astype(np.int32)


def freeze(k_bits, v_bits, vl_idx, window: int, group: int = 64, fmts=(FMT_INT4, FMT_INT4),
           staging_capacity: int = 128) -> dict:
    """Algorithm 4.  k_bits, v_bits: uint16 [B,Hkv,N,D] (bf16 bit patterns); vl_idx int32
    [B,Hkv,k], each row strictly ascending in [0, N - W).  Returns the four buffers:
      k_win, v_win   uint16 [B,Hkv,W',D]   the last W' = min(W, N) rows
      k_vl, v_vl     uint16 [B,Hkv,k,D]    rows vl_idx, in that order
      kq_codes, kq_scales, vq_codes, vq_scales   the other prefix rows, compacted in ascending
                     position order and quantized per group of `group` compacted rows
      iq             int32 [B,Hkv,nQ]      their original positions
      k_s, v_s       uint16 [B,Hkv,W_s,D]  empty staging buffer (zeros), n_s = 0
    """
    k_bits = np.ascontiguousarray(k_bits, dtype=np.uint16)
    v_bits = np.ascontiguousarray(v_bits, dtype=np.uint16)
    B, H, N, D = k_bits.shape
    Wc = min(window, N)
    P = N - Wc
    kk = 0 if vl_idx is None else vl_idx.shape[2]
    nQ = P - kk
    iq = np.zeros((B, H, nQ), dtype=np.int32)
    k_vl = np.zeros((B, H, kk, D), dtype=np.uint16)
    v_vl = np.zeros((B, H, kk, D), dtype=np.uint16)
    kc = np.zeros((B, H, nQ, D), dtype=np.uint16)
    vc = np.zeros((B, H, nQ, D), dtype=np.uint16)
    for b in range(B):
        for h in range(H):
            row = vl_idx[b, h] if kk else np.zeros(0, dtype=np.int32)
            assert np.all(np.diff(row) > 0) and (kk == 0 or (row[0] >= 0 and row[-1] < P))
            iq[b, h] = quantized_positions(N, Wc, row)
            k_vl[b, h], v_vl[b, h] = k_bits[b, h, row], v_bits[b, h, row]
            kc[b, h], vc[b, h] = k_bits[b, h, iq[b, h]], v_bits[b, h, iq[b, h]]
    kq_codes, kq_scales = quantize(kc, fmts[0], group)
    vq_codes, vq_scales = quantize(vc, fmts[1], group)
    return dict(B=B, Hkv=H, N=N, D=D, window=Wc, k=kk, nQ=nQ, group=group, fmts=tuple(fmts), iq=iq,
                k_win=k_bits[:, :, P:].copy(), v_win=v_bits[:, :, P:].copy(), k_vl=k_vl, v_vl=v_vl,
                kq_codes=kq_codes, kq_scales=kq_scales, vq_codes=vq_codes, vq_scales=vq_scales,
                k_s=np.zeros((B, H, staging_capacity, D), dtype=np.uint16),
                v_s=np.zeros((B, H, staging_capacity, D), dtype=np.uint16), n_s=0)


def append_staging(cache: dict, k_new_bits, v_new_bits) -> None:
    """Places one new token's key and value rows ([B,Hkv,D]) in the staging buffer."""
    n = cache["n_s"]
    assert n < cache["k_s"].shape[2], "staging buffer full"
    cache["k_s"][:, :, n] = k_new_bits
    cache["v_s"][:, :, n] = v_new_bits
    cache["n_s"] = n + 1


def cache_code_bytes(cache: dict) -> dict:
    """Bytes of key/value payload per buffer (scales excluded), for the memory accounting."""
    per = cache["B"] * cache["Hkv"] * cache["D"]
    bk, bv = _BITS[cache["fmts"][0]], _BITS[cache["fmts"][1]]
    return dict(quantized=per * cache["nQ"] * (bk + bv) // 8, vertical=per * cache["k"] * 4,
                window=per * cache["window"] * 4, staging=per * cache["k_s"].shape[2] * 4)


def _segments(cache: dict, b: int, h: int):
    """The four key/value segments of one (b, kv head) as fp64 matrices, in Algorithm 3's order."""
    g = cache["group"]
    kq = dequantize(cache["kq_codes"][b, h], cache["kq_scales"][b, h], cache["fmts"][0], g)
    vq = dequantize(cache["vq_codes"][b, h], cache["vq_scales"][b, h], cache["fmts"][1], g)
    n_s = cache["n_s"]
    return [(kq, vq),
            (bf16_to_f64(cache["k_vl"][b, h]), bf16_to_f64(cache["v_vl"][b, h])),
            (bf16_to_f64(cache["k_s"][b, h, :n_s]), bf16_to_f64(cache["v_s"][b, h, :n_s])),
            (bf16_to_f64(cache["k_win"][b, h]), bf16_to_f64(cache["v_win"][b, h]))]


def decode_attention(q_bits, cache: dict, alpha: float | None = None):
    """Section 3.3 as a definition: o = softmax(alpha * q [K^Q_hat; K^VL; K^S; K^Win]^T) [V...].
    q_bits uint16 [B,Hq,D].  Returns (out fp64 [B,Hq,D], lse fp64 [B,Hq])."""
    q = bf16_to_f64(q_bits)
    B, Hq, D = q.shape
    g = Hq // cache["Hkv"]
    alpha = 1.0 / np.sqrt(D) if alpha is None else alpha
    out = np.zeros((B, Hq, D))
    lse = np.zeros((B, Hq))
    for b in range(B):
        for h in range(Hq):
            segs = _segments(cache, b, h // g)
            K = np.concatenate([s[0] for s in segs], axis=0)
            V = np.concatenate([s[1] for s in segs], axis=0)
            s = alpha * (K @ q[b, h])
            m = s.max()
            p = np.exp(s - m)
            out[b, h] = (p @ V) / p.sum()
            lse[b, h] = m + np.log(p.sum())
    return out, lse


def flash_os(P, V, state):
    """FlashOS of Algorithms 2-3: one online-softmax update of (m, l, acc) with the score tile
    P [g, n] and the value tile V [n, D]."""
    m, l, acc = state
    if P.shape[1] == 0:
        return state
    m_new = np.maximum(m, P.max(axis=1))
    corr = np.where(np.isneginf(m), 0.0, np.exp(m - m_new))
    p = np.exp(P - m_new[:, None])
    return m_new, l * corr + p.sum(axis=1), acc * corr[:, None] + p @ V


def reduce_softmax(states):
    """ReduceSoftmax of Algorithm 3: merges split states computed from empty states."""
    m = np.max(np.stack([s[0] for s in states]), axis=0)
    l = np.zeros_like(m)
    acc = np.zeros_like(states[0][2])
    for ms, ls, accs in states:
        w = np.where(np.isneginf(ms), 0.0, np.exp(ms - m))
        l += ls * w
        acc += accs * w[:, None]
    return m, l, acc


def decode_attention_segmented(q_bits, cache: dict, alpha: float | None = None, splits: int = 4,
                               tile: int = 64):
    """Algorithm 3 step by step: the g query heads of a KV head are packed into one [g, D] block,
    the quantized prefix is cut into `splits` chunks, each scanned tile by tile from an empty
    state, the chunk states are merged, and the vertical-line, staging and window segments
    continue from the merged state.  Returns (out [B,Hq,D], lse [B,Hq])."""
    q = bf16_to_f64(q_bits)
    B, Hq, D = q.shape
    Hkv = cache["Hkv"]
    g = Hq // Hkv
    alpha = 1.0 / np.sqrt(D) if alpha is None else alpha
    out = np.zeros((B, Hq, D))
    lse = np.zeros((B, Hq))

    def scan(qt, K, V, state):
        for t0 in range(0, K.shape[0], tile):
            state = flash_os(alpha * (qt @ K[t0:t0 + tile].T), V[t0:t0 + tile], state)
        return state

    for b in range(B):
        for hk in range(Hkv):
            qt = q[b, hk * g:(hk + 1) * g]
            segs = _segments(cache, b, hk)
            empty = (np.full(g, -np.inf), np.zeros(g), np.zeros((g, D)))
            kq, vq = segs[0]
            bounds = np.linspace(0, kq.shape[0], splits + 1).astype(int)
            chunk_states = [scan(qt, kq[a:z], vq[a:z], empty) for a, z in zip(bounds[:-1], bounds[1:])]
            state = reduce_softmax(chunk_states)
            for K, V in segs[1:]:
                state = scan(qt, K, V, state)
            m, l, acc = state
            out[b, hk * g:(hk + 1) * g] = acc / l[:, None]
            lse[b, hk * g:(hk + 1) * g] = m + np.log(l)
    return out, lse
