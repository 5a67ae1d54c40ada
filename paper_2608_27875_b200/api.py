"""Thin Python binding of the C-ABI library (``include/hyq.h``): argument
marshalling only.  torch supplies device memory and the current stream; every
step of the path runs in the library's kernels.  There is no CPU fallback: the
first call raises if ``libhyq.so`` has not been built."""
from __future__ import annotations

import ctypes
import os

import torch

from .workloads import FMT_FP8_E4M3, FMT_INT4, FMT_INT8  # noqa: F401

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libhyq.so")

HYQ_OK = 0
IMPL_AUTO, IMPL_TCGEN05, IMPL_SIMT = 0, 1, 2
WINDOW_SLIDING, WINDOW_FIXED_TAIL = 0, 1
EXPORTS = ("hyq_status_string", "hyq_version", "hyq_paper_k", "hyq_select_vertical_workspace",
           "hyq_select_vertical", "hyq_select_vertical_static", "hyq_select_vertical_mass_workspace",
           "hyq_select_vertical_mass", "hyq_quantize_blocks", "hyq_hybrid_attention_prefill_workspace",
           "hyq_hybrid_attention_prefill", "hyq_test_set_attention_hooks", "hyq_test_read_attention_restarts", "hyq_select_vertical_varlen",
           "hyq_quantize_blocks_varlen", "hyq_hybrid_attention_prefill_varlen")


class HyqError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {status_string(code)} (status {code})")


class AttnArgs(ctypes.Structure):
    """Mirror of ``hyq_attn_args``."""
    _fields_ = ([("struct_size", ctypes.c_uint32)] +
                [(n, ctypes.c_int32) for n in ("B", "Hq", "Hkv", "L", "D", "window", "k", "block_tokens",
                                               "q_format", "k_format", "v_format", "out_dtype", "impl")] +
                [("softmax_scale", ctypes.c_float)] +
                [(n, ctypes.c_void_p) for n in ("q", "k_", "v", "q_codes", "k_codes", "v_codes", "q_scales",
                                                "k_scales", "v_scales", "vl_idx", "out", "lse", "status_word",
                                                "workspace")] +
                [("workspace_bytes", ctypes.c_size_t), ("ev_kernel_start", ctypes.c_void_p),
                 ("ev_kernel_stop", ctypes.c_void_p), ("Lq", ctypes.c_int32), ("window_mode", ctypes.c_int32)])


_lib = None


def lib() -> ctypes.CDLL:
    """The loaded shared library; raises if it is missing (no fallback)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2608_27875_b200.build`")
        L = ctypes.CDLL(LIB_PATH)
        L.hyq_status_string.restype = ctypes.c_char_p
        L.hyq_status_string.argtypes = [ctypes.c_int]
        L.hyq_version.restype = ctypes.c_int
        L.hyq_paper_k.restype = ctypes.c_int
        L.hyq_paper_k.argtypes = [ctypes.c_int, ctypes.c_int, ctypes.c_double]
        L.hyq_select_vertical_workspace.argtypes = [ctypes.c_int] * 8 + [ctypes.POINTER(ctypes.c_size_t)]
        L.hyq_select_vertical.argtypes = ([ctypes.c_void_p] * 2 + [ctypes.c_int] * 9 +
                                          [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_size_t, ctypes.c_void_p])
        L.hyq_select_vertical_static.argtypes = ([ctypes.c_void_p] * 2 + [ctypes.c_int] * 9 +
                                                 [ctypes.c_void_p, ctypes.c_void_p])
        L.hyq_select_vertical_mass_workspace.argtypes = [ctypes.c_int] * 9 + [ctypes.POINTER(ctypes.c_size_t)]
        L.hyq_select_vertical_mass.argtypes = ([ctypes.c_void_p] * 2 + [ctypes.c_int] * 9 + [ctypes.c_float] +
                                               [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_size_t, ctypes.c_void_p])
        L.hyq_quantize_blocks.argtypes = ([ctypes.c_void_p] + [ctypes.c_int] * 6 +
                                          [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p])
        L.hyq_hybrid_attention_prefill_workspace.argtypes = [ctypes.POINTER(AttnArgs), ctypes.POINTER(ctypes.c_size_t)]
        L.hyq_hybrid_attention_prefill.argtypes = [ctypes.POINTER(AttnArgs), ctypes.c_void_p]
        L.hyq_test_set_attention_hooks.argtypes = [ctypes.c_longlong, ctypes.c_int]
        L.hyq_test_read_attention_restarts.argtypes = [ctypes.POINTER(ctypes.c_ulonglong), ctypes.c_int]
        i32p = ctypes.POINTER(ctypes.c_int32)
        L.hyq_select_vertical_varlen.argtypes = ([ctypes.c_void_p] * 2 + [ctypes.c_int, i32p] + [ctypes.c_int] * 5 + [i32p] +
                                                 [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_size_t, ctypes.c_void_p])
        L.hyq_quantize_blocks_varlen.argtypes = ([ctypes.c_void_p, ctypes.c_int, i32p] + [ctypes.c_int] * 4 +
                                                 [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p])
        L.hyq_hybrid_attention_prefill_varlen.argtypes = [ctypes.POINTER(AttnArgs), ctypes.c_int, i32p, i32p, ctypes.c_void_p]
        _lib = L
    return _lib


def status_string(code: int) -> str:
    return lib().hyq_status_string(int(code)).decode()


def _check(code: int, where: str):
    if code != HYQ_OK:
        raise HyqError(code, where)


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _dev(t: torch.Tensor, dtype, name: str) -> torch.Tensor:
    if not (t.is_cuda and t.dtype == dtype and t.is_contiguous()):
        raise ValueError(f"{name}: expected a contiguous CUDA tensor of {dtype}, got {t.dtype} on {t.device}")
    return t


def hyq_paper_k(Lk: int, window: int, ratio: float) -> int:
    return int(lib().hyq_paper_k(Lk, window, ratio))


def hyq_select_vertical_workspace(B, Hq, Hkv, Lq, Lk, D, window, k) -> int:
    n = ctypes.c_size_t(0)
    _check(lib().hyq_select_vertical_workspace(B, Hq, Hkv, Lq, Lk, D, window, k, ctypes.byref(n)),
           "hyq_select_vertical_workspace")
    return int(n.value)


def hyq_select_vertical(q: torch.Tensor, k: torch.Tensor, window: int, k_sel: int, n_tail: int = 0,
                        workspace: torch.Tensor | None = None, out: torch.Tensor | None = None) -> torch.Tensor:
    """Algorithm 1.  q [B,Hq,L,D], k [B,Hkv,L,D] bf16 CUDA -> int32 [B,Hq,k_sel] ascending."""
    _dev(q, torch.bfloat16, "q"), _dev(k, torch.bfloat16, "k")
    B, Hq, Lq, D = q.shape
    _, Hkv, Lk, _ = k.shape
    P = max(0, Lk - window)
    k_eff = k_sel if P > 0 else 0
    if out is None:
        out = torch.empty(B, Hq, k_eff, dtype=torch.int32, device=q.device)
    need = hyq_select_vertical_workspace(B, Hq, Hkv, Lq, Lk, D, window, k_eff)
    if workspace is None:
        workspace = torch.empty(max(need, 16), dtype=torch.uint8, device=q.device)
    _check(lib().hyq_select_vertical(q.data_ptr(), k.data_ptr(), B, Hq, Hkv, Lq, Lk, D, window, n_tail, k_eff,
                                     out.data_ptr(), workspace.data_ptr(), workspace.numel(), _stream()),
           "hyq_select_vertical")
    return out


def hyq_select_vertical_mass(q: torch.Tensor, k: torch.Tensor, window: int, k_sel: int, n_queries: int = 0,
                             softmax_scale: float = 0.0, workspace: torch.Tensor | None = None,
                             out: torch.Tensor | None = None) -> torch.Tensor:
    """Eq. 4-5: top-k of the softmax column mass of the last ``n_queries`` queries.  q [B,Hq,Lq,D],
    k [B,Hkv,Lk,D] bf16 CUDA -> int32 [B,Hq,k_sel] ascending."""
    _dev(q, torch.bfloat16, "q"), _dev(k, torch.bfloat16, "k")
    B, Hq, Lq, D = q.shape
    _, Hkv, Lk, _ = k.shape
    k_eff = k_sel if Lk - window > 0 else 0
    if out is None:
        out = torch.empty(B, Hq, k_eff, dtype=torch.int32, device=q.device)
    n = ctypes.c_size_t(0)
    _check(lib().hyq_select_vertical_mass_workspace(B, Hq, Hkv, Lq, Lk, D, window, n_queries, k_eff, ctypes.byref(n)),
           "hyq_select_vertical_mass_workspace")
    if workspace is None:
        workspace = torch.empty(max(int(n.value), 16), dtype=torch.uint8, device=q.device)
    _check(lib().hyq_select_vertical_mass(q.data_ptr(), k.data_ptr(), B, Hq, Hkv, Lq, Lk, D, window, n_queries, k_eff,
                                          softmax_scale, out.data_ptr(), workspace.data_ptr(), workspace.numel(),
                                          _stream()), "hyq_select_vertical_mass")
    return out


SELECT_STATIC_SCRATCH_BYTES = 8 << 20


def hyq_select_vertical_static(q: torch.Tensor, k: torch.Tensor, window: int, k_sel: int, n_tail: int = 0,
                               out: torch.Tensor | None = None) -> torch.Tensor:
    """Algorithm 1 with the library's built-in scratch array instead of a workspace: for callers that
    cannot allocate device memory at call time.  Pass ``out`` to make the call allocation-free on the
    Python side as well.  Calls on one device must not overlap; problems needing more than
    ``SELECT_STATIC_SCRATCH_BYTES`` of scratch raise ``HyqError`` (workspace too small)."""
    _dev(q, torch.bfloat16, "q"), _dev(k, torch.bfloat16, "k")
    B, Hq, Lq, D = q.shape
    _, Hkv, Lk, _ = k.shape
    k_eff = k_sel if Lk - window > 0 else 0
    if out is None:
        out = torch.empty(B, Hq, k_eff, dtype=torch.int32, device=q.device)
    _check(lib().hyq_select_vertical_static(q.data_ptr(), k.data_ptr(), B, Hq, Hkv, Lq, Lk, D, window, n_tail, k_eff,
                                            out.data_ptr(), _stream()), "hyq_select_vertical_static")
    return out


def hyq_test_read_attention_restarts(reset: bool = False) -> int:
    """Test hook: CTAs of the tensor-core kernel that have gone through their keys a second time (synchronises the device)."""
    n = ctypes.c_ulonglong(0)
    _check(lib().hyq_test_read_attention_restarts(ctypes.byref(n), 1 if reset else 0), "hyq_test_read_attention_restarts")
    return int(n.value)


def hyq_test_set_attention_hooks(wait_limit_clocks: int = 0, drop_load_position: int = -1) -> None:
    """Test hook: clock limit of a device-side barrier wait (0: default) and the walk position whose K/V copy the
    tensor-core kernel's producer leaves out (-1: none).  Process-wide; reset with the defaults."""
    _check(lib().hyq_test_set_attention_hooks(int(wait_limit_clocks), int(drop_load_position)), "hyq_test_set_attention_hooks")


def code_row_bytes(fmt: int, D: int) -> int:
    return D // 2 if fmt == FMT_INT4 else D


def hyq_quantize_blocks(x: torch.Tensor, fmt: int, block_tokens: int = 64, codes: torch.Tensor | None = None,
                        scales: torch.Tensor | None = None):
    """Algorithm 2 Stage 2.  x [B,H,L,D] bf16 CUDA -> (codes uint8 [B,H,L,D or D/2], scales fp32 [B,H,nb])."""
    _dev(x, torch.bfloat16, "x")
    B, H, L, D = x.shape
    nb = -(-L // block_tokens)
    if codes is None:
        codes = torch.empty(B, H, L, code_row_bytes(fmt, D), dtype=torch.uint8, device=x.device)
    if scales is None:
        scales = torch.empty(B, H, nb, dtype=torch.float32, device=x.device)
    _check(lib().hyq_quantize_blocks(x.data_ptr(), B, H, L, D, block_tokens, fmt, codes.data_ptr(),
                                     scales.data_ptr(), _stream()), "hyq_quantize_blocks")
    return codes, scales


def make_attn_args(q, k, v, q_codes, k_codes, v_codes, q_scales, k_scales, v_scales, fmts, vl_idx, window,
                   out, lse=None, status_word=None, workspace=None, impl=IMPL_AUTO, softmax_scale=0.0,
                   block_tokens=64, window_mode=WINDOW_SLIDING) -> AttnArgs:
    B, Hq, Lq, D = q.shape                  # Lq query rows against the k.shape[2] keys (end-aligned query block)
    a = AttnArgs()
    a.struct_size = ctypes.sizeof(AttnArgs)
    a.B, a.Hq, a.Hkv, a.L, a.D = B, Hq, k.shape[1], k.shape[2], D
    a.Lq = Lq
    a.window_mode = window_mode
    a.window, a.k, a.block_tokens = window, (0 if vl_idx is None else vl_idx.shape[2]), block_tokens
    a.q_format, a.k_format, a.v_format = fmts
    a.out_dtype = 1 if out.dtype == torch.float32 else 0
    a.impl = impl
    a.softmax_scale = softmax_scale
    a.q, a.k_, a.v = q.data_ptr(), k.data_ptr(), v.data_ptr()
    a.q_codes, a.k_codes, a.v_codes = q_codes.data_ptr(), k_codes.data_ptr(), v_codes.data_ptr()
    a.q_scales, a.k_scales, a.v_scales = q_scales.data_ptr(), k_scales.data_ptr(), v_scales.data_ptr()
    a.vl_idx = None if (vl_idx is None or vl_idx.numel() == 0) else vl_idx.data_ptr()
    a.out = out.data_ptr()
    a.lse = None if lse is None else lse.data_ptr()
    a.status_word = None if status_word is None else status_word.data_ptr()
    a.workspace = None if workspace is None else workspace.data_ptr()
    a.workspace_bytes = 0 if workspace is None else workspace.numel()
    return a


def hyq_hybrid_attention_prefill_workspace(args: AttnArgs) -> int:
    n = ctypes.c_size_t(0)
    _check(lib().hyq_hybrid_attention_prefill_workspace(ctypes.byref(args), ctypes.byref(n)),
           "hyq_hybrid_attention_prefill_workspace")
    return int(n.value)


def hyq_hybrid_attention_prefill(q, k, v, q_codes, k_codes, v_codes, q_scales, k_scales, v_scales, fmts,
                                 vl_idx, window: int, out: torch.Tensor | None = None, out_dtype=torch.float32,
                                 lse: torch.Tensor | None = None, status_word: torch.Tensor | None = None,
                                 workspace: torch.Tensor | None = None, impl: int = IMPL_AUTO,
                                 softmax_scale: float = 0.0, window_mode: int = WINDOW_SLIDING,
                                 block_tokens: int = 64) -> torch.Tensor:
    """Eq. 6-7 / Algorithm 2 Stage 3.  q may hold fewer rows than k, v: the last Lq query rows of the context
    (Algorithm 2's query block).  Returns out [B,Hq,Lq,D] (fp32 by default)."""
    for t, dt, n in ((q, torch.bfloat16, "q"), (k, torch.bfloat16, "k"), (v, torch.bfloat16, "v"),
                     (q_codes, torch.uint8, "q_codes"), (k_codes, torch.uint8, "k_codes"),
                     (v_codes, torch.uint8, "v_codes"), (q_scales, torch.float32, "q_scales"),
                     (k_scales, torch.float32, "k_scales"), (v_scales, torch.float32, "v_scales")):
        _dev(t, dt, n)
    if vl_idx is not None:
        _dev(vl_idx, torch.int32, "vl_idx")
    if out is None:
        out = torch.empty(q.shape, dtype=out_dtype, device=q.device)
    args = make_attn_args(q, k, v, q_codes, k_codes, v_codes, q_scales, k_scales, v_scales, fmts, vl_idx, window,
                          out, lse, status_word, workspace, impl, softmax_scale, block_tokens=block_tokens,
                          window_mode=window_mode)
    if workspace is None:
        need = hyq_hybrid_attention_prefill_workspace(args)
        workspace = torch.empty(max(need, 16), dtype=torch.uint8, device=q.device)
        args.workspace, args.workspace_bytes = workspace.data_ptr(), workspace.numel()
    _check(lib().hyq_hybrid_attention_prefill(ctypes.byref(args), _stream()), "hyq_hybrid_attention_prefill")
    return out


def hybrid_prefill(q, k, v, window: int, k_sel: int, fmts=(FMT_INT8, FMT_INT8, FMT_INT8), impl: int = IMPL_AUTO,
                   out_dtype=torch.float32):
    """The whole path on device tensors: select -> quantize Q, K, V -> fused attention."""
    idx = hyq_select_vertical(q, k, window, k_sel)
    qc, qs = hyq_quantize_blocks(q, fmts[0])
    kc, ks = hyq_quantize_blocks(k, fmts[1])
    vc, vs = hyq_quantize_blocks(v, fmts[2])
    out = hyq_hybrid_attention_prefill(q, k, v, qc, kc, vc, qs, ks, vs, fmts, idx, window, impl=impl,
                                       out_dtype=out_dtype)
    return dict(idx=idx, q_codes=qc, k_codes=kc, v_codes=vc, q_scales=qs, k_scales=ks, v_scales=vs, out=out)


# ---- ragged batches --------------------------------------------------------------------------------------------
def _i32(xs):
    return (ctypes.c_int32 * len(xs))(*[int(x) for x in xs])


def pack_sequences(seqs) -> tuple[torch.Tensor, list[int]]:
    """[H, L_s, D] tensors -> one flat packed buffer (each sequence a contiguous [H, L_s, D] block) and the token
    offsets cu_seqlens."""
    cu = [0]
    for t in seqs:
        cu.append(cu[-1] + t.shape[1])
    return torch.cat([t.contiguous().reshape(-1) for t in seqs]), cu


def hybrid_prefill_varlen(qs, ks, vs, window: int, k_per_seq, fmts=(FMT_INT8, FMT_INT8, FMT_INT8), block_tokens: int = 64,
                          out_dtype=torch.float32):
    """The whole path over a ragged batch: ``qs[s]`` is [Hq, L_s, D], ``ks[s]`` / ``vs[s]`` are [Hkv, L_s, D] (bf16,
    CUDA).  Packs the prompts, runs the three *_varlen calls and returns per-sequence views of the results:
    a list of dicts with idx [Hq, k_s], codes, scales and out [Hq, L_s, D]."""
    n = len(qs)
    Hq, _, D = qs[0].shape
    Hkv = ks[0].shape[0]
    dev = qs[0].device
    qp, cu = pack_sequences(qs)
    kp, _ = pack_sequences(ks)
    vp, _ = pack_sequences(vs)
    lens = [cu[s + 1] - cu[s] for s in range(n)]
    k_per_seq = [int(k) if lens[s] - window > 0 else 0 for s, k in enumerate(k_per_seq)]
    cu_c, k_c = _i32(cu), _i32(k_per_seq)
    total, nbs = cu[-1], [-(-L_ // block_tokens) for L_ in lens]
    idx = torch.empty(max(1, Hq * sum(k_per_seq)), dtype=torch.int32, device=dev)
    need = max([hyq_select_vertical_workspace(1, Hq, Hkv, L_, L_, D, window, k_) for L_, k_ in zip(lens, k_per_seq)] + [16])
    ws = torch.empty(need, dtype=torch.uint8, device=dev)
    _check(lib().hyq_select_vertical_varlen(qp.data_ptr(), kp.data_ptr(), n, cu_c, Hq, Hkv, D, window, 0, k_c, idx.data_ptr(),
                                            ws.data_ptr(), ws.numel(), _stream()), "hyq_select_vertical_varlen")
    codes, scales = [], []
    for x, H, f in ((qp, Hq, fmts[0]), (kp, Hkv, fmts[1]), (vp, Hkv, fmts[2])):
        c = torch.empty(H * total * code_row_bytes(f, D), dtype=torch.uint8, device=dev)
        sc = torch.empty(H * sum(nbs), dtype=torch.float32, device=dev)
        _check(lib().hyq_quantize_blocks_varlen(x.data_ptr(), n, cu_c, H, D, block_tokens, f, c.data_ptr(), sc.data_ptr(), _stream()),
               "hyq_quantize_blocks_varlen")
        codes.append(c)
        scales.append(sc)
    out = torch.empty(Hq * total * D, dtype=out_dtype, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    a = AttnArgs()
    a.struct_size = ctypes.sizeof(AttnArgs)
    a.B, a.Hq, a.Hkv, a.L, a.D, a.Lq = 1, Hq, Hkv, max(lens), D, 0
    a.window, a.k, a.block_tokens = window, max(k_per_seq), block_tokens
    a.q_format, a.k_format, a.v_format = fmts
    a.out_dtype, a.impl, a.softmax_scale, a.window_mode = (1 if out_dtype == torch.float32 else 0), IMPL_AUTO, 0.0, WINDOW_SLIDING
    a.q, a.k_, a.v = qp.data_ptr(), kp.data_ptr(), vp.data_ptr()
    a.q_codes, a.k_codes, a.v_codes = (c.data_ptr() for c in codes)
    a.q_scales, a.k_scales, a.v_scales = (s_.data_ptr() for s_ in scales)
    a.vl_idx, a.out, a.status_word = idx.data_ptr(), out.data_ptr(), status.data_ptr()
    a.k = k_per_seq[lens.index(max(lens))]
    wsa = torch.empty(max(16, hyq_hybrid_attention_prefill_workspace(a)), dtype=torch.uint8, device=dev)   # the longest sequence's need
    a.workspace, a.workspace_bytes = wsa.data_ptr(), wsa.numel()
    _check(lib().hyq_hybrid_attention_prefill_varlen(ctypes.byref(a), n, cu_c, k_c, _stream()), "hyq_hybrid_attention_prefill_varlen")
    res, ko, no = [], 0, 0
    for s in range(n):
        L_, k_, nb = lens[s], k_per_seq[s], nbs[s]
        view = lambda buf, H, row, t0=cu[s], L_=L_: buf[H * row * t0:H * row * (t0 + L_)].view(H, L_, row)   # noqa: E731
        res.append(dict(
            idx=idx[Hq * ko:Hq * (ko + k_)].view(Hq, k_),
            q_codes=view(codes[0], Hq, code_row_bytes(fmts[0], D)), k_codes=view(codes[1], Hkv, code_row_bytes(fmts[1], D)),
            v_codes=view(codes[2], Hkv, code_row_bytes(fmts[2], D)),
            q_scales=scales[0][Hq * no:Hq * (no + nb)].view(Hq, nb), k_scales=scales[1][Hkv * no:Hkv * (no + nb)].view(Hkv, nb),
            v_scales=scales[2][Hkv * no:Hkv * (no + nb)].view(Hkv, nb), out=view(out, Hq, D)))
        ko += k_
        no += nb
    torch.cuda.synchronize()
    if int(status.item()) != 0:
        raise HyqError(int(status.item()), "hyq_hybrid_attention_prefill_varlen (device)")
    return res
