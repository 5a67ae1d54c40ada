"""Helpers shared by the GPU parity tests (marshalling only)."""
import numpy as np
import torch

import oracle
from paper_2608_27875_b200 import api, build, workloads as wl

# tolerance of the attention output against the fp64 oracle: max-abs error and
# sum|err| / sum|ref| (the workload definition fixes both)
MAX_ABS_TOL = 1e-2
MEAN_REL_TOL = 2e-3


def ensure_built():
    build.build()
    return api.lib()


def rand_bf16(shape, seed, scale=1.0):
    g = torch.Generator().manual_seed(seed)
    return (torch.randn(*shape, generator=g) * scale).to(torch.bfloat16)


def errors(got: np.ndarray, ref: np.ndarray):
    d = np.abs(got.astype(np.float64) - ref)
    return float(d.max()), float(d.sum() / np.abs(ref).sum())


def oracle_quant_all(Q, K, V, fmts, block_tokens=64):
    return [oracle.quantize(wl.bits(t), f, block_tokens) for t, f in zip((Q, K, V), fmts)]


def gpu_attention(Q, K, V, qz, fmts, idx, window, impl, out_dtype=torch.float32, lse=False, window_mode=0, block_tokens=64):
    """Runs the library's attention on the oracle's codes/scales/indices (so that this step is
    compared on identical inputs)."""
    dev = "cuda"
    (qc, qs), (kc, ks), (vc, vs) = qz
    t = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(dev)   # noqa: E731
    idx_t = None if idx is None or idx.shape[2] == 0 else t(idx)
    lse_t = torch.empty(Q.shape[:3], dtype=torch.float32, device=dev) if lse else None
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    out = api.hyq_hybrid_attention_prefill(Q.to(dev), K.to(dev), V.to(dev), t(qc), t(kc), t(vc), t(qs), t(ks), t(vs),
                                           fmts, idx_t, window, impl=impl, out_dtype=out_dtype, lse=lse_t,
                                           status_word=status, window_mode=window_mode, block_tokens=block_tokens)
    torch.cuda.synchronize()
    assert int(status.item()) == 0, "kernel reported a device-side error"
    return (out.cpu(), lse_t.cpu()) if lse else out.cpu()
