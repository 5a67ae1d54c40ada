"""Seeded synthetic inputs shaped like long-context prefill layers.

This module holds no arithmetic of the method itself: it only draws Q/K/V and
plants structure that real prefills show (an attention sink at position 0, a
few persistently attended "vertical-line" key columns, optional outlier
channels in K).  Both the CUDA path and the CPU checker are fed from here so
that they see identical bf16 bit patterns.

Recipe, per tensor and per (b, head): a torch CPU generator seeded
``seed*10**6 + tensor_id*10**5 + b*10**3 + h`` (tensor_id Q=0, K=1, V=2, u=3,
pos=4) draws fp32 standard normals.  For each (b, kv head): a unit direction u;
``n_plant`` planted key positions (position 0 plus distinct uniform positions in
[1, L-W)); optionally K channels {17,49,81,113} are multiplied by 20; planted
keys get ``+4u``; every query row of the g query heads of that kv head gets
``+1.5u``.  V is untouched.  Everything is then rounded to bf16.
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import numpy as np
import torch

FMT_INT8, FMT_FP8_E4M3, FMT_INT4 = 0, 1, 2
OUTLIER_CHANNELS = (17, 49, 81, 113)


@dataclass(frozen=True)
class Workload:
    name: str
    B: int
    Hq: int
    Hkv: int
    L: int
    D: int
    window: int
    k: int
    n_plant: int
    q_fmt: int = FMT_INT8
    k_fmt: int = FMT_INT8
    v_fmt: int = FMT_INT8
    outlier_channels: bool = False
    seed: int = 1000

    @property
    def fmts(self):
        return (self.q_fmt, self.k_fmt, self.v_fmt)

    @property
    def causal_pairs(self) -> int:
        return self.B * self.Hq * self.L * (self.L + 1) // 2

    @property
    def flops(self) -> int:
        return 4 * self.D * self.causal_pairs

    def scaled(self, **kw) -> "Workload":
        return replace(self, **kw)


def _pct(L: int, pct: int) -> int:
    return -(-pct * L // 100)


CONFIGS = {
    "c0": Workload("c0", 1, 2, 2, 2048, 128, 128, 32, 16, seed=1000),
    "c1": Workload("c1", 1, 32, 8, 8192, 128, 512, _pct(8192, 2), 64, seed=1001),
    "c2": Workload("c2", 1, 32, 8, 32768, 128, 1024, _pct(32768, 2), 256,
                   q_fmt=FMT_INT4, k_fmt=FMT_INT4, v_fmt=FMT_FP8_E4M3, seed=1002),
    "c3": Workload("c3", 1, 32, 8, 131072, 128, 1024, _pct(131072, 1), 512, seed=1003),
    "c4": Workload("c4", 4, 40, 8, 16384, 128, 512, _pct(16384, 3), 128, outlier_channels=True, seed=1004),
}


def _gen(seed: int, tensor_id: int, b: int, h: int) -> torch.Generator:
    g = torch.Generator(device="cpu")
    g.manual_seed(seed * 10**6 + tensor_id * 10**5 + b * 10**3 + h)
    return g


def planted_positions(w: Workload, b: int, kvh: int) -> torch.Tensor:
    P = max(0, w.L - w.window)
    n = min(w.n_plant, P)
    if n <= 0:
        return torch.zeros(0, dtype=torch.long)
    rest = 1 + torch.randperm(max(P - 1, 0), generator=_gen(w.seed, 4, b, kvh))[: n - 1]
    return torch.cat([torch.zeros(1, dtype=torch.long), rest])


def make_inputs(w: Workload, heads=None):
    """Returns (Q, K, V) bf16 CPU tensors [B,Hq,L,D], [B,Hkv,L,D], [B,Hkv,L,D].

    ``heads``: optional iterable of kv-head indices; when given, only those kv
    heads (and their query heads) are generated, with the bits they have in the
    full workload (used to check a few heads of a very large configuration)."""
    g = w.Hq // w.Hkv
    kv_list = list(range(w.Hkv)) if heads is None else list(heads)
    Q = torch.empty(w.B, len(kv_list) * g, w.L, w.D, dtype=torch.bfloat16)
    K = torch.empty(w.B, len(kv_list), w.L, w.D, dtype=torch.bfloat16)
    V = torch.empty_like(K)
    for b in range(w.B):
        for n, kvh in enumerate(kv_list):
            u = torch.randn(w.D, generator=_gen(w.seed, 3, b, kvh))
            u = u / u.norm()
            k = torch.randn(w.L, w.D, generator=_gen(w.seed, 1, b, kvh))
            if w.outlier_channels:
                k[:, list(OUTLIER_CHANNELS)] *= 20.0
            pos = planted_positions(w, b, kvh)
            k[pos] += 4.0 * u
            K[b, n] = k.to(torch.bfloat16)
            V[b, n] = torch.randn(w.L, w.D, generator=_gen(w.seed, 2, b, kvh)).to(torch.bfloat16)
            for r in range(g):
                h = kvh * g + r
                q = torch.randn(w.L, w.D, generator=_gen(w.seed, 0, b, h))
                q += 1.5 * u
                Q[b, n * g + r] = q.to(torch.bfloat16)
    return Q, K, V


def bits(t: torch.Tensor) -> np.ndarray:
    """bf16 tensor -> uint16 numpy array of its bit patterns (no copy of meaning)."""
    assert t.dtype == torch.bfloat16
    return t.contiguous().view(torch.uint16).numpy()


def sample_rows(L: int, window: int, n_random: int = 64, seed: int = 7, edge: int = 8) -> np.ndarray:
    """A row sample that touches every structural boundary of the path: the
    first and last rows, rows around the window edge, around 64/128-multiples,
    plus seeded random rows.  Sorted, unique, int32."""
    rs = set()
    for c in (0, L - 1):
        rs.update(range(max(0, c - edge), min(L, c + edge + 1)))
    for c in (window - 1, window, 64, 128, 127, L // 2, (L // 128) * 128 - 1, (L // 2 // 128) * 128):
        rs.update(range(max(0, c - 2), min(L, c + 3)))
    rng = np.random.default_rng(seed)
    rs.update(int(x) for x in rng.integers(0, L, size=n_random))
    return np.array(sorted(rs), dtype=np.int32)
