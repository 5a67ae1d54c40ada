"""How the path spreads over several GPUs: by (batch, KV head) units, with no exchange step.

Selection is per query head, quantization per (b, head, block) and attention per (b, query head), so a
(batch, KV head) unit together with its g query heads is independent of every other unit.  Each rank
takes a contiguous, balanced range of units; nothing is communicated on the data path.  The only
collective is the max-over-ranks of a timing (or any scalar) for reporting.
"""
from __future__ import annotations

import torch


def unit_range(n_units: int, world: int, rank: int) -> tuple[int, int]:
    """Contiguous balanced split: the first ``n_units % world`` ranks get one unit more."""
    if not (0 <= rank < world):
        raise ValueError("rank out of range")
    base, extra = divmod(n_units, world)
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)


def shard_units(B: int, Hkv: int, world: int, rank: int) -> list[tuple[int, int]]:
    """The (b, kv_head) units of ``rank``; unit u = b * Hkv + kv_head."""
    lo, hi = unit_range(B * Hkv, world, rank)
    return [(u // Hkv, u % Hkv) for u in range(lo, hi)]


def query_heads_of(kv_head: int, Hq: int, Hkv: int) -> range:
    g = Hq // Hkv
    return range(kv_head * g, (kv_head + 1) * g)


def max_over_ranks(value: float, device: torch.device | str = "cpu") -> float:
    """Max of a scalar over all ranks of the default process group (identity without one)."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def run_sharded(Q: torch.Tensor, K: torch.Tensor, V: torch.Tensor, window: int, k_sel: int, fmts, prefill_fn=None,
                out: torch.Tensor | None = None, gather: bool = False, world: int | None = None,
                rank: int | None = None, device: torch.device | str | None = None) -> torch.Tensor:
    """One prefill batch over the ranks of the default process group, head-sharded.

    ``Q [B,Hq,L,D]``, ``K, V [B,Hkv,L,D]`` are the whole batch (every rank holds it, e.g. in host memory).  Each
    rank runs the whole path - select, quantize, fused attention - on its own (batch, KV head) units through
    ``prefill_fn(q, k, v, window, k_sel, fmts) -> out [1,g,L,D]`` (default: the library's ``api.hybrid_prefill`` on
    ``device``) and writes the result into its slices of ``out [B,Hq,L,D]`` (allocated if not given; the slices
    of other ranks are left as they are).  Nothing is exchanged on the data path.  With ``gather=True`` the
    slices are then all-gathered (one plain collective per unit count, padded to the largest share) so that
    every rank ends up with the complete ``out`` - what a tensor-parallel consumer would ask for.

    Returns ``out``.  ``world`` / ``rank`` default to the process group's (1 / 0 without one)."""
    import torch.distributed as dist
    have_pg = dist.is_available() and dist.is_initialized()
    world = (dist.get_world_size() if have_pg else 1) if world is None else world
    rank = (dist.get_rank() if have_pg else 0) if rank is None else rank
    B, Hq, L, D = Q.shape
    Hkv = K.shape[1]
    if prefill_fn is None:
        from . import api
        dev = torch.device("cuda", torch.cuda.current_device()) if device is None else torch.device(device)

        def prefill_fn(q, k_, v, w_, ks_, f_):
            return api.hybrid_prefill(q.to(dev, non_blocking=True), k_.to(dev, non_blocking=True), v.to(dev, non_blocking=True),
                                      w_, ks_, f_)["out"]
    if out is None:
        out = torch.zeros(B, Hq, L, D, dtype=torch.float32, device=Q.device if device is None else device)
    mine = shard_units(B, Hkv, world, rank)
    for b, hk in mine:
        hs = query_heads_of(hk, Hq, Hkv)
        o = prefill_fn(Q[b:b + 1, hs.start:hs.stop].contiguous(), K[b:b + 1, hk:hk + 1].contiguous(),
                       V[b:b + 1, hk:hk + 1].contiguous(), window, k_sel, fmts)
        out[b:b + 1, hs.start:hs.stop].copy_(torch.as_tensor(o).to(out.dtype), non_blocking=True)
    if gather and world > 1:
        g = Hq // Hkv
        n_max = -(-(B * Hkv) // world)
        send = torch.zeros(n_max, g, L, D, dtype=out.dtype, device=out.device)
        for n, (b, hk) in enumerate(mine):
            send[n].copy_(out[b, hk * g:(hk + 1) * g])
        recv = [torch.empty_like(send) for _ in range(world)]
        dist.all_gather(recv, send)
        for r in range(world):
            for n, (b, hk) in enumerate(shard_units(B, Hkv, world, r)):
                out[b, hk * g:(hk + 1) * g].copy_(recv[r][n])
    return out
