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
