"""The multi-GPU layout of the path, checked on CPU with a world-size-2 gloo group: every (batch, KV head)
unit lands on exactly one rank, the shards reproduce the unsharded result with no exchange, and the
reported time is the max over ranks."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_2608_27875_b200 import sharding, workloads as wl


def test_unit_ranges_partition_the_units():
    for n in (1, 7, 8, 32, 33):
        for world in (1, 2, 3, 8):
            ranges = [sharding.unit_range(n, world, r) for r in range(world)]
            assert ranges[0][0] == 0 and ranges[-1][1] == n
            assert all(a[1] == b[0] for a, b in zip(ranges, ranges[1:]))
            sizes = [hi - lo for lo, hi in ranges]
            assert max(sizes) - min(sizes) <= 1
    assert sharding.shard_units(2, 3, 2, 1) == [(1, 0), (1, 1), (1, 2)]
    assert list(sharding.query_heads_of(2, 12, 4)) == [6, 7, 8]
    with pytest.raises(ValueError):
        sharding.unit_range(4, 2, 2)


W = wl.CONFIGS["c0"].scaled(B=2, Hq=6, Hkv=3, L=192, window=32, k=6, n_plant=4, seed=77)
ROWS = np.array([0, 31, 32, 100, 191], dtype=np.int32)


def _unit_result(b, kvh):
    """Oracle result of one (b, kv head) unit computed from that unit's tensors alone."""
    Q, K, V = wl.make_inputs(W.scaled(B=b + 1), heads=[kvh])
    Q, K, V = Q[b:b + 1], K[b:b + 1], V[b:b + 1]
    r = oracle.hybrid_prefill(wl.bits(Q), wl.bits(K), wl.bits(V), W.window, W.k, W.fmts, rows=ROWS)
    return r["idx"][0], r["out"][0]


def _worker(rank, world, port, ret):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        g = W.Hq // W.Hkv
        mine = {}
        for b, kvh in sharding.shard_units(W.B, W.Hkv, world, rank):
            mine[(b, kvh)] = _unit_result(b, kvh)
        gathered = [None] * world
        dist.all_gather_object(gathered, mine)           # reporting only: the data path exchanged nothing
        t_max = sharding.max_over_ranks(10.0 + rank)
        if rank == 0:
            full = {}
            for part in gathered:
                assert not (set(part) & set(full))         # every unit on exactly one rank
                full.update(part)
            idx = np.zeros((W.B, W.Hq, W.k), dtype=np.int32)
            out = np.zeros((W.B, W.Hq, len(ROWS), W.D))
            for (b, kvh), (i_, o_) in full.items():
                idx[b, kvh * g:(kvh + 1) * g] = i_
                out[b, kvh * g:(kvh + 1) * g] = o_
            ret["idx"], ret["out"], ret["t_max"], ret["n_units"] = idx, out, t_max, len(full)
    finally:
        dist.destroy_process_group()


def test_two_ranks_reproduce_the_unsharded_result():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ret = mp.Manager().dict()
    mp.spawn(_worker, args=(2, port, ret), nprocs=2, join=True)
    Q, K, V = wl.make_inputs(W)
    ref = oracle.hybrid_prefill(wl.bits(Q), wl.bits(K), wl.bits(V), W.window, W.k, W.fmts, rows=ROWS)
    assert ret["n_units"] == W.B * W.Hkv
    np.testing.assert_array_equal(ret["idx"], ref["idx"])
    np.testing.assert_allclose(ret["out"], ref["out"], rtol=0, atol=1e-13)
    assert ret["t_max"] == 11.0                            # max over ranks of (10, 11)


# ---- the wrapper the product uses (sharding.run_sharded), with the oracle standing in for the device calls ---------
def _oracle_prefill(q, k, v, window, k_sel, fmts):
    r = oracle.hybrid_prefill(wl.bits(q), wl.bits(k), wl.bits(v), window, k_sel, fmts)
    return torch.from_numpy(r["out"])


def _wrapper_worker(rank, world, port, ret):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        Q, K, V = wl.make_inputs(W)
        own = sharding.run_sharded(Q, K, V, W.window, W.k, W.fmts, prefill_fn=_oracle_prefill,
                                   out=torch.zeros(W.B, W.Hq, W.L, W.D, dtype=torch.float64))
        full = sharding.run_sharded(Q, K, V, W.window, W.k, W.fmts, prefill_fn=_oracle_prefill,
                                    out=torch.zeros(W.B, W.Hq, W.L, W.D, dtype=torch.float64), gather=True)
        ret[rank] = (own.numpy(), full.numpy())
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("world", [2, 3])
def test_run_sharded_fills_each_ranks_slices_and_gathers_the_whole_output(world):
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ret = mp.Manager().dict()
    mp.spawn(_wrapper_worker, args=(world, port, ret), nprocs=world, join=True)
    Q, K, V = wl.make_inputs(W)
    ref = oracle.hybrid_prefill(wl.bits(Q), wl.bits(K), wl.bits(V), W.window, W.k, W.fmts)["out"]
    g = W.Hq // W.Hkv
    for rank in range(world):
        own, full = ret[rank]
        np.testing.assert_allclose(full, ref, rtol=0, atol=1e-13)               # after the gather: everything, everywhere
        mask = np.zeros((W.B, W.Hq), dtype=bool)
        for b, kvh in sharding.shard_units(W.B, W.Hkv, world, rank):
            mask[b, kvh * g:(kvh + 1) * g] = True
        np.testing.assert_allclose(own[mask], ref[mask], rtol=0, atol=1e-13)    # without it: the rank's own slices ...
        assert not own[~mask].any()                                             # ... and nothing else touched
    # without a process group the wrapper runs every unit itself
    solo = sharding.run_sharded(Q, K, V, W.window, W.k, W.fmts, prefill_fn=_oracle_prefill,
                                out=torch.zeros(W.B, W.Hq, W.L, W.D, dtype=torch.float64))
    np.testing.assert_allclose(solo.numpy(), ref, rtol=0, atol=1e-13)


# ---- the decode side shards by the same (batch, KV head) units ------------------------------------------------
def _decode_inputs():
    g = torch.Generator().manual_seed(91)
    B, Hq, Hkv, N, D = 2, 6, 3, 150, 16
    k = torch.randn(B, Hkv, N, D, generator=g).to(torch.bfloat16)
    v = torch.randn(B, Hkv, N, D, generator=g).to(torch.bfloat16)
    q = torch.randn(B, Hq, D, generator=g).to(torch.bfloat16)
    rng = np.random.default_rng(92)
    idx = np.stack([np.stack([np.sort(rng.choice(N - 20, 7, replace=False)) for _ in range(Hkv)]) for _ in range(B)]).astype(np.int32)
    return q, k, v, idx


def _decode_worker(rank, world, port, ret):
    from oracle import decode as od
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        q, k, v, idx = _decode_inputs()
        g = q.shape[1] // k.shape[1]
        mine = {}
        for b, kvh in sharding.shard_units(k.shape[0], k.shape[1], world, rank):
            # Freeze and one token on this unit's tensors alone
            cache = od.freeze(wl.bits(k[b:b + 1, kvh:kvh + 1]), wl.bits(v[b:b + 1, kvh:kvh + 1]), idx[b:b + 1, kvh:kvh + 1], 20, group=16)
            out, _ = od.decode_attention(wl.bits(q[b:b + 1, kvh * g:(kvh + 1) * g]), cache)
            mine[(b, kvh)] = out[0]
        gathered = [None] * world
        dist.all_gather_object(gathered, mine)
        if rank == 0:
            full = {}
            for part in gathered:
                assert not (set(part) & set(full))
                full.update(part)
            out = np.zeros((q.shape[0], q.shape[1], q.shape[2]))
            for (b, kvh), o_ in full.items():
                out[b, kvh * g:(kvh + 1) * g] = o_
            ret["out"], ret["n_units"] = out, len(full)
    finally:
        dist.destroy_process_group()


def test_two_ranks_reproduce_the_unsharded_decode_step():
    from oracle import decode as od
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ret = mp.Manager().dict()
    mp.spawn(_decode_worker, args=(2, port, ret), nprocs=2, join=True)
    q, k, v, idx = _decode_inputs()
    ref, _ = od.decode_attention(wl.bits(q), od.freeze(wl.bits(k), wl.bits(v), idx, 20, group=16))
    assert ret["n_units"] == k.shape[0] * k.shape[1]
    np.testing.assert_allclose(ret["out"], ref, rtol=0, atol=1e-13)
