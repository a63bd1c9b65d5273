"""N>1 path on CPU: two gloo ranks shard the independent units with no data-path collective."""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    from oracle import cask_oracle as orc
    from paper_2604_10900_b200 import workloads as wl
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = wl.WORKLOADS["tiny"].with_(layers=3, kv_heads=2, decode=300)
    units = wl.unit_list(w)
    mine = wl.shard_units(units, rank, world)
    gathered = [None] * world
    dist.all_gather_object(gathered, mine)
    # each rank runs the event on its shard only
    hb = wl.make_batch(w, mine, threads=1)
    o = orc.event_batch(hb.k, hb.v, hb.q, hb.tok_off, hb.P, hb.B, hb.reserve)
    tokens = torch.tensor([float(hb.T.sum())], dtype=torch.float64)
    dist.all_reduce(tokens, op=dist.ReduceOp.SUM)
    t = torch.tensor([1.0 + rank], dtype=torch.float64)       # a stand-in for this rank's device time
    dist.barrier()
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    if rank == 0:
        q.put(dict(gathered=gathered, tokens=tokens.item(), tmax=t.item()))
    q.put(dict(rank=rank, units=mine, n_out=o["n_out"].tolist(), kind=o["kind"].tolist()))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_shard_units_without_exchange():
    sys.path.insert(0, ROOT)
    from oracle import cask_oracle as orc
    from paper_2604_10900_b200 import workloads as wl
    orc.lib()                                   # build the oracle once, before the ranks race for it
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    msgs = [q.get(timeout=120) for _ in range(world + 1)]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    head = next(m for m in msgs if "gathered" in m)
    per_rank = sorted((m for m in msgs if "rank" in m), key=lambda m: m["rank"])
    w = wl.WORKLOADS["tiny"].with_(layers=3, kv_heads=2, decode=300)
    units = wl.unit_list(w)
    assert [u for part in head["gathered"] for u in part] == units          # disjoint cover, order kept
    assert head["tmax"] == 2.0                                               # max over ranks
    assert head["tokens"] == float(len(units) * (w.prefix + 300))           # whole-job token count
    # the shards together give exactly what one process computes for all units
    hb = wl.make_batch(w, units, threads=1)
    full = orc.event_batch(hb.k, hb.v, hb.q, hb.tok_off, hb.P, hb.B, hb.reserve)
    assert sum((m["n_out"] for m in per_rank), []) == full["n_out"].tolist()
    assert sum((m["kind"] for m in per_rank), []) == full["kind"].tolist()


def test_weak_scaling_ranks_get_distinct_sequences():
    sys.path.insert(0, ROOT)
    from paper_2604_10900_b200 import workloads as wl
    w = wl.WORKLOADS["reasoning8k_b384"].with_(layers=1, kv_heads=1, decode=64, prefix=16)
    k0, _, _ = wl.make_unit(w, 0, 0, 0)
    k1, _, _ = wl.make_unit(w, 1, 0, 0)
    assert k0.shape == k1.shape and not np.array_equal(k0, k1)
