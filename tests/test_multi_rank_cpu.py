"""world_size-2 `gloo` test on CPU of the multi-GPU path's host logic (token-sharded replicas, no data-path
collective): ranks evaluate disjoint token shards independently and the gathered result equals the single-rank
result on the whole batch; the job's step time is the max over ranks."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2609_36070_b200 import inputs, sharding
from paper_2609_36070_b200.inputs import MoEConfig


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        from oracle import mok_ref
        cfg = MoEConfig("mr", T=50, H=16, E=6, k=2, I=8, I_s=8, seed=5)
        d = inputs.make_inputs(cfg, threads=1)                   # every rank: the same weights and the same full batch
        b, e = sharding.shard_rows(cfg.T, world, rank)
        x_local = np.ascontiguousarray(d["x"][b:e])
        out_local, idx_local, _ = mok_ref.forward(x_local, d["W_r"], None, d["W_gate_up"], d["W_down"], d["W_sgu"],
                                                  d["W_sd"], cfg.k)
        gathered = [None] * world
        dist.all_gather_object(gathered, (b, e, out_local))
        ms = sharding.max_over_ranks(10.0 + 5.0 * rank, dist)     # rank 1 is the slow one
        dist.barrier()
        if rank == 0:
            full, _, _ = mok_ref.forward(d["x"], d["W_r"], None, d["W_gate_up"], d["W_down"], d["W_sgu"], d["W_sd"], cfg.k)
            ok = all(np.array_equal(full[bb:ee], oo) for bb, ee, oo in gathered)
            covered = sorted((bb, ee) for bb, ee, _ in gathered)
            q.put((ok, covered, ms, sharding.aggregate_tokens_per_s(cfg.T, world, ms)))
        # per-rank token streams of the weak-scaling benchmark differ between ranks and are reproducible
        x_r = sharding.rank_tokens(cfg, rank)
        assert np.array_equal(x_r, sharding.rank_tokens(cfg, rank))
        if rank > 0:
            assert not np.array_equal(x_r, d["x"])
    finally:
        dist.destroy_process_group()


def test_token_sharded_replicas_need_no_exchange():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.SimpleQueue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(120)
        assert p.exitcode == 0
    ok, covered, ms, value = q.get()
    assert ok                                                     # shards, evaluated independently, reproduce the whole batch
    assert covered == [(0, 25), (25, 50)]
    assert ms == 15.0                                             # the slowest rank sets the step time
    assert value == 2 * 50 / 15e-3


def test_shard_rows_partition():
    for total, world in [(10, 3), (7, 7), (5, 8), (16384, 4)]:
        spans = [sharding.shard_rows(total, world, r) for r in range(world)]
        assert spans[0][0] == 0 and spans[-1][1] == total
        assert all(a[1] == b[0] for a, b in zip(spans, spans[1:]))
        sizes = [e - b for b, e in spans]
        assert max(sizes) - min(sizes) <= 1
