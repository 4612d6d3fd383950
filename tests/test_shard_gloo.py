"""Multi-rank host logic on CPU (gloo, world_size 2): token sharding covers the batch exactly once,
ranks draw distinct synthetic batches, the elapsed-time reduction is a MAX, and sharded oracle runs
reassemble to the unsharded result (tokens are independent: no data-path collective is needed)."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2604_14156_b200 import shard


def test_token_slices_partition_the_batch():
    for n in (1, 2, 7, 64, 65):
        for world in (1, 2, 3, 8):
            cover = []
            for r in range(world):
                b, e = shard.token_slice(n, world, r)
                cover += list(range(b, e))
            assert cover == list(range(n))
            sizes = [shard.token_slice(n, world, r)[1] - shard.token_slice(n, world, r)[0] for r in range(world)]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        shard.token_slice(4, 2, 2)
    assert len({shard.batch_stream(r, j, 16) for r in range(4) for j in range(16)}) == 64


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, q):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        import oracle
        from gen import workloads as W
        cfg = W.CONFIGS["tiny_f32"].with_(B=7)
        L = W.make_layer(cfg)
        x = W.make_tokens(cfg, L.A).h
        b, e = shard.token_slice(cfg.B, world, rank)
        local = oracle.layer_step(L, x[b:e], group=cfg.group, k=cfg.k, T=cfg.T)
        full = shard.gather_rows(torch.from_numpy(local.x_out), cfg.B).numpy()
        sup = shard.gather_rows(torch.from_numpy(local.support.astype(np.int64)), cfg.B).numpy()
        elapsed = shard.max_over_ranks(1.0 + rank)   # slowest rank decides
        dist.barrier()
        if rank == 0:
            ref = oracle.layer_step(L, x, group=cfg.group, k=cfg.k, T=cfg.T)
            q.put((bool(np.array_equal(full, ref.x_out)), bool(np.array_equal(sup, ref.support)), elapsed))
    finally:
        dist.destroy_process_group()


def test_sharded_step_reassembles_and_time_is_max_over_ranks():
    import oracle
    oracle.build()
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    same_out, same_sup, elapsed = q.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert same_out and same_sup
    assert elapsed == 2.0
