"""Multi-rank host logic on CPU: world_size-2 gloo ranks shard a prompt batch, predict, gather.

The per-rank compute is the oracle (there is no GPU here); what is under test is the partition,
the packing of each rank's prompts, the gather back into global prompt order and the
max-over-ranks / sum-over-ranks reduction the benchmark uses.
"""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2602_11812_b200 import inputs as gen
from paper_2602_11812_b200 import shard


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, q):
    from oracle import egtp_oracle as orc
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        wl = gen.config_mid(V=96, d=32, m_h=16, B=11, max_len=64)
        parts = shard.partition_prompts(wl.lengths, world)
        mine = parts[rank]
        rows, off = shard.local_batch(wl.hidden, wl.offsets, mine)
        y = orc.egtp_predict(rows, off, wl.W, wl.head)["yhat"] if len(mine) else np.zeros(0)
        y_all = shard.gather_predictions(torch.from_numpy(y.astype(np.float32)), mine, wl.B)
        t_max, units = shard.reduce_time_and_work(10.0 + rank, float(rows.shape[0]), torch.device("cpu"))
        # the vocabulary-parallel exchange: every rank contributes a [rows, 3] block, all ranks receive all blocks
        part = torch.full((5, 3), float(rank), dtype=torch.float32) + torch.arange(15, dtype=torch.float32).reshape(5, 3)
        gathered = shard.all_gather_partials(part)
        g_ok = gathered.shape == (world, 5, 3) and all(bool(torch.equal(gathered[r], part - rank + r)) for r in range(world))
        if rank == 0:
            ref = orc.egtp_predict(wl.hidden, wl.offsets, wl.W, wl.head)["yhat"]
            q.put(dict(ok=bool(np.allclose(y_all.numpy(), ref, rtol=1e-6, atol=1e-6)) and g_ok, t_max=t_max, units=units,
                       T=wl.T))
    finally:
        dist.destroy_process_group()


def test_partition_is_balanced_and_complete():
    lengths = gen.lengths_pareto(3, 64, 1.2, 128, 128, 8192)
    for world in (1, 2, 3, 8):
        parts = shard.partition_prompts(lengths, world)
        assert sorted(np.concatenate(parts).tolist()) == list(range(64))
        loads = [int(lengths[p].sum()) for p in parts]
        assert max(loads) - min(loads) <= int(lengths.max())         # LPT bound
    assert [p.tolist() for p in shard.partition_prompts([5, 5, 5], 2)] == [[0, 2], [1]]
    assert shard.vocab_shards(151936, 4) == [(0, 37888), (37888, 76032), (76032, 113920), (113920, 151936)]
    assert shard.vocab_shards(100, 3, multiple=256) == [(0, 0), (0, 0), (0, 100)]
    rows, off = shard.local_batch(np.arange(20).reshape(10, 2), np.array([0, 3, 4, 10]), np.array([2, 0]))
    assert off.tolist() == [0, 6, 9] and rows[:, 0].tolist() == [8, 10, 12, 14, 16, 18, 0, 2, 4]


@pytest.mark.timeout(180)
def test_two_gloo_ranks_shard_predict_gather():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = q.get(timeout=150)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert res["ok"] and res["t_max"] == 11.0 and res["units"] == res["T"]
