"""World-size-2 gloo test of the multi-GPU host logic (batch-sharded replicas: rank-specific
batches, barrier, max over ranks, aggregate throughput).  Runs on CPU."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2312_07987_b200 import inputs, sharding


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    cfg = inputs.CONFIGS["tiny_f32"]
    inp = inputs.make_inputs(cfg)
    xb = sharding.rank_batch(inp.x, rank)
    # every rank keeps the same multiset of token rows (so the same gate margins), in its own order
    same_rows = np.array_equal(np.sort(xb.reshape(-1, cfg.d_model), axis=0), np.sort(inp.x.reshape(-1, cfg.d_model), axis=0))
    dist.barrier()
    my_ms = 10.0 + 5.0 * rank                       # pretend device time of this rank
    worst, = sharding.max_over_ranks([my_ms])
    value = sharding.aggregate_throughput(cfg.n_tokens, world, worst * 1e-3)
    gathered = [None] * world
    dist.all_gather_object(gathered, (float(xb.sum()), bool(np.array_equal(xb, inp.x))))
    if rank == 0:
        out.put(dict(worst=worst, value=value, same_rows=same_rows, gathered=gathered))
    elif not same_rows:
        raise AssertionError("rank batch changed the token rows")
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_replicas_on_gloo():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = out.get(timeout=120)
    for p in procs:
        p.join(timeout=120)
        assert p.exitcode == 0
    assert res["worst"] == 15.0                      # max over ranks, not rank 0's own time
    assert abs(res["value"] - 2 * 64 / 15e-3) < 1e-6  # units of all ranks over the slowest time
    assert res["same_rows"]
    (s0, id0), (s1, id1) = res["gathered"]
    assert id0 and not id1                           # rank 0 keeps x, rank 1 gets its own order
    assert abs(s0 - s1) < 1e-3


def test_max_over_ranks_without_process_group_is_identity():
    assert sharding.max_over_ranks([1.5, 2.5]) == [1.5, 2.5]
