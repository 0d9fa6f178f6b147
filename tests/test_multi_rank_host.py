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


def test_bench_starts_its_own_ranks_when_asked_for_several_gpus():
    """`python bench.py --gpus 2` without a torchrun environment re-launches itself as two ranks
    (torch.distributed.run, rendezvous on 127.0.0.1).  The reference arm needs no GPU, so the
    launcher path runs here: rank 0 alone prints the line, the other rank exits 0."""
    import json
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    res = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--gpus", "2", "--impl", "reference",
                          "--config", "tiny_f32", "--steps", "2", "--warmup", "0"],
                         capture_output=True, text=True, timeout=300, env=env, cwd=root)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [l for l in res.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1, res.stdout
    rec = json.loads(lines[0])
    assert rec["impl"] == "reference" and rec["n_gpus"] == 2
    assert rec["config"]["workload"] == "tiny_f32" and rec["config"]["batch_per_gpu"] == 1
