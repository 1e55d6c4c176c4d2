"""N > 1 on CPU: two gloo ranks shard the requests of one workload (no collective on the data path), run
the oracle on their shards, and the aggregate equals the single-process result."""
import os
import socket
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def run_shard(w_args, requests, steps):
    """Oracle over the given requests of the workload; returns (hits + misses, misses, per-request misses)."""
    sys.path.insert(0, ROOT)
    from oracle import Oracle, FLAG_NO_BYTES
    from paper_2608_07009_b200 import inputs
    w = inputs.c2_dsa_decode(**w_args)
    N = w.num_requests
    tr = inputs.Trace(w)                       # every rank draws the full trace and keeps its rows
    orcs = {r: Oracle(1, w.num_layers, 1, w.cache_slots, w.top_k, w.entry_bytes, [w.capacity[r]], [w.init_len[r]],
                      None, FLAG_NO_BYTES) for r in requests}
    total, miss, per_req = 0, 0, {r: 0 for r in requests}
    for _ in range(steps):
        sel, appended, _ = tr.step()
        for r in requests:
            if appended:
                orcs[r].append()
            for layer in range(w.num_layers):
                _, h, m = orcs[r].resolve(layer, sel[layer, r][None])
                total += int(h[0]) + int(m[0])
                miss += int(m[0])
                per_req[r] += int(m[0])
    tr.close()
    return total, miss, per_req


W_ARGS = dict(num_requests=5, num_layers=2, steps=6, context=3000)
STEPS = 6


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    from paper_2608_07009_b200 import sharding
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    mine = sharding.requests_of_rank(W_ARGS["num_requests"], world, rank)
    total, miss, _ = run_shard(W_ARGS, mine, STEPS)
    elapsed = 1.0 + rank                        # stand-in for a device time: the slowest rank must win
    t_max, total_all = sharding.aggregate(elapsed, total)
    _, miss_all = sharding.aggregate(elapsed, miss)
    if rank == 0:
        out.put((mine, t_max, total_all, miss_all))
    else:
        out.put((mine, None, None, None))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_shard_requests_and_aggregate():
    sys.path.insert(0, ROOT)
    from paper_2608_07009_b200 import sharding
    world = 2
    shards = [sharding.requests_of_rank(5, world, r) for r in range(world)]
    assert sorted(sum(shards, [])) == list(range(5)) and not set(shards[0]) & set(shards[1])
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    results = [out.get(timeout=120) for _ in range(world)]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    agg = [x for x in results if x[1] is not None][0]
    total_ref, miss_ref, _ = run_shard(W_ARGS, list(range(5)), STEPS)
    assert agg[1] == 2.0                         # max over ranks
    assert agg[2] == total_ref and agg[3] == miss_ref
    assert total_ref == STEPS * 5 * 2 * 2048
