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


def _oracle_selections(bench, args, rank):
    """What rank `rank` of bench.py's multi-rank job resolves: its own workload (bench.make_workload), by the oracle."""
    from oracle import Oracle, FLAG_NO_BYTES
    from paper_2608_07009_b200 import inputs
    w = bench.make_workload(args, rank, steps=args.steps + 1)
    orc = Oracle(w.num_requests, w.num_layers, w.layers_per_group, w.cache_slots, w.top_k, w.entry_bytes, w.capacity,
                 w.init_len, None, FLAG_NO_BYTES)
    tr = inputs.Trace(w)
    n, first = 0, None
    for _ in range(args.steps):
        sel, appended, _ = tr.step()
        if first is None:
            first = [int(x) for x in sel[0][0][:4]]
        if appended:
            orc.append()
        for layer in range(w.num_layers):
            _, h, m = orc.resolve(layer, sel[layer // w.layers_per_group])
            n += int(h.sum()) + int(m.sum())
    tr.close()
    orc.close()
    return n, first


def test_bench_gpus_flag_starts_that_many_ranks():
    """`bench.py --gpus 2` without a launcher must start two ranks itself (never run one rank in their place): here
    with the oracle as the per-rank worker and gloo in place of NCCL, through the same make_workload / aggregate
    calls as the GPU arm."""
    import json
    import subprocess
    sys.path.insert(0, ROOT)
    import bench
    argv = ["--impl", "sharding-dry-run", "--gpus", "2", "--workload", "c2", "--requests", "3", "--layers", "2",
            "--context", "2000", "--steps", "3"]
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK")}
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py")] + argv, env=env, capture_output=True, text=True,
                         timeout=300)
    assert out.returncode == 0, out.stderr[-2000:]
    line = json.loads([ln for ln in out.stdout.splitlines() if ln.startswith("{")][-1])
    args = bench.parse_args(argv)
    want = [_oracle_selections(bench, args, r) for r in range(2)]
    assert line["n_gpus"] == 2
    assert line["selections"] == want[0][0] + want[1][0] and line["selections_rank0"] == want[0][0]
    assert line["first_rows"] == [want[0][1], want[1][1]] and want[0][1] != want[1][1]   # every rank serves its own requests
    assert line["config"]["num_requests"] == 3 and line["config"]["num_layers"] == 2


def test_bench_refuses_more_gpus_than_there_are():
    import subprocess
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK")}
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "64", "--steps", "1"], env=env,
                         capture_output=True, text=True, timeout=300)
    assert out.returncode != 0 and "--gpus 64" in out.stderr and not out.stdout.strip()


def test_cpu_list_parsing_for_numa_binding():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.parse_cpulist("0-3,8,10-11\n") == {0, 1, 2, 3, 8, 10, 11}
    assert bench.parse_cpulist("") == set()
