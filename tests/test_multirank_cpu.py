"""The N > 1 path on CPU: two gloo ranks.  The layer shards by token with no exchange (replicas), so the
only cross-rank step is the reduction of the timing into a whole-job throughput; ranks that shard a batch
must also reproduce the single-rank result row for row (checked here on the oracle, which is what a rank
without a GPU can run)."""
import os
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    import dsmoe_inputs as gi
    import oracle
    # timing reduction: the job is as slow as its slowest rank, tokens add up
    value, ms, n = bench.job_throughput(dist, 10.0 * (rank + 1), 1000, device="cpu")
    # token sharding: each rank evaluates its own slice of the batch with replicated weights
    s = gi.LayerSpec("mr", T=12, d=32, H=16, E=4, dtype="bf16", mode=gi.MODE_TOPK, K=2)
    x, (Wr, br), (W1, W2) = gi.tokens(s), gi.router(s), gi.experts(s)
    lo, hi = rank * s.T // world, (rank + 1) * s.T // world
    S = oracle.router_scores(x[lo:hi], Wr, br)
    mask, _ = oracle.select(S, s.mode, K=s.K)
    part = oracle.layer(x[lo:hi], W1, W2, S, mask)
    gathered = [None] * world
    dist.all_gather_object(gathered, part)          # test-side check only, not part of the data path
    q.put((rank, value, ms, n, np.concatenate(gathered)))
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_shard_by_token_and_reduce_the_timing():
    world, port = 2, 29000 + os.getpid() % 2000
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    got = [q.get(timeout=120) for _ in range(world)]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    sys.path.insert(0, ROOT)
    import dsmoe_inputs as gi
    import oracle
    s = gi.LayerSpec("mr", T=12, d=32, H=16, E=4, dtype="bf16", mode=gi.MODE_TOPK, K=2)
    x, (Wr, br), (W1, W2) = gi.tokens(s), gi.router(s), gi.experts(s)
    S = oracle.router_scores(x, Wr, br)
    mask, _ = oracle.select(S, s.mode, K=s.K)
    full = oracle.layer(x, W1, W2, S, mask)
    for rank, value, ms, n, joined in got:
        assert n == 2 and ms == 20.0                       # max over ranks
        assert value == pytest.approx(2000 / 20e-3)        # all tokens over the slowest rank's time
        assert np.array_equal(joined, full)                # sharding by token changes nothing


def test_bench_gpus_2_starts_two_ranks_itself():
    """`bench.py --gpus 2` outside torchrun starts its own ranks; --rendezvous-only runs that launch path, the
    process group (gloo here, NCCL on GPUs) and the timing reduction without any GPU work."""
    import json
    import subprocess
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    env["CUDA_VISIBLE_DEVICES"] = ""                        # the CPU path, also on a box with GPUs
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--rendezvous-only"],
                       capture_output=True, text=True, timeout=300, env=env)
    assert r.returncode == 0, r.stderr[-2000:]
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["n_gpus"] == 2 and line["backend"] == "gloo"
    assert line["ms_per_step"] == 20.0 and line["value"] == pytest.approx(2000 / 20e-3)
