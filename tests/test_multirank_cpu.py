"""The N > 1 path of the benchmark is replicas only (images are independent, no exchange step): each rank
rolls out its own batch, the job's step time is the max over ranks and its throughput the sum of the ranks'
tokens over that time.  Checked here with two gloo ranks on CPU."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    from paper_2608_18183_b200 import synth
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = synth.WORKLOADS["tiny"]
    toks, k, lab = bench.rank_inputs(w, rank)
    tokens_local = int((w.shape.T - k).sum()) + rank  # make the ranks differ
    ms = bench.max_over_ranks(10.0 + 5.0 * rank, dist, "cpu")
    value, total = bench.job_tokens_per_s(tokens_local, 3, dist, "cpu", ms)
    out.put((rank, toks.tobytes(), ms, value, total, tokens_local))
    dist.barrier()
    dist.destroy_process_group()


def test_two_replica_ranks_aggregate_as_a_weak_scaling_job():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, t0, ms0, v0, tot0, n0), (r1, t1, ms1, v1, tot1, n1) = res
    assert t0 != t1                       # each rank has its own batch
    assert ms0 == ms1 == 15.0             # the slowest rank sets the step time
    assert tot0 == tot1 == 3 * (n0 + n1)  # the job's tokens are the sum over ranks
    assert abs(v0 - tot0 / 15e-3) < 1e-6 and v0 == v1


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(7.5, None, "cpu") == 7.5
    v, tot = bench.job_tokens_per_s(100, 4, None, "cpu", 20.0)
    assert tot == 400 and abs(v - 20000.0) < 1e-9
