"""Host side of the multi-GPU path on CPU: two gloo ranks.

The path shards without any exchange of data (every batch element, KV-head group and layer is
independent), so `bench.py --gpus N` runs N replicas; what the ranks share is a barrier, the
maximum of their device times and rank 0's report.  These tests run that logic as two
processes over gloo."""
import os
import socket
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import bench
    from paper_2507_19608_b200 import workloads as WL
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        # every rank draws its own replica of the workload
        w = WL.Workload("t", 1, 2, 1, 64, 64, "bf16", 0.95, 0.5, 16, (), 2000)
        q = WL.make_qkv(w, layer=bench.replica_layer(rank), n_decode=0)["q"]
        digests = [None] * world
        dist.all_gather_object(digests, float(np.abs(q).sum()))
        # the job's step time is the slowest rank's
        mine = 10.0 + 5.0 * rank
        dist.barrier()
        slowest = bench.max_over_ranks(mine, dist, "cpu")
        dist.barrier()
        if rank == 0:
            out.put((digests, slowest, bench.job_value(world, w.B * w.T, slowest)))
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_are_independent_replicas_timed_by_the_slowest():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.SimpleQueue()
    procs = [ctx.Process(target=_rank_main, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(120)
        assert p.exitcode == 0
    digests, slowest, value = out.get()
    assert digests[0] != digests[1]                    # different seeds: no rank repeats another's work
    assert slowest == 15.0                             # max over ranks, not rank 0's own 10.0
    assert abs(value - 2 * 64 / 15e-3) < 1e-6          # whole-job tokens/s over the slowest rank's time


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5, None, "cpu") == 3.5
    assert bench.job_value(1, 1024, 0.05) == 1024 / 0.05e-3
