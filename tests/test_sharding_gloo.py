"""The multi-rank path of the benchmark on CPU: two gloo ranks shard the batched workload by instance and reduce
their timings the way bench.py does (MAX of the times, SUM of the counts).  No GPU is involved."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2505_06641_b200 import shard, synth


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _rank_main(rank, world, port, per_rank, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        first, count = shard.instance_shard(rank, world, per_rank)
        w = synth.make_workload("C4", n_instances=count, first_instance=first, n_requests=40)
        # stand-ins for a rank's measurements: a time that differs per rank, and its request / launch counts
        ms, (n_total, launches) = shard.reduce_step_stats(10.0 + rank, [w.n_requests, 7], "cpu")
        dist.barrier()
        out[rank] = dict(first=first, count=count, ms=ms, n_total=n_total, launches=launches,
                         deadline=w.deadline_ns.copy(), feats_sum=float(w.feats.astype(np.float64).sum()))
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_shard_instances_and_reduce_like_the_benchmark():
    world, per_rank = 2, 3
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_rank_main, args=(world, _free_port(), per_rank, out), nprocs=world, join=True)
    res = [out[r] for r in range(world)]
    # disjoint, contiguous instance ranges that cover the job
    assert [(r["first"], r["count"]) for r in res] == [(0, 3), (3, 3)]
    # every rank reports the slowest rank's time and the job-wide totals
    assert all(r["ms"] == 11.0 for r in res)
    assert all(r["n_total"] == 2 * 3 * 40 and r["launches"] == 14 for r in res)
    # the shards are exactly the slices of the one-rank workload with the same global instance numbers
    whole = synth.make_workload("C4", n_instances=world * per_rank, n_requests=40)
    inst = np.asarray(whole.instance)
    for r in range(world):
        sel = (inst >= res[r]["first"]) & (inst < res[r]["first"] + per_rank)
        assert np.array_equal(whole.deadline_ns[sel], res[r]["deadline"])
        assert np.isclose(whole.feats[sel].astype(np.float64).sum(), res[r]["feats_sum"])


def test_single_process_reduction_is_the_identity():
    assert shard.reduce_step_stats(3.5, [4, 5], "cpu") == (3.5, [4, 5])
    assert shard.instance_shard(2, 4, 100) == (200, 100)
