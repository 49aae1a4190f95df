"""The N>1 plumbing of bench.py with two gloo ranks on CPU: the path shards over the batch (every
rank its own seeded images, weights replicated by construction of the seeds' layer part), has no
data-path collective, and reports whole-job throughput over the slowest rank's time."""
import os
import socket
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import bench
    from paper_2111_00153_b200 import synth
    dist.init_process_group("gloo", rank=rank, world_size=world)
    L = synth.resnet18_convs()[-1]
    W, x = bench.host_layer(3, L, 2, rank)
    local_ms = 10.0 + 5.0 * rank                      # rank 1 is the slow one
    ms = bench.max_over_ranks(local_ms, world, "cpu")
    dist.barrier()
    out[rank] = (float(np.abs(W).sum()), float(x.sum()), ms, bench.whole_job_tops(10 ** 12, world, ms))
    dist.destroy_process_group()


def test_two_ranks_shard_the_batch_and_take_the_slowest_time():
    world = 2
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, _free_port(), out), nprocs=world, join=True)
    (w0, x0, ms0, v0), (w1, x1, ms1, v1) = out[0], out[1]
    assert x0 != x1 and w0 != w1          # every rank draws its own batch (and layer instance)
    assert ms0 == ms1 == 15.0             # max over ranks, seen by both
    assert v0 == v1 == world * 1e12 / 15e-3 / 1e12


def test_single_rank_needs_no_process_group():
    import bench
    assert bench.max_over_ranks(7.0, 1, "cpu") == 7.0
    assert bench.whole_job_tops(2 * 10 ** 12, 1, 1000.0) == 2.0
