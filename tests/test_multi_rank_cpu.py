"""The N>1 plumbing of bench.py with two gloo ranks on CPU: the path shards over the batch (every
rank its own seeded images, the weights seeded by layer only and therefore replicated), has no
data-path collective, and reports whole-job throughput over the slowest rank's time."""
import json
import os
import socket
import subprocess
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
    assert x0 != x1 and w0 == w1          # every rank draws its own batch; the weights are replicated
    assert ms0 == ms1 == 15.0             # max over ranks, seen by both
    assert v0 == v1 == world * 1e12 / 15e-3 / 1e12


def test_single_rank_needs_no_process_group():
    import bench
    assert bench.max_over_ranks(7.0, 1, "cpu") == 7.0
    assert bench.whole_job_tops(2 * 10 ** 12, 1, 1000.0) == 2.0


def test_gpus_flag_starts_the_ranks_itself():
    """`bench.py --gpus 2` without a launcher's environment re-executes itself as two ranks; in the
    GPU-free self-check mode the ranks report replicated weights, distinct batches and the slowest time."""
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--check-ranks"],
                       env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stderr[-2000:]
    line = [l for l in r.stdout.splitlines() if l.startswith("{")][-1]
    out = json.loads(line)
    assert out["n_ranks"] == 2 and out["weights_replicated"] and out["inputs_differ"]
    assert out["max_ms"] == 15.0 and out["whole_job_tops_at_1e12_ops"] == 2 * 1e12 / 15e-3 / 1e12
