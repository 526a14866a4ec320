"""bench.py --gpus N runs N independent replicas (no data-path collective): the whole-job value is all
ranks' tokens over the slowest rank's time. Checked with two gloo ranks on CPU."""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    seconds, units = (2.0, 100.0) if rank == 0 else (3.0, 140.0)     # rank 1 is slower and emitted more
    t, u = bench.aggregate_replicas(seconds, units, world)
    out[rank] = (t, u)
    dist.destroy_process_group()


def test_two_gloo_ranks_max_time_sum_tokens():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    out = mp.Manager().dict()
    mp.spawn(_worker, args=(2, port, out), nprocs=2, join=True)
    assert out[0] == out[1] == (3.0, 240.0)


def test_single_rank_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.aggregate_replicas(1.5, 7, 1) == (1.5, 7.0)
