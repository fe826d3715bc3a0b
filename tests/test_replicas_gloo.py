"""The only multi-GPU logic of the benchmark is the replica bookkeeping: N independent replicas,
timing = the slowest rank, throughput = the sum over replicas.  Checked with two gloo ranks on CPU."""
import os
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = bench.max_over_ranks(100.0 + 50.0 * rank, device="cpu")
    out[rank] = (ms, bench.aggregate_images_per_s(64, ms, world))
    dist.barrier()
    dist.destroy_process_group()


def test_two_replicas_report_the_slowest_rank_and_the_sum():
    import socket
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    out = mp.Manager().dict()
    mp.spawn(_worker, args=(2, port, out), nprocs=2, join=True)
    for r in (0, 1):
        ms, ips = out[r]
        assert ms == 150.0                                   # max over ranks, seen by every rank
        assert abs(ips - 2 * 64 / 0.150) < 1e-9              # whole-job images/s of two replicas


def test_single_process_passthrough():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(12.5, device="cpu") == 12.5
    assert bench.aggregate_images_per_s(64, 500.0, 1) == 128.0
