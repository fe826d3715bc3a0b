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


def test_bench_starts_its_own_replicas_when_no_launcher_did():
    """`python bench.py --gpus 2` with no WORLD_SIZE in the environment starts two rank processes itself
    (checked on the reference arm, which needs no GPU: rank 0 alone works and prints, rank 1 exits 0)."""
    import json
    import os
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK")}
    r = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--gpus", "2", "--impl", "reference", "--config", "tiny",
                        "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [ln for ln in r.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["n_gpus"] == 2 and d["value"] > 0
