"""The N > 1 path of the benchmark is N independent replicas; what crosses ranks is only the
timing reduction.  Run it on CPU with two gloo ranks."""
import os
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
    ms_local = 100.0 if rank == 0 else 250.0            # rank 1 is the slow replica
    dist.barrier()
    ms, value = bench.replicas_throughput(ms_local, steps=5, world=world, device="cpu")
    out.put((rank, ms, value))
    dist.barrier()
    dist.destroy_process_group()


def test_replica_throughput_uses_the_slowest_rank():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ms, value in got:
        assert ms == 250.0                                 # max over ranks
        assert abs(value - 2 * 5 / 0.25) < 1e-9            # both replicas' epochs over the slowest time


def test_single_rank_is_a_plain_ratio():
    sys.path.insert(0, ROOT)
    import bench
    ms, value = bench.replicas_throughput(200.0, steps=4, world=1, device="cpu")
    assert ms == 200.0 and abs(value - 20.0) < 1e-12
