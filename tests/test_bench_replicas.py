"""bench.py at N > 1 runs N independent replicas (the path has no exchange step): the only
cross-rank logic is the barrier and the max-over-ranks of the timings.  Checked here with two
gloo ranks on CPU."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank_main(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    mine = 10.0 + 5.0 * rank            # rank 1 is the slow replica
    dist.barrier()
    slowest = bench.max_over_ranks(mine, world, torch.device("cpu"))
    value = bench.whole_job_tokens_per_s(8, 16, world, slowest / 1e3)
    out.put((rank, slowest, value))
    dist.destroy_process_group()


def test_two_replicas_report_the_slowest_time_and_the_whole_job():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, slowest, value in res:
        assert slowest == 15.0                        # every rank sees the max
        assert abs(value - 2 * 8 * 16 / 0.015) < 1e-6  # both replicas' tokens over the slowest replica's time


def test_single_rank_is_the_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5, 1, torch.device("cpu")) == 3.5
    assert bench.whole_job_tokens_per_s(8, 16, 1, 0.5) == 256.0
