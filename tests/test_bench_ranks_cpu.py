"""The multi-rank bookkeeping of bench.py on CPU: two gloo ranks, no GPU.  Every rank runs a
replica (the path shards by rows with no exchange), the job's time is the slowest rank's and
the job's bytes are the sum over the ranks."""
import os
import sys

import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _rank(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    my_ms = 10.0 + 5.0 * rank                    # rank 1 is the slow one
    total = bench.max_over_ranks(my_ms, world)
    out.put((rank, total, bench.whole_job_value(1_000_000_000, 3, world, total)))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_take_the_slowest_time_and_add_the_bytes():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_rank, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, total, value in got:
        assert total == 15.0                      # max over ranks, on every rank
        assert abs(value - 2 * 3 * 1.0 / 15e-3) < 1e-9   # 2 ranks x 3 steps x 1 GB / 15 ms


def test_single_rank_is_the_identity():
    import bench
    assert bench.max_over_ranks(7.5, 1) == 7.5
    assert abs(bench.whole_job_value(2_000_000_000, 10, 1, 20.0) - 1000.0) < 1e-9
