"""The N > 1 path of bench.py is 'replicas only': no data-path collective, only a barrier and a
max-over-ranks of the timings.  Exercised here with two gloo ranks on CPU."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    mine = [10.0 + rank, 30.0 - 5 * rank]          # rank 0: (10, 30)   rank 1: (11, 25)
    dist.barrier()
    red = bench.max_over_ranks(mine)
    value = bench.whole_job_throughput(16, 100, world, red[0])
    out.put((rank, red, value))
    dist.destroy_process_group()


def test_two_gloo_ranks_agree_on_max_time_and_aggregate_rate():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, red, value in res:
        assert red == [11.0, 30.0]                              # slowest rank per timing, same on every rank
        assert abs(value - 2 * 16 * 100 / 11e-3) < 1e-6        # all ranks' tokens over the slowest rank's time


def test_single_rank_is_identity():
    import bench
    assert bench.max_over_ranks([3.5, 4.0]) == [3.5, 4.0]
    assert bench.whole_job_throughput(16, 10, 1, 2.0) == 16 * 10 / 2e-3
