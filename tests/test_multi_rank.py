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


def test_bench_gpus_flag_starts_the_ranks_itself():
    """`python bench.py --gpus 2` with no launcher environment must start two ranks (not one rank that reports
    n_gpus = 1).  Driven through the file's real entry point with the CPU stand-in step (--op plumbing, gloo): rank r
    sleeps (1 + r) ms per step, so the reported time must be the slower rank's and the rate both ranks' units over it."""
    import json
    import subprocess
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--op", "plumbing", "--steps", "30",
                        "--tokens", "16"], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [ln for ln in r.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1, r.stdout          # rank 0 alone prints
    out = json.loads(lines[0])
    assert out["n_gpus"] == 2
    assert out["ms_per_step"] >= 2.0 > out["ms_rank0"]            # the slowest rank defines the step
    assert abs(out["value"] - 2 * 16 / (out["ms_per_step"] * 1e-3)) < 1e-6 * out["value"]


def test_bench_refuses_a_world_size_that_contradicts_gpus():
    import subprocess
    env = dict(os.environ, WORLD_SIZE="2", RANK="0", LOCAL_RANK="0")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "4", "--op", "plumbing"], env=env,
                       capture_output=True, text=True, timeout=120)
    assert r.returncode != 0 and "WORLD_SIZE" in (r.stderr + r.stdout)
