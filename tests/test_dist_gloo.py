"""The multi-rank bookkeeping of bench.py, run as two gloo ranks on the CPU.

The path shards as independent replicas (no data-path collective): each rank decodes its own
batch, the job time is the max over ranks and the job throughput the sum of the tokens.
"""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _worker(rank, world, port, q):
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    local_ms = [12.0, 20.0][rank]
    mx = bench.reduce_max_ms(local_ms, dist, torch.device("cpu"))
    q.put((rank, mx, bench.job_throughput(world, 8, 16, mx)))
    dist.barrier()
    dist.destroy_process_group()


def test_max_over_ranks_and_whole_job_throughput():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, mx, val in res:
        assert mx == 20.0                                  # the slowest replica sets the time
        assert val == 2 * 8 * 16 / 20e-3                   # tokens of both ranks / that time


def test_single_rank_needs_no_process_group():
    import bench
    assert bench.reduce_max_ms(5.0, None, torch.device("cpu")) == 5.0
    assert bench.job_throughput(1, 8, 4, 2.0) == 16000.0


def test_reference_arm_other_ranks_exit_without_work():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2"],
                       capture_output=True, text=True, env=env, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""


def test_timed_window_is_whole_blocks_whatever_the_arguments():
    import bench
    L, s = 4, 4                                            # cache copies, refresh interval
    for warm, steps in [(5, 20), (4, 16), (0, 1), (3, 17), (16, 32), (33, 7)]:
        Wn, Kn = bench.aligned_window(warm, steps, L * s)
        assert Wn >= max(warm, 1) and Kn >= max(steps, 1)
        assert Wn % (L * s) == 0 and Kn % (L * s) == 0
        # step i is decode step i // L of cache i % L: it retrieves iff (i // L) % s == 0
        retrievals = sum((i // L) % s == 0 for i in range(Wn, Wn + Kn))
        assert retrievals * s == Kn                        # the schedule's steady state, exactly
        for l in range(L):                                 # every cache's first step in the window retrieves
            first = next(i for i in range(Wn, Wn + Kn) if i % L == l)
            assert (first // L) % s == 0
    assert bench.aligned_window(5, 20, 16) == (16, 32)
