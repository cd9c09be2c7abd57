"""The N > 1 path of bench.py on CPU: two gloo ranks on 127.0.0.1.  The hot path itself does not
shard (replicas only), so what is multi-rank is the timing rule -- the job's time is the maximum
over ranks, the job's value the sum of all replicas' elements -- and the reference arm, which
only rank 0 runs."""
import os
import socket
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    my_ms = 10.0 * (rank + 1)                      # rank 1 is the slow one
    dist.barrier()
    ms = bench.max_over_ranks(my_ms, world, torch.device("cpu"))
    value = bench.job_value(world, elems_per_step=1000, steps=4, seconds=ms * 1e-3)
    out.put((rank, ms, value))
    dist.destroy_process_group()


def test_time_is_max_over_ranks_and_value_is_the_sum():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ms, value in res:
        assert ms == 20.0                           # the slowest rank's time, on every rank
        assert abs(value - 2 * 1000 * 4 / 0.020) < 1e-6


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""          # other ranks exit 0 without work
