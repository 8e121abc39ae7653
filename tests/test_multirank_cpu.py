"""The N > 1 path of the benchmark on CPU: the store has no exchange step, so ranks are independent replicas
and only the result is combined (slowest rank's time, sum of the bytes).  Runs two gloo ranks."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = [10.0, 12.5][rank]
    nbytes = [4.0e9, 6.0e9][rank]
    res = bench.whole_job_throughput(dist, ms, nbytes, "cpu")
    mx = bench.reduce_over_ranks(dist, rank + 1, "max", "cpu")
    dist.barrier()
    out.put((rank, res, mx))
    dist.destroy_process_group()


def test_two_replicas_combine_as_max_time_and_sum_of_bytes():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = [q.get(timeout=120) for _ in procs]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, (ms, nbytes, gbps), mx in got:
        assert ms == 12.5 and nbytes == 1.0e10 and mx == 2.0
        assert abs(gbps - 1.0e10 / 12.5e-3 / 1e9) < 1e-9


def test_single_process_needs_no_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.whole_job_throughput(None, 5.0, 1e9, "cpu") == (5.0, 1e9, 1e9 / 5e-3 / 1e9)


def test_reference_arm_prints_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1", "--warmup", "0"],
                       env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""


def test_gpus_flag_starts_that_many_replicas():
    """`bench.py --gpus 2` outside any launcher must itself start two ranks (here with the CPU stub of the step and
    gloo) and report n_gpus 2, the slowest rank's time and the sum of the work."""
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--stub-cpu", "--steps", "4", "--warmup", "0"],
                       env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    out = json.loads(lines[0])
    assert out["n_gpus"] == 2 and out["config"]["replicas"] == 2
    assert out["ms_per_step"] == 12.5 / 4                      # max over ranks of 10.0 and 12.5 ms
    assert abs(out["value"] - 2 * 4.0e9 * 4 / 12.5e-3 / 1e9) < 0.1
