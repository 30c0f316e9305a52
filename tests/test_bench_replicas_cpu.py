"""The multi-GPU arm of bench.py is "replicas only": ranks share nothing on the data path, the
job's time is the slowest rank's and its work the sum over ranks.  Checked here with two gloo
ranks on the CPU."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    ms, units = bench.whole_job(10.0 + 5.0 * rank, 7.0, dist, "cpu")
    out.put((rank, ms, units))
    dist.barrier()
    dist.destroy_process_group()


def test_two_replicas_take_the_slowest_time_and_sum_the_work():
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
    assert [g[0] for g in got] == [0, 1]
    for _, ms, units in got:
        assert ms == 15.0          # MAX over ranks
        assert units == 14.0       # whole-job work


def test_gpus_flag_starts_its_own_replica_processes():
    """`python bench.py --gpus 2` run as a plain process (no torchrun around it, WORLD_SIZE
    unset) starts two ranks itself; the line rank 0 prints says n_gpus 2, the slowest rank's
    time and the summed work."""
    import json
    import subprocess
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_PORT")}
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--impl", "replicas-selftest"],
                       capture_output=True, text=True, timeout=300, env=env)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [json.loads(l) for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    assert lines[0]["n_gpus"] == 2 and lines[0]["ms_per_step"] == 15.0 and lines[0]["units"] == 14.0


def test_single_process_is_the_identity():
    import bench
    assert bench.whole_job(3.5, 2.0) == (3.5, 2.0)
